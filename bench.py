#!/usr/bin/env python
"""Benchmark: encoder forward+backward audio frames per second on B200.

One "step" = one encoder_fwd_bwd call (every layer forward, then backward) over one synthetic batch.
Default workload: the bf16 QuartzNet-5x5-style encoder, B=32, T=1600 input frames, full lengths
(config 4); `--config 5` runs the ragged B=64, T=3200 encoder.  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config 4|5] [--impl reference]
                  [--no-cpu-baseline] [--no-e2e] [--host-launches] [--block C_in,C_out,K,B,T]

The timed steps replay one captured CUDA graph of the step (`--host-launches`: every kernel launched from the host
instead; the line reports the other mode's time beside the timed one).

Besides the step throughput the line carries `roofline_per_class`: for every kernel class of the step
its CUDA-event time, launches, algorithmic bytes and flops (every tensor the class must read or write
once, 16-bit activations, valid frames only), the bound that binds it (the slower of its flops at the
measured tensor peak and its bytes at the measured HBM peak) and the fraction of that bound it reaches;
`roofline` repeats the entry of the class with the largest share of the step.

N > 1 (under torchrun): every rank runs an independent replica of the same workload on its own GPU
(the path has no exchange step); value = N * frames / max-over-ranks time.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import synth_inputs as si  # noqa: E402

METRIC = "encoder fwd+bwd audio frames/sec"
UNIT = "frames/s"
TOLERANCE = {"fp32": "max |err| <= 1e-4 * max(|ref|, RMS ref) per tensor",
             "16bit": "max |err| <= 2e-2 * RMS(ref over valid frames) per tensor; for tensors stored in bf16/fp16 the "
                      "elements whose half unit in the last place exceeds that allowance get the half unit added"}


def kernels_sha():
    """Hash of the kernel sources: ties a committed counter summary to the kernels it was taken on."""
    import hashlib
    h = hashlib.sha256()
    d = os.path.join(ROOT, "paper_1909_09577_b200", "csrc")
    for fn in sorted(os.listdir(d)):
        if fn.endswith((".cu", ".cuh", ".h")):
            h.update(open(os.path.join(d, fn), "rb").read())
    return h.hexdigest()[:16]


def dram_traffic_ratios():
    """Measured DRAM bytes / algorithmic bytes per kernel class, from the committed ncu summary
    profiles/dram_traffic_by_class.txt (lines `class <name> dram_bytes <x> algorithmic_bytes <y>` taken on
    one block of the workload, plus `kernels_sha <hash of the kernel sources at capture time>`).  Returns
    {} when the file is absent or the kernel sources have changed since the counters were taken."""
    path = os.path.join(ROOT, "profiles", "dram_traffic_by_class.txt")
    if not os.path.exists(path):
        return {}
    ratios, sha = {}, None
    for line in open(path):
        f = line.split()
        if len(f) >= 2 and f[0] == "kernels_sha":
            sha = f[1]
        if len(f) >= 6 and f[0] == "class" and f[2] == "dram_bytes" and f[4] == "algorithmic_bytes":
            ratios[f[1]] = float(f[3]) / float(f[5])
    return ratios if sha == kernels_sha() else {}


def class_rooflines(prof, nsteps, valid_frac, peaks, traffic_ratio):
    """Per kernel class: time, launches, algorithmic work on valid frames, binding bound and fraction.
    The launchers count padded frames (they cannot see the lengths); every per-position cost scales
    with the valid fraction, which the caller knows from the host copy of the lengths."""
    out = {}
    tot = sum(v["ms"] for v in prof.values()) or 1.0
    for k, v in prof.items():
        ms = v["ms"] / nsteps
        by, fl = v["bytes"] * valid_frac / nsteps, v["flops"] * valid_frac / nsteps
        t_hbm = by / (peaks["hbm_gbs"] * 1e9) * 1e3
        t_ten = fl / (peaks["bf16_tflops_sustained"] * 1e12) * 1e3
        bound = "tensor" if (k.startswith("pw_") and t_ten > t_hbm) else "hbm"
        gbs, tfs = by / ms / 1e6, fl / ms / 1e9
        lps = v["launches"] / nsteps
        out[k] = {"ms_per_step": ms, "launches_per_step": lps, "share": v["ms"] / tot,
                  "algorithmic_bytes": by, "flops": fl, "GB/s": gbs, "TFLOP/s": tfs, "bound": bound,
                  "frac": (t_ten if bound == "tensor" else t_hbm) / ms if ms > 0 else None,
                  "hbm_frac": gbs / peaks["hbm_gbs"], "tensor_frac": tfs / peaks["bf16_tflops_sustained"],
                  "traffic": traffic_ratio[k] * by / lps if k in traffic_ratio and lps else None}
    return out


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.rows = []
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(gpu_index)],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], None, set()
        for ts, line in self.rows:
            f = [q.strip() for q in line.split(",")]
            if len(f) < 9:
                continue
            try:
                clk = float(f[1]); mx = float(f[2])
            except ValueError:
                continue
            if t0 - 0.05 <= ts <= t1 + 0.15:
                sm.append(clk)
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        if not sm:   # region shorter than the sampling period: use all samples
            for ts, line in self.rows:
                f = [q.strip() for q in line.split(",")]
                try:
                    sm.append(float(f[1]))
                except Exception:
                    pass
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


def max_over_ranks(ms, device=None):
    """Slowest rank's time (every rank gets it); a no-op outside a process group."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(frames_per_rank_step, steps, ms_max, world):
    """Whole-job frames per second: every rank ran `steps` independent replicas' steps in ms_max."""
    return world * frames_per_rank_step * steps / (ms_max * 1e-3)


def oracle_sample(w, B_sample, repeats=1):
    """Times the fp64 oracle (as it stands) on a B_sample-sample slice of the workload.
    Returns (frames per second, threads used, description)."""
    from oracle import sepconv_oracle as O
    ws = si.Workload(w.name, w.dtype, B_sample, w.T, w.layers, w.seed, w.len_lo, w.len_hi, w.affine)
    d = si.draw(ws)
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count() or 1
    t0 = time.perf_counter()
    for _ in range(repeats):
        saved, lens = O.encoder_fwd(ws.layers, d.x, d.lengths, d.params)
        O.encoder_bwd(ws.layers, d.g, lens, d.params, saved)
    dt = (time.perf_counter() - t0) / repeats
    frames = B_sample * w.T
    return frames / dt, cores, dt, f"{B_sample} of {w.B} samples of {w.name} (T={w.T}), full encoder fwd+bwd, numpy fp64"


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = si.config(args.config)
    Bs = 1
    # each step = one bounded sample; warmup + steps kept to a few minutes in total
    vals = []
    cores = 1
    desc = ""
    for i in range(args.warmup + args.steps):
        v, cores, dt, desc = oracle_sample(w, Bs)
        if i >= args.warmup:
            vals.append((v, dt))
    fps = float(np.mean([v for v, _ in vals]))
    ms = float(np.mean([dt for _, dt in vals]) * 1e3)
    line = {"metric": METRIC, "value": fps, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "impl": "reference",
            "config": {"workload": w.name, "B": w.B, "T_in": w.T, "sample": desc},
            "cpu_baseline": {"value": fps, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": fps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=4, choices=[4, 5])
    ap.add_argument("--block", default=None,
                    help="profile aid: time one sepconv block instead of the encoder, as C_in,C_out,K,B,T "
                         "(e.g. 512,512,63,32,800); residual projection from the block input")
    ap.add_argument("--no-e2e", action="store_true", help="skip the end-to-end (host buffers) leg")
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--breakdown", default=None, help="also write the per-kernel-class table to this text file")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--gemm-mode", type=int, default=0)
    ap.add_argument("--tile-shape", type=int, default=None, help="tile shape of the pointwise contractions (0..5, see sepconv_set_tile_shape)")
    ap.add_argument("--dp", action="store_true",
                    help="with N > 1 ranks: data-parallel step -- every rank its own batch, per-replica batch statistics, "
                         "and an NCCL all-reduce of the gradient blob inside the step (default: independent replicas)")
    ap.add_argument("--stream-priority", type=int, default=0,
                    help="priority of the stream the step is captured on (0 = default, -1 = above the library's second stream)")
    ap.add_argument("--no-pdl", action="store_true", help="launch kernels without programmatic stream serialization")
    ap.add_argument("--no-overlap", action="store_true",
                    help="every kernel on one stream in program order (default: weight gradients and the residual "
                         "projection overlap the critical path on the library's second stream)")
    ap.add_argument("--host-launches", action="store_true",
                    help="launch every kernel of every step from the host, with programmatic dependent launch (default: the "
                         "step is captured once as a CUDA graph and replayed; the other mode's time is reported beside it)")
    ap.add_argument("--graph", action="store_true", help=argparse.SUPPRESS)
    ap.add_argument("--no-graph", action="store_true", help=argparse.SUPPRESS)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    args.no_graph = args.host_launches or args.no_graph
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist
    import paper_1909_09577_b200 as api

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)

    w = si.config(args.config)
    if args.block:
        ci, co, k, bb, tt = [int(q) for q in args.block.split(",")]
        w = si.Workload(f"block_{ci}_{co}_k{k}_B{bb}_T{tt}", "bf16", bb, tt,
                        [si.LayerCfg(ci, co, K=k, residual="proj")], seed=5)
    d = si.draw(w)
    ctx = api.Context(local)
    ctx.set_gemm_mode(args.gemm_mode)
    ctx.set_overlap(not args.no_overlap, not args.no_pdl)
    if args.tile_shape is not None:
        ctx.set_tile_shape(args.tile_shape)
    spec = api.EncoderSpec(w.layers, w.B, w.T, w.dtype)
    td = api.binding.TORCH_DTYPE[spec.code]
    blob = spec.pack_params(d.params, dev)
    # host (pinned) copies of the per-step inputs and of the per-step results
    x_h = torch.from_numpy(d.x).to(td).pin_memory()
    g_h = torch.from_numpy(d.g).to(td).pin_memory()
    len_h = torch.from_numpy(d.lengths).pin_memory()
    x_d, g_d, len_d = x_h.to(dev), g_h.to(dev), len_h.to(dev)
    logits = torch.empty((w.B, spec.C_out, spec.T_out), dtype=td, device=dev)
    grads = torch.zeros(spec.grad_bytes, dtype=torch.uint8, device=dev)
    ws = torch.empty(api.encoder_workspace_bytes(spec), dtype=torch.uint8, device=dev)
    logits_h = torch.empty(logits.shape, dtype=td).pin_memory()
    grads_h = torch.empty(spec.grad_bytes, dtype=torch.uint8).pin_memory()
    stream = torch.cuda.current_stream()

    dp_exchange = args.dp and world > 1
    if dp_exchange:
        from paper_1909_09577_b200 import data_parallel as dp
        args.no_graph = True          # the collective is launched from the host every step

    def step():
        api.encoder_fwd_bwd(ctx, spec, x_d, len_d, blob, g_d, grads_blob=grads, workspace=ws, logits=logits)
        if dp_exchange:
            dp.all_reduce_gradients(grads)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps, finish=None):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        t0 = time.time()
        e0.record(stream)
        for _ in range(steps):
            fn()
        if finish:
            finish()
        e1.record(stream)
        barrier()
        t1 = time.time()
        ms = max_over_ranks(e0.elapsed_time(e1), dev)
        return ms, t0, t1

    for _ in range(args.warmup):
        step()
    assert ctx.last_status() == 0
    launches_per_step = None
    if not args.no_graph:
        # The step is a fixed sequence of stream-ordered launches on fixed buffers: capture it once and
        # replay it, which removes the per-launch host cost and most of the inter-kernel gaps.
        l0 = ctx.launch_count()
        graph = torch.cuda.CUDAGraph()
        cap_stream = torch.cuda.Stream(priority=args.stream_priority)
        cap_stream.wait_stream(torch.cuda.current_stream())
        with torch.cuda.graph(graph, stream=cap_stream):
            api.encoder_fwd_bwd(ctx, spec, x_d, len_d, blob, g_d, grads_blob=grads, workspace=ws, logits=logits,
                                stream=cap_stream)
        launches_per_step = ctx.launch_count() - l0
        eager_step = step

        def step():
            graph.replay()
        for _ in range(2):
            step()
        assert ctx.last_status() == 0

    # ---- device-resident timing ------------------------------------------------------------------
    sampler = ClockSampler(local) if rank == 0 else None
    l0 = ctx.launch_count()
    ms, t0, t1 = timed(step, args.steps)
    launches = (ctx.launch_count() - l0) if args.no_graph else launches_per_step * args.steps
    clocks = sampler.stop(t0, t1) if sampler else None
    other_ms = None
    if args.no_graph and not dp_exchange:
        # for context: the same K steps replayed as one captured CUDA graph (no per-launch host cost)
        try:
            graph = torch.cuda.CUDAGraph()
            cap_stream = torch.cuda.Stream(priority=args.stream_priority)
            cap_stream.wait_stream(torch.cuda.current_stream())
            with torch.cuda.graph(graph, stream=cap_stream):
                api.encoder_fwd_bwd(ctx, spec, x_d, len_d, blob, g_d, grads_blob=grads, workspace=ws, logits=logits,
                                    stream=cap_stream)
            for _ in range(3):
                graph.replay()
            other_ms, _, _ = timed(graph.replay, args.steps)
            other_ms /= args.steps
        except Exception as e:      # the comparison figure is optional
            other_ms = None
    elif not dp_exchange:
        # for context: the same K steps launched kernel by kernel from the host (programmatic dependent launch)
        for _ in range(2):
            eager_step()
        other_ms, _, _ = timed(eager_step, args.steps)
        other_ms /= args.steps
    # Per-kernel-class CUDA-event brackets cannot sit inside a replayed graph: every class is timed right
    # after the timed region, same buffers and kernels, launched one by one from the host.
    # The profiled steps run every kernel alone, in program order (overlap off): a class's time is its kernels'
    # own duration, not that of whatever shared the GPU with them.
    nprof = max(3, args.steps // 4)
    ctx.set_overlap(False, False)
    ctx.profile_begin("all", max_launches=600 * nprof)
    for _ in range(nprof):
        (step if args.no_graph else eager_step)()
    prof = ctx.profile_end()
    ctx.set_overlap(not args.no_overlap, not args.no_pdl)

    # ---- end to end: pinned host inputs in, logits + gradients out, every step --------------------
    # Every step copies its inputs from pinned host memory and its logits and gradients back to pinned host memory.
    # Two buffer sets alternate and the copies run on two streams of their own, so that the copies of steps k - 1 and
    # k + 1 overlap the kernels of step k; the timed region starts before the first copy and ends after the last.
    if args.no_e2e:
        ms_e2e = float("nan")
    else:
        h2d_s, d2h_s = torch.cuda.Stream(), torch.cuda.Stream()
        sets = []
        for _ in range(2):
            q = {"x": x_h.to(dev), "g": g_h.to(dev), "len": len_h.to(dev), "logits": torch.empty_like(logits),
                 "grads": torch.zeros_like(grads), "logits_h": torch.empty(logits.shape, dtype=td).pin_memory(),
                 "grads_h": torch.empty(spec.grad_bytes, dtype=torch.uint8).pin_memory(),
                 "ev_in": torch.cuda.Event(), "ev_comp": torch.cuda.Event(), "ev_out": torch.cuda.Event(), "used": False}

            def run(q=q, strm=None):
                api.encoder_fwd_bwd(ctx, spec, q["x"], q["len"], blob, q["g"], grads_blob=q["grads"], workspace=ws,
                                    logits=q["logits"], **({"stream": strm} if strm is not None else {}))
            if args.no_graph:
                q["run"] = run
            else:
                gq = torch.cuda.CUDAGraph()
                cs = torch.cuda.Stream(priority=args.stream_priority)
                cs.wait_stream(torch.cuda.current_stream())
                with torch.cuda.graph(gq, stream=cs):
                    run(strm=cs)
                q["graph"] = gq
                q["run"] = gq.replay
            sets.append(q)
        torch.cuda.synchronize()
        counter = [0]

        def step_e2e():
            q = sets[counter[0] & 1]
            counter[0] += 1
            with torch.cuda.stream(h2d_s):
                if q["used"]:
                    h2d_s.wait_event(q["ev_comp"])      # the previous step on this set has read its inputs
                q["x"].copy_(x_h, non_blocking=True)
                q["g"].copy_(g_h, non_blocking=True)
                q["len"].copy_(len_h, non_blocking=True)
                q["ev_in"].record(h2d_s)
            stream.wait_event(q["ev_in"])
            if q["used"]:
                stream.wait_event(q["ev_out"])          # ... and its results have left the device buffers
            q["run"]()
            if dp_exchange:
                dp.all_reduce_gradients(q["grads"])
            q["ev_comp"].record(stream)
            with torch.cuda.stream(d2h_s):
                d2h_s.wait_event(q["ev_comp"])
                q["logits_h"].copy_(q["logits"], non_blocking=True)
                q["grads_h"].copy_(q["grads"], non_blocking=True)
                q["ev_out"].record(d2h_s)
            q["used"] = True

        def finish_e2e():
            for q in sets:
                if q["used"]:
                    stream.wait_event(q["ev_out"])

        for _ in range(4):
            step_e2e()
        finish_e2e()
        ms_e2e, _, _ = timed(step_e2e, args.steps, finish_e2e)
        assert ctx.last_status() == 0
        assert torch.equal(sets[0]["logits_h"], sets[1]["logits_h"]) and torch.equal(sets[0]["grads_h"], sets[1]["grads_h"])
    h2d = x_h.numel() * x_h.element_size() + g_h.numel() * g_h.element_size() + len_h.numel() * 4
    d2h = logits_h.numel() * logits_h.element_size() + grads_h.numel()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    frames = w.B * w.T
    peaks = measured_peaks()
    value = job_throughput(frames, args.steps, ms, world)
    e2e = job_throughput(frames, args.steps, ms_e2e, world)
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
            "config": {"workload": w.name, "B": w.B, "T_in": w.T, "layers": len(w.layers),
                       "valid_frames": int(d.lengths.sum()), "l2": "per-step working set (GBs) exceeds L2",
                       "parallelism": ("dp%d: per-replica batch statistics, gradient all-reduce (NCCL)" % world) if dp_exchange
                       else ("replicas" if world > 1 else "single"),
                       "launch": "host launches, programmatic dependent launch" if args.no_graph else "CUDA graph replay",
                       ("graph_replay_ms_per_step" if args.no_graph else "host_launch_ms_per_step"): other_ms,
                       "overlap": "off" if args.no_overlap else "weight gradients and residual projection on a second stream"},
            "clocks": clocks, "gpu_launches": int(launches),
            "e2e": {"value": e2e, "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                    "ms_per_step": ms_e2e / args.steps,
                    "note": "inputs from pinned host memory and logits + gradients back to pinned host memory every step; two "
                            "buffer sets, copies on their own streams overlap the neighbouring steps' kernels"}}
    valid_frac = float(d.lengths.sum()) / float(w.B * w.T)
    per_class = class_rooflines(prof, nprof, valid_frac, peaks, dram_traffic_ratios())
    line["tolerance"] = TOLERANCE
    line["roofline_per_class"] = per_class
    line["roofline_note"] = ("class times: CUDA events around every launch of %d host-launched steps run right after the "
                             "timed region, one stream, no overlap (they sum to %.3f ms/step against %.3f ms for the "
                             "timed step, in which independent kernels overlap); bytes and "
                             "flops are algorithmic, valid frames only; peaks: %s HBM %.0f GB/s, bf16 %.0f TFLOP/s sustained"
                             % (nprof, sum(v["ms_per_step"] for v in per_class.values()), ms / args.steps,
                                peaks["source"], peaks["hbm_gbs"], peaks["bf16_tflops_sustained"]))
    if per_class:
        top = max(per_class, key=lambda k: per_class[k]["share"])
        e = per_class[top]
        tens = e["bound"] == "tensor"
        line["roofline"] = {"kernel": top, "bound": e["bound"], "achieved": e["TFLOP/s"] if tens else e["GB/s"],
                            "peak": peaks["bf16_tflops_sustained"] if tens else peaks["hbm_gbs"],
                            "unit": "TFLOP/s" if tens else "GB/s", "frac": e["frac"], "traffic": e["traffic"],
                            "peak_source": peaks["source"], "launches": e["launches_per_step"] * nprof,
                            "avg_ms": e["ms_per_step"] / e["launches_per_step"], "share_of_step": e["share"]}
    if args.breakdown:
        with open(args.breakdown, "w") as f:
            f.write(f"# per-kernel-class CUDA-event time, {w.name}, {nprof} host-launched steps; "
                    f"timed step ({'host launches' if args.no_graph else 'graph replay'}) {ms / args.steps:.3f} ms\n")
            f.write("class launches/step ms/step share GB/s TFLOP/s bound frac\n")
            for k, v in sorted(per_class.items(), key=lambda kv: -kv[1]["share"]):
                f.write(f"{k} {v['launches_per_step']:.0f} {v['ms_per_step']:.4f} {v['share']:.3f} {v['GB/s']:.0f} "
                        f"{v['TFLOP/s']:.1f} {v['bound']} {v['frac']:.3f}\n")
    if not args.no_cpu_baseline and world == 1:
        v, cores, dt, desc = oracle_sample(w, 1)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc,
                                "seconds": dt, "note": "a one-sample slice: its batch statistics run over that sample "
                                                       "alone, so it is the same arithmetic per frame, not the same batch"}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
