#!/usr/bin/env python
"""Benchmark: encoder forward+backward audio frames per second on B200.

One "step" = one encoder_fwd_bwd call (every layer forward, then backward) over one synthetic batch.
Default workload: the bf16 QuartzNet-5x5-style encoder, B=32, T=1600 input frames, full lengths
(config 4); `--config 5` runs the ragged B=64, T=3200 encoder.  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config 4|5] [--impl reference]
                  [--profile-class NAME|all] [--no-cpu-baseline]

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
# The kernel class that takes the largest share of the step (see profiles/); its roofline is reported.
DOMINANT_CLASS = "pw_fwd"
# measured DRAM bytes / algorithmic bytes of that class's kernel (profiles/block512_dram_traffic.txt:
# the 512->512 forward contraction read 26.8 MB and wrote 0.1 MB to DRAM for 78.6 MB of operands and
# results -- the fp32 result stays in the 126 MB L2 for the kernel that consumes it); scales with the
# elements processed
TRAFFIC_RATIO = {"pw_fwd": 26.9 / 78.6}


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
    ap.add_argument("--profile-class", default=DOMINANT_CLASS)
    ap.add_argument("--breakdown", default=None, help="write a per-kernel-class event-time table to this file")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--gemm-mode", type=int, default=0)
    ap.add_argument("--no-graph", action="store_true",
                    help="launch every kernel from the host each step instead of replaying a captured CUDA graph")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
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

    def step():
        api.encoder_fwd_bwd(ctx, spec, x_d, len_d, blob, g_d, grads_blob=grads, workspace=ws, logits=logits)

    def step_e2e():
        x_d.copy_(x_h, non_blocking=True)
        g_d.copy_(g_h, non_blocking=True)
        len_d.copy_(len_h, non_blocking=True)
        step()
        logits_h.copy_(logits, non_blocking=True)
        grads_h.copy_(grads, non_blocking=True)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        t0 = time.time()
        e0.record(stream)
        for _ in range(steps):
            fn()
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
        cap_stream = torch.cuda.Stream()
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

    # ---- device-resident timing; the dominant kernel class is bracketed with events meanwhile ----
    sampler = ClockSampler(local) if rank == 0 else None
    l0 = ctx.launch_count()
    if args.no_graph:
        ctx.profile_begin(args.profile_class, max_launches=8192)
    ms, t0, t1 = timed(step, args.steps)
    if args.no_graph:
        prof = ctx.profile_end()
        launches = ctx.launch_count() - l0
    else:
        launches = launches_per_step * args.steps
        # per-kernel event brackets cannot sit inside a replayed graph: the dominant kernel class is
        # timed right after, same buffers and kernels, launched one by one
        ctx.profile_begin(args.profile_class, max_launches=8192)
        for _ in range(max(3, args.steps // 2)):
            eager_step()
        prof = ctx.profile_end()
    clocks = sampler.stop(t0, t1) if sampler else None

    # ---- end to end: pinned host inputs in, logits + gradients out, every step --------------------
    if args.no_e2e:
        ms_e2e = float("nan")
    else:
        for _ in range(2):
            step_e2e()
        ms_e2e, _, _ = timed(step_e2e, args.steps)
    h2d = x_h.numel() * x_h.element_size() + g_h.numel() * g_h.element_size() + len_h.numel() * 4
    d2h = logits_h.numel() * logits_h.element_size() + grads_h.numel()

    if args.breakdown and rank == 0:
        ctx.profile_begin("all", max_launches=8192)
        nb = 3
        for _ in range(nb):
            (step if args.no_graph else eager_step)()
        allp = ctx.profile_end()
        tot = sum(v["ms"] for v in allp.values())
        with open(args.breakdown, "w") as f:
            f.write(f"# per-kernel-class CUDA-event time, {w.name}, {nb} steps; sum {tot / nb:.3f} ms/step\n")
            f.write("class launches/step ms/step share GB/s TFLOP/s\n")
            for k, v in sorted(allp.items(), key=lambda kv: -kv[1]["ms"]):
                f.write(f"{k} {v['launches'] / nb:.0f} {v['ms'] / nb:.4f} {v['ms'] / tot:.3f} "
                        f"{v['bytes'] / v['ms'] / 1e6:.0f} {v['flops'] / v['ms'] / 1e9:.1f}\n")

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
                       "parallelism": "replicas" if world > 1 else "single",
                       "launch": "host launches" if args.no_graph else "CUDA graph replay"},
            "clocks": clocks, "gpu_launches": int(launches),
            "e2e": {"value": e2e, "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                    "ms_per_step": ms_e2e / args.steps}}
    pc = prof.get(args.profile_class)
    if pc:
        per_ms = pc["ms"] / pc["launches"]
        gbs = pc["bytes"] / pc["ms"] / 1e6
        tfs = pc["flops"] / pc["ms"] / 1e9
        alu_peak = 148 * 128 * 1.965e9 / 1e12     # T FMA/s: SMs x fp32 lanes x max clock
        if args.profile_class.startswith("dw_"):
            line["roofline"] = {"kernel": args.profile_class, "bound": "alu", "achieved": tfs / 2, "peak": alu_peak,
                                "unit": "TFMA/s", "frac": tfs / 2 / alu_peak,
                                "traffic": (TRAFFIC_RATIO[args.profile_class] * pc["bytes"] / pc["launches"]
                                            if args.profile_class in TRAFFIC_RATIO else None),
                                "hbm_gbs": gbs, "hbm_frac": gbs / peaks["hbm_gbs"], "peak_source": "derived: 148 SMs x 128 lanes x 1.965 GHz",
                                "launches": pc["launches"], "avg_ms": per_ms}
        elif (args.profile_class.startswith("pw_") and args.gemm_mode == 0
              and tfs / peaks["bf16_tflops_sustained"] > gbs / peaks["hbm_gbs"]):
            # the class's FLOPs at the tensor peak take longer than its bytes at the HBM peak
            line["roofline"] = {"kernel": args.profile_class, "bound": "tensor", "achieved": tfs,
                                "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                                "frac": tfs / peaks["bf16_tflops_sustained"],
                                "traffic": (TRAFFIC_RATIO[args.profile_class] * pc["bytes"] / pc["launches"]
                                            if args.profile_class in TRAFFIC_RATIO else None),
                                "hbm_gbs": gbs, "hbm_frac": gbs / peaks["hbm_gbs"],
                                "peak_source": peaks["source"], "launches": pc["launches"], "avg_ms": per_ms}
        else:
            line["roofline"] = {"kernel": args.profile_class, "bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"],
                                "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                                "traffic": (TRAFFIC_RATIO[args.profile_class] * pc["bytes"] / pc["launches"]
                                            if args.profile_class in TRAFFIC_RATIO else None),
                                "tflops": tfs, "tensor_frac": tfs / peaks["bf16_tflops_sustained"],
                                "peak_source": peaks["source"], "launches": pc["launches"], "avg_ms": per_ms}
    if not args.no_cpu_baseline and world == 1:
        v, cores, dt, desc = oracle_sample(w, 1)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc,
                                "seconds": dt}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
