"""Helpers shared by the GPU parity tests: moving seeded inputs to the device, running one block
through the C ABI, the tolerance rule, and the ReLU-gate protocol for gradients."""
from __future__ import annotations

import numpy as np
import torch

import synth_inputs as si
from oracle import sepconv_oracle as O

TD = {"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16}
# Tolerances: fp32 path max relative error 1e-4 (relative to max(|ref|, RMS(ref)));
# 16-bit paths max abs error <= 2e-2 * RMS(ref), per tensor.
TOL = {"f32": 1e-4, "f16": 2e-2, "bf16": 2e-2}
# ReLU gates the oracle may take from the GPU (pre-activation inside the tolerance band of zero): at most
# this fraction of the valid elements, plus five.  Measured rates are 1e-4 and below; the band itself
# holds about 1.6 % of a unit-variance pre-activation, so a rate near that would mean the GPU's
# pre-activations are noise at the scale of the band.
ADOPT_CAP = 1e-3


def dev(a: np.ndarray, dtype: str, device="cuda"):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(TD[dtype]).to(device)


def params_dev(p, dtype, device="cuda"):
    return {k: dev(v, dtype if k in si.IO_DTYPE_PARAMS else "f32", device) for k, v in p.items()}


def host(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def masked(t: torch.Tensor, valid) -> np.ndarray:
    """Host copy of a saved tensor with the frames beyond each sample's length (which the library
    leaves unspecified) set to zero."""
    m = torch.from_numpy(np.ascontiguousarray(np.broadcast_to(valid, tuple(t.shape)))).to(t.device)
    return host(torch.where(m, t, torch.zeros_like(t)))


def rms(a) -> float:
    a = np.asarray(a, dtype=np.float64)
    return float(np.sqrt(np.mean(a * a))) if a.size else 0.0


def half_ulp(ref, storage):
    """Half a unit in the last place of `storage` ("bf16": 8 significand bits, "f16": 11) at |ref|."""
    a = np.abs(np.asarray(ref, dtype=np.float64))
    bits = {"bf16": 8, "f16": 11}[storage]
    e = np.floor(np.log2(np.where(a > 0, a, 1.0)))
    if storage == "f16":
        e = np.maximum(e, -14)           # subnormal range: fixed spacing
    return np.where(a > 0, 2.0 ** (e - bits), 0.0)


def err_ratio(got, ref, dtype, mask=None, storage=None, stored_addend=None) -> float:
    """Error divided by the allowed error; <= 1 passes.  The error is taken over every element; the
    RMS that scales the allowance is taken over the valid (unpadded) frames when a mask is given,
    since padded frames are structural zeros on both sides.

    fp32:   |got - ref| <= 1e-4 * max(|ref|, RMS(ref)).
    16-bit: |got - ref| <= 2e-2 * RMS(ref)  (the plain bound).

    storage: the 16-bit type the tensor is stored in, if any (y, dx, dx_res, logits).  The plain bound
    is applied to every element whose half unit in the last place of that type, at the reference
    value, is at most half the plain allowance: there the final rounding takes at most half of the
    budget and the representation cannot be the excuse.  For the remaining large-magnitude elements
    the final rounding alone can use up (or exceed) the plain allowance whatever the arithmetic
    before it (bf16 at |ref| >= 4 RMS: half a unit is 0.008..0.03 RMS), so the allowance there is the
    plain one plus that half unit.  (With the threshold at the full allowance, elements whose half
    unit is within a few per cent of the allowance fail by those few per cent: measured 1.02 and
    1.08 on small blocks whose pre-rounding error is below 0.1 of the allowance.)

    stored_addend: reference values of a second tensor of the same storage type that is summed into
    this one (the projection residual's input gradient, which is a stored tensor of the activation
    type before it is added to the depthwise path's gradient).  Its own half unit is added to the
    allowance: that rounding happens whatever the arithmetic around it."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (got.shape, ref.shape)
    if ref.size == 0:
        return 0.0
    assert np.all(np.isfinite(got)), "non-finite values in the GPU result"
    r = rms(ref if mask is None else ref[np.broadcast_to(mask, ref.shape)])
    if dtype == "f32":
        denom = TOL[dtype] * np.maximum(np.abs(ref), r)
        denom = np.where(denom == 0, 1e-30, denom)
        return float(np.max(np.abs(got - ref) / denom))
    scale = TOL[dtype] * r
    if storage is not None:
        hu = half_ulp(ref, storage)
        allow = np.where(hu <= 0.5 * scale, scale, scale + hu)
        if stored_addend is not None:
            allow = allow + half_ulp(stored_addend, storage)
        allow = np.where(allow > 0, allow, 1e-300)
        return float(np.max(np.abs(got - ref) / allow))
    d = float(np.max(np.abs(got - ref)))
    return d / scale if scale > 0 else (0.0 if d == 0 else np.inf)


class Report:
    def __init__(self, dtype):
        self.dtype = dtype
        self.rows = []
        self.plain = []      # the same ratios with the plain bound on every element, for the record

    def add(self, name, got, ref, mask=None, stored=False, stored_addend=None):
        """stored=True: the tensor lives in the 16-bit activation type (y, dx, ...); see err_ratio."""
        storage = self.dtype if (stored and self.dtype != "f32") else None
        self.rows.append((name, err_ratio(got, ref, self.dtype, mask, storage, stored_addend if storage else None)))
        if storage is not None:
            self.plain.append((name, err_ratio(got, ref, self.dtype, mask)))

    def worst(self):
        return max(self.rows, key=lambda r: r[1]) if self.rows else ("", 0.0)

    def check(self, limit=1.0):
        bad = [(n, round(e, 3)) for n, e in self.rows if not e <= limit]
        assert not bad, f"outside tolerance (error/allowed): {bad}; all: {[(n, round(e, 3)) for n, e in self.rows]}"

    def __str__(self):
        t = ", ".join(f"{n}={e:.3f}" for n, e in self.rows)
        if self.plain:
            t += " | plain bound on every element: " + ", ".join(f"{n}={e:.3f}" for n, e in self.plain)
        return t


def adopt_gate(L, S, gate_gpu, dtype):
    """ReLU-gate protocol: where the oracle's pre-activation lies within the forward tolerance band of
    zero either gate is the derivative of an in-tolerance forward value, so the oracle's backward uses
    the GPU's decision there; a disagreement anywhere else is an error.  Returns (gate, n_adopted,
    n_hard_mismatch)."""
    valid = np.broadcast_to(S["valid"], S["a"].shape)
    a = S["a"]
    band = np.abs(a) <= TOL[dtype] * rms(a[valid])
    gate_o = a > 0
    mism = (gate_o != gate_gpu) & valid
    hard = int(np.sum(mism & ~band))
    gate = np.where(band, gate_gpu, gate_o)
    return gate, int(np.sum(mism & band)), hard


def gpu_gate(L, y_gpu, saved_gpu, params):
    """The ReLU decision the GPU took, reconstructed from its own outputs."""
    if L.res_before_relu or L.residual == "none":
        return host(y_gpu) > 0
    vh = (saved_gpu["v"].float() - saved_gpu["mean"][None, :, None]) * saved_gpu["invstd"][None, :, None]
    return (torch.addcmul(params["beta"].float()[None, :, None], params["gamma"].float()[None, :, None], vh)
            > 0).cpu().numpy()


def run_block(ctx, api, L, dtype, x, lengths, params, g, x_res=None, want_dx_res=False, dx_add=None):
    """Runs one block forward+backward through the C ABI and compares every tensor with the oracle.
    Returns the Report."""
    B, _, T = x.shape
    desc = api.block_desc(L, B, T, dtype)
    xd, pd = dev(x, dtype), params_dev(params, dtype)
    ld = torch.from_numpy(np.asarray(lengths, dtype=np.int32)).cuda()
    xrd = dev(x_res, dtype) if x_res is not None else None
    y, out_len, saved = api.sepconv_fwd(ctx, desc, xd, ld, pd, x_res=xrd)
    S = O.block_fwd(L, x, lengths, params, res_src=x_res)
    assert ctx.last_status() == 0
    np.testing.assert_array_equal(out_len.cpu().numpy(), S["out_len"])
    rep = Report(dtype)
    vm = S["valid"]
    if L.has_dw:
        rep.add("u", host(saved["u"]), S["u"], vm)
    if L.has_bn:
        rep.add("v", masked(saved["v"], vm), np.where(vm, S["v"], 0.0), vm)
        rep.add("mean", host(saved["mean"]), S["mean"])
        rep.add("invstd", host(saved["invstd"]), S["invstd"])
    if L.residual == "proj":
        rep.add("vr", masked(saved["vr"], vm), np.where(vm, S["vr"], 0.0), vm)
        rep.add("mean_r", host(saved["mean_r"]), S["mean_r"])
        rep.add("invstd_r", host(saved["invstd_r"]), S["invstd_r"])
    yh = host(y)
    rep.add("y", yh, S["y"], vm, stored=True)
    assert np.all(yh[~np.broadcast_to(S["valid"], yh.shape)] == 0), "padded output frames must be zero"

    gate = None
    adopted = hard = 0
    if L.has_relu:
        gate, adopted, hard = adopt_gate(L, S, gpu_gate(L, y, saved, pd), dtype)
    G = O.block_bwd(L, g, lengths, params, S, gate=gate)
    gd = dev(g, dtype)
    dxa = dev(dx_add, dtype) if dx_add is not None else None
    dx, dx_res, grads = api.sepconv_bwd(ctx, desc, gd, xd, y, ld, pd, saved, x_res=xrd, dx_add=dxa,
                                        want_dx_res=want_dx_res)
    assert ctx.last_status() == 0
    ref_dx = G["dx"]
    addend = None
    if "dx_res" in G and not want_dx_res:
        ref_dx = ref_dx + G["dx_res"]
        if L.residual == "proj":
            addend = G["dx_res"]       # computed, stored in the activation type, then summed into dx
    if dx_add is not None:
        ref_dx = ref_dx + np.where(O.time_mask(lengths, T), dx_add, 0.0)
    rep.add("dx", host(dx), ref_dx, O.time_mask(lengths, T), stored=True, stored_addend=addend)
    if want_dx_res:
        rep.add("dx_res", host(dx_res), G["dx_res"], vm, stored=True)
    for name in params:
        rep.add("d" + name, host(grads["d" + name]), G["d" + name])
    rep.adopted, rep.hard = adopted, hard
    rep.out = dict(y=y, saved=saved, dx=dx, dx_res=dx_res, grads=grads, out_len=out_len)
    n_valid = int(np.broadcast_to(S["valid"], S["a"].shape).sum())
    assert hard == 0, f"{hard} ReLU gates differ outside the tolerance band"
    assert adopted <= ADOPT_CAP * n_valid + 5, f"too many adopted gates: {adopted}/{n_valid}"
    return rep


# ---------------------------------------------------------------------------------------------------
# Teacher-forced chain.  The GPU runs first (every layer forward, then every layer backward, on its own
# stored tensors); after that each layer's comparison with the oracle is an independent task -- the
# oracle evaluates that layer on the GPU's stored input -- so the tasks can run side by side in a pool of
# CPU processes (the oracle is plain numpy and mostly single-threaded).
# ---------------------------------------------------------------------------------------------------
def _cpu(t):
    return None if t is None else t.detach().cpu()


def layer_task(t):
    """One layer, teacher-forced: the oracle on the stored input against the GPU's stored outputs.
    `t` holds CPU tensors / numpy arrays only.  Returns a picklable summary of the Report."""
    L, dtype = t["L"], t["dtype"]
    x, lengths, params = host(t["x"]), t["lengths"], t["params"]
    x_res = host(t["x_res"]) if t["x_res"] is not None else None
    S = O.block_fwd(L, x, lengths, params, res_src=x_res)
    rep = Report(dtype)
    assert np.array_equal(t["out_len"], S["out_len"]), "output lengths differ"
    vm = S["valid"]
    sv = t["saved"]
    if L.has_dw:
        rep.add("u", host(sv["u"]), S["u"], vm)
    if L.has_bn:
        rep.add("v", masked(sv["v"], vm), np.where(vm, S["v"], 0.0), vm)
    if L.residual == "proj":
        rep.add("vr", masked(sv["vr"], vm), np.where(vm, S["vr"], 0.0), vm)
    rep.add("y", host(t["y"]), S["y"], vm, stored=True)
    gate = None
    adopted = hard = 0
    if L.has_relu:
        gate, adopted, hard = adopt_gate(L, S, gpu_gate(L, t["y"], sv, t["pd"]), dtype)
    G = O.block_bwd(L, host(t["g"]), lengths, params, S, gate=gate)
    T = x.shape[2]
    ref_dx = G["dx"]
    addend = None
    if "dx_res" in G and not t["want_res"]:
        ref_dx = ref_dx + G["dx_res"]
        if L.residual == "proj":
            addend = G["dx_res"]
    if t["dx_add"] is not None:
        ref_dx = ref_dx + np.where(O.time_mask(lengths, T), host(t["dx_add"]), 0.0)
    rep.add("dx", host(t["dx"]), ref_dx, O.time_mask(lengths, T), stored=True, stored_addend=addend)
    if t["want_res"]:
        rep.add("dx_res", host(t["dx_res"]), G["dx_res"], vm, stored=True)
    for name in params:
        rep.add("d" + name, host(t["grads"]["d" + name]), G["d" + name])
    return dict(rows=rep.rows, plain=rep.plain, adopted=adopted, hard=hard, index=t["index"])


def _limit_threads(n):
    """Pool initialiser: keep each worker's BLAS to a few threads so that the workers do not fight."""
    global _THREAD_LIMIT
    try:
        from threadpoolctl import threadpool_limits
        _THREAD_LIMIT = threadpool_limits(limits=n)
    except Exception:
        _THREAD_LIMIT = None


def make_pool(workers=10, blas_threads=2):
    """A spawn pool for oracle tasks (a forked child of a process that has touched CUDA hangs)."""
    import multiprocessing as mp
    return mp.get_context("spawn").Pool(workers, initializer=_limit_threads, initargs=(blas_threads,))


def report_from(summary, dtype):
    rep = Report(dtype)
    rep.rows, rep.plain = list(summary["rows"]), list(summary["plain"])
    rep.adopted, rep.hard = summary["adopted"], summary["hard"]
    return rep


def run_chain(ctx, api, w, d, check=True, oracle_layers=None, pool=None):
    """Teacher-forced chain: every layer runs through sepconv_fwd / sepconv_bwd on the GPU's own
    previous output, and the oracle evaluates the same layer on the same (stored) input (in `pool`
    when one is given).  Returns (per-layer reports, dict of final GPU tensors)."""
    layers = w.layers
    n = len(layers)
    xs = [dev(d.x, w.dtype)]                       # what the GPU stored, layer by layer
    lens = [np.asarray(d.lengths)]
    fwd = []
    for i, L in enumerate(layers):
        B, _, T = xs[i].shape
        desc = api.block_desc(L, B, T, w.dtype)
        pd = params_dev(d.params[i], w.dtype)
        ld = torch.from_numpy(np.asarray(lens[i], dtype=np.int32)).cuda()
        j = L.res_from if L.res_from is not None else i
        xr = xs[j] if (L.residual != "none" and j != i) else None
        y, out_len, saved = api.sepconv_fwd(ctx, desc, xs[i], ld, pd, x_res=xr)
        fwd.append(dict(desc=desc, xd=xs[i], pd=pd, ld=ld, xr=xr, y=y, saved=saved, j=j))
        xs.append(y)
        lens.append(out_len.cpu().numpy())
    tasks = [None] * n
    g = dev(d.g, w.dtype)
    pending = {}
    grads_all = [None] * n
    final_dx = None
    for i in reversed(range(n)):
        L, f = layers[i], fwd[i]
        want_res = f["xr"] is not None
        dx_add = pending.pop(i, None)
        dx, dx_res, grads = api.sepconv_bwd(ctx, f["desc"], g, f["xd"], f["y"], f["ld"], f["pd"], f["saved"],
                                            x_res=f["xr"], dx_add=dx_add, want_dx_res=want_res)
        if want_res:          # several layers may feed one source: their residual gradients are summed as stored tensors
            pending[f["j"]] = dx_res if f["j"] not in pending else pending[f["j"]] + dx_res
        grads_all[i] = grads
        if oracle_layers is None or i in oracle_layers:
            tasks[i] = dict(index=i, L=L, dtype=w.dtype, x=_cpu(f["xd"]), lengths=lens[i], params=d.params[i],
                            x_res=_cpu(f["xr"]), out_len=lens[i + 1], saved={k: _cpu(v) for k, v in f["saved"].items()},
                            pd={k: _cpu(v) for k, v in f["pd"].items()}, y=_cpu(f["y"]), g=_cpu(g), dx=_cpu(dx),
                            dx_res=_cpu(dx_res), dx_add=_cpu(dx_add), want_res=want_res,
                            grads={k: _cpu(v) for k, v in grads.items()})
        g = dx
        final_dx = dx
    assert ctx.last_status() == 0
    todo = [t for t in tasks if t is not None]
    results = pool.map(layer_task, todo, chunksize=1) if pool is not None else [layer_task(t) for t in todo]
    reports = [None] * n
    for r in results:
        rep = report_from(r, w.dtype)
        if check:
            assert rep.hard == 0, f"layer {r['index']}: {rep.hard} ReLU gates differ outside the tolerance band"
            rep.check()
        reports[r["index"]] = rep
    return reports, dict(logits=fwd[-1]["y"], dx=final_dx, grads=grads_all, out_len=lens[-1],
                         ys=[f["y"] for f in fwd], saved=[f["saved"] for f in fwd], pds=[f["pd"] for f in fwd])


# ---------------------------------------------------------------------------------------------------
# End to end: the oracle on its own activations, and the control that says what to expect of it.
# ---------------------------------------------------------------------------------------------------
def end_to_end_task(t):
    """The oracle run end to end on its own activations against the one-call encoder's results.
    t: layers, dtype, x, lengths, params, g (numpy), ys (per-layer GPU outputs, CPU tensors), gate_extra
    (per layer: saved v / mean / invstd and gamma / beta where the ReLU decision is not y > 0), logits, dx, grads
    (per layer dict of CPU tensors).  Returns per-layer rows and the adopted / differing gate counts."""
    layers, dtype = t["layers"], t["dtype"]
    saved, lens = O.encoder_fwd(layers, t["x"], t["lengths"], t["params"])
    out = dict(y=[], plain=[], grads=[], adopted=0, hard=0, gates=0)
    gates = []
    for i, L in enumerate(layers):
        ref, vm = saved[i]["y"], saved[i]["valid"]
        out["y"].append(err_ratio(host(t["ys"][i]), ref, dtype, vm, dtype if dtype != "f32" else None))
        out["plain"].append(err_ratio(host(t["ys"][i]), ref, dtype, vm))
        if not L.has_relu:
            gates.append(None)
            continue
        ge = t["gate_extra"][i]
        gg = gpu_gate(L, t["ys"][i], ge, ge) if ge is not None else host(t["ys"][i]) > 0
        gt, a_, h_ = adopt_gate(L, saved[i], gg, dtype)
        gates.append(gt)
        out["adopted"] += a_; out["hard"] += h_; out["gates"] += int(np.broadcast_to(vm, ref.shape).sum())
    grads, dx_ref, _ = O.encoder_bwd(layers, t["g"], lens, t["params"], saved, gates=gates)
    T = t["x"].shape[2]
    st = dtype if dtype != "f32" else None
    out["dx"] = err_ratio(host(t["dx"]), dx_ref, dtype, O.time_mask(t["lengths"], T), st)
    out["dx_plain"] = err_ratio(host(t["dx"]), dx_ref, dtype, O.time_mask(t["lengths"], T))
    for i in range(len(layers)):
        out["grads"].append([("d" + name, err_ratio(host(t["grads"][i]["d" + name]), grads[i]["d" + name], dtype))
                             for name in t["params"][i]])
    return out


def storage_control_task(t):
    """What correctly rounded storage alone does to this network: the oracle's own arithmetic, exact, but with
    every layer's output rounded to the activation type before the next layer reads it (and, backward, every
    layer's input gradient likewise), against the oracle without any rounding.  A batch-normalised ReLU
    network at random initialisation amplifies a perturbation of its activations by a roughly constant
    factor per layer, so this error grows geometrically with depth whatever the implementation; the
    control measures that growth on the workload at hand.  Returns per-layer ratios as end_to_end_task.
    The two chains (exact, rounded) run in two threads: numpy releases the interpreter lock in its loops."""
    from concurrent.futures import ThreadPoolExecutor
    layers, dtype = t["layers"], t["dtype"]
    n = len(layers)
    rnd = lambda a: si.quantise(np.asarray(a, dtype=np.float32), dtype).astype(np.float64)

    def exact_chain():
        saved, lens = O.encoder_fwd(layers, t["x"], t["lengths"], t["params"])
        grads, dx, _ = O.encoder_bwd(layers, t["g"], lens, t["params"], saved)
        return [(S["y"], S["valid"]) for S in saved], grads, dx

    def rounded_chain():
        acts = [np.asarray(t["x"], dtype=np.float64)]
        lens = [np.asarray(t["lengths"], dtype=np.int64)]
        Sq = []
        for i, L in enumerate(layers):
            res = acts[L.res_from if L.res_from is not None else i] if L.residual != "none" else None
            S = O.block_fwd(L, acts[i], lens[i], t["params"][i], res_src=res)
            S["y"] = rnd(S["y"])
            Sq.append(S)
            acts.append(S["y"])
            lens.append(S["out_len"])
        grads_q = [None] * n
        pend = {}
        cur = np.asarray(t["g"], dtype=np.float64)
        for i in reversed(range(n)):      # its own gates; input gradients rounded to the activation type
            L = layers[i]
            G = O.block_bwd(L, cur, lens[i], t["params"][i], Sq[i])
            dx = G["dx"]
            if "dx_res" in G:
                j = L.res_from if L.res_from is not None else i
                pend[j] = pend.get(j, 0.0) + rnd(G.pop("dx_res"))
            if i in pend:
                dx = dx + pend.pop(i)
            cur = rnd(dx)
            grads_q[i] = G
        return [S["y"] for S in Sq], grads_q, cur

    with ThreadPoolExecutor(2) as ex:
        fa, fb = ex.submit(exact_chain), ex.submit(rounded_chain)
        (ys, gp, dxp), (yq, gq, dxq) = fa.result(), fb.result()
    st = dtype if dtype != "f32" else None
    T = t["x"].shape[2]
    out = dict(y=[err_ratio(yq[i], ys[i][0], dtype, ys[i][1], st) for i in range(n)], grads=[])
    out["dx"] = err_ratio(dxq, dxp, dtype, O.time_mask(t["lengths"], T), st)
    for i in range(n):
        out["grads"].append([("d" + name, err_ratio(gq[i]["d" + name], gp[i]["d" + name], dtype)) for name in t["params"][i]])
    return out
