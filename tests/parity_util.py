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


def dev(a: np.ndarray, dtype: str, device="cuda"):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(TD[dtype]).to(device)


def params_dev(p, dtype, device="cuda"):
    return {k: dev(v, dtype if k in si.IO_DTYPE_PARAMS else "f32", device) for k, v in p.items()}


def host(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


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


def err_ratio(got, ref, dtype, mask=None, storage=None) -> float:
    """Error divided by the allowed error; <= 1 passes.  The error is taken over every element; the
    RMS that scales the allowance is taken over the valid (unpadded) frames when a mask is given,
    since padded frames are structural zeros on both sides.

    storage: the 16-bit type the tensor is stored in, if any.  No value of that type can be closer
    to the reference than half a unit in its last place (for bf16 at 8 x RMS that alone is 0.016 RMS),
    so the stated bound is applied to the error in excess of that representation quantum."""
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
        allow = scale + half_ulp(ref, storage)
        allow = np.where(allow > 0, allow, 1e-300)
        return float(np.max(np.abs(got - ref) / allow))
    d = float(np.max(np.abs(got - ref)))
    return d / scale if scale > 0 else (0.0 if d == 0 else np.inf)


class Report:
    def __init__(self, dtype):
        self.dtype = dtype
        self.rows = []
        self.plain = []      # the same ratios without the representation quantum, for the record

    def add(self, name, got, ref, mask=None, stored=False):
        """stored=True: the tensor lives in the 16-bit activation type (y, dx, ...); see err_ratio."""
        storage = self.dtype if (stored and self.dtype != "f32") else None
        self.rows.append((name, err_ratio(got, ref, self.dtype, mask, storage)))
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
            t += " | without quantum: " + ", ".join(f"{n}={e:.3f}" for n, e in self.plain)
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
    vh = saved_gpu["vhat"].float()
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
        rep.add("vhat", host(saved["vhat"]), np.where(vm, S["vhat"], 0.0), vm)
        rep.add("mean", host(saved["mean"]), S["mean"])
        rep.add("invstd", host(saved["invstd"]), S["invstd"])
    if L.residual == "proj":
        rep.add("vhat_r", host(saved["vhat_r"]), np.where(vm, S["vhat_r"], 0.0), vm)
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
    if "dx_res" in G and not want_dx_res:
        ref_dx = ref_dx + G["dx_res"]
    if dx_add is not None:
        ref_dx = ref_dx + np.where(O.time_mask(lengths, T), dx_add, 0.0)
    rep.add("dx", host(dx), ref_dx, O.time_mask(lengths, T), stored=True)
    if want_dx_res:
        rep.add("dx_res", host(dx_res), G["dx_res"], vm, stored=True)
    for name in params:
        rep.add("d" + name, host(grads["d" + name]), G["d" + name])
    rep.adopted, rep.hard = adopted, hard
    rep.out = dict(y=y, saved=saved, dx=dx, dx_res=dx_res, grads=grads, out_len=out_len)
    n_valid = int(np.broadcast_to(S["valid"], S["a"].shape).sum())
    assert hard == 0, f"{hard} ReLU gates differ outside the tolerance band"
    assert adopted <= 0.05 * n_valid + 5, f"too many adopted gates: {adopted}/{n_valid}"
    return rep


def run_chain(ctx, api, w, d, check=True, oracle_layers=None):
    """Teacher-forced chain: every layer runs through sepconv_fwd / sepconv_bwd on the GPU's own
    previous output, and the oracle evaluates the same layer on the same (stored) input.  Returns
    (per-layer reports, dict of final GPU tensors)."""
    layers = w.layers
    n = len(layers)
    acts = [d.x]                     # numpy float32 copies of what the GPU stored
    lens = [d.lengths]
    outs = []
    # forward pass first (the backward needs the last layer's upstream gradient)
    fwd = []
    for i, L in enumerate(layers):
        B, _, T = acts[i].shape
        desc = api.block_desc(L, B, T, w.dtype)
        xd = dev(acts[i], w.dtype)
        pd = params_dev(d.params[i], w.dtype)
        ld = torch.from_numpy(np.asarray(lens[i], dtype=np.int32)).cuda()
        j = L.res_from if L.res_from is not None else i
        xr = dev(acts[j], w.dtype) if (L.residual != "none" and j != i) else None
        y, out_len, saved = api.sepconv_fwd(ctx, desc, xd, ld, pd, x_res=xr)
        fwd.append(dict(desc=desc, xd=xd, pd=pd, ld=ld, xr=xr, y=y, saved=saved, j=j))
        acts.append(y.float().cpu().numpy())
        lens.append(out_len.cpu().numpy())
    reports = [None] * n
    g = d.g
    pending = {}
    grads_all = [None] * n
    for i in reversed(range(n)):
        L = layers[i]
        f = fwd[i]
        x_res_np = acts[f["j"]] if f["xr"] is not None else None
        if oracle_layers is not None and i not in oracle_layers:
            # GPU only: keeps the gradient flowing without the (slow) oracle evaluation of this layer
            want_res = f["xr"] is not None
            dx_add = pending.pop(i, None)
            dx, dx_res, grads = api.sepconv_bwd(ctx, f["desc"], dev(g, w.dtype), f["xd"], f["y"], f["ld"], f["pd"],
                                                f["saved"], x_res=f["xr"], dx_add=dx_add, want_dx_res=want_res)
            if want_res:
                pending[f["j"]] = dx_res
            grads_all[i] = grads
            g = dx.float().cpu().numpy()
            final_dx = dx
            continue
        S = O.block_fwd(L, acts[i], lens[i], d.params[i], res_src=x_res_np)
        rep = Report(w.dtype)
        np.testing.assert_array_equal(lens[i + 1], S["out_len"])
        vm = S["valid"]
        if L.has_dw:
            rep.add("u", host(f["saved"]["u"]), S["u"], vm)
        if L.has_bn:
            rep.add("vhat", host(f["saved"]["vhat"]), np.where(vm, S["vhat"], 0.0), vm)
        if L.residual == "proj":
            rep.add("vhat_r", host(f["saved"]["vhat_r"]), np.where(vm, S["vhat_r"], 0.0), vm)
        rep.add("y", acts[i + 1], S["y"], vm, stored=True)
        gate = None
        adopted = hard = 0
        if L.has_relu:
            gate, adopted, hard = adopt_gate(L, S, gpu_gate(L, f["y"], f["saved"], f["pd"]), w.dtype)
        G = O.block_bwd(L, g, lens[i], d.params[i], S, gate=gate)
        want_res = f["xr"] is not None
        dx_add = pending.pop(i, None)
        dx, dx_res, grads = api.sepconv_bwd(ctx, f["desc"], dev(g, w.dtype), f["xd"], f["y"], f["ld"], f["pd"],
                                            f["saved"], x_res=f["xr"], dx_add=dx_add, want_dx_res=want_res)
        ref_dx = G["dx"]
        if "dx_res" in G and not want_res:
            ref_dx = ref_dx + G["dx_res"]
        if dx_add is not None:
            ref_dx = ref_dx + np.where(O.time_mask(lens[i], acts[i].shape[2]), host(dx_add), 0.0)
        rep.add("dx", host(dx), ref_dx, O.time_mask(lens[i], acts[i].shape[2]), stored=True)
        if want_res:
            rep.add("dx_res", host(dx_res), G["dx_res"], vm, stored=True)
            pending[f["j"]] = dx_res
        for name in d.params[i]:
            rep.add("d" + name, host(grads["d" + name]), G["d" + name])
        rep.adopted, rep.hard = adopted, hard
        if check:
            assert hard == 0, f"layer {i}: {hard} ReLU gates differ outside the tolerance band"
            rep.check()
        reports[i] = rep
        grads_all[i] = grads
        g = dx.float().cpu().numpy()
        final_dx = dx
    assert ctx.last_status() == 0
    return reports, dict(logits=fwd[-1]["y"], dx=final_dx, grads=grads_all, out_len=lens[-1],
                         ys=[f["y"] for f in fwd], saved=[f["saved"] for f in fwd], pds=[f["pd"] for f in fwd])
