"""sepconv_fwd_static -- the forward block call for callers that may not allocate device memory
(fixed-memory real-time pipelines, plugins under a framework that owns the device heap).  It must
give exactly what sepconv_fwd gives, call after call, although all calls share one built-in scratch
array that still holds the previous call's data."""
import numpy as np
import pytest
import torch

import synth_inputs as si
from tests import parity_util as U

pytestmark = pytest.mark.gpu


def _run_pair(api, ctx, L, B, T, dtype, seed, first_call_on_device=False):
    w = si.Workload("static", dtype, B, T, [L], seed, len_lo=T // 3, len_hi=T, affine="random")
    d = si.draw(w)
    desc = api.block_desc(L, B, T, dtype)
    xd, pd = U.dev(d.x, dtype), U.params_dev(d.params[0], dtype)
    ld = torch.from_numpy(d.lengths).cuda()
    y_ref, len_ref, saved_ref = api.sepconv_fwd(ctx, desc, xd, ld, pd)
    # caller-owned outputs, allocated before the call under test
    y = torch.full_like(y_ref, float("nan"))
    out_len = torch.zeros_like(len_ref)
    saved = {k: torch.full_like(v, float("nan")) for k, v in saved_ref.items()}
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    free_before = torch.cuda.mem_get_info()[0]          # the driver's view: sees any allocation, not only torch's
    api.sepconv_fwd_static(ctx, desc, xd, ld, pd, y, out_len, saved)
    assert ctx.last_status() == 0
    assert torch.cuda.memory_allocated() == before
    if not first_call_on_device:                        # the first call loads the module that holds the array
        assert torch.cuda.mem_get_info()[0] == free_before
    rep = U.Report(dtype)
    rep.add("y", U.host(y), U.host(y_ref))
    # frames at and beyond a sample's output length are unspecified in the saved pointwise results
    valid = (torch.arange(y.shape[2], device="cuda")[None, None, :] < len_ref[:, None, None]).cpu().numpy()
    for k in saved_ref:
        if k in ("v", "vr"):
            rep.add(k, U.masked(saved[k], valid), U.masked(saved_ref[k], valid))
        else:
            rep.add(k, U.host(saved[k]), U.host(saved_ref[k]))
    rep.check()
    assert torch.equal(out_len, len_ref)
    assert torch.equal(y, y_ref)          # same kernels, same order: identical bits


def test_static_scratch_forward_matches_twice():
    import paper_1909_09577_b200 as api
    ctx = api.Context(0)
    try:
        # two calls in a row with different shapes and types: the second starts from the first one's leftovers
        _run_pair(api, ctx, si.LayerCfg(48, 64, K=33, residual="proj"), 4, 200, "bf16", seed=31, first_call_on_device=True)
        _run_pair(api, ctx, si.LayerCfg(32, 32, K=9, residual="identity"), 3, 120, "f32", seed=32)
        _run_pair(api, ctx, si.LayerCfg(48, 64, K=33, residual="proj"), 4, 200, "bf16", seed=33)
    finally:
        ctx.close()


def test_static_scratch_rejects_large_blocks():
    import paper_1909_09577_b200 as api
    ctx = api.Context(0)
    try:
        L = si.config(3).layers[0]                  # at B = 64 it needs more scratch than the built-in array holds
        desc = api.block_desc(L, 64, 400, "bf16")
        assert api.sepconv_workspace_bytes(desc)[0] > api.binding.STATIC_SCRATCH_BYTES
        x = torch.zeros((64, 256, 400), dtype=torch.bfloat16, device="cuda")
        y = torch.zeros((64, 512, 400), dtype=torch.bfloat16, device="cuda")
        lens = torch.full((64,), 400, dtype=torch.int32, device="cuda")
        with pytest.raises(api.SepconvError) as e:
            api.sepconv_fwd_static(ctx, desc, x, lens, {"wd": x, "wp": x, "gamma": x, "beta": x, "wr": x,
                                                        "gamma_r": x, "beta_r": x}, y, lens, {"u": x})
        assert e.value.code == -7
    finally:
        ctx.close()
