"""GPU parity of the two steps that follow the training hot path: the decoder tail (log-softmax over the classes
on the logits layer, forward and backward) and the evaluation-mode forward (fixed running statistics)."""
import numpy as np
import pytest
import torch

import synth_inputs as si
from oracle import sepconv_oracle as O
from tests import parity_util as U

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    import paper_1909_09577_b200 as api
    return api


@pytest.fixture(scope="module")
def ctx(api):
    c = api.Context(0)
    yield c
    c.close()


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
@pytest.mark.parametrize("shape", [(64, 29, 3, 50), (1024, 29, 4, 264), (40, 7, 2, 33)])
def test_decoder_tail_block(api, ctx, dtype, shape):
    """Linear + bias + log-softmax layer: log_probs, dx, dwp and dbias against the oracle (run_block drives
    sepconv_fwd / sepconv_bwd and the oracle from the same layer description)."""
    Ci, Co, B, T = shape
    L = si.LayerCfg(Ci, Co, K=1, has_dw=False, has_bn=False, has_relu=False, has_bias=True, log_softmax=True)
    d = si.draw(si.Workload("tail", dtype, B, T, [L], 41, len_lo=max(1, T // 4), len_hi=T, affine="random"))
    rep = U.run_block(ctx, api, L, dtype, d.x, d.lengths, d.params[0], d.g)
    print(f"\ndecoder tail {shape} {dtype}: {rep}")
    rep.check()
    y = U.host(rep.out["y"])
    valid = O.time_mask(O.out_lengths(d.lengths, 1), T)
    p = np.exp(y).sum(axis=1)                             # probabilities sum to one on valid frames
    assert np.all(np.abs(p[valid[:, 0, :]] - 1.0) < (1e-5 if dtype == "f32" else 3e-2))


def test_encoder_with_log_probs(api, ctx):
    """Tiny encoder ending in log-probabilities: one call equals the chain of block calls bit for bit, and every
    layer meets the per-layer tolerance teacher-forced."""
    w = si.tiny_encoder(dtype="bf16", B=8, T=512, ragged=True, width=32)
    last = w.layers[-1]
    w.layers[-1] = si.LayerCfg(last.C_in, last.C_out, K=1, has_dw=False, has_bn=False, has_relu=False, has_bias=True,
                               log_softmax=True)
    d = si.draw(w)
    reports, chain = U.run_chain(ctx, api, w, d)
    spec = api.EncoderSpec(w.layers, w.B, w.T, w.dtype)
    blob = spec.pack_params(d.params, "cuda")
    logp, out_len, gblob, dx = api.encoder_fwd_bwd(ctx, spec, U.dev(d.x, w.dtype), torch.from_numpy(d.lengths).cuda(), blob,
                                                   U.dev(d.g, w.dtype), want_dx=True)
    assert ctx.last_status() == 0
    assert torch.equal(logp, chain["logits"]) and torch.equal(dx, chain["dx"])
    for i in range(len(w.layers)):
        for name in d.params[i]:
            assert torch.equal(spec.grad_view(gblob, i, name), chain["grads"][i]["d" + name]), (i, name)


def _running(rng, L):
    r = {}
    if L.has_bn:
        r["mean"] = rng.standard_normal(L.C_out).astype(np.float32) * 0.3
        r["var"] = rng.uniform(0.5, 2.0, L.C_out).astype(np.float32)
    if L.residual == "proj":
        r["mean_r"] = rng.standard_normal(L.C_out).astype(np.float32) * 0.3
        r["var_r"] = rng.uniform(0.5, 2.0, L.C_out).astype(np.float32)
    return r


INFER_CASES = [
    (dict(C_in=24, C_out=40, K=9, residual="proj"), 3, 77),
    (dict(C_in=256, C_out=256, K=33, residual="identity"), 16, 328),
    (dict(C_in=64, C_out=256, K=33, stride=2), 4, 400),
    (dict(C_in=512, C_out=1024, K=1, has_dw=False), 2, 264),
    (dict(C_in=1024, C_out=29, K=1, has_dw=False, has_bn=False, has_relu=False, has_bias=True, log_softmax=True), 3, 200),
    (dict(C_in=24, C_out=40, K=5, stride=2, has_dw=False, full_conv=True), 3, 78),        # non-separable convolution
]


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
@pytest.mark.parametrize("case", range(len(INFER_CASES)))
def test_infer_block(api, ctx, dtype, case):
    kw, B, T = INFER_CASES[case]
    L = si.LayerCfg(**kw)
    d = si.draw(si.Workload("infer", dtype, B, T, [L], 50 + case, len_lo=max(1, T // 4), len_hi=T, affine="random"))
    run = _running(np.random.default_rng(60 + case), L)
    desc = api.block_desc(L, B, T, dtype)
    rd = {k: torch.from_numpy(v).cuda() for k, v in run.items()}
    y, out_len = api.sepconv_infer(ctx, desc, U.dev(d.x, dtype), torch.from_numpy(d.lengths).cuda(),
                                   U.params_dev(d.params[0], dtype), rd)
    assert ctx.last_status() == 0
    S = O.block_infer(L, d.x, d.lengths, d.params[0], run)
    np.testing.assert_array_equal(out_len.cpu().numpy(), S["out_len"])
    rep = U.Report(dtype)
    rep.add("y", U.host(y), S["y"], S["valid"], stored=True)
    print(f"\ninfer case {case} {dtype}: {rep}")
    rep.check()
    assert np.all(U.host(y)[~np.broadcast_to(S["valid"], y.shape)] == 0)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_infer_encoder(api, ctx, dtype):
    """Evaluation-mode forward of a whole (tiny) encoder in one call, ending in log-probabilities, against the
    oracle's evaluation-mode encoder; end to end, so bounded at the stated multiple."""
    w = si.tiny_encoder(dtype=dtype, B=4, T=256, ragged=True, width=32)
    last = w.layers[-1]
    w.layers[-1] = si.LayerCfg(last.C_in, last.C_out, K=1, has_dw=False, has_bn=False, has_relu=False, has_bias=True,
                               log_softmax=True)
    d = si.draw(w)
    rng = np.random.default_rng(77)
    running = [_running(rng, L) for L in w.layers]
    spec = api.EncoderSpec(w.layers, w.B, w.T, w.dtype)
    blob = spec.pack_params(d.params, "cuda")
    rblob, roffs = spec.pack_running(running, "cuda")
    out, out_len = api.encoder_infer(ctx, spec, U.dev(d.x, dtype), torch.from_numpy(d.lengths).cuda(), blob, rblob, roffs)
    assert ctx.last_status() == 0
    acts, lens = O.encoder_infer(w.layers, d.x, d.lengths, d.params, running)
    np.testing.assert_array_equal(out_len.cpu().numpy(), lens[-1])
    valid = O.time_mask(lens[-1], acts[-1].shape[2])
    rep = U.Report(dtype)
    rep.add("log_probs", U.host(out), acts[-1], valid, stored=True)
    print(f"\ninfer encoder {dtype}: {rep}")
    rep.check(limit=4.0 if dtype != "f32" else 1.0)
