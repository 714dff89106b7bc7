"""Pins for the fp64 oracle: each test checks it against something other than itself --
pure-Python brute force, PyTorch CPU float64 operators + autograd, finite differences,
closed forms and a hand-worked example."""
import itertools
import math
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import synth_inputs as si
from oracle import sepconv_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rand_params(rng, L):
    p = {}
    for name, shp in L.param_shapes().items():
        if name in ("gamma", "gamma_r"):
            p[name] = rng.uniform(0.5, 1.5, shp)
        else:
            p[name] = rng.uniform(-1.0, 1.0, shp)
    return p


# ----------------------------------------------------------------------------------------------
# P1: brute force, pure Python, written straight from the index definition
# ----------------------------------------------------------------------------------------------
def brute_block(L, x, lengths, p, res_src=None):
    B, Ci, T = x.shape
    taps = L.has_dw or L.full_conv
    s = L.stride if taps else 1
    K = L.K if taps else 1
    dil = L.dilation if taps else 1
    P = (dil * (K - 1)) // 2                 # zeros on the left; the right side gets the rest
    Tp = (T - 1) // s + 1
    Co = L.C_out
    lenp = [-(-int(l) // s) for l in lengths]
    xt = lambda b, c, t: (x[b][c][t] if 0 <= t < T and t < lengths[b] else 0.0)
    u = [[[0.0] * Tp for _ in range(Ci)] for _ in range(B)]
    for b, c, t in itertools.product(range(B), range(Ci), range(Tp)):
        if t >= lenp[b]:
            continue
        if L.has_dw:
            u[b][c][t] = sum(p["wd"][c][k] * xt(b, c, t * s + k * dil - P) for k in range(K))
        else:
            u[b][c][t] = xt(b, c, t)

    def pw_bn(src, w, gamma, beta, bias, C_src, use_bn):
        v = [[[0.0] * Tp for _ in range(Co)] for _ in range(B)]
        for b, o, t in itertools.product(range(B), range(Co), range(Tp)):
            v[b][o][t] = sum(w[o][c] * src[b][c][t] for c in range(C_src)) + (bias[o] if bias is not None else 0.0)
        if not use_bn:
            return v
        N = sum(lenp)
        out = [[[0.0] * Tp for _ in range(Co)] for _ in range(B)]
        for o in range(Co):
            vals = [v[b][o][t] for b in range(B) for t in range(lenp[b])]
            mu = sum(vals) / N
            var = sum((q - mu) ** 2 for q in vals) / N
            for b in range(B):
                for t in range(lenp[b]):
                    out[b][o][t] = gamma[o] * (v[b][o][t] - mu) / math.sqrt(var + L.eps) + beta[o]
        return out

    if L.full_conv:
        # the non-separable convolution written as a pointwise contraction over the C_in * K shifted copies of x
        cols = [[[xt(b, c, t * s + k * dil - P) for t in range(Tp)] for c in range(Ci) for k in range(K)] for b in range(B)]
        wflat = [[p["wp"][o][c][k] for c in range(Ci) for k in range(K)] for o in range(Co)]
        bn = pw_bn(cols, wflat, p.get("gamma"), p.get("beta"), p.get("bias") if L.has_bias else None, Ci * K, L.has_bn)
    else:
        bn = pw_bn(u, p["wp"], p.get("gamma"), p.get("beta"), p.get("bias") if L.has_bias else None,
                   Ci, L.has_bn)
    r = None
    if L.residual != "none":
        rs = x if res_src is None else res_src
        Cr = rs.shape[1]
        xr = [[[rs[b][c][t] if t < lenp[b] else 0.0 for t in range(Tp)] for c in range(Cr)] for b in range(B)]
        r = xr if L.residual == "identity" else pw_bn(xr, p["wr"], p["gamma_r"], p["beta_r"], None, Cr, True)
    y = np.zeros((B, Co, Tp))
    for b, o, t in itertools.product(range(B), range(Co), range(Tp)):
        if t >= lenp[b]:
            continue
        a = bn[b][o][t]
        if r is not None and L.res_before_relu:
            a += r[b][o][t]
        q = max(a, 0.0) if L.has_relu else a
        if r is not None and not L.res_before_relu:
            q += r[b][o][t]
        y[b, o, t] = q
    return y


TINY = [
    dict(C_in=3, C_out=3, K=5, stride=1, residual="identity"),
    dict(C_in=3, C_out=4, K=3, stride=1, residual="proj"),
    dict(C_in=2, C_out=3, K=5, stride=2, residual="none"),
    dict(C_in=3, C_out=3, K=1, stride=1, residual="identity", res_before_relu=False),
    dict(C_in=3, C_out=2, K=1, has_dw=False, has_bn=False, has_relu=False, has_bias=True),
    dict(C_in=2, C_out=4, K=3, stride=1, residual="proj", res_before_relu=False),
    dict(C_in=3, C_out=3, K=4, stride=1, residual="identity"),            # even K: one more zero on the right
    dict(C_in=2, C_out=3, K=3, stride=1, dilation=2, residual="proj"),
    dict(C_in=2, C_out=2, K=2, stride=2, dilation=3, residual="none"),
    # non-separable convolution (the original Jasper block's)
    dict(C_in=3, C_out=3, K=3, has_dw=False, full_conv=True, residual="identity"),
    dict(C_in=2, C_out=3, K=4, stride=2, dilation=2, has_dw=False, full_conv=True, residual="none"),
    dict(C_in=2, C_out=2, K=3, has_dw=False, full_conv=True, has_bn=False, has_relu=False, has_bias=True),
]


@pytest.mark.parametrize("kw", TINY)
@pytest.mark.parametrize("ragged", [False, True])
def test_p1_forward_matches_brute_force(kw, ragged):
    rng = np.random.default_rng(5)
    L = si.LayerCfg(**kw)
    B, T = 2, 9
    x = rng.standard_normal((B, L.C_in, T))
    lengths = np.array([9, 9]) if not ragged else np.array([9, 4])
    p = rand_params(rng, L)
    S = O.block_fwd(L, x, lengths, p)
    yb = brute_block(L, x, lengths, p)
    np.testing.assert_allclose(S["y"], yb, rtol=1e-11, atol=1e-12)


@pytest.mark.parametrize("kw", TINY)
def test_p4_gradients_match_finite_differences_of_brute_force(kw):
    """Central differences of the *brute-force* forward against the oracle's analytic backward:
    pins every gradient (dx incl. the residual path, dwd, dwp, dgamma, dbeta, dbias, dwr,
    dgamma_r, dbeta_r) to an independent forward."""
    rng = np.random.default_rng(9)
    L = si.LayerCfg(**kw)
    B, T = 2, 7
    lengths = np.array([7, 4])
    for attempt in range(20):     # redraw until no pre-activation sits near the ReLU kink
        x = rng.standard_normal((B, L.C_in, T))
        p = rand_params(rng, L)
        S = O.block_fwd(L, x, lengths, p)
        if not L.has_relu or np.min(np.abs(S["a"][np.broadcast_to(S["valid"], S["a"].shape)])) > 2e-3:
            break
    g = rng.standard_normal(S["y"].shape)
    _, G = O.block_fwd_bwd(L, x, lengths, p, g)
    h = 1e-6

    def loss(xx, pp):
        return float(np.sum(brute_block(L, xx, lengths, pp) * g))

    def fd(arr, setter):
        out = np.zeros_like(arr)
        it = np.nditer(arr, flags=["multi_index"])
        for _ in it:
            i = it.multi_index
            a0 = arr[i]
            arr[i] = a0 + h
            lp = setter()
            arr[i] = a0 - h
            lm = setter()
            arr[i] = a0
            out[i] = (lp - lm) / (2 * h)
        return out

    dx_fd = fd(x, lambda: loss(x, p))
    np.testing.assert_allclose(G["dx"], dx_fd, rtol=2e-6, atol=2e-7)
    for name in p:
        d_fd = fd(p[name], lambda: loss(x, p))
        np.testing.assert_allclose(G["d" + name], d_fd, rtol=2e-6, atol=2e-7, err_msg=name)


# ----------------------------------------------------------------------------------------------
# P2 / P3: PyTorch CPU float64 operators + autograd (textbook grouped conv, 1x1 conv, batch_norm)
# ----------------------------------------------------------------------------------------------
def torch_layer_packed(L, xs, p, res_list):
    """xs: list of per-sample [C, len_b] tensors (already truncated).  Depthwise per sample, then
    all valid frames packed along time into [1, C, N] for pointwise + batch_norm + residual + ReLU."""
    s = L.stride if L.has_dw else 1
    us = []
    for xb in xs:
        if L.has_dw:
            P = (L.K - 1) // 2
            us.append(F.conv1d(xb[None], p["wd"][:, None, :], stride=s, padding=P, groups=L.C_in)[0])
        else:
            us.append(xb)
    lens = [u.shape[1] for u in us]
    pack = torch.cat(us, dim=1)[None]
    v = F.conv1d(pack, p["wp"][:, :, None], bias=p.get("bias") if L.has_bias else None)
    if L.has_bn:
        v = F.batch_norm(v, None, None, p["gamma"], p["beta"], training=True, eps=L.eps)
    r = None
    if L.residual != "none":
        rp = torch.cat(res_list, dim=1)[None]
        if L.residual == "identity":
            r = rp
        else:
            r = F.batch_norm(F.conv1d(rp, p["wr"][:, :, None]), None, None, p["gamma_r"], p["beta_r"],
                             training=True, eps=L.eps)
    a = v + r if (r is not None and L.res_before_relu) else v
    y = torch.relu(a) if L.has_relu else a
    if r is not None and not L.res_before_relu:
        y = y + r
    return list(torch.split(y[0], lens, dim=1))


def torch_network(layers, x, lengths, params):
    """Returns (list of per-layer per-sample outputs, leaf tensors)."""
    xt = torch.tensor(x, dtype=torch.float64, requires_grad=True)
    pt = [{k: torch.tensor(np.asarray(v), dtype=torch.float64, requires_grad=True) for k, v in p.items()}
          for p in params]
    acts = [[xt[b, :, :int(lengths[b])] for b in range(x.shape[0])]]
    for i, L in enumerate(layers):
        res = None
        if L.residual != "none":
            res = acts[L.res_from if L.res_from is not None else i]
        acts.append(torch_layer_packed(L, acts[i], pt[i], res))
    return acts, xt, pt


def pad_stack(seq, T):
    out = np.zeros((len(seq), seq[0].shape[0], T))
    for b, a in enumerate(seq):
        out[b, :, :a.shape[1]] = a.detach().numpy()
    return out


BLOCKS = [
    dict(C_in=6, C_out=6, K=7, residual="identity"),
    dict(C_in=5, C_out=8, K=9, residual="proj"),
    dict(C_in=4, C_out=6, K=5, stride=2, residual="none"),
    dict(C_in=5, C_out=7, K=3, residual="proj", res_before_relu=False),
    dict(C_in=6, C_out=3, K=1, has_dw=False, has_bn=False, has_relu=False, has_bias=True),
    dict(C_in=4, C_out=4, K=11, residual="none"),
]


@pytest.mark.parametrize("kw", BLOCKS)
@pytest.mark.parametrize("ragged", [False, True])
def test_p2_p3_block_matches_torch_autograd(kw, ragged):
    """ragged=False is the textbook special case (all lengths full); ragged=True is the
    truncate-and-pack equivalence: each sample processed alone on its valid frames, statistics over
    the packed frames."""
    rng = np.random.default_rng(21)
    L = si.LayerCfg(**kw)
    B, T = 4, 24
    lengths = np.full(B, T) if not ragged else np.array([24, 13, 7, 18])
    x = rng.standard_normal((B, L.C_in, T))
    p = rand_params(rng, L)
    S = O.block_fwd(L, x, lengths, p)
    Tp = S["y"].shape[2]
    g = rng.standard_normal(S["y"].shape)
    _, G = O.block_fwd_bwd(L, x, lengths, p, g)

    acts, xt, pt = torch_network([L], x, lengths, [p])
    y_t = pad_stack(acts[1], Tp)
    np.testing.assert_allclose(S["y"], y_t, rtol=1e-10, atol=1e-11)
    loss = sum((yb * torch.tensor(g[b, :, :yb.shape[1]])).sum() for b, yb in enumerate(acts[1]))
    loss.backward()
    np.testing.assert_allclose(G["dx"], xt.grad.numpy(), rtol=1e-9, atol=1e-10)
    for name in p:
        np.testing.assert_allclose(G["d" + name], pt[0][name].grad.numpy(), rtol=1e-9, atol=1e-10,
                                   err_msg=name)


@pytest.mark.parametrize("ragged", [False, True])
def test_encoder_matches_torch_autograd(ragged):
    w = si.tiny_encoder(B=3, T=40, ragged=ragged, width=8)
    d = si.draw(w)
    saved, lens = O.encoder_fwd(w.layers, d.x, d.lengths, d.params)
    grads, dx, _ = O.encoder_bwd(w.layers, d.g, lens, d.params, saved)
    acts, xt, pt = torch_network(w.layers, d.x, d.lengths, d.params)
    for i in range(len(w.layers)):
        np.testing.assert_allclose(saved[i]["y"], pad_stack(acts[i + 1], saved[i]["y"].shape[2]),
                                   rtol=1e-9, atol=1e-10)
    assert [a.shape[1] for a in acts[-1]] == list(lens[-1])
    loss = sum((yb * torch.tensor(d.g[b, :, :yb.shape[1]].astype(np.float64))).sum()
               for b, yb in enumerate(acts[-1]))
    loss.backward()
    np.testing.assert_allclose(dx, xt.grad.numpy(), rtol=1e-8, atol=1e-10)
    for i in range(len(w.layers)):
        for name in d.params[i]:
            np.testing.assert_allclose(grads[i]["d" + name], pt[i][name].grad.numpy(),
                                       rtol=1e-8, atol=1e-10, err_msg=f"layer {i} {name}")


# ----------------------------------------------------------------------------------------------
# P5: invariants;  P6: degenerate cases
# ----------------------------------------------------------------------------------------------
def _block(seed=3, **kw):
    rng = np.random.default_rng(seed)
    L = si.LayerCfg(**kw)
    B, T = 5, 32
    lengths = np.array([32, 11, 1, 20, 27])
    x = rng.standard_normal((B, L.C_in, T))
    p = rand_params(rng, L)
    return L, x, lengths, p, rng


def test_p5_padding_stays_zero_and_is_ignored():
    L, x, lengths, p, rng = _block(C_in=6, C_out=8, K=9, residual="proj")
    S = O.block_fwd(L, x, lengths, p)
    assert np.all(S["y"][~np.broadcast_to(S["valid"], S["y"].shape)] == 0)
    x2 = x.copy()
    pad = ~np.broadcast_to(O.time_mask(lengths, x.shape[2]), x.shape)
    x2[pad] = rng.standard_normal(int(pad.sum())) * 100
    S2 = O.block_fwd(L, x2, lengths, p)
    np.testing.assert_array_equal(S["y"], S2["y"])
    g = rng.standard_normal(S["y"].shape)
    _, G = O.block_fwd_bwd(L, x, lengths, p, g)
    assert np.all(G["dx"][pad] == 0)
    g2 = g.copy()
    g2[~np.broadcast_to(S["valid"], g.shape)] += 7.0       # upstream grad in padding is ignored
    _, G2 = O.block_fwd_bwd(L, x, lengths, p, g2)
    for k in G:
        np.testing.assert_array_equal(G[k], G2[k])


def test_p5_bn_moments_closed_form():
    L, x, lengths, p, rng = _block(C_in=6, C_out=8, K=9, residual="none")
    S = O.block_fwd(L, x, lengths, p)
    valid = np.broadcast_to(S["valid"], S["v"].shape)
    bn = p["gamma"][None, :, None] * S["vhat"] + p["beta"][None, :, None]
    for o in range(L.C_out):
        vals = bn[:, o, :][valid[:, o, :]]
        assert vals.size == int(O.out_lengths(lengths, 1).sum())
        np.testing.assert_allclose(vals.mean(), p["beta"][o], atol=1e-12)
        np.testing.assert_allclose(vals.var(), p["gamma"][o] ** 2 * S["var"][o] / (S["var"][o] + L.eps),
                                   rtol=1e-12)
    # zero mean / unit variance of vhat up to the eps factor
    vh = S["vhat"][:, 0, :][valid[:, 0, :]]
    np.testing.assert_allclose(vh.mean(), 0, atol=1e-12)
    np.testing.assert_allclose(vh.var(), S["var"][0] / (S["var"][0] + L.eps), rtol=1e-12)


def test_p5_bn_backward_orthogonality_and_linearity():
    L, x, lengths, p, rng = _block(C_in=6, C_out=8, K=9, residual="none")
    S = O.block_fwd(L, x, lengths, p)
    g = rng.standard_normal(S["y"].shape)
    G = O.block_bwd(L, g, lengths, p, S)
    # reconstruct gv through the pointwise adjoint identity: dwp = sum gv u^T, so use bn_bwd directly
    ga = np.where(S["valid"] & (S["a"] > 0), g, 0.0)
    gv, dgamma, dbeta = O.bn_bwd(ga, S["vhat"], S["valid"], p["gamma"], S["invstd"], S["N"])
    np.testing.assert_allclose(gv.sum(axis=(0, 2)), 0, atol=1e-12)
    lhs = (gv * S["vhat"]).sum(axis=(0, 2))
    rhs = p["gamma"] * dgamma * L.eps * (S["var"] + L.eps) ** -1.5
    np.testing.assert_allclose(lhs, rhs, rtol=1e-9, atol=1e-13)
    # backward is linear in g (a loss scale passes straight through)
    G3 = O.block_bwd(L, 1024.0 * g, lengths, p, S)
    for k in G:
        np.testing.assert_allclose(G3[k], 1024.0 * G[k], rtol=1e-12, atol=1e-12)


def test_p5_batch_permutation_equivariance():
    L, x, lengths, p, rng = _block(C_in=6, C_out=6, K=5, residual="identity")
    perm = np.array([3, 0, 4, 2, 1])
    S = O.block_fwd(L, x, lengths, p)
    Sp = O.block_fwd(L, x[perm], lengths[perm], p)
    np.testing.assert_allclose(Sp["y"], S["y"][perm], rtol=1e-12, atol=1e-13)


def test_p6_degenerate_cases():
    rng = np.random.default_rng(4)
    B, C, T = 3, 5, 16
    lengths = np.array([16, 9, 12])
    x = rng.standard_normal((B, C, T))
    # K=1 with unit taps: depthwise is the identity, block = pointwise + BN + ReLU
    L1 = si.LayerCfg(C, 7, K=1)
    p1 = rand_params(rng, L1)
    p1["wd"] = np.ones((C, 1))
    L1b = si.LayerCfg(C, 7, K=1, has_dw=False)
    np.testing.assert_allclose(O.block_fwd(L1, x, lengths, p1)["y"],
                               O.block_fwd(L1b, x, lengths, {k: v for k, v in p1.items() if k != "wd"})["y"],
                               rtol=1e-13)
    # wp = I: v equals the depthwise output
    L2 = si.LayerCfg(C, C, K=5)
    p2 = rand_params(rng, L2)
    p2["wp"] = np.eye(C)
    S = O.block_fwd(L2, x, lengths, p2)
    np.testing.assert_array_equal(S["v"], S["u"])
    # a single delta tap in the middle: depthwise is a per-channel scale
    p3 = dict(p2)
    wd = np.zeros((C, 5))
    wd[:, 2] = np.arange(1, C + 1)
    p3["wd"] = wd
    S3 = O.block_fwd(L2, x, lengths, p3)
    np.testing.assert_allclose(S3["u"], S3["xm"] * np.arange(1, C + 1)[None, :, None])
    # a delta at tap 0 reads x[t - P]: shifts right by P (cross-correlation, not flipped)
    wd = np.zeros((C, 5))
    wd[:, 0] = 1.0
    u = O.depthwise_fwd(x, wd, 1)
    np.testing.assert_array_equal(u[:, :, 2:], x[:, :, :-2])
    assert np.all(u[:, :, :2] == 0)


def test_lengths_and_stride():
    assert O.out_time(1600, 33, 2) == 800 and O.out_time(400, 63, 1) == 400 and O.out_time(9, 5, 2) == 5
    np.testing.assert_array_equal(O.out_lengths([1, 2, 3, 200, 3199], 2), [1, 1, 2, 100, 1600])
    # stride 2 keeps every other output of stride 1
    rng = np.random.default_rng(0)
    x = rng.standard_normal((1, 2, 10)); wd = rng.standard_normal((2, 5))
    np.testing.assert_allclose(O.depthwise_fwd(x, wd, 2), O.depthwise_fwd(x, wd, 1)[:, :, ::2])


def test_single_valid_frame_batch():
    """N = 1: variance 0, vhat 0, output = relu(beta)."""
    L = si.LayerCfg(2, 3, K=3)
    rng = np.random.default_rng(1)
    p = rand_params(rng, L)
    S = O.block_fwd(L, rng.standard_normal((1, 2, 6)), np.array([1]), p)
    np.testing.assert_allclose(S["y"][0, :, 0], np.maximum(p["beta"], 0))
    assert np.all(S["y"][0, :, 1:] == 0)


# ----------------------------------------------------------------------------------------------
# P7: hand-worked example
# ----------------------------------------------------------------------------------------------
def _golden():
    vals = {}
    with open(os.path.join(GOLDEN, "micro_example_T4.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            k, *v = line.split()
            vals[k] = np.array([float(q) for q in v])
    return vals


def test_p7_hand_worked_example():
    gold = _golden()
    x = np.array([[[1.0, 2, 3, 4]]])
    p = dict(wd=np.ones((1, 3)), wp=np.ones((1, 1)), gamma=np.ones(1), beta=np.zeros(1))
    g = np.ones((1, 1, 4))
    L = si.LayerCfg(1, 1, K=3, residual="identity", eps=0.0)
    S, G = O.block_fwd_bwd(L, x, [4], p, g)
    tol = dict(rtol=0, atol=1.5e-6)
    np.testing.assert_allclose(S["u"].ravel(), gold["eps0.u"], **tol)
    np.testing.assert_allclose(S["mean"], gold["eps0.mean"], **tol)
    np.testing.assert_allclose(S["var"], gold["eps0.var"], **tol)
    np.testing.assert_allclose(S["vhat"].ravel(), gold["eps0.vhat"], **tol)
    np.testing.assert_allclose(S["y"].ravel(), gold["eps0.y"], **tol)
    np.testing.assert_allclose(G["dbeta"], gold["eps0.dbeta"], **tol)
    np.testing.assert_allclose(G["dgamma"], gold["eps0.dgamma"], **tol)
    np.testing.assert_allclose(G["dwd"].ravel(), gold["eps0.dwd"], **tol)
    np.testing.assert_allclose(G["dx"].ravel(), gold["eps0.dx"], **tol)
    ga = np.array([[[0.0, 1, 1, 1]]])
    gv, _, _ = O.bn_bwd(ga, S["vhat"], S["valid"], p["gamma"], S["invstd"], 4)
    np.testing.assert_allclose(gv.ravel(), gold["eps0.gv"], **tol)
    L2 = si.LayerCfg(1, 1, K=3, residual="identity", eps=0.0, res_before_relu=False)
    np.testing.assert_allclose(O.block_fwd(L2, x, [4], p)["y"].ravel(), gold["eps0.y_relu_then_add"], **tol)
    L3 = si.LayerCfg(1, 1, K=3, residual="identity", eps=1e-3)
    np.testing.assert_allclose(O.block_fwd(L3, x, [4], p)["vhat"].ravel(), gold["eps1e-3.vhat"], **tol)


# ----------------------------------------------------------------------------------------------
# Decoder tail: log-softmax over the classes
# ----------------------------------------------------------------------------------------------
def test_log_softmax_matches_torch_and_closed_forms():
    rng = np.random.default_rng(21)
    z = rng.standard_normal((3, 29, 11)) * 3.0
    lp = O.log_softmax_fwd(z)
    zt = torch.tensor(z, requires_grad=True)
    ref = F.log_softmax(zt, dim=1)
    np.testing.assert_allclose(lp, ref.detach().numpy(), rtol=0, atol=1e-13)
    # probabilities sum to one at every position; shifting z by a per-position constant changes nothing
    np.testing.assert_allclose(np.exp(lp).sum(axis=1), 1.0, atol=1e-13)
    np.testing.assert_allclose(O.log_softmax_fwd(z + rng.standard_normal((3, 1, 11)) * 50), lp, atol=1e-11)
    # two classes: the closed form -log(1 + exp(z1 - z0))
    z2 = rng.standard_normal((2, 2, 5))
    np.testing.assert_allclose(O.log_softmax_fwd(z2)[:, 0], -np.log1p(np.exp(z2[:, 1] - z2[:, 0])), atol=1e-13)
    # adjoint against autograd; rows of the gradient sum to zero
    g = rng.standard_normal(z.shape)
    ref.backward(torch.tensor(g))
    dz = O.log_softmax_bwd(g, lp)
    np.testing.assert_allclose(dz, zt.grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(dz.sum(axis=1), 0.0, atol=1e-12)


def test_decoder_tail_layer_fwd_bwd():
    """Linear + bias + log-softmax layer under a padding mask: against torch on the packed valid frames,
    and every gradient against central differences."""
    rng = np.random.default_rng(22)
    L = si.LayerCfg(6, 5, K=1, has_dw=False, has_bn=False, has_relu=False, has_bias=True, log_softmax=True)
    B, T = 3, 7
    lengths = np.array([7, 3, 1])
    x = rng.standard_normal((B, 6, T))
    p = {"wp": rng.uniform(-1, 1, (5, 6)), "bias": rng.uniform(-1, 1, (5,))}
    g = rng.standard_normal((B, 5, T))
    S = O.block_fwd(L, x, lengths, p)
    G = O.block_bwd(L, g, lengths, p, S)
    valid = S["valid"]
    assert np.all(S["y"][~np.broadcast_to(valid, S["y"].shape)] == 0)
    xt = torch.tensor(x, requires_grad=True)
    wt = torch.tensor(p["wp"], requires_grad=True)
    bt = torch.tensor(p["bias"], requires_grad=True)
    m = torch.tensor(np.broadcast_to(valid, (B, 5, T)).copy())
    yt = torch.where(m, F.log_softmax(torch.einsum("oc,bct->bot", wt, xt) + bt[None, :, None], dim=1), torch.zeros(()).double())
    np.testing.assert_allclose(S["y"], yt.detach().numpy(), atol=1e-12)
    (yt * torch.tensor(g)).sum().backward()
    np.testing.assert_allclose(G["dx"], xt.grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(G["dwp"], wt.grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(G["dbias"], bt.grad.numpy(), atol=1e-12)
    # central differences of the loss sum(y * g) w.r.t. one weight and one input element
    def loss(xx, pp):
        return float(np.sum(O.block_fwd(L, xx, lengths, pp)["y"] * g))
    h = 1e-6
    pp = {k: v.copy() for k, v in p.items()}; pp["wp"][2, 3] += h
    pm = {k: v.copy() for k, v in p.items()}; pm["wp"][2, 3] -= h
    assert abs((loss(x, pp) - loss(x, pm)) / (2 * h) - G["dwp"][2, 3]) < 1e-6
    xp = x.copy(); xp[1, 4, 2] += h
    xm = x.copy(); xm[1, 4, 2] -= h
    assert abs((loss(xp, p) - loss(xm, p)) / (2 * h) - G["dx"][1, 4, 2]) < 1e-6


# ----------------------------------------------------------------------------------------------
# Evaluation mode: fixed running statistics
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("residual", ["none", "identity", "proj"])
def test_infer_matches_torch_eval_and_folded_weights(residual):
    rng = np.random.default_rng(31)
    Co = 6 if residual == "identity" else 5
    L = si.LayerCfg(6, Co, K=5, residual=residual)
    B, T = 3, 12
    lengths = np.array([12, 5, 9])
    x = rng.standard_normal((B, 6, T))
    p = rand_params(rng, L)
    run = {"mean": rng.standard_normal(Co), "var": rng.uniform(0.5, 2.0, Co),
           "mean_r": rng.standard_normal(Co), "var_r": rng.uniform(0.5, 2.0, Co)}
    S = O.block_infer(L, x, lengths, p, run)
    valid = S["valid"]
    # torch: grouped conv, 1x1 conv, batch_norm in eval mode, on the masked input
    xm = torch.tensor(np.where(O.time_mask(lengths, T), x, 0.0))
    u = F.conv1d(xm, torch.tensor(p["wd"])[:, None, :], padding=2, groups=6)
    u = torch.where(torch.tensor(np.broadcast_to(valid, u.shape).copy()), u, torch.zeros(()).double())
    v = F.conv1d(u, torch.tensor(p["wp"])[:, :, None])
    bn = F.batch_norm(v, torch.tensor(run["mean"]), torch.tensor(run["var"]), torch.tensor(p["gamma"]),
                      torch.tensor(p["beta"]), training=False, eps=L.eps)
    if residual == "identity":
        bn = bn + xm
    if residual == "proj":
        vr = F.conv1d(xm, torch.tensor(p["wr"])[:, :, None])
        bn = bn + F.batch_norm(vr, torch.tensor(run["mean_r"]), torch.tensor(run["var_r"]), torch.tensor(p["gamma_r"]),
                               torch.tensor(p["beta_r"]), training=False, eps=L.eps)
    ref = torch.where(torch.tensor(np.broadcast_to(valid, bn.shape).copy()), F.relu(bn), torch.zeros(()).double())
    np.testing.assert_allclose(S["y"], ref.numpy(), atol=1e-12)
    # folding: the fixed normalisation is an affine map per channel, so it folds into the pointwise weights
    k = p["gamma"] / np.sqrt(run["var"] + L.eps)
    Lf = si.LayerCfg(6, Co, K=5, has_bn=False, has_relu=False, has_bias=True)
    pf = {"wd": p["wd"], "wp": p["wp"] * k[:, None], "bias": p["beta"] - run["mean"] * k}
    folded = O.block_fwd(Lf, x, lengths, pf)["y"]
    if residual == "none":
        np.testing.assert_allclose(S["y"], np.maximum(folded, 0.0), atol=1e-12)
    # with the batch's own statistics as "running" statistics it is the training-mode forward
    St = O.block_fwd(L, x, lengths, p)
    own = {"mean": St["mean"], "var": St["var"], "mean_r": St.get("mean_r"), "var_r": St.get("var_r")}
    np.testing.assert_allclose(O.block_infer(L, x, lengths, p, own)["y"], St["y"], atol=1e-12)


@pytest.mark.parametrize("K,dil", [(4, 1), (3, 2), (2, 3), (6, 2), (5, 3)])
def test_same_padding_convention_matches_torch(K, dil):
    """Even K and dilated taps against torch's grouped conv1d with padding='same' (stride 1), forward and both
    gradients: pins where the zeros go when dilation*(K-1) is odd."""
    rng = np.random.default_rng(40 + K + dil)
    x = rng.standard_normal((2, 3, 11))
    w = rng.standard_normal((3, K))
    g = rng.standard_normal((2, 3, 11))
    u = O.depthwise_fwd(x, w, 1, dil)
    xt, wt = torch.tensor(x, requires_grad=True), torch.tensor(w, requires_grad=True)
    ref = F.conv1d(xt, wt[:, None, :], padding="same", dilation=dil, groups=3)
    np.testing.assert_allclose(u, ref.detach().numpy(), atol=1e-12)
    ref.backward(torch.tensor(g))
    gx, dwd = O.depthwise_bwd(g, x, w, 1, dil)
    np.testing.assert_allclose(gx, xt.grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(dwd, wt.grad.numpy(), atol=1e-12)
    assert O.out_time(11, K, 1, dil) == 11 and O.out_time(11, K, 2, dil) == 6


@pytest.mark.parametrize("K,stride,dil", [(3, 1, 1), (4, 1, 1), (5, 2, 1), (3, 1, 2), (4, 2, 3)])
def test_full_conv_matches_torch(K, stride, dil):
    """The non-separable convolution against torch's dense conv1d (explicit zero padding: dilation*(K-1) in total,
    the odd one on the right), forward and both gradients."""
    rng = np.random.default_rng(60 + K + stride + dil)
    x = rng.standard_normal((2, 3, 11))
    w = rng.standard_normal((4, 3, K))
    Tp = O.out_time(11, K, stride, dil)
    g = rng.standard_normal((2, 4, Tp))
    v = O.conv_fwd(x, w, stride, dil)
    xt, wt = torch.tensor(x, requires_grad=True), torch.tensor(w, requires_grad=True)
    pl, pr = O.same_padding(K, dil)
    ref = F.conv1d(F.pad(xt, (pl, pr)), wt, stride=stride, dilation=dil)
    assert ref.shape[2] == Tp
    np.testing.assert_allclose(v, ref.detach().numpy(), atol=1e-12)
    ref.backward(torch.tensor(g))
    gx, dw = O.conv_bwd(g, x, w, stride, dil)
    np.testing.assert_allclose(gx, xt.grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(dw, wt.grad.numpy(), atol=1e-12)
    if stride == 1:
        np.testing.assert_allclose(v, F.conv1d(xt, wt, padding="same", dilation=dil).detach().numpy(), atol=1e-12)


def test_full_conv_with_factorised_weights_is_the_separable_block():
    """w[o,c,k] = wp[o,c] * wd[c,k] makes the non-separable convolution the depthwise step followed by the pointwise
    step: the two variants of the block then agree on every output and input gradient, and the full weight gradient
    contracts to the two separable ones.  K = 1 is the pointwise layer itself."""
    rng = np.random.default_rng(71)
    B, T = 3, 12
    for kw in (dict(K=5, stride=1), dict(K=3, stride=2), dict(K=4, stride=1, dilation=2)):
        Ls = si.LayerCfg(4, 5, residual="proj", **kw)
        Lf = si.LayerCfg(4, 5, residual="proj", has_dw=False, full_conv=True, **kw)
        x = rng.standard_normal((B, 4, T))
        lengths = np.array([T, T, T])          # the separable path zeroes u beyond len'; with full lengths nothing is beyond
        ps = rand_params(rng, Ls)
        pf = {k: v for k, v in ps.items() if k != "wd"}
        pf["wp"] = ps["wp"][:, :, None] * ps["wd"][None, :, :]
        res = rng.standard_normal((B, 4, O.out_time(T, kw["K"], kw["stride"], kw.get("dilation", 1))))
        g = rng.standard_normal((B, 5, res.shape[2]))
        Ss, Sf = O.block_fwd(Ls, x, lengths, ps, res_src=res), O.block_fwd(Lf, x, lengths, pf, res_src=res)
        np.testing.assert_allclose(Sf["v"], Ss["v"], atol=1e-11)
        np.testing.assert_allclose(Sf["y"], Ss["y"], atol=1e-11)
        Gs, Gf = O.block_bwd(Ls, g, lengths, ps, Ss), O.block_bwd(Lf, g, lengths, pf, Sf)
        np.testing.assert_allclose(Gf["dx"], Gs["dx"], atol=1e-10)
        np.testing.assert_allclose(Gf["dx_res"], Gs["dx_res"], atol=1e-10)
        np.testing.assert_allclose(np.einsum("ock,ck->oc", Gf["dwp"], ps["wd"]), Gs["dwp"], atol=1e-10)
        np.testing.assert_allclose(np.einsum("ock,oc->ck", Gf["dwp"], ps["wp"]), Gs["dwd"], atol=1e-10)
        for n in ("dgamma", "dbeta", "dwr", "dgamma_r", "dbeta_r"):
            np.testing.assert_allclose(Gf[n], Gs[n], atol=1e-10, err_msg=n)
    Lp = si.LayerCfg(4, 5, K=1, has_dw=False)
    Lq = si.LayerCfg(4, 5, K=1, has_dw=False, full_conv=True)
    x = rng.standard_normal((B, 4, T)); lengths = np.array([T, 5, 9])
    pp = rand_params(rng, Lp)
    pq = dict(pp); pq["wp"] = pp["wp"][:, :, None]
    np.testing.assert_allclose(O.block_fwd(Lq, x, lengths, pq)["y"], O.block_fwd(Lp, x, lengths, pp)["y"], atol=1e-12)


def test_running_stats():
    rm, rv = O.running_stats_update(np.zeros(2), np.ones(2), np.array([1.0, 2.0]), np.array([4.0, 9.0]), 10)
    np.testing.assert_allclose(rm, [0.1, 0.2])
    np.testing.assert_allclose(rv, [0.9 + 0.1 * 4 * 10 / 9, 0.9 + 0.1 * 9 * 10 / 9])


def test_running_stats_match_torch_batch_norm():
    """The running-statistics reading (momentum 0.1, unbiased variance into the running buffer) against torch's own
    update: batch_norm in training mode on the valid frames of a ragged batch packed into one [1, C, N] tensor
    (masked statistics reduce to plain statistics there), starting from non-trivial running buffers."""
    rng = np.random.default_rng(77)
    B, C, T = 3, 5, 11
    lengths = np.array([11, 4, 7])
    v = rng.normal(size=(B, C, T)) * rng.uniform(0.5, 2.0, size=(1, C, 1)) + rng.normal(size=(1, C, 1))
    mean, var, N = O.bn_stats(v, O.time_mask(lengths, T))
    rm0, rv0 = rng.normal(size=C), rng.uniform(0.5, 1.5, size=C)
    rm, rv = O.running_stats_update(rm0, rv0, mean, var, N)
    packed = torch.from_numpy(np.concatenate([v[b, :, :lengths[b]] for b in range(B)], axis=1)[None])
    trm, trv = torch.from_numpy(rm0.copy()), torch.from_numpy(rv0.copy())
    F.batch_norm(packed, trm, trv, training=True, momentum=0.1, eps=1e-3)
    np.testing.assert_allclose(rm, trm.numpy(), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(rv, trv.numpy(), rtol=1e-12, atol=1e-12)


def test_inputs_are_seeded_and_representable():
    a, b = si.draw(si.config(2)), si.draw(si.config(2))
    np.testing.assert_array_equal(a.x, b.x)
    np.testing.assert_array_equal(a.x, a.x.astype(np.float16).astype(np.float32))
    assert a.lengths.min() >= 200 and a.lengths.max() <= 400
    c = si.draw(si.config(3))
    np.testing.assert_array_equal(c.x, torch.from_numpy(c.x).to(torch.bfloat16).float().numpy())
    assert si.n_params(si.quartznet5x5_layers()) == 6713181
