"""fp64 CPU oracle for the time-channel separable convolution block and encoder.

TEST INFRASTRUCTURE ONLY.  Nothing on the product path may import this module;
it exists so that tests, the smoke check and the benchmark's CPU-baseline leg
have an independent statement of what the block computes.  It shares no code
with the CUDA path and is deliberately plain: every function is the
mathematical definition written out with numpy in float64, in the order the
definition states it, with no blocking, fusion or reordering.

Where the definition comes from.  The paper (NeMo, arXiv 1909.09577) gives the
module boundary -- ``encoded, encoded_len = jasper_encoder(audio_signal, length)``
(section 4.1.1), tensors as [batch, channel, time] arrays with tagged axes
(section 3.2, Table 1) and the mixed-precision policy (section 3.3) -- but no
equations for the Jasper-like encoder it cites.  The block itself is therefore
the standard one: per-channel depthwise cross-correlation over time with "same"
zero padding, a 1x1 channel-mixing convolution, training-mode batch
normalisation over the valid (unpadded) frames, a residual add and ReLU, all
under a per-sample padding mask.  The readings taken where that statement is
open (cross-correlation rather than flipped convolution, biased variance with
eps inside the root, residual joined before the ReLU by default, output length
ceil(len/stride), ...) are marked "reading:" below.

Pins (tests/test_oracle_pins.py): brute-force pure-Python evaluation on tiny
inputs, PyTorch CPU float64 autograd for the all-lengths-full special case and
for the truncate-and-pack form of ragged batches, central finite differences
for every gradient, closed-form batch-norm invariants, degenerate cases, and a
hand-worked four-frame example stored under tests/golden/.
Parity unpinned: nothing in the paper prints a value for this path, so the
conventions listed as readings are pinned only to the textbook/library
operators named above, not to the paper.

Layout: activations [B, C, T] (time contiguous), lengths int [B] in input frames.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


# ----------------------------------------------------------------------------
# Lengths and masks
# ----------------------------------------------------------------------------
def same_padding(K: int, dilation: int = 1):
    """Zeros added left and right so that a stride-1 correlation keeps the length: dilation*(K-1) in
    total.  reading: for an even total (odd K, or even dilation) it splits evenly; otherwise the extra
    zero goes to the right (left = total // 2), the convention of the common "same" padding."""
    total = dilation * (K - 1)
    return total // 2, total - total // 2


def out_time(T: int, K: int, stride: int, dilation: int = 1) -> int:
    """Frames produced by a K-tap, "same"-padded correlation (taps `dilation` frames apart) with the
    given stride: floor((T + pad_total - dilation*(K-1) - 1) / stride) + 1 = floor((T-1)/stride) + 1."""
    pl, pr = same_padding(K, dilation)
    return (T + pl + pr - dilation * (K - 1) - 1) // stride + 1


def out_lengths(lengths, stride: int):
    """reading: a sample of ``len`` valid frames has ceil(len/stride) valid output frames,
    i.e. what it would produce if processed alone (this is the ``encoded_len`` port)."""
    lengths = np.asarray(lengths, dtype=np.int64)
    return (lengths + stride - 1) // stride


def time_mask(lengths, T: int):
    """m[b, t] = 1 if t < len[b] else 0, shape [B, 1, T] (boolean)."""
    return (np.arange(T)[None, :] < np.asarray(lengths)[:, None])[:, None, :]


# ----------------------------------------------------------------------------
# The four linear pieces and their adjoints
# ----------------------------------------------------------------------------
def depthwise_fwd(xm, wd, stride: int, dilation: int = 1):
    """u[b,c,t] = sum_k wd[c,k] * xm[b,c,t*stride + k*dilation - P], zero outside [0,T), P = left padding.
    reading: cross-correlation (taps are not flipped)."""
    B, C, T = xm.shape
    K = wd.shape[1]
    P, Pr = same_padding(K, dilation)
    Tp = out_time(T, K, stride, dilation)
    xp = np.zeros((B, C, T + P + Pr), F64)
    xp[:, :, P:P + T] = xm
    u = np.zeros((B, C, Tp), F64)
    span = (Tp - 1) * stride + 1
    for k in range(K):
        u += wd[None, :, k, None] * xp[:, :, k * dilation:k * dilation + span:stride]
    return u


def depthwise_bwd(gu, xm, wd, stride: int, dilation: int = 1):
    """Adjoint of depthwise_fwd: returns (gx, dwd).
    gx[b,c,tau] = sum over (k,t) with t*stride+k*dilation-P = tau of wd[c,k]*gu[b,c,t];
    dwd[c,k]    = sum_{b,t} gu[b,c,t] * xm[b,c,t*stride+k*dilation-P]."""
    B, C, T = xm.shape
    K = wd.shape[1]
    P, Pr = same_padding(K, dilation)
    Tp = gu.shape[2]
    xp = np.zeros((B, C, T + P + Pr), F64)
    xp[:, :, P:P + T] = xm
    gxp = np.zeros_like(xp)
    dwd = np.zeros((C, K), F64)
    span = (Tp - 1) * stride + 1
    for k in range(K):
        o = k * dilation
        gxp[:, :, o:o + span:stride] += wd[None, :, k, None] * gu
        dwd[:, k] = np.sum(gu * xp[:, :, o:o + span:stride], axis=(0, 2))
    return gxp[:, :, P:P + T], dwd


def conv_fwd(xm, w, stride: int, dilation: int = 1):
    """Non-separable 1-D convolution over time (the convolution of the original Jasper block, which the
    separable block factorises; paper section 4.1.1):
        v[b,o,t] = sum_{c,k} w[o,c,k] * xm[b,c,t*stride + k*dilation - P],
    zero outside [0,T), P = left padding.  Same conventions as depthwise_fwd (cross-correlation, "same"
    padding, stride on the convolution)."""
    B, C, T = xm.shape
    K = w.shape[2]
    P, Pr = same_padding(K, dilation)
    Tp = out_time(T, K, stride, dilation)
    xp = np.zeros((B, C, T + P + Pr), F64)
    xp[:, :, P:P + T] = xm
    v = np.zeros((B, w.shape[0], Tp), F64)
    span = (Tp - 1) * stride + 1
    for k in range(K):
        v += np.einsum("oc,bct->bot", w[:, :, k], xp[:, :, k * dilation:k * dilation + span:stride], optimize=True)
    return v


def conv_bwd(gv, xm, w, stride: int, dilation: int = 1):
    """Adjoint of conv_fwd: returns (gx, dw).
    gx[b,c,tau] = sum over (o,k,t) with t*stride+k*dilation-P = tau of w[o,c,k]*gv[b,o,t];
    dw[o,c,k]   = sum_{b,t} gv[b,o,t] * xm[b,c,t*stride+k*dilation-P]."""
    B, C, T = xm.shape
    K = w.shape[2]
    P, Pr = same_padding(K, dilation)
    Tp = gv.shape[2]
    xp = np.zeros((B, C, T + P + Pr), F64)
    xp[:, :, P:P + T] = xm
    gxp = np.zeros_like(xp)
    dw = np.zeros(w.shape, F64)
    span = (Tp - 1) * stride + 1
    for k in range(K):
        o = k * dilation
        gxp[:, :, o:o + span:stride] += np.einsum("oc,bot->bct", w[:, :, k], gv, optimize=True)
        dw[:, :, k] = np.einsum("bot,bct->oc", gv, xp[:, :, o:o + span:stride], optimize=True)
    return gxp[:, :, P:P + T], dw


def pointwise_fwd(u, wp):
    """v[b,o,t] = sum_c wp[o,c] * u[b,c,t]."""
    return np.einsum("oc,bct->bot", wp, u, optimize=True)


def pointwise_bwd(gv, u, wp):
    """(gu, dwp): gu[b,c,t] = sum_o wp[o,c]*gv[b,o,t]; dwp[o,c] = sum_{b,t} gv[b,o,t]*u[b,c,t]."""
    gu = np.einsum("oc,bot->bct", wp, gv, optimize=True)
    dwp = np.einsum("bot,bct->oc", gv, u, optimize=True)
    return gu, dwp


# ----------------------------------------------------------------------------
# Masked training-mode batch normalisation
# ----------------------------------------------------------------------------
def bn_stats(v, valid):
    """Per-channel mean and biased variance over valid frames only (two-pass).
    reading: variance uses 1/N with N = number of valid (b,t) positions."""
    N = int(valid.sum())
    mean = np.sum(np.where(valid, v, 0.0), axis=(0, 2)) / N
    d = np.where(valid, v - mean[None, :, None], 0.0)
    var = np.sum(d * d, axis=(0, 2)) / N
    return mean, var, N


def bn_fwd(v, valid, gamma, beta, eps):
    """reading: eps sits inside the square root."""
    mean, var, N = bn_stats(v, valid)
    invstd = 1.0 / np.sqrt(var + eps)
    vhat = (v - mean[None, :, None]) * invstd[None, :, None]
    out = gamma[None, :, None] * vhat + beta[None, :, None]
    return out, vhat, mean, var, invstd, N


def bn_bwd(ga, vhat, valid, gamma, invstd, N):
    """ga is already zero outside the valid frames.
    dbeta = sum ga; dgamma = sum ga*vhat;
    gv = gamma*invstd*(ga - dbeta/N - vhat*dgamma/N) on valid frames, 0 elsewhere."""
    dbeta = np.sum(ga, axis=(0, 2))
    dgamma = np.sum(np.where(valid, ga * vhat, 0.0), axis=(0, 2))
    gv = (gamma * invstd)[None, :, None] * (
        ga - dbeta[None, :, None] / N - vhat * dgamma[None, :, None] / N)
    gv = np.where(valid, gv, 0.0)
    return gv, dgamma, dbeta


# ----------------------------------------------------------------------------
# Decoder tail: log-softmax over the class (channel) axis.  The paper's CTC decoder module turns
# the encoder output into ``log_probs`` (section 4.1.1); its last step, after the 1x1 convolution
# that produces the class scores z, is  log_probs[b,c,t] = z[b,c,t] - log(sum_c' exp(z[b,c',t])).
# ----------------------------------------------------------------------------
def log_softmax_fwd(z):
    """Per (b, t) position over axis 1, written as the definition with the usual max shift
    (exp(z - max) is the same ratio; it only avoids overflow)."""
    zmax = np.max(z, axis=1, keepdims=True)
    return z - zmax - np.log(np.sum(np.exp(z - zmax), axis=1, keepdims=True))


def log_softmax_bwd(g, logp):
    """Adjoint: d z[c] = g[c] - softmax[c] * sum_c' g[c'],  softmax = exp(log_probs)."""
    return g - np.exp(logp) * np.sum(g, axis=1, keepdims=True)


# ----------------------------------------------------------------------------
# One layer:  [mask] -> [depthwise] -> pointwise [+bias] -> [BN] -> [+residual] -> [ReLU] -> mask
#             (or, for the decoder tail:  ... pointwise + bias -> log-softmax over channels -> mask)
# ----------------------------------------------------------------------------
def _p(params, name):
    return np.asarray(params[name], dtype=F64)


def block_fwd(L, x, lengths, params, res_src=None):
    """Forward of one layer described by ``L`` (fields: C_in, C_out, K, stride, has_dw, has_bn,
    has_relu, has_bias, residual in {"none","identity","proj"}, res_before_relu, eps).

    x        [B, C_in, T]  input; frames t >= len[b] are ignored (masked to zero first)
    res_src  source of the residual branch (defaults to x); masked the same way
    Returns a dict with every intermediate so that tests can compare stage by stage:
      xm, u, v, mean, var, invstd, vhat, (xr, vr, mean_r, var_r, invstd_r, vhat_r), r, a, y,
      out_len, valid, N.
    """
    x = np.asarray(x, dtype=F64)
    B, C_in, T = x.shape
    full = bool(getattr(L, "full_conv", False))         # block variant: one non-separable K-tap convolution
    taps = L.has_dw or full
    s = L.stride if taps else 1
    K = L.K if taps else 1
    dil = getattr(L, "dilation", 1) if taps else 1
    Tp = out_time(T, K, s, dil)
    lengths = np.asarray(lengths, dtype=np.int64)
    out_len = out_lengths(lengths, s)
    valid = time_mask(out_len, Tp)                      # m'
    S = {"out_len": out_len, "valid": valid}

    # mask on the conv input
    xm = np.where(time_mask(lengths, T), x, 0.0)
    S["xm"] = xm
    if full:
        v = conv_fwd(xm, _p(params, "wp"), s, dil)      # wp is [C_out, C_in, K] here
    else:
        u = depthwise_fwd(xm, _p(params, "wd"), s, dil) if L.has_dw else xm
        u = np.where(valid, u, 0.0)                     # frames beyond len' are never used
        S["u"] = u
        v = pointwise_fwd(u, _p(params, "wp"))
    if L.has_bias:
        v = v + _p(params, "bias")[None, :, None]
    S["v"] = v
    if L.has_bn:
        bn, vhat, mean, var, invstd, N = bn_fwd(v, valid, _p(params, "gamma"), _p(params, "beta"),
                                                L.eps)
        S.update(vhat=vhat, mean=mean, var=var, invstd=invstd, N=N)
    else:
        bn = v
        S["N"] = int(valid.sum())

    # residual branch
    if L.residual == "none":
        r = None
    else:
        rs = x if res_src is None else np.asarray(res_src, dtype=F64)
        if rs.shape[2] != Tp:
            raise ValueError("residual needs the same number of frames as the output")
        xr = np.where(valid, rs, 0.0)
        S["xr"] = xr
        if L.residual == "identity":
            if xr.shape[1] != L.C_out:
                raise ValueError("identity residual needs C_res == C_out")
            r = xr
        else:
            vr = pointwise_fwd(xr, _p(params, "wr"))
            r, vhat_r, mean_r, var_r, invstd_r, _ = bn_fwd(
                vr, valid, _p(params, "gamma_r"), _p(params, "beta_r"), L.eps)
            S.update(vr=vr, vhat_r=vhat_r, mean_r=mean_r, var_r=var_r, invstd_r=invstd_r)
    S["r"] = r

    # reading: the residual joins before the activation unless res_before_relu is False
    if r is not None and L.res_before_relu:
        a = bn + r
    else:
        a = bn
    S["a"] = a                                          # the ReLU's argument
    y = np.maximum(a, 0.0) if L.has_relu else a
    if r is not None and not L.res_before_relu:
        y = y + r
    if getattr(L, "log_softmax", False):
        # decoder tail (only legal on a linear layer): reading: padded frames read as zero, like
        # every other output of the path
        y = log_softmax_fwd(y)
    S["y"] = np.where(valid, y, 0.0)
    return S


def block_infer(L, x, lengths, params, running, res_src=None):
    """Forward of one layer in evaluation mode (the paper's `eval` / `infer` actions, section 3.1): the
    batch statistics are replaced by fixed running statistics,
        bn = gamma * (v - running_mean) / sqrt(running_var + eps) + beta,
    everything else as in block_fwd.  ``running`` = dict(mean, var[, mean_r, var_r]).  Returns y only
    (plus out_len, valid)."""
    x = np.asarray(x, dtype=F64)
    B, C_in, T = x.shape
    full = bool(getattr(L, "full_conv", False))
    taps = L.has_dw or full
    s = L.stride if taps else 1
    K = L.K if taps else 1
    dil = getattr(L, "dilation", 1) if taps else 1
    Tp = out_time(T, K, s, dil)
    lengths = np.asarray(lengths, dtype=np.int64)
    out_len = out_lengths(lengths, s)
    valid = time_mask(out_len, Tp)
    xm = np.where(time_mask(lengths, T), x, 0.0)
    if full:
        v = conv_fwd(xm, _p(params, "wp"), s, dil)
    else:
        u = depthwise_fwd(xm, _p(params, "wd"), s, dil) if L.has_dw else xm
        u = np.where(valid, u, 0.0)
        v = pointwise_fwd(u, _p(params, "wp"))
    if L.has_bias:
        v = v + _p(params, "bias")[None, :, None]

    def fixed_bn(t, mean, var, gamma, beta):
        k = gamma / np.sqrt(np.asarray(var, F64) + L.eps)
        return k[None, :, None] * (t - np.asarray(mean, F64)[None, :, None]) + beta[None, :, None]

    bn = fixed_bn(v, running["mean"], running["var"], _p(params, "gamma"), _p(params, "beta")) if L.has_bn else v
    r = None
    if L.residual != "none":
        rs = x if res_src is None else np.asarray(res_src, dtype=F64)
        xr = np.where(valid, rs, 0.0)
        if L.residual == "identity":
            r = xr
        else:
            r = fixed_bn(pointwise_fwd(xr, _p(params, "wr")), running["mean_r"], running["var_r"],
                         _p(params, "gamma_r"), _p(params, "beta_r"))
    a = bn + r if (r is not None and L.res_before_relu) else bn
    y = np.maximum(a, 0.0) if L.has_relu else a
    if r is not None and not L.res_before_relu:
        y = y + r
    if getattr(L, "log_softmax", False):
        y = log_softmax_fwd(y)
    return {"y": np.where(valid, y, 0.0), "out_len": out_len, "valid": valid}


def encoder_infer(layers, x, lengths, params, running):
    """Evaluation-mode forward through every layer; ``running[i]`` as for block_infer."""
    acts = [np.asarray(x, dtype=F64)]
    lens = [np.asarray(lengths, dtype=np.int64)]
    for i, L in enumerate(layers):
        res = acts[L.res_from if L.res_from is not None else i] if L.residual != "none" else None
        S = block_infer(L, acts[i], lens[i], params[i], running[i], res_src=res)
        acts.append(S["y"])
        lens.append(S["out_len"])
    return acts, lens


def block_bwd(L, g, lengths, params, S, gate=None):
    """Backward of block_fwd.  ``g`` = dLoss/dy, ``S`` = block_fwd's dict.
    ``gate`` (bool [B,C_out,T'], optional) overrides the ReLU gate [a > 0]; derivative at a == 0
    is 0 by convention.
    Returns dict: dx (w.r.t. x), dx_res (w.r.t. res_src when the residual has a source), and the
    parameter gradients present for this layer.  When the residual source is x itself the caller
    adds dx and dx_res."""
    g = np.asarray(g, dtype=F64)
    valid = S["valid"]
    full = bool(getattr(L, "full_conv", False))
    s = L.stride if (L.has_dw or full) else 1
    T = S["xm"].shape[2]
    G = {}
    gm = np.where(valid, g, 0.0)                        # output mask
    if getattr(L, "log_softmax", False):
        gm = np.where(valid, log_softmax_bwd(gm, S["y"]), 0.0)
    if L.has_relu:
        if gate is None:
            gate = S["a"] > 0.0
        ga = np.where(gate, gm, 0.0)
    else:
        ga = gm
    # gradient reaching the residual sum r
    if S["r"] is None:
        gr = None
    else:
        gr = ga if L.res_before_relu else gm

    if L.has_bn:
        gv, G["dgamma"], G["dbeta"] = bn_bwd(ga, S["vhat"], valid, _p(params, "gamma"),
                                             S["invstd"], S["N"])
    else:
        gv = ga
    if L.has_bias:
        G["dbias"] = np.sum(gv, axis=(0, 2))
    if full:
        gx, G["dwp"] = conv_bwd(np.where(valid, gv, 0.0), S["xm"], _p(params, "wp"), s, getattr(L, "dilation", 1))
    else:
        gu, G["dwp"] = pointwise_bwd(gv, S["u"], _p(params, "wp"))
        if L.has_dw:
            gx, G["dwd"] = depthwise_bwd(gu, S["xm"], _p(params, "wd"), s, getattr(L, "dilation", 1))
        else:
            gx = gu
    G["dx"] = np.where(time_mask(lengths, T), gx, 0.0)

    if gr is not None:
        if L.residual == "identity":
            gxr = gr
        else:
            gvr, G["dgamma_r"], G["dbeta_r"] = bn_bwd(gr, S["vhat_r"], valid, _p(params, "gamma_r"),
                                                      S["invstd_r"], S["N"])
            gxr, G["dwr"] = pointwise_bwd(gvr, S["xr"], _p(params, "wr"))
        G["dx_res"] = np.where(valid, gxr, 0.0)
    return G


def block_fwd_bwd(L, x, lengths, params, g):
    """Single-block convenience: residual source is x, so dx includes the residual path."""
    S = block_fwd(L, x, lengths, params)
    G = block_bwd(L, g, lengths, params, S)
    if "dx_res" in G:
        G["dx"] = G["dx"] + G.pop("dx_res")
    return S, G


# ----------------------------------------------------------------------------
# Encoder: a fixed list of layers; a layer with res_from=j takes its residual from layer j's input
# ----------------------------------------------------------------------------
def encoder_fwd(layers, x, lengths, params):
    """Returns (list of per-layer dicts, list of per-layer input lengths incl. the final one)."""
    acts = [np.asarray(x, dtype=F64)]
    lens = [np.asarray(lengths, dtype=np.int64)]
    saved = []
    for i, L in enumerate(layers):
        res = None
        if L.residual != "none":
            res = acts[L.res_from if L.res_from is not None else i]
        S = block_fwd(L, acts[i], lens[i], params[i], res_src=res)
        saved.append(S)
        acts.append(S["y"])
        lens.append(S["out_len"])
    return saved, lens


def encoder_bwd(layers, g, lens, params, saved, gates=None):
    """Returns (list of per-layer gradient dicts, dx w.r.t. the encoder input, list of the
    upstream gradient each layer received)."""
    n = len(layers)
    grads = [None] * n
    pending = {}                      # layer index -> gradient to add to that layer's input
    g_in = [None] * n
    cur = np.asarray(g, dtype=F64)
    for i in reversed(range(n)):
        L = layers[i]
        g_in[i] = cur
        G = block_bwd(L, cur, lens[i], params[i], saved[i],
                      gate=None if gates is None else gates[i])
        dx = G["dx"]
        if "dx_res" in G:
            j = L.res_from if L.res_from is not None else i
            pending[j] = pending.get(j, 0.0) + G.pop("dx_res")
        if i in pending:
            dx = dx + pending.pop(i)
        G["dx"] = dx
        grads[i] = G
        cur = dx
    return grads, cur, g_in


def running_stats_update(rm, rv, mean, var, N, momentum=0.1):
    """reading: running_var takes the unbiased variance (N/(N-1)); momentum 0.1."""
    unb = var * (N / (N - 1.0)) if N > 1 else var
    return (1 - momentum) * rm + momentum * mean, (1 - momentum) * rv + momentum * unb
