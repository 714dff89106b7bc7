"""Seeded synthetic workloads for the time-channel separable convolution path.

This module only *describes* workloads and draws random numbers: layer lists,
tensor shapes, per-sample lengths, inputs, parameters and upstream gradients,
plus the round-to-nearest-even quantisation of those draws to the storage type.
It holds none of the block's arithmetic.  Both the CPU oracle's tests and the
CUDA path's tests/benchmarks draw their inputs here so that the two sides see
bit-identical values.

The inputs stand in for the ASR data layer's outputs (a batch of 64-channel
spectrogram features plus per-sample lengths, paper section 4.1.1 and the
``Spectrogram:64`` axis of Table 1); no speech data is used.

Draw order for one workload (numpy ``default_rng(seed)``, PCG64):
  1. lengths (if ragged)         integers, inclusive bounds
  2. x                           N(0,1), float32, then quantised
  3. per layer, in layer order:  wd, wp, gamma, beta, bias, wr, gamma_r, beta_r
                                 (only those the layer has)
  4. upstream gradient g         N(0,1), float32, then quantised
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional

import numpy as np

F32, F16, BF16 = "f32", "f16", "bf16"


# --------------------------------------------------------------------------
# Quantisation of drawn values to the storage type (round to nearest even).
# --------------------------------------------------------------------------
def bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 array -> uint16 array holding the bfloat16 bit patterns (RNE)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32)


def quantise(a: np.ndarray, dtype: str) -> np.ndarray:
    """Round float32 draws to ``dtype`` and return them widened back to float32."""
    a = np.asarray(a, dtype=np.float32)
    if dtype == F32:
        return a
    if dtype == F16:
        return a.astype(np.float16).astype(np.float32)
    if dtype == BF16:
        return bf16_to_f32(bf16_bits(a)).reshape(a.shape)
    raise ValueError(dtype)


# --------------------------------------------------------------------------
# Workload description
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class LayerCfg:
    """One layer: [depthwise] -> pointwise [+bias] -> [BN] -> [+residual] -> [ReLU]."""
    C_in: int
    C_out: int
    K: int = 1
    stride: int = 1
    has_dw: bool = True
    has_bn: bool = True
    has_relu: bool = True
    has_bias: bool = False
    residual: str = "none"          # "none" | "identity" | "proj"
    res_from: Optional[int] = None  # index of the layer whose INPUT feeds the residual (None: own input)
    res_before_relu: bool = True
    eps: float = 1e-3
    log_softmax: bool = False       # decoder tail on a linear layer: log-softmax over the channels
    dilation: int = 1               # frames between neighbouring taps of the depthwise step
    full_conv: bool = False         # block variant: one non-separable K-tap convolution [C_out, C_in, K] (needs has_dw=False)

    def param_shapes(self) -> Dict[str, tuple]:
        s: Dict[str, tuple] = {}
        if self.has_dw:
            s["wd"] = (self.C_in, self.K)
        s["wp"] = (self.C_out, self.C_in, self.K) if self.full_conv else (self.C_out, self.C_in)
        if self.has_bn:
            s["gamma"] = (self.C_out,)
            s["beta"] = (self.C_out,)
        if self.has_bias:
            s["bias"] = (self.C_out,)
        if self.residual == "proj":
            c_res = self.C_res
            s["wr"] = (self.C_out, c_res)
            s["gamma_r"] = (self.C_out,)
            s["beta_r"] = (self.C_out,)
        return s

    # channel count of the residual source; set by the workload builder
    C_res_override: Optional[int] = None

    @property
    def C_res(self) -> int:
        return self.C_res_override if self.C_res_override is not None else self.C_in


PARAM_ORDER = ("wd", "wp", "gamma", "beta", "bias", "wr", "gamma_r", "beta_r")
# Parameters stored in the activation type (the conv weights); the rest stay float32.
IO_DTYPE_PARAMS = ("wd", "wp", "wr")


@dataclass
class Workload:
    name: str
    dtype: str
    B: int
    T: int
    layers: List[LayerCfg]
    seed: int
    len_lo: Optional[int] = None   # None: all lengths = T
    len_hi: Optional[int] = None
    affine: str = "unit"           # "unit": gamma=1, beta=0, bias=0 | "random"

    @property
    def C_in(self) -> int:
        return self.layers[0].C_in

    def out_T(self) -> int:
        T = self.T
        for L in self.layers:
            if L.has_dw or L.full_conv:
                T = (T - 1) // L.stride + 1      # "same" padding: dilation * (K - 1) zeros in total
        return T


def quartznet5x5_layers(log_probs: bool = False) -> List[LayerCfg]:
    """QuartzNet-5x5-style encoder plus the two pointwise layers that end in 29 logits
    (log_probs=True: in 29 log-probabilities, the decoder module's output)."""
    layers: List[LayerCfg] = [LayerCfg(64, 256, K=33, stride=2)]
    plan = [(256, 33), (256, 39), (512, 51), (512, 63), (512, 75)]
    c_prev = 256
    for c_out, k in plan:
        first = len(layers)
        for r in range(5):
            c_in = c_prev if r == 0 else c_out
            if r < 4:
                layers.append(LayerCfg(c_in, c_out, K=k))
            else:
                layers.append(LayerCfg(c_in, c_out, K=k, residual="proj", res_from=first,
                                       C_res_override=c_prev))
        c_prev = c_out
    layers.append(LayerCfg(512, 512, K=87))
    layers.append(LayerCfg(512, 1024, K=1, has_dw=False))
    layers.append(LayerCfg(1024, 29, K=1, has_dw=False, has_bn=False, has_relu=False, has_bias=True,
                           log_softmax=log_probs))
    return layers


def config(i: int, affine: str = "unit") -> Workload:
    """The five benchmark/parity configurations, numbered 1..5 (seed = i-1)."""
    if i == 1:
        return Workload("cfg1_block_f32", F32, 2, 128,
                        [LayerCfg(64, 64, K=33, residual="identity")], seed=0, affine=affine)
    if i == 2:
        return Workload("cfg2_block_f16_ragged", F16, 32, 400,
                        [LayerCfg(256, 256, K=33, residual="identity")], seed=1,
                        len_lo=200, len_hi=400, affine=affine)
    if i == 3:
        return Workload("cfg3_block_bf16_proj", BF16, 32, 400,
                        [LayerCfg(256, 512, K=63, residual="proj")], seed=2,
                        len_lo=100, len_hi=400, affine=affine)
    if i == 4:
        return Workload("cfg4_encoder_bf16", BF16, 32, 1600, quartznet5x5_layers(), seed=3,
                        affine=affine)
    if i == 5:
        return Workload("cfg5_encoder_bf16_ragged", BF16, 64, 3200, quartznet5x5_layers(), seed=4,
                        len_lo=200, len_hi=3200, affine=affine)
    raise ValueError(i)


def tiny_encoder(dtype: str = BF16, B: int = 3, T: int = 96, seed: int = 11,
                 ragged: bool = True, affine: str = "random", width: int = 64) -> Workload:
    """A narrow, shallow encoder with the same structure (stride-2 prologue, two blocks with
    projection residuals from the block input, epilogue, pointwise+BN, logits+bias)."""
    w = width
    layers = [LayerCfg(16, w, K=5, stride=2)]
    c_prev = w
    for c_out, k in [(w, 7), (2 * w, 9)]:
        first = len(layers)
        for r in range(3):
            c_in = c_prev if r == 0 else c_out
            if r < 2:
                layers.append(LayerCfg(c_in, c_out, K=k))
            else:
                layers.append(LayerCfg(c_in, c_out, K=k, residual="proj", res_from=first,
                                       C_res_override=c_prev))
        c_prev = c_out
    layers.append(LayerCfg(c_prev, c_prev, K=11))
    layers.append(LayerCfg(c_prev, 2 * c_prev, K=1, has_dw=False))
    layers.append(LayerCfg(2 * c_prev, 29, K=1, has_dw=False, has_bn=False, has_relu=False,
                           has_bias=True))
    return Workload("tiny_encoder", dtype, B, T, layers, seed,
                    len_lo=(T // 4 if ragged else None), len_hi=(T if ragged else None),
                    affine=affine)


# --------------------------------------------------------------------------
# Drawing
# --------------------------------------------------------------------------
def _kaiming_uniform(rng, shape, fan_in):
    b = np.sqrt(6.0 / fan_in)
    return rng.uniform(-b, b, size=shape).astype(np.float32)


def draw_layer_params(rng, L: LayerCfg, dtype: str, affine: str) -> Dict[str, np.ndarray]:
    """Float32 arrays; the conv weights already carry values representable in ``dtype``."""
    p: Dict[str, np.ndarray] = {}
    shapes = L.param_shapes()
    for name in PARAM_ORDER:
        if name not in shapes:
            continue
        shp = shapes[name]
        if name == "wd":
            a = quantise(_kaiming_uniform(rng, shp, L.K), dtype)
        elif name == "wp":
            a = quantise(_kaiming_uniform(rng, shp, L.C_in * (L.K if L.full_conv else 1)), dtype)
        elif name == "wr":
            a = quantise(_kaiming_uniform(rng, shp, L.C_res), dtype)
        elif name in ("gamma", "gamma_r"):
            a = (rng.uniform(0.5, 1.5, size=shp).astype(np.float32) if affine == "random"
                 else np.ones(shp, np.float32))
        else:  # beta, beta_r, bias
            a = (rng.uniform(-0.5, 0.5, size=shp).astype(np.float32) if affine == "random"
                 else np.zeros(shp, np.float32))
        p[name] = a
    return p


@dataclass
class Drawn:
    workload: Workload
    lengths: np.ndarray                      # int32 [B], in input frames
    x: np.ndarray                            # float32 [B, C_in, T], values representable in dtype
    params: List[Dict[str, np.ndarray]]      # one dict per layer (float32 arrays)
    g: np.ndarray                            # float32 [B, C_last, T_out]


def draw(w: Workload) -> Drawn:
    rng = np.random.default_rng(w.seed)
    if w.len_lo is None:
        lengths = np.full((w.B,), w.T, dtype=np.int32)
    else:
        lengths = rng.integers(w.len_lo, w.len_hi, size=w.B, endpoint=True).astype(np.int32)
    x = quantise(rng.standard_normal((w.B, w.C_in, w.T), dtype=np.float32), w.dtype)
    params = [draw_layer_params(rng, L, w.dtype, w.affine) for L in w.layers]
    g = quantise(rng.standard_normal((w.B, w.layers[-1].C_out, w.out_T()), dtype=np.float32),
                 w.dtype)
    return Drawn(w, lengths, x, params, g)


def n_params(layers: List[LayerCfg]) -> int:
    return int(sum(int(np.prod(s)) for L in layers for s in L.param_shapes().values()))
