"""GPU parity of sepconv_fwd / sepconv_bwd (through the C ABI) against the fp64 oracle."""
import numpy as np
import pytest
import torch

import synth_inputs as si
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


def _draw_block(L, B, T, dtype, seed, ragged, affine="random", lo_frac=0.25):
    w = si.Workload("t", dtype, B, T, [L], seed, len_lo=max(1, int(T * lo_frac)) if ragged else None,
                    len_hi=T if ragged else None, affine=affine)
    return si.draw(w)


SMALL = [
    # (layer kwargs, B, T, ragged)
    (dict(C_in=8, C_out=8, K=5, residual="identity"), 3, 40, True),
    (dict(C_in=24, C_out=40, K=9, residual="proj"), 3, 77, True),          # T not a multiple of 8
    (dict(C_in=16, C_out=32, K=33, stride=2, residual="none"), 2, 130, True),
    (dict(C_in=16, C_out=32, K=7, stride=2, residual="none"), 2, 131, True),   # odd T with stride 2
    (dict(C_in=16, C_out=16, K=11, residual="identity", res_before_relu=False), 2, 64, True),
    (dict(C_in=16, C_out=24, K=3, residual="proj", res_before_relu=False), 2, 64, True),
    (dict(C_in=64, C_out=29, K=1, has_dw=False, has_bn=False, has_relu=False, has_bias=True), 3, 50, True),
    (dict(C_in=32, C_out=64, K=1, has_dw=False), 3, 48, True),
    (dict(C_in=8, C_out=8, K=87, residual="none"), 2, 300, True),          # halo wider than some samples
    (dict(C_in=130, C_out=70, K=15, residual="proj"), 2, 520, False),      # several tiles + ragged channel tail
    (dict(C_in=8, C_out=8, K=3, has_relu=False), 2, 33, True),
    # block variants: even K (the odd zero of the "same" padding goes to the right), dilated taps, both with stride 2
    (dict(C_in=16, C_out=24, K=4, residual="proj"), 3, 72, True),
    (dict(C_in=16, C_out=16, K=11, dilation=3, residual="identity"), 3, 120, True),
    (dict(C_in=8, C_out=16, K=6, dilation=2, stride=2, residual="none"), 2, 131, True),
    # block variant: one non-separable K-tap convolution (tiles with channel and frame tails, stride 2, dilation,
    # even K, a linear layer with bias)
    (dict(C_in=24, C_out=40, K=5, has_dw=False, full_conv=True, residual="proj"), 3, 77, True),
    (dict(C_in=70, C_out=70, K=11, has_dw=False, full_conv=True, residual="identity"), 5, 150, True),
    (dict(C_in=16, C_out=24, K=4, stride=2, dilation=2, has_dw=False, full_conv=True, residual="none"), 6, 131, True),
    (dict(C_in=16, C_out=8, K=3, has_dw=False, full_conv=True, has_bn=False, has_relu=False, has_bias=True), 2, 40, True),
]


@pytest.fixture(params=[0, 1], ids=["tensorcore", "simt"])
def gemm_mode(request, ctx):
    """0: tensor-core contractions where the shape allows; 1: plain SIMT contractions everywhere."""
    ctx.set_gemm_mode(request.param)
    yield request.param
    ctx.set_gemm_mode(0)


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
@pytest.mark.parametrize("case", range(len(SMALL)))
def test_small_blocks(api, ctx, dtype, case, gemm_mode):
    if dtype == "f32" and gemm_mode == 1:
        pytest.skip("fp32 always uses the SIMT contractions")
    kw, B, T, ragged = SMALL[case]
    L = si.LayerCfg(**kw)
    d = _draw_block(L, B, T, dtype, seed=100 + case, ragged=ragged)
    rep = U.run_block(ctx, api, L, dtype, d.x, d.lengths, d.params[0], d.g)
    rep.check()


TC_SHAPES = [
    # shapes that exercise the tensor-core tiling: channel tails, several k-blocks, T' tails, tiny C_out
    (dict(C_in=64, C_out=256, K=33, stride=2, residual="none"), 4, 400, True),
    (dict(C_in=256, C_out=256, K=5, residual="identity"), 3, 328, True),
    (dict(C_in=320, C_out=200, K=5, residual="proj"), 2, 136, True),
    (dict(C_in=1024, C_out=29, K=1, has_dw=False, has_bn=False, has_relu=False, has_bias=True), 3, 200, True),
    (dict(C_in=512, C_out=1024, K=1, has_dw=False), 2, 264, True),
    (dict(C_in=72, C_out=136, K=3, residual="proj"), 5, 64, False),
    # tensor-core tap gradient: sample chunks with a ragged tail, T' that is no multiple of 128, wide halos,
    # more (channel, split) units than SMs
    (dict(C_in=24, C_out=16, K=87, residual="none"), 20, 328, True),
    (dict(C_in=16, C_out=24, K=121, residual="proj"), 40, 136, True),
    (dict(C_in=160, C_out=8, K=39, residual="none"), 33, 1000, True),
    (dict(C_in=8, C_out=8, K=5, residual="identity"), 16, 128, False),
    # TMA-fed depthwise: a single tap, the widest supported halo (tap gradient falls back to SIMT), rows
    # shorter than one 128-frame block, two sample chunks of 32 with time-block groups cut short by T
    (dict(C_in=8, C_out=16, K=1, residual="none"), 16, 64, True),
    (dict(C_in=8, C_out=8, K=129, residual="none"), 17, 264, True),
    (dict(C_in=16, C_out=8, K=33, residual="proj"), 18, 72, True),
    (dict(C_in=8, C_out=8, K=75, residual="identity"), 64, 1160, True),
    # large enough for the streaming batch-norm kernels (ring of bulk copies): no residual, ragged rows,
    # a row length that is no multiple of the 256-vector chunk
    (dict(C_in=128, C_out=136, K=33, residual="none"), 32, 328, True),
]


@pytest.mark.parametrize("dtype", ["bf16", "f16"])
@pytest.mark.parametrize("case", range(len(TC_SHAPES)))
def test_tensorcore_shapes(api, ctx, dtype, case):
    kw, B, T, ragged = TC_SHAPES[case]
    L = si.LayerCfg(**kw)
    d = _draw_block(L, B, T, dtype, seed=200 + case, ragged=ragged, lo_frac=0.1)
    rep = U.run_block(ctx, api, L, dtype, d.x, d.lengths, d.params[0], d.g)
    print(f"\ntc shape {case} {dtype}: {rep}")
    rep.check()


@pytest.mark.parametrize("shape", [0, 1, 2, 3, 4, 5])
@pytest.mark.parametrize("case", [2, 4])
def test_tile_shapes(api, ctx, shape, case):
    """Every tile shape of the flattened-block contraction (forward with statistics, input gradient): a projection
    block with channel tails on both sides, and a 512 -> 1024 pointwise layer (several M tiles per CTA range)."""
    kw, B, T, ragged = TC_SHAPES[case]
    L = si.LayerCfg(**kw)
    d = _draw_block(L, 8 * B, T, "bf16", seed=300 + case, ragged=ragged, lo_frac=0.1)
    ctx.set_tile_shape(shape)
    try:
        rep = U.run_block(ctx, api, L, "bf16", d.x, d.lengths, d.params[0], d.g)
    finally:
        ctx.set_tile_shape(0)
    print(f"\ntile shape {shape} case {case}: {rep}")
    rep.check()


@pytest.mark.parametrize("shape", [0, 1, 2, 3, 5])
def test_tile_shapes_large_batch(api, ctx, shape):
    """More than 256 samples: the block offsets no longer fit beside the sixteen epilogue warps' staging buffers (nor
    beside two CTAs per SM), so shapes 0, 3 and 5 take their eight-warp / one-CTA forms."""
    L = si.LayerCfg(C_in=136, C_out=144, K=9, residual="proj")
    d = _draw_block(L, 272, 72, "bf16", seed=411, ragged=True, lo_frac=0.1)
    ctx.set_tile_shape(shape)
    try:
        rep = U.run_block(ctx, api, L, "bf16", d.x, d.lengths, d.params[0], d.g)
    finally:
        ctx.set_tile_shape(0)
    print(f"\nlarge batch, tile shape {shape}: {rep}")
    rep.check()


def test_batch_beyond_the_flattened_block_list(api, ctx):
    """More than 2048 samples: the contraction leaves the flattened-block kernel (its shared-memory copy of the block
    offsets is bounded) for the per-sample tiled one."""
    L = si.LayerCfg(C_in=8, C_out=16, K=5, residual="none")
    d = _draw_block(L, 2100, 16, "f16", seed=412, ragged=True, lo_frac=0.1)
    rep = U.run_block(ctx, api, L, "f16", d.x, d.lengths, d.params[0], d.g)
    print(f"\n2100 samples: {rep}")
    rep.check()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_len_one_and_full(api, ctx, dtype):
    L = si.LayerCfg(16, 16, K=9, residual="identity")
    d = _draw_block(L, 4, 64, dtype, seed=7, ragged=False)
    d.lengths[:] = [1, 64, 2, 63]
    U.run_block(ctx, api, L, dtype, d.x, d.lengths, d.params[0], d.g).check()


def test_external_residual_and_dx_add(api, ctx):
    """Residual taken from another tensor (as the encoder's blocks do), its gradient returned
    separately, and an extra gradient folded into dx."""
    rng = np.random.default_rng(3)
    L = si.LayerCfg(32, 48, K=7, residual="proj", C_res_override=16)
    d = _draw_block(L, 3, 96, "bf16", seed=8, ragged=True)
    x_res = si.quantise(rng.standard_normal((3, 16, 96)).astype(np.float32), "bf16")
    dx_add = si.quantise(rng.standard_normal((3, 32, 96)).astype(np.float32), "bf16")
    U.run_block(ctx, api, L, "bf16", d.x, d.lengths, d.params[0], d.g, x_res=x_res, want_dx_res=True,
                dx_add=dx_add).check()


@pytest.mark.parametrize("i", [1, 2, 3])
@pytest.mark.parametrize("affine", ["unit", "random"])
def test_benchmark_block_configs(api, ctx, i, affine, gemm_mode):
    """Configs 1-3 at full size, seeds as specified; reports error/allowed per tensor."""
    w = si.config(i, affine=affine)
    d = si.draw(w)
    rep = U.run_block(ctx, api, w.layers[0], w.dtype, d.x, d.lengths, d.params[0], d.g)
    print(f"\nconfig {i} ({affine}, gemm_mode {gemm_mode}) error/allowed: {rep}; adopted gates {rep.adopted}")
    rep.check()
    if affine == "unit":
        # the configuration exactly as specified also meets the plain bound on every element of every stored
        # tensor -- except dx of config 3, whose projection-residual gradient is rounded to bf16 once more
        # before it is summed in (a second half unit in the last place, see parity_util.err_ratio)
        bad = [(n, round(e, 3)) for n, e in rep.plain if e > 1.0 and not (i == 3 and n == "dx")]
        assert not bad, bad


def test_gradient_accumulation(api, ctx):
    L = si.LayerCfg(16, 24, K=5, residual="proj")
    d = _draw_block(L, 2, 48, "f32", seed=5, ragged=True)
    desc = api.block_desc(L, 2, 48, "f32")
    xd, pd = U.dev(d.x, "f32"), U.params_dev(d.params[0], "f32")
    ld = torch.from_numpy(d.lengths).cuda()
    y, _, saved = api.sepconv_fwd(ctx, desc, xd, ld, pd)
    gd = U.dev(d.g, "f32")
    _, _, g1 = api.sepconv_bwd(ctx, desc, gd, xd, y, ld, pd, saved)
    g2 = {k: v.clone() for k, v in g1.items()}
    api.sepconv_bwd(ctx, desc, gd, xd, y, ld, pd, saved, grads=g2, accumulate=True)
    for k in g1:
        torch.testing.assert_close(g2[k], 2 * g1[k], rtol=1e-6, atol=1e-7)


def test_bitwise_repeatable(api, ctx):
    w = si.config(3)
    d = si.draw(w)
    L = w.layers[0]
    desc = api.block_desc(L, w.B, w.T, w.dtype)
    xd, pd = U.dev(d.x, w.dtype), U.params_dev(d.params[0], w.dtype)
    ld = torch.from_numpy(d.lengths).cuda()
    gd = U.dev(d.g, w.dtype)
    outs = []
    for _ in range(2):
        y, _, saved = api.sepconv_fwd(ctx, desc, xd, ld, pd)
        dx, _, grads = api.sepconv_bwd(ctx, desc, gd, xd, y, ld, pd, saved)
        outs.append([y, dx] + [grads[k] for k in sorted(grads)])
    for a, b in zip(*outs):
        assert torch.equal(a, b)


def test_running_stats(api, ctx):
    from oracle import sepconv_oracle as O
    L = si.LayerCfg(8, 12, K=5)
    d = _draw_block(L, 3, 40, "f32", seed=2, ragged=True)
    desc = api.block_desc(L, 3, 40, "f32")
    rm = torch.zeros(12, device="cuda"); rv = torch.ones(12, device="cuda")
    api.sepconv_fwd(ctx, desc, U.dev(d.x, "f32"), torch.from_numpy(d.lengths).cuda(), U.params_dev(d.params[0], "f32"),
                    running_mean=rm, running_var=rv)
    S = O.block_fwd(L, d.x, d.lengths, d.params[0])
    erm, erv = O.running_stats_update(np.zeros(12), np.ones(12), S["mean"], S["var"], S["N"])
    np.testing.assert_allclose(rm.cpu().numpy(), erm, rtol=1e-4, atol=1e-6)
    np.testing.assert_allclose(rv.cpu().numpy(), erv, rtol=1e-4, atol=1e-6)


def test_invalid_length_sets_status(api, ctx):
    L = si.LayerCfg(8, 8, K=3)
    d = _draw_block(L, 2, 32, "f32", seed=1, ragged=False)
    desc = api.block_desc(L, 2, 32, "f32")
    bad = torch.tensor([0, 40], dtype=torch.int32, device="cuda")
    api.sepconv_fwd(ctx, desc, U.dev(d.x, "f32"), bad, U.params_dev(d.params[0], "f32"))
    assert ctx.last_status() == -8
    assert ctx.last_status() == 0      # cleared by the read
