"""The boundary's error behaviour, through the C ABI on a device: every validation code of the header, the
two device-side status codes, and the bounded-wait exit.  Nothing here faults or hangs the GPU: invalid
arguments are turned into status codes by the host checks before anything is enqueued."""
import ctypes as C

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


class Call:
    """One sepconv_fwd call on a small bf16 block, every argument replaceable."""

    def __init__(self, api, ctx, dtype="bf16"):
        self.api, self.ctx = api, ctx
        self.L = si.LayerCfg(16, 24, K=5, residual="proj")
        B, T = 2, 64
        w = si.Workload("b", dtype, B, T, [self.L], 9, len_lo=20, len_hi=T, affine="random")
        self.d = si.draw(w)
        self.desc = api.block_desc(self.L, B, T, dtype)
        self.x = U.dev(self.d.x, dtype)
        self.p = U.params_dev(self.d.params[0], dtype)
        self.lens = torch.from_numpy(self.d.lengths).cuda()
        self.y = torch.empty((B, 24, T), dtype=self.x.dtype, device="cuda")
        nt = torch.float16
        self.saved = {"u": torch.empty((B, 16, T), dtype=torch.float16, device="cuda"),
                      "v": torch.empty((B, 24, T), dtype=nt, device="cuda"),
                      "vr": torch.empty((B, 24, T), dtype=nt, device="cuda")}
        for n in ("mean", "invstd", "mean_r", "invstd_r"):
            self.saved[n] = torch.empty((24,), dtype=torch.float32, device="cuda")
        self.ws = torch.empty(api.sepconv_workspace_bytes(self.desc)[0], dtype=torch.uint8, device="cuda")

    def run(self, x_arg=None, y_arg=None, ws_ptr=None, ws_bytes=None, null_x=False):
        b = self.api.binding
        sv = b.sc_block_saved()
        for n, _ in b.sc_block_saved._fields_:
            setattr(sv, n, self.saved[n].data_ptr() if n in self.saved else None)
        p = b._params_struct(self.p)
        xa = None if null_x else (x_arg if x_arg is not None else b.tensor_arg(self.x))
        ya = y_arg if y_arg is not None else b.tensor_arg(self.y)
        return self.ctx.lib.sepconv_fwd(self.ctx.h, C.byref(self.desc), xa, None, self.lens.data_ptr(), C.byref(p), ya,
                                        None, C.byref(sv), None, None,
                                        self.ws.data_ptr() if ws_ptr is None else ws_ptr,
                                        self.ws.numel() if ws_bytes is None else ws_bytes,
                                        int(torch.cuda.current_stream().cuda_stream))


def test_valid_call_is_ok(api, ctx):
    c = Call(api, ctx)
    assert c.run() == 0
    assert ctx.last_status() == 0


def test_transposed_strides_and_swapped_tags(api, ctx):
    c = Call(api, ctx)
    xt = c.x.transpose(1, 2).contiguous().transpose(1, 2)          # [B, C, T] sizes, time not contiguous
    assert c.run(x_arg=api.binding.tensor_arg(xt)) == -4
    assert c.run(x_arg=api.binding.tensor_arg(c.x, tags=(0, 2, 1))) == -4      # [batch, time, channel] tags


def test_wrong_channel_count_dtype_and_tags(api, ctx):
    c = Call(api, ctx)
    x40 = torch.zeros((2, 40, 64), dtype=c.x.dtype, device="cuda")                # 40 channels into a 16-channel port
    assert c.run(x_arg=api.binding.tensor_arg(x40)) == -3
    assert c.run(x_arg=api.binding.tensor_arg(c.x.half())) == -2                  # float16 tensor, bfloat16 block
    assert c.run(x_arg=api.binding.tensor_arg(c.x, tags=(0, 1, 1))) == -2         # not a batch/channel/time tensor


def test_null_misaligned_and_short_workspace(api, ctx):
    c = Call(api, ctx)
    assert c.run(null_x=True) == -1
    off = api.binding.tensor_arg(c.x)
    off._obj.ptr = c.x.data_ptr() + 2                                              # two bytes off a 16-byte boundary
    assert c.run(x_arg=off) == -5
    assert c.run(ws_bytes=c.ws.numel() - 257) == -7                                # less than the planned scratch
    assert c.run(ws_ptr=0) == -7
    assert ctx.last_status() == 0                                                  # nothing was enqueued


def test_value_beyond_half_range_sets_status(api, ctx):
    c = Call(api, ctx)
    big = (c.x.float() * 1.0e6).to(c.x.dtype)           # u = wd * x leaves the float16 range
    assert c.run(x_arg=api.binding.tensor_arg(big)) == 0
    assert ctx.last_status() == -12
    assert ctx.last_status() == 0


def test_separate_residual_source_needs_dx_res(api, ctx):
    L = si.LayerCfg(16, 16, K=3, residual="identity")
    d = si.draw(si.Workload("r", "f32", 2, 32, [L], 3))
    desc = api.block_desc(L, 2, 32, "f32")
    x, p = U.dev(d.x, "f32"), U.params_dev(d.params[0], "f32")
    lens = torch.from_numpy(d.lengths).cuda()
    other = torch.randn_like(x)
    y, _, saved = api.sepconv_fwd(ctx, desc, x, lens, p, x_res=other)
    with pytest.raises(api.SepconvError) as e:
        api.sepconv_bwd(ctx, desc, U.dev(d.g, "f32"), x, y, lens, p, saved, x_res=other, want_dx_res=False)
    assert e.value.code == -6


def test_bounded_wait_runs_out_and_context_survives(api, ctx):
    ctx.selftest_bounded_wait()
    assert ctx.last_status() == -9
    assert ctx.last_status() == 0
    c = Call(api, ctx)                                   # the context is still usable
    assert c.run() == 0 and ctx.last_status() == 0
