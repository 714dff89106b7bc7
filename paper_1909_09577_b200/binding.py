"""ctypes binding of libsepconv_b200.so.

Argument marshalling only: torch tensors supply device memory and the current stream; every step of
the computation runs inside the library's CUDA kernels.  There is no fallback: if the shared library
is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libsepconv_b200.so")

SC_F32, SC_F16, SC_BF16 = 0, 1, 2
DTYPE_CODE = {"f32": SC_F32, "f16": SC_F16, "bf16": SC_BF16}
TORCH_DTYPE = {SC_F32: torch.float32, SC_F16: torch.float16, SC_BF16: torch.bfloat16}
RES_CODE = {"none": 0, "identity": 1, "proj": 2}
PARAM_ORDER = ("wd", "wp", "gamma", "beta", "bias", "wr", "gamma_r", "beta_r")
IO_PARAMS = ("wd", "wp", "wr")


class SepconvError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


class sc_tensor(C.Structure):
    _fields_ = [("ptr", C.c_void_p), ("dtype", C.c_int32), ("rank", C.c_int32),
                ("size", C.c_int64 * 3), ("stride", C.c_int64 * 3), ("tag", C.c_int32 * 3)]


class sc_block_desc(C.Structure):
    _fields_ = [("B", C.c_int32), ("C_in", C.c_int32), ("C_out", C.c_int32), ("T_in", C.c_int32),
                ("K", C.c_int32), ("stride", C.c_int32), ("io_dtype", C.c_int32),
                ("residual", C.c_int32), ("C_res", C.c_int32),
                ("has_dw", C.c_int32), ("has_bn", C.c_int32), ("has_relu", C.c_int32),
                ("has_bias", C.c_int32), ("res_before_relu", C.c_int32),
                ("bn_eps", C.c_float), ("bn_momentum", C.c_float), ("log_softmax", C.c_int32), ("dilation", C.c_int32),
                ("full_conv", C.c_int32)]

    @property
    def T_out(self) -> int:
        s = self.stride if (self.has_dw or self.full_conv) else 1
        return (self.T_in - 1) // s + 1


class sc_block_params(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in PARAM_ORDER]


class sc_block_saved(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("u", "v", "mean", "invstd", "vr", "mean_r", "invstd_r")]


class sc_block_grads(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("dwd", "dwp", "dgamma", "dbeta", "dbias", "dwr", "dgamma_r", "dbeta_r")]


class sc_encoder_desc(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("layers", C.POINTER(sc_block_desc)), ("res_from", C.POINTER(C.c_int32))]


_lib = None

EXPORTS = ("sepconv_set_overlap", "sepconv_set_tile_shape", "sepconv_fwd_static", "sepconv_selftest_bounded_wait", "sepconv_infer", "sepconv_infer_workspace_bytes",
           "encoder_infer", "encoder_infer_workspace_bytes", "sepconv_profile_begin", "sepconv_profile_end", "sepconv_kernel_class_count",
           "sepconv_kernel_class_name", "sepconv_ctx_create", "sepconv_ctx_destroy", "sepconv_last_status", "sepconv_strerror",
           "sepconv_workspace_bytes", "sepconv_fwd", "sepconv_bwd", "encoder_workspace_bytes",
           "encoder_fwd_bwd", "sepconv_set_gemm_mode", "sepconv_launch_count")


def load_library(path: str = LIB_PATH):
    """Loads the shared library (never builds it, never falls back)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(path):
        raise FileNotFoundError(
            f"{path} not found: build it with `python -m paper_1909_09577_b200.build` "
            "(there is no CPU or PyTorch fallback)")
    lib = C.CDLL(path)
    lib.sepconv_strerror.restype = C.c_char_p
    lib.sepconv_strerror.argtypes = [C.c_int]
    lib.sepconv_ctx_create.argtypes = [C.POINTER(C.c_void_p), C.c_int]
    lib.sepconv_ctx_destroy.argtypes = [C.c_void_p]
    lib.sepconv_ctx_destroy.restype = None
    lib.sepconv_last_status.argtypes = [C.c_void_p, C.c_void_p]
    lib.sepconv_set_gemm_mode.argtypes = [C.c_void_p, C.c_int]
    lib.sepconv_selftest_bounded_wait.argtypes = [C.c_void_p, C.c_void_p]
    lib.sepconv_set_overlap.argtypes = [C.c_void_p, C.c_int]
    lib.sepconv_set_tile_shape.argtypes = [C.c_void_p, C.c_int]
    lib.sepconv_launch_count.argtypes = [C.c_void_p]
    lib.sepconv_launch_count.restype = C.c_int64
    lib.sepconv_workspace_bytes.argtypes = [C.POINTER(sc_block_desc), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
    lib.sepconv_fwd.argtypes = [C.c_void_p, C.POINTER(sc_block_desc), C.POINTER(sc_tensor), C.POINTER(sc_tensor),
                                C.c_void_p, C.POINTER(sc_block_params), C.POINTER(sc_tensor), C.c_void_p,
                                C.POINTER(sc_block_saved), C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t,
                                C.c_void_p]
    lib.sepconv_fwd_static.argtypes = [C.c_void_p, C.POINTER(sc_block_desc), C.POINTER(sc_tensor),
                                       C.POINTER(sc_tensor), C.c_void_p, C.POINTER(sc_block_params),
                                       C.POINTER(sc_tensor), C.c_void_p, C.POINTER(sc_block_saved), C.c_void_p]
    lib.sepconv_bwd.argtypes = [C.c_void_p, C.POINTER(sc_block_desc), C.POINTER(sc_tensor), C.POINTER(sc_tensor),
                                C.POINTER(sc_tensor), C.POINTER(sc_tensor), C.c_void_p,
                                C.POINTER(sc_block_params), C.POINTER(sc_block_saved), C.POINTER(sc_tensor),
                                C.POINTER(sc_tensor), C.POINTER(sc_tensor), C.POINTER(sc_block_grads), C.c_int,
                                C.c_void_p, C.c_size_t, C.c_void_p]
    lib.encoder_workspace_bytes.argtypes = [C.POINTER(sc_encoder_desc), C.POINTER(C.c_size_t)]
    lib.encoder_fwd_bwd.argtypes = [C.c_void_p, C.POINTER(sc_encoder_desc), C.POINTER(sc_tensor), C.c_void_p,
                                    C.c_void_p, C.POINTER(C.c_int64), C.POINTER(sc_tensor),
                                    C.POINTER(sc_tensor), C.c_void_p, C.c_void_p, C.POINTER(C.c_int64),
                                    C.POINTER(sc_tensor), C.c_int, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.sepconv_infer_workspace_bytes.argtypes = [C.POINTER(sc_block_desc), C.POINTER(C.c_size_t)]
    lib.sepconv_infer.argtypes = [C.c_void_p, C.POINTER(sc_block_desc), C.POINTER(sc_tensor), C.POINTER(sc_tensor),
                                  C.c_void_p, C.POINTER(sc_block_params), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                  C.POINTER(sc_tensor), C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.encoder_infer_workspace_bytes.argtypes = [C.POINTER(sc_encoder_desc), C.POINTER(C.c_size_t)]
    lib.encoder_infer.argtypes = [C.c_void_p, C.POINTER(sc_encoder_desc), C.POINTER(sc_tensor), C.c_void_p, C.c_void_p,
                                  C.POINTER(C.c_int64), C.c_void_p, C.POINTER(C.c_int64), C.POINTER(sc_tensor), C.c_void_p,
                                  C.c_void_p, C.c_size_t, C.c_void_p]
    lib.sepconv_profile_begin.argtypes = [C.c_void_p, C.c_int, C.c_int]
    lib.sepconv_profile_end.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_int64),
                                        C.POINTER(C.c_double), C.POINTER(C.c_double)]
    lib.sepconv_kernel_class_name.restype = C.c_char_p
    lib.sepconv_kernel_class_name.argtypes = [C.c_int]
    _lib = lib
    return lib


def strerror(code: int) -> str:
    return load_library().sepconv_strerror(code).decode()


def _check(code: int, where: str):
    if code != 0:
        raise SepconvError(code, where)


def _stream_ptr(stream) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


def tensor_arg(t: Optional[torch.Tensor], tags=(0, 1, 2)):
    """torch [B,C,T] tensor -> sc_tensor (by reference); None -> NULL."""
    if t is None:
        return None
    code = {torch.float32: SC_F32, torch.float16: SC_F16, torch.bfloat16: SC_BF16}.get(t.dtype, -1)
    st = sc_tensor()
    st.ptr = t.data_ptr()
    st.dtype = code
    st.rank = t.dim()
    for i in range(min(3, t.dim())):
        st.size[i] = t.shape[i]
        st.stride[i] = t.stride(i)
        st.tag[i] = tags[i]
    return C.byref(st)


def block_desc(L, B: int, T: int, dtype: str) -> sc_block_desc:
    """Descriptor from any object with the layer fields (C_in, C_out, K, stride, has_dw, ...)."""
    d = sc_block_desc()
    d.B, d.C_in, d.C_out, d.T_in = B, L.C_in, L.C_out, T
    d.K, d.stride = L.K, L.stride
    d.io_dtype = DTYPE_CODE[dtype] if isinstance(dtype, str) else int(dtype)
    d.residual = RES_CODE[L.residual]
    d.C_res = getattr(L, "C_res", L.C_in) if L.residual != "none" else 0
    d.has_dw, d.has_bn, d.has_relu, d.has_bias = int(L.has_dw), int(L.has_bn), int(L.has_relu), int(L.has_bias)
    d.res_before_relu = int(L.res_before_relu)
    d.bn_eps = float(L.eps)
    d.bn_momentum = 0.1
    d.log_softmax = int(getattr(L, "log_softmax", False))
    d.dilation = int(getattr(L, "dilation", 1))
    d.full_conv = int(getattr(L, "full_conv", False))
    return d


class Context:
    """Owns an sc_ctx on one CUDA device."""

    def __init__(self, device: int = 0):
        self.lib = load_library()
        self.device = device
        h = C.c_void_p()
        _check(self.lib.sepconv_ctx_create(C.byref(h), device), "sepconv_ctx_create")
        self.h = h

    def close(self):
        if getattr(self, "h", None):
            self.lib.sepconv_ctx_destroy(self.h)
            self.h = None

    __del__ = close

    def last_status(self, stream=None) -> int:
        return int(self.lib.sepconv_last_status(self.h, _stream_ptr(stream)))

    def selftest_bounded_wait(self, stream=None):
        """Enqueues the kernel whose bounded wait must run out (see sepconv.h)."""
        _check(self.lib.sepconv_selftest_bounded_wait(self.h, _stream_ptr(stream)), "sepconv_selftest_bounded_wait")

    def set_overlap(self, second_stream: bool = True, dependent_launch: bool = True):
        """second_stream: independent kernels on the context's second stream; dependent_launch: every kernel
        launched so that its set-up overlaps the previous kernel's tail.  Both default to on."""
        _check(self.lib.sepconv_set_overlap(self.h, int(bool(second_stream)) | (int(bool(dependent_launch)) << 1)),
               "sepconv_set_overlap")

    def set_tile_shape(self, shape: int):
        _check(self.lib.sepconv_set_tile_shape(self.h, shape), "sepconv_set_tile_shape")

    def set_gemm_mode(self, mode: int):
        _check(self.lib.sepconv_set_gemm_mode(self.h, mode), "sepconv_set_gemm_mode")

    def launch_count(self) -> int:
        return int(self.lib.sepconv_launch_count(self.h))

    def kernel_classes(self):
        return [self.lib.sepconv_kernel_class_name(i).decode() for i in range(self.lib.sepconv_kernel_class_count())]

    def profile_begin(self, kernel_class="all", max_launches: int = 4096):
        """Start bracketing launches of one kernel class (name, or "all") with CUDA events."""
        cls = -1 if kernel_class == "all" else self.kernel_classes().index(kernel_class)
        _check(self.lib.sepconv_profile_begin(self.h, cls, max_launches), "sepconv_profile_begin")

    def profile_end(self, stream=None):
        """Synchronise and return {class name: dict(ms, launches, bytes, flops)} for bracketed classes."""
        n = self.lib.sepconv_kernel_class_count()
        ms, cnt = (C.c_double * n)(), (C.c_int64 * n)()
        by, fl = (C.c_double * n)(), (C.c_double * n)()
        _check(self.lib.sepconv_profile_end(self.h, _stream_ptr(stream), ms, cnt, by, fl), "sepconv_profile_end")
        names = self.kernel_classes()
        return {names[i]: dict(ms=ms[i], launches=int(cnt[i]), bytes=by[i], flops=fl[i])
                for i in range(n) if cnt[i] > 0}


def sepconv_workspace_bytes(desc: sc_block_desc):
    f, b = C.c_size_t(), C.c_size_t()
    _check(load_library().sepconv_workspace_bytes(C.byref(desc), C.byref(f), C.byref(b)), "sepconv_workspace_bytes")
    return int(f.value), int(b.value)


def _workspace(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)


def _params_struct(params: Dict[str, torch.Tensor]) -> sc_block_params:
    p = sc_block_params()
    for n in PARAM_ORDER:
        setattr(p, n, params[n].data_ptr() if n in params and params[n] is not None else None)
    return p


def sepconv_fwd(ctx: Context, desc: sc_block_desc, x: torch.Tensor, lengths: torch.Tensor,
                params: Dict[str, torch.Tensor], x_res: Optional[torch.Tensor] = None,
                running_mean=None, running_var=None, workspace: Optional[torch.Tensor] = None, stream=None,
                y: Optional[torch.Tensor] = None, saved: Optional[Dict[str, torch.Tensor]] = None):
    """Returns (y, out_lengths, saved).  Buffers are allocated with torch unless passed in."""
    dev = x.device
    td = TORCH_DTYPE[desc.io_dtype]
    B, Co, Ci, Tp = desc.B, desc.C_out, desc.C_in, desc.T_out
    if y is None:
        y = torch.empty((B, Co, Tp), dtype=td, device=dev)
    out_len = torch.empty((B,), dtype=torch.int32, device=dev)
    if saved is None:
        ut = torch.float16 if (desc.has_dw and desc.has_bn and desc.io_dtype != SC_F32) else td
        saved = {"u": torch.empty((B, Ci, Tp), dtype=ut, device=dev)}
        nt = torch.float32 if desc.io_dtype == SC_F32 else torch.float16   # type of the saved pointwise results
        if desc.has_bn:
            saved["v"] = torch.empty((B, Co, Tp), dtype=nt, device=dev)
            saved["mean"] = torch.empty((Co,), dtype=torch.float32, device=dev)
            saved["invstd"] = torch.empty((Co,), dtype=torch.float32, device=dev)
        if desc.residual == 2:
            saved["vr"] = torch.empty((B, Co, Tp), dtype=nt, device=dev)
            saved["mean_r"] = torch.empty((Co,), dtype=torch.float32, device=dev)
            saved["invstd_r"] = torch.empty((Co,), dtype=torch.float32, device=dev)
    sv = sc_block_saved()
    for n, _ in sc_block_saved._fields_:
        setattr(sv, n, saved[n].data_ptr() if n in saved else None)
    if workspace is None:
        workspace = _workspace(sepconv_workspace_bytes(desc)[0], dev)
    p = _params_struct(params)
    rc = ctx.lib.sepconv_fwd(ctx.h, C.byref(desc), tensor_arg(x), tensor_arg(x_res), lengths.data_ptr(),
                             C.byref(p), tensor_arg(y), out_len.data_ptr(), C.byref(sv),
                             running_mean.data_ptr() if running_mean is not None else None,
                             running_var.data_ptr() if running_var is not None else None,
                             workspace.data_ptr(), workspace.numel(), _stream_ptr(stream))
    _check(rc, "sepconv_fwd")
    return y, out_len, saved


def sepconv_infer(ctx: Context, desc: sc_block_desc, x: torch.Tensor, lengths: torch.Tensor,
                  params: Dict[str, torch.Tensor], running: Dict[str, torch.Tensor],
                  x_res: Optional[torch.Tensor] = None, stream=None):
    """Evaluation-mode forward.  running: float32 device tensors "mean", "var" (and "mean_r", "var_r" for a
    projection residual).  Returns (y, out_lengths)."""
    dev = x.device
    y = torch.empty((desc.B, desc.C_out, desc.T_out), dtype=TORCH_DTYPE[desc.io_dtype], device=dev)
    out_len = torch.empty((desc.B,), dtype=torch.int32, device=dev)
    n = C.c_size_t()
    _check(ctx.lib.sepconv_infer_workspace_bytes(C.byref(desc), C.byref(n)), "sepconv_infer_workspace_bytes")
    ws = _workspace(int(n.value), dev)
    p = _params_struct(params)
    ptr = lambda k: running[k].data_ptr() if k in running and running[k] is not None else None
    rc = ctx.lib.sepconv_infer(ctx.h, C.byref(desc), tensor_arg(x), tensor_arg(x_res), lengths.data_ptr(), C.byref(p),
                               ptr("mean"), ptr("var"), ptr("mean_r"), ptr("var_r"), tensor_arg(y), out_len.data_ptr(),
                               ws.data_ptr(), ws.numel(), _stream_ptr(stream))
    _check(rc, "sepconv_infer")
    return y, out_len


STATIC_SCRATCH_BYTES = 8 << 20


def sepconv_fwd_static(ctx: Context, desc: sc_block_desc, x: torch.Tensor, lengths: torch.Tensor,
                       params: Dict[str, torch.Tensor], y: torch.Tensor, out_lengths: torch.Tensor,
                       saved: Dict[str, torch.Tensor], x_res: Optional[torch.Tensor] = None, stream=None):
    """sepconv_fwd for callers that cannot allocate: every buffer (y, out_lengths, saved) is passed in
    and the scratch is the library's built-in fixed array.  This wrapper allocates nothing either."""
    sv = sc_block_saved()
    for n, _ in sc_block_saved._fields_:
        setattr(sv, n, saved[n].data_ptr() if n in saved else None)
    p = _params_struct(params)
    rc = ctx.lib.sepconv_fwd_static(ctx.h, C.byref(desc), tensor_arg(x), tensor_arg(x_res), lengths.data_ptr(),
                                    C.byref(p), tensor_arg(y), out_lengths.data_ptr(), C.byref(sv),
                                    _stream_ptr(stream))
    _check(rc, "sepconv_fwd_static")


def sepconv_bwd(ctx: Context, desc: sc_block_desc, dy: torch.Tensor, x: torch.Tensor, y: torch.Tensor,
                lengths: torch.Tensor, params: Dict[str, torch.Tensor], saved: Dict[str, torch.Tensor],
                x_res: Optional[torch.Tensor] = None, dx_add: Optional[torch.Tensor] = None,
                want_dx_res: bool = False, grads: Optional[Dict[str, torch.Tensor]] = None,
                accumulate: bool = False, workspace: Optional[torch.Tensor] = None, stream=None):
    """Returns (dx, dx_res or None, grads)."""
    dev = x.device
    td = TORCH_DTYPE[desc.io_dtype]
    dx = torch.empty_like(x)
    dx_res = None
    if want_dx_res:
        Cres = desc.C_res if desc.C_res > 0 else desc.C_in
        dx_res = torch.empty((desc.B, Cres, desc.T_out), dtype=td, device=dev)
    if grads is None:
        grads = {"d" + n: torch.zeros(params[n].shape, dtype=torch.float32, device=dev)
                 for n in PARAM_ORDER if n in params and params[n] is not None}
    g = sc_block_grads()
    for n, _ in sc_block_grads._fields_:
        setattr(g, n, grads[n].data_ptr() if n in grads else None)
    sv = sc_block_saved()
    for n, _ in sc_block_saved._fields_:
        setattr(sv, n, saved[n].data_ptr() if n in saved else None)
    if workspace is None:
        workspace = _workspace(sepconv_workspace_bytes(desc)[1], dev)
    p = _params_struct(params)
    rc = ctx.lib.sepconv_bwd(ctx.h, C.byref(desc), tensor_arg(dy), tensor_arg(x), tensor_arg(x_res), tensor_arg(y),
                             lengths.data_ptr(), C.byref(p), C.byref(sv), tensor_arg(dx), tensor_arg(dx_res),
                             tensor_arg(dx_add), C.byref(g), int(accumulate), workspace.data_ptr(),
                             workspace.numel(), _stream_ptr(stream))
    _check(rc, "sepconv_bwd")
    return dx, dx_res, grads


class EncoderSpec:
    """Host-side description of an encoder: layer descriptors, residual sources and the layout of the
    flat parameter / gradient blobs (conv weights in the activation type, the rest float32; every
    array starts on a 256-byte boundary)."""

    def __init__(self, layers: Sequence, B: int, T: int, dtype: str):
        self.layers = list(layers)
        self.B, self.T, self.dtype = B, T, dtype
        self.code = DTYPE_CODE[dtype]
        n = len(self.layers)
        self._descs = (sc_block_desc * n)()
        self._res = (C.c_int32 * n)()
        self.param_offsets = (C.c_int64 * (8 * n))()
        self.grad_offsets = (C.c_int64 * (8 * n))()
        self.shapes: List[Dict[str, tuple]] = []
        es = 4 if dtype == "f32" else 2
        po = go = 0
        t = T
        for i, L in enumerate(self.layers):
            d = block_desc(L, B, t, dtype)
            self._descs[i] = d
            t = d.T_out
            rf = getattr(L, "res_from", None)
            self._res[i] = -1 if rf is None else rf
            shp = L.param_shapes()
            self.shapes.append(shp)
            for j, name in enumerate(PARAM_ORDER):
                if name not in shp:
                    self.param_offsets[8 * i + j] = -1
                    self.grad_offsets[8 * i + j] = -1
                    continue
                cnt = int(np.prod(shp[name]))
                self.param_offsets[8 * i + j] = po
                self.grad_offsets[8 * i + j] = go
                po += (cnt * (es if name in IO_PARAMS else 4) + 255) // 256 * 256
                go += (cnt * 4 + 255) // 256 * 256
        self.param_bytes, self.grad_bytes = po, go
        self.T_out = t
        self.C_out = self.layers[-1].C_out
        self.desc = sc_encoder_desc(n, self._descs, self._res)

    def pack_params(self, params: Sequence[Dict[str, np.ndarray]], device) -> torch.Tensor:
        blob = torch.zeros(self.param_bytes, dtype=torch.uint8, device=device)
        td = TORCH_DTYPE[self.code]
        for i, p in enumerate(params):
            for j, name in enumerate(PARAM_ORDER):
                off = self.param_offsets[8 * i + j]
                if off < 0:
                    continue
                src = torch.as_tensor(np.ascontiguousarray(p[name], dtype=np.float32))
                src = src.to(td if name in IO_PARAMS else torch.float32).contiguous().to(device)
                raw = src.view(torch.uint8).reshape(-1)
                blob[off:off + raw.numel()] = raw
        return blob

    def pack_running(self, running: Sequence[Optional[Dict[str, np.ndarray]]], device):
        """Flat float32 blob of the per-layer running statistics (mean, var, mean_r, var_r) and the host
        offsets array that encoder_infer takes."""
        offs = (C.c_int64 * (4 * len(self.layers)))()
        chunks, pos = [], 0
        for i, r in enumerate(running):
            for j, name in enumerate(("mean", "var", "mean_r", "var_r")):
                if r is None or name not in r or r[name] is None:
                    offs[4 * i + j] = -1
                    continue
                a = np.ascontiguousarray(r[name], dtype=np.float32)
                offs[4 * i + j] = pos
                chunks.append((pos, a))
                pos += (a.nbytes + 255) // 256 * 256
        blob = torch.zeros(max(pos, 256), dtype=torch.uint8, device=device)
        for off, a in chunks:
            blob[off:off + a.nbytes] = torch.from_numpy(a).view(torch.uint8).reshape(-1).to(device)
        return blob, offs

    def param_view(self, blob: torch.Tensor, i: int, name: str) -> torch.Tensor:
        j = PARAM_ORDER.index(name)
        off = self.param_offsets[8 * i + j]
        td = TORCH_DTYPE[self.code] if name in IO_PARAMS else torch.float32
        cnt = int(np.prod(self.shapes[i][name]))
        return blob[off:off + cnt * td.itemsize].view(td).reshape(self.shapes[i][name])

    def grad_view(self, blob: torch.Tensor, i: int, name: str) -> torch.Tensor:
        j = PARAM_ORDER.index(name)
        off = self.grad_offsets[8 * i + j]
        cnt = int(np.prod(self.shapes[i][name]))
        return blob[off:off + cnt * 4].view(torch.float32).reshape(self.shapes[i][name])


def encoder_workspace_bytes(spec: EncoderSpec) -> int:
    n = C.c_size_t()
    _check(load_library().encoder_workspace_bytes(C.byref(spec.desc), C.byref(n)), "encoder_workspace_bytes")
    return int(n.value)


def encoder_infer(ctx: Context, spec: EncoderSpec, x: torch.Tensor, lengths: torch.Tensor, params_blob: torch.Tensor,
                  running_blob: torch.Tensor, running_offsets, workspace: Optional[torch.Tensor] = None, stream=None):
    """Evaluation-mode forward through every layer.  Returns (out, out_lengths)."""
    dev = x.device
    out = torch.empty((spec.B, spec.C_out, spec.T_out), dtype=TORCH_DTYPE[spec.code], device=dev)
    out_len = torch.empty((spec.B,), dtype=torch.int32, device=dev)
    if workspace is None:
        n = C.c_size_t()
        _check(ctx.lib.encoder_infer_workspace_bytes(C.byref(spec.desc), C.byref(n)), "encoder_infer_workspace_bytes")
        workspace = _workspace(int(n.value), dev)
    rc = ctx.lib.encoder_infer(ctx.h, C.byref(spec.desc), tensor_arg(x), lengths.data_ptr(), params_blob.data_ptr(),
                               spec.param_offsets, running_blob.data_ptr(), running_offsets, tensor_arg(out),
                               out_len.data_ptr(), workspace.data_ptr(), workspace.numel(), _stream_ptr(stream))
    _check(rc, "encoder_infer")
    return out, out_len


def encoder_fwd_bwd(ctx: Context, spec: EncoderSpec, x: torch.Tensor, lengths: torch.Tensor,
                    params_blob: torch.Tensor, dlogits: torch.Tensor, grads_blob: Optional[torch.Tensor] = None,
                    want_dx: bool = False, accumulate: bool = False, workspace: Optional[torch.Tensor] = None,
                    logits: Optional[torch.Tensor] = None, stream=None):
    """Returns (logits, out_lengths, grads_blob, dx or None)."""
    dev = x.device
    td = TORCH_DTYPE[spec.code]
    if logits is None:
        logits = torch.empty((spec.B, spec.C_out, spec.T_out), dtype=td, device=dev)
    out_len = torch.empty((spec.B,), dtype=torch.int32, device=dev)
    if grads_blob is None:
        grads_blob = torch.zeros(spec.grad_bytes, dtype=torch.uint8, device=dev)
    dx = torch.empty_like(x) if want_dx else None
    if workspace is None:
        workspace = _workspace(encoder_workspace_bytes(spec), dev)
    rc = ctx.lib.encoder_fwd_bwd(ctx.h, C.byref(spec.desc), tensor_arg(x), lengths.data_ptr(),
                                 params_blob.data_ptr(), spec.param_offsets, tensor_arg(dlogits),
                                 tensor_arg(logits), out_len.data_ptr(), grads_blob.data_ptr(),
                                 spec.grad_offsets, tensor_arg(dx), int(accumulate), workspace.data_ptr(),
                                 workspace.numel(), _stream_ptr(stream))
    _check(rc, "encoder_fwd_bwd")
    return logits, out_len, grads_blob, dx
