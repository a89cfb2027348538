"""Thin ctypes binding over ``libqf.so`` — argument marshalling only; every step of the path runs
in the CUDA kernels behind the C ABI declared in ``include/qf.h``. Function names match the C
entry points. Tensors are torch CUDA tensors (used purely as device-memory handles); work is
enqueued on torch's current stream. There is no CPU fallback: if the library cannot be loaded or a
call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
from ctypes import c_char_p, c_float, c_int, c_int32, c_int64, c_size_t, c_uint32, c_void_p
from pathlib import Path

import torch

FMT_NONE, FMT_NVFP4, FMT_MXFP4, FMT_Q4_K = 0, 1, 2, 3
DT_BF16, DT_F32 = 0, 1
OP_QDQ, OP_LINEAR_FWD, OP_LINEAR_BWD, OP_GROUPED_FWD, OP_GROUPED_BWD, OP_QDQ_BATCHED = 0, 1, 2, 3, 4, 5
TENSOR_SCALE_GIVEN = 0x1
W_TSCALE_GIVEN, A_TSCALE_GIVEN, ACCUMULATE_DW, FUSED_QDQ, AMAX_RUNNING = 0x1, 0x2, 0x4, 0x8, 0x10
REUSE_W_HAT, REUSE_X_HAT = 0x20, 0x40
MXFP4_NO_CLIP = 0x80
SCALES_TILED = 0x100
TENSOR_SCALE_SPECULATIVE = W_TSCALE_SPECULATIVE = 0x200
BLOCK = {FMT_NVFP4: 16, FMT_MXFP4: 32, FMT_Q4_K: 256}
FORMATS = {"none": FMT_NONE, "nvfp4": FMT_NVFP4, "mxfp4": FMT_MXFP4, "q4_k": FMT_Q4_K}

LIB_PATH = Path(__file__).resolve().parent / "libqf.so"

EXPORTS = [
    "qf_status_string", "qf_version", "qf_workspace_bytes", "qf_read_status", "qf_qdq", "qf_dequant", "qf_amax",
    "qf_fq_linear_fwd", "qf_fq_linear_bwd", "qf_fq_grouped_linear_fwd", "qf_fq_grouped_linear_bwd", "qf_selftest_cvt",
    "qf_selftest_div", "qf_fq_linear_fwd_noalloc", "qf_selftest_mxfp4_bf16", "qf_selftest_timeout", "qf_pack_bytes", "qf_pack", "qf_unpack", "qf_nvfp4_tensor_scale", "qf_qdq_lora",
    "qf_fp4_matmul_native", "qf_qdq_batched",
]
NOALLOC_SCRATCH_BYTES = 32 << 20
LAYOUT_GGUF_Q4_K, LAYOUT_FP4_SWIZZLED_SCALES = 1, 2


class QfError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (qf_status_t={code})")


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libqf.so, building it first if the sources are newer. Raises if that is impossible."""
    global _lib
    if _lib is None:
        from . import build as _build
        path = _build.build()
        L = ctypes.CDLL(str(path))
        L.qf_status_string.restype = c_char_p
        L.qf_status_string.argtypes = [c_int]
        L.qf_version.restype = c_int
        L.qf_workspace_bytes.restype = c_size_t
        L.qf_workspace_bytes.argtypes = [c_int, c_int64, c_int64, c_int64, c_int]
        L.qf_read_status.restype = c_int
        L.qf_read_status.argtypes = [c_void_p, c_void_p, ctypes.POINTER(c_int)]
        L.qf_qdq.restype = c_int
        L.qf_qdq.argtypes = [c_int, c_void_p, c_int64, c_int64, c_void_p, c_void_p, c_void_p, c_void_p, c_uint32,
                             c_void_p, c_size_t, c_void_p]
        L.qf_qdq_batched.restype = c_int
        L.qf_qdq_batched.argtypes = [c_int, c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_uint32,
                                     c_void_p, c_size_t, c_void_p]
        L.qf_dequant.restype = c_int
        L.qf_dequant.argtypes = [c_int, c_void_p, c_void_p, c_void_p, c_int64, c_int64, c_void_p, c_void_p]
        L.qf_amax.restype = c_int
        L.qf_amax.argtypes = [c_void_p, c_int64, c_void_p, c_void_p]
        L.qf_fq_linear_fwd.restype = c_int
        L.qf_fq_linear_fwd.argtypes = [c_void_p, c_void_p, c_void_p, c_int, c_int64, c_int64, c_int64, c_int, c_int,
                                       c_void_p, c_void_p, c_void_p, c_uint32, c_void_p, c_size_t, c_void_p]
        L.qf_fq_linear_bwd.restype = c_int
        L.qf_fq_linear_bwd.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_int, c_int64, c_int64,
                                       c_int64, c_int, c_int, c_void_p, c_void_p, c_uint32, c_void_p, c_size_t, c_void_p]
        L.qf_fq_grouped_linear_fwd.restype = c_int
        L.qf_fq_grouped_linear_fwd.argtypes = [c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_int, c_int64, c_int64,
                                               c_int64, c_int, c_int, c_void_p, c_void_p, c_uint32, c_void_p, c_size_t,
                                               c_void_p]
        L.qf_fq_grouped_linear_bwd.restype = c_int
        L.qf_fq_grouped_linear_bwd.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_int, c_void_p,
                                               c_int, c_int64, c_int64, c_int64, c_int, c_int, c_void_p, c_void_p,
                                               c_uint32, c_void_p, c_size_t, c_void_p]
        L.qf_selftest_cvt.restype = c_int
        L.qf_selftest_cvt.argtypes = [c_void_p, c_int64, c_void_p, c_void_p, c_void_p]
        L.qf_fq_linear_fwd_noalloc.restype = c_int
        L.qf_fq_linear_fwd_noalloc.argtypes = [c_void_p, c_void_p, c_void_p, c_int, c_int64, c_int64, c_int64, c_int, c_int,
                                               c_void_p, c_void_p, c_uint32, c_void_p]
        L.qf_qdq_lora.restype = c_int
        L.qf_qdq_lora.argtypes = [c_int, c_void_p, c_void_p, c_void_p, c_int, c_float, c_int64, c_int64, c_void_p, c_void_p,
                                  c_void_p, c_void_p, c_uint32, c_void_p, c_size_t, c_void_p]
        L.qf_nvfp4_tensor_scale.restype = c_int
        L.qf_nvfp4_tensor_scale.argtypes = [c_void_p, c_void_p, c_int, c_void_p, c_void_p, c_uint32, c_void_p]
        L.qf_pack_bytes.restype = c_size_t
        L.qf_pack_bytes.argtypes = [c_int, c_int, c_int64, c_int64]
        L.qf_pack.restype = c_int
        L.qf_pack.argtypes = [c_int, c_int, c_void_p, c_void_p, c_int64, c_int64, c_void_p, c_void_p]
        L.qf_unpack.restype = c_int
        L.qf_unpack.argtypes = [c_int, c_int, c_void_p, c_int64, c_int64, c_void_p, c_void_p, c_void_p]
        L.qf_fp4_matmul_native.restype = c_int
        L.qf_fp4_matmul_native.argtypes = [c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int64, c_int64,
                                           c_int64, c_void_p, c_uint32, c_void_p, c_size_t, c_void_p]
        L.qf_selftest_timeout.restype = c_int
        L.qf_selftest_timeout.argtypes = [c_void_p, c_size_t, c_int64, c_void_p]
        L.qf_selftest_mxfp4_bf16.restype = c_int
        L.qf_selftest_mxfp4_bf16.argtypes = [c_void_p, c_void_p]
        L.qf_selftest_div.restype = c_int
        L.qf_selftest_div.argtypes = [c_void_p, c_int64, c_void_p, c_int64, c_void_p, c_void_p]
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().qf_status_string(int(code)).decode()


def _check(code: int, where: str):
    if code != 0:
        raise QfError(code, where)


def _ptr(t):
    return None if t is None else c_void_p(t.data_ptr())


def _stream():
    return c_void_p(torch.cuda.current_stream().cuda_stream)


def _dt(dtype: torch.dtype) -> int:
    if dtype == torch.bfloat16:
        return DT_BF16
    if dtype == torch.float32:
        return DT_F32
    raise TypeError(f"unsupported output dtype {dtype}")


def _bf16(t: torch.Tensor, name: str) -> torch.Tensor:
    if t.dtype != torch.bfloat16 or not t.is_cuda or not t.is_contiguous():
        raise TypeError(f"{name} must be a contiguous CUDA BF16 tensor")
    return t


def qf_workspace_bytes(op: int, M: int, N: int, K: int, groups: int = 1) -> int:
    return int(lib().qf_workspace_bytes(op, M, N, K, groups))


def workspace(op: int, M: int, N: int, K: int, groups: int = 1, device="cuda") -> torch.Tensor:
    return torch.empty(qf_workspace_bytes(op, M, N, K, groups), dtype=torch.uint8, device=device)


def qf_read_status(ws: torch.Tensor) -> int:
    out = c_int(0)
    _check(lib().qf_read_status(_ptr(ws), _stream(), ctypes.byref(out)), "qf_read_status")
    return out.value


def scales_shape(fmt: int, rows: int, cols: int):
    return (rows, cols // 256, 16) if fmt == FMT_Q4_K else (rows, cols // BLOCK[fmt])


def qf_qdq(fmt: int, x: torch.Tensor, *, want_out=True, want_codes=True, want_scales=True, tensor_scale=None,
           ws: torch.Tensor | None = None, out=None, codes=None, scales=None, ts_out=None, flags: int = 0):
    """(C, theta) = Q(x), x_hat = Q^-1(C, theta). Returns dict(out, codes, scales, tensor_scale); the
    tensor scale (NVFP4) is a 1-element float32 CUDA tensor, read if ``tensor_scale`` is given.
    ``flags`` may carry MXFP4_NO_CLIP."""
    x = _bf16(x, "x")
    rows, cols = x.shape
    dev = x.device
    if want_out and out is None:
        out = torch.empty_like(x)
    if want_codes and codes is None:
        codes = torch.empty((rows, cols // 2), dtype=torch.uint8, device=dev)
    if want_scales and scales is None:
        scales = torch.empty(scales_shape(fmt, rows, cols), dtype=torch.uint8, device=dev)
    speculative = bool(flags & TENSOR_SCALE_SPECULATIVE)
    flags &= MXFP4_NO_CLIP | TENSOR_SCALE_SPECULATIVE
    ts = None
    if fmt == FMT_NVFP4:
        if tensor_scale is not None:
            ts = tensor_scale if isinstance(tensor_scale, torch.Tensor) else torch.tensor([tensor_scale], dtype=torch.float32, device=dev)
            if not speculative:                      # speculative: the tensor holds a guess and receives the derived scale
                flags |= TENSOR_SCALE_GIVEN
        else:
            ts = ts_out if ts_out is not None else torch.empty(1, dtype=torch.float32, device=dev)
    if ws is None:
        ws = workspace(OP_QDQ, rows, 0, cols, device=dev)
    _check(lib().qf_qdq(fmt, _ptr(x), rows, cols, _ptr(out), _ptr(codes), _ptr(scales), _ptr(ts), flags, _ptr(ws),
                        ws.numel(), _stream()), "qf_qdq")
    return {"out": out, "codes": codes, "scales": scales, "tensor_scale": ts}


class QdqBatch:
    """Marshalled argument arrays of a batched call (built once, reusable call after call: the tensors it was built
    from must stay alive). ``out`` / ``codes`` / ``scales`` are lists of tensors; ``tensor_scales`` is a float32
    CUDA tensor with one entry per input (NVFP4)."""

    def __init__(self, fmt: int, xs, *, want_out=True, want_codes=True, want_scales=True, tensor_scales=None, ws=None):
        self.fmt, self.xs = fmt, [_bf16(x, "x") for x in xs]
        n = self.n = len(self.xs)
        dev = self.xs[0].device if n else "cuda"
        self.out = [torch.empty_like(x) for x in self.xs] if want_out else None
        self.codes = [torch.empty((x.shape[0], x.shape[1] // 2), dtype=torch.uint8, device=dev) for x in self.xs] if want_codes else None
        self.scales = [torch.empty(scales_shape(fmt, *x.shape), dtype=torch.uint8, device=dev) for x in self.xs] if want_scales else None
        self.tensor_scales = tensor_scales
        if fmt == FMT_NVFP4 and tensor_scales is None:
            self.tensor_scales = torch.zeros(max(n, 1), dtype=torch.float32, device=dev)
        self.ws = ws if ws is not None else workspace(OP_QDQ_BATCHED, 0, 0, 0, n, device=dev)
        arr = lambda ts: None if ts is None else (c_void_p * max(n, 1))(*[t.data_ptr() for t in ts])
        self._in, self._out, self._codes, self._scales = arr(self.xs), arr(self.out), arr(self.codes), arr(self.scales)
        self._rows = (c_int64 * max(n, 1))(*[x.shape[0] for x in self.xs])
        self._cols = (c_int64 * max(n, 1))(*[x.shape[1] for x in self.xs])

    def run(self, flags: int = 0):
        _check(lib().qf_qdq_batched(self.fmt, self.n, self._in, self._rows, self._cols, self._out, self._codes, self._scales,
                                    _ptr(self.tensor_scales), flags, _ptr(self.ws), self.ws.numel(), _stream()), "qf_qdq_batched")
        return self


def qf_qdq_batched(fmt: int, xs, *, flags: int = 0, **kw) -> QdqBatch:
    """qf_qdq over a list of tensors in one call; returns the QdqBatch holding the outputs."""
    return QdqBatch(fmt, xs, **kw).run(flags)


def qf_dequant(fmt: int, codes: torch.Tensor, scales: torch.Tensor, tensor_scale, rows: int, cols: int) -> torch.Tensor:
    out = torch.empty((rows, cols), dtype=torch.bfloat16, device=codes.device)
    _check(lib().qf_dequant(fmt, _ptr(codes), _ptr(scales), _ptr(tensor_scale), rows, cols, _ptr(out), _stream()), "qf_dequant")
    return out


def qf_amax(x: torch.Tensor) -> torch.Tensor:
    x = _bf16(x, "x")
    out = torch.empty(1, dtype=torch.float32, device=x.device)
    _check(lib().qf_amax(_ptr(x), x.numel(), _ptr(out), _stream()), "qf_amax")
    return out


def qf_fq_linear_fwd(X, W, wq_fmt: int, aq_fmt: int, *, y_dtype=torch.bfloat16, w_tscale=None, a_tscale=None,
                     a_amax_out=None, flags: int = 0, ws=None, Y=None) -> torch.Tensor:
    """Y = QDQ_a(X) . QDQ_w(W)^T."""
    X, W = _bf16(X, "X"), _bf16(W, "W")
    M, K = X.shape
    N = W.shape[0]
    if Y is None:
        Y = torch.empty((M, N), dtype=y_dtype, device=X.device)
    if ws is None:
        ws = workspace(OP_LINEAR_FWD, M, N, K, device=X.device)
    _check(lib().qf_fq_linear_fwd(_ptr(X), _ptr(W), _ptr(Y), _dt(Y.dtype), M, N, K, wq_fmt, aq_fmt, _ptr(w_tscale),
                                  _ptr(a_tscale), _ptr(a_amax_out), flags, _ptr(ws), ws.numel(), _stream()),
           "qf_fq_linear_fwd")
    return Y


def qf_fq_linear_bwd(dY, X, W, wq_fmt: int, aq_fmt: int, *, dx_dtype=torch.bfloat16, dw_dtype=torch.float32,
                     want_dx=True, want_dw=True, w_tscale=None, a_tscale=None, flags: int = 0, ws=None, dX=None, dW=None):
    """(dX, dW) with dX = dY . QDQ_w(W) and dW = dY^T . QDQ_a(X) (straight-through estimator)."""
    dY = _bf16(dY, "dY")
    M, N = dY.shape
    K = (W if W is not None else X).shape[1]
    if want_dx and dX is None:
        dX = torch.empty((M, K), dtype=dx_dtype, device=dY.device)
    if want_dw and dW is None:
        dW = torch.empty((N, K), dtype=dw_dtype, device=dY.device)
    if ws is None:
        ws = workspace(OP_LINEAR_BWD, M, N, K, device=dY.device)
    _check(lib().qf_fq_linear_bwd(_ptr(dY), _ptr(X), _ptr(W), _ptr(dX), _dt(dX.dtype) if dX is not None else 0, _ptr(dW),
                                  _dt(dW.dtype) if dW is not None else 0, M, N, K, wq_fmt, aq_fmt, _ptr(w_tscale),
                                  _ptr(a_tscale), flags, _ptr(ws), ws.numel(), _stream()), "qf_fq_linear_bwd")
    return dX, dW


def qf_fq_grouped_linear_fwd(X, W, group_offsets, wq_fmt: int, aq_fmt: int, *, y_dtype=torch.bfloat16, w_tscale=None,
                             a_tscale=None, flags: int = 0, ws=None, Y=None) -> torch.Tensor:
    X, W = _bf16(X, "X"), _bf16(W, "W")
    rows, K = X.shape
    G, N, _ = W.shape
    if Y is None:
        Y = torch.empty((rows, N), dtype=y_dtype, device=X.device)
    if ws is None:
        ws = workspace(OP_GROUPED_FWD, rows, N, K, G, device=X.device)
    _check(lib().qf_fq_grouped_linear_fwd(_ptr(X), _ptr(W), _ptr(Y), _dt(Y.dtype), _ptr(group_offsets), G, rows, N, K,
                                          wq_fmt, aq_fmt, _ptr(w_tscale), _ptr(a_tscale), flags, _ptr(ws), ws.numel(),
                                          _stream()), "qf_fq_grouped_linear_fwd")
    return Y


def qf_fq_grouped_linear_bwd(dY, X, W, group_offsets, wq_fmt: int, aq_fmt: int, *, dx_dtype=torch.bfloat16,
                             dw_dtype=torch.float32, want_dx=True, want_dw=True, w_tscale=None, a_tscale=None,
                             flags: int = 0, ws=None, dX=None, dW=None):
    dY = _bf16(dY, "dY")
    rows, N = dY.shape
    G, _, K = W.shape
    if want_dx and dX is None:
        dX = torch.empty((rows, K), dtype=dx_dtype, device=dY.device)
    if want_dw and dW is None:
        dW = torch.empty((G, N, K), dtype=dw_dtype, device=dY.device)
    if ws is None:
        ws = workspace(OP_GROUPED_BWD, rows, N, K, G, device=dY.device)
    _check(lib().qf_fq_grouped_linear_bwd(_ptr(dY), _ptr(X), _ptr(W), _ptr(dX), _dt(dX.dtype) if dX is not None else 0,
                                          _ptr(dW), _dt(dW.dtype) if dW is not None else 0, _ptr(group_offsets), G, rows,
                                          N, K, wq_fmt, aq_fmt, _ptr(w_tscale), _ptr(a_tscale), flags, _ptr(ws),
                                          ws.numel(), _stream()), "qf_fq_grouped_linear_bwd")
    return dX, dW


def qf_selftest_cvt(x: torch.Tensor):
    """E2M1 and E4M3 codes the hardware conversion instructions produce for each FP32 input."""
    assert x.dtype == torch.float32 and x.is_cuda and x.is_contiguous()
    e2 = torch.empty(x.numel(), dtype=torch.uint8, device=x.device)
    e4 = torch.empty(x.numel(), dtype=torch.uint8, device=x.device)
    _check(lib().qf_selftest_cvt(_ptr(x), x.numel(), _ptr(e2), _ptr(e4), _stream()), "qf_selftest_cvt")
    return e2, e4


def qf_selftest_div(xs: torch.Tensor, ys: torch.Tensor) -> int:
    """Number of (x, y) pairs for which the kernels' reciprocal-based division differs from the IEEE divide."""
    assert xs.dtype == torch.float32 and ys.dtype == torch.float32 and xs.is_cuda and ys.is_cuda
    out = torch.zeros(1, dtype=torch.int64, device=xs.device)
    _check(lib().qf_selftest_div(_ptr(xs), xs.numel(), _ptr(ys), ys.numel(), _ptr(out), _stream()), "qf_selftest_div")
    return int(out.item())


def qf_fq_linear_fwd_noalloc(X, W, Y, wq_fmt: int, aq_fmt: int, *, w_tscale=None, a_tscale=None, flags: int = 0) -> torch.Tensor:
    """Y = QDQ_a(X) . QDQ_w(W)^T through the entry point that allocates nothing: the caller passes the
    output tensor, and the transient fake-quantized copies live in a 32 MiB buffer built into the
    library (one per GPU, shared by all calls — do not let two such calls overlap on the GPU). Meant
    for hosts that may not allocate device memory at call time; this wrapper therefore creates no tensor."""
    X, W = _bf16(X, "X"), _bf16(W, "W")
    M, K = X.shape
    N = W.shape[0]
    _check(lib().qf_fq_linear_fwd_noalloc(_ptr(X), _ptr(W), _ptr(Y), _dt(Y.dtype), M, N, K, wq_fmt, aq_fmt, _ptr(w_tscale),
                                          _ptr(a_tscale), flags, _stream()), "qf_fq_linear_fwd_noalloc")
    return Y


def qf_selftest_mxfp4_bf16() -> int:
    """Mismatches between the conversion-free MXFP4 rounding and the conversion-instruction route (all inputs)."""
    out = torch.zeros(1, dtype=torch.int64, device="cuda")
    _check(lib().qf_selftest_mxfp4_bf16(_ptr(out), _stream()), "qf_selftest_mxfp4_bf16")
    return int(out.item())


def qf_selftest_timeout(limit_cycles: int = 1 << 20):
    """Runs the bounded-wait self-test; returns (status word, gave-up flag) read back from the workspace."""
    ws = workspace(OP_QDQ, 0, 0, 0)
    _check(lib().qf_selftest_timeout(_ptr(ws), ws.numel(), limit_cycles, _stream()), "qf_selftest_timeout")
    status = qf_read_status(ws)
    return status, int(ws.view(torch.int32)[16].item())


def qf_pack_bytes(layout: int, fmt: int, rows: int, cols: int) -> int:
    return int(lib().qf_pack_bytes(layout, fmt, rows, cols))


def qf_pack(layout: int, fmt: int, codes, scales, rows: int, cols: int) -> torch.Tensor:
    """Engine-native re-layout of quantized weights: GGUF Q4_K records, or swizzled FP4 block scales."""
    packed = torch.empty(qf_pack_bytes(layout, fmt, rows, cols), dtype=torch.uint8, device=scales.device)
    _check(lib().qf_pack(layout, fmt, _ptr(codes), _ptr(scales), rows, cols, _ptr(packed), _stream()), "qf_pack")
    return packed


def qf_unpack(layout: int, fmt: int, packed: torch.Tensor, rows: int, cols: int):
    codes = torch.empty((rows, cols // 2), dtype=torch.uint8, device=packed.device) if layout == LAYOUT_GGUF_Q4_K else None
    scales = torch.empty(scales_shape(fmt, rows, cols), dtype=torch.uint8, device=packed.device)
    _check(lib().qf_unpack(layout, fmt, _ptr(packed), rows, cols, _ptr(codes), _ptr(scales), _stream()), "qf_unpack")
    return codes, scales


def qf_nvfp4_tensor_scale(tensors, amax_state: torch.Tensor, *, running: bool = False, want_scale: bool = True):
    """Shared NVFP4 tensor scale over several BF16 tensors (fused projections) and/or over steps (running
    activation maximum). Updates ``amax_state`` (1-element float32 CUDA tensor) and returns the scale tensor."""
    n = len(tensors)
    ptrs = (c_void_p * max(n, 1))(*[t.data_ptr() for t in tensors])
    sizes = (c_int64 * max(n, 1))(*[t.numel() for t in tensors])
    scale = torch.empty(1, dtype=torch.float32, device=amax_state.device) if want_scale else None
    _check(lib().qf_nvfp4_tensor_scale(ptrs, sizes, n, _ptr(amax_state), _ptr(scale), AMAX_RUNNING if running else 0, _stream()),
           "qf_nvfp4_tensor_scale")
    return scale


def qf_qdq_lora(fmt: int, W: torch.Tensor, B: torch.Tensor, A: torch.Tensor, lora_scale: float = 1.0, *, tensor_scale=None,
                ws=None, flags: int = 0):
    """Quantize-dequantize of the merged weight W + lora_scale * B @ A without materialising the merge."""
    W, B, A = _bf16(W, "W"), _bf16(B, "B"), _bf16(A, "A")
    rows, cols = W.shape
    rank = A.shape[0]
    dev = W.device
    out = torch.empty_like(W)
    codes = torch.empty((rows, cols // 2), dtype=torch.uint8, device=dev)
    scales = torch.empty(scales_shape(fmt, rows, cols), dtype=torch.uint8, device=dev)
    flags, ts = flags & MXFP4_NO_CLIP, None
    if fmt == FMT_NVFP4:
        if tensor_scale is not None:
            ts, flags = tensor_scale, flags | TENSOR_SCALE_GIVEN
        else:
            ts = torch.empty(1, dtype=torch.float32, device=dev)
    if ws is None:
        ws = workspace(OP_QDQ, rows, 0, cols, device=dev)
    _check(lib().qf_qdq_lora(fmt, _ptr(W), _ptr(B), _ptr(A), rank, float(lora_scale), rows, cols, _ptr(out), _ptr(codes),
                             _ptr(scales), _ptr(ts), flags, _ptr(ws), ws.numel(), _stream()), "qf_qdq_lora")
    return {"out": out, "codes": codes, "scales": scales, "tensor_scale": ts}


def qf_fp4_matmul_native(fmt: int, a: dict, b: dict, K: int, *, flags: int = 0, ws=None) -> torch.Tensor:
    """Y = deq(A) . deq(B)^T on the block-scaled FP4 tensor cores, from the dicts qf_qdq returned for
    A [M, K] and B [N, K] (codes, scales and, for NVFP4, tensor_scale). Returns float32 [M, N].
    With SCALES_TILED in ``flags`` the two ``scales`` entries are qf_pack's tiled block scales."""
    M, N = a["codes"].shape[0], b["codes"].shape[0]
    dev = a["codes"].device
    Y = torch.empty((M, N), dtype=torch.float32, device=dev)
    if ws is None:
        ws = workspace(OP_QDQ, M, 0, K, device=dev)
    _check(lib().qf_fp4_matmul_native(fmt, _ptr(a["codes"]), _ptr(a["scales"]), _ptr(a.get("tensor_scale")), _ptr(b["codes"]),
                                      _ptr(b["scales"]), _ptr(b.get("tensor_scale")), M, N, K, _ptr(Y), flags, _ptr(ws), ws.numel(),
                                      _stream()), "qf_fp4_matmul_native")
    return Y
