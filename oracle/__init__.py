"""CPU oracle for the fake-quantization hot path — TEST INFRASTRUCTURE ONLY.

Plain, slow, host-only restatement of what the path computes (the paper's Section 3.2: the
quantizer interface, the NVFP4 / MXFP4 / Q4_K formats, the quantization-aware layer and its
straight-through backward). Only the tests, the smoke check and the benchmark's CPU-baseline leg
may import this package. The CUDA library never does and shares no code with it.

The arithmetic lives in ``qf_oracle.cpp`` (plain C++, compiled here with g++); this module only
builds it, loads it with ctypes and marshals numpy arrays. BF16 tensors travel as ``uint16``
arrays holding the raw bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "qf_oracle.cpp"
_LIB = _HERE / "libqf_oracle.so"

FMT_NONE, FMT_NVFP4, FMT_MXFP4, FMT_Q4_K = 0, 1, 2, 3
BLOCK = {FMT_NVFP4: 16, FMT_MXFP4: 32, FMT_Q4_K: 256}


def build(force: bool = False) -> Path:
    """Compile the oracle. No fast-math, no FMA contraction: every FP32 operation is one IEEE op."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
        cmd = ["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
               "-shared", "-fPIC", str(_SRC), "-o", str(tmp)]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(str(build()))
        c = ctypes
        L.orc_e2m1_encode.restype = c.c_uint8
        L.orc_e2m1_encode.argtypes = [c.c_float]
        L.orc_e2m1_value.restype = c.c_float
        L.orc_e2m1_value.argtypes = [c.c_uint8]
        L.orc_e4m3_encode.restype = c.c_uint8
        L.orc_e4m3_encode.argtypes = [c.c_float]
        L.orc_e4m3_value.restype = c.c_float
        L.orc_e4m3_value.argtypes = [c.c_uint8]
        L.orc_bf16_round.restype = c.c_uint16
        L.orc_bf16_round.argtypes = [c.c_float]
        L.orc_fp16_round_sat.restype = c.c_uint16
        L.orc_fp16_round_sat.argtypes = [c.c_float]
        L.orc_fp16_value.restype = c.c_float
        L.orc_fp16_value.argtypes = [c.c_uint16]
        L.orc_num_threads.restype = c.c_int
        L.orc_amax.restype = c.c_float
        L.orc_amax.argtypes = [c.c_void_p, c.c_int64]
        L.orc_qdq.restype = c.c_int
        L.orc_qdq.argtypes = [c.c_int, c.c_void_p, c.c_int64, c.c_int64, c.c_void_p, c.c_void_p,
                              c.c_void_p, c.c_void_p, c.c_int, c.c_int]
        L.orc_dequant.restype = c.c_int
        L.orc_dequant.argtypes = [c.c_int, c.c_void_p, c.c_void_p, c.c_void_p, c.c_int64, c.c_int64,
                                  c.c_void_p]
        for name in ("orc_matmul_fwd", "orc_matmul_dgrad"):
            f = getattr(L, name)
            f.restype = None
            f.argtypes = [c.c_void_p, c.c_void_p, c.c_int64, c.c_int64, c.c_int64, c.c_void_p]
        L.orc_matmul_wgrad.restype = None
        L.orc_matmul_wgrad.argtypes = [c.c_void_p, c.c_void_p, c.c_int64, c.c_int64, c.c_int64,
                                       c.c_void_p, c.c_int64, c.c_void_p]
        L.orc_lora_merge.restype = None
        L.orc_lora_merge.argtypes = [c.c_void_p, c.c_void_p, c.c_void_p, c.c_int64, c.c_int64, c.c_int64, c.c_float, c.c_void_p]
        _lib = L
    return _lib


def num_threads() -> int:
    return int(lib().orc_num_threads())


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _bf16_arr(x) -> np.ndarray:
    a = np.ascontiguousarray(x)
    if a.dtype != np.uint16:
        raise TypeError("BF16 tensors are passed as uint16 bit patterns")
    return a


# ---- scalar helpers (pinned one by one in the tests) ------------------------------------------

def e2m1_encode(v: float) -> int:
    return int(lib().orc_e2m1_encode(float(v)))


def e2m1_value(c: int) -> float:
    return float(lib().orc_e2m1_value(int(c)))


def e4m3_encode(q: float) -> int:
    return int(lib().orc_e4m3_encode(float(q)))


def e4m3_value(c: int) -> float:
    return float(lib().orc_e4m3_value(int(c)))


def bf16_round(f: float) -> int:
    return int(lib().orc_bf16_round(float(f)))


def fp16_round_sat(f: float) -> int:
    return int(lib().orc_fp16_round_sat(float(f)))


def fp16_value(h: int) -> float:
    return float(lib().orc_fp16_value(int(h)))


def bf16_to_f32(a: np.ndarray) -> np.ndarray:
    """Exact widening of BF16 bit patterns to float32 (a format conversion, no arithmetic)."""
    return (a.astype(np.uint32) << 16).view(np.float32)


def amax(x) -> float:
    x = _bf16_arr(x)
    return float(lib().orc_amax(_p(x), x.size))


# ---- quantizer interface: Q(X) -> (C, theta), Q^-1(C, theta) -> X_hat ------------------------

def scales_shape(fmt: int, rows: int, cols: int):
    if fmt == FMT_Q4_K:
        return (rows, cols // 256, 16)
    return (rows, cols // BLOCK[fmt])


def qdq(fmt: int, x, tensor_scale: float | None = None, mxfp4_noclip: bool = False):
    """Quantize-dequantize a BF16 [rows, cols] tensor. Returns a dict with ``out`` (uint16 BF16
    bits), ``codes`` (uint8, two 4-bit codes per byte), ``scales`` (uint8 metadata) and
    ``tensor_scale`` (float32, NVFP4 only; given or derived from the tensor's absolute maximum).
    ``mxfp4_noclip`` picks the MXFP4 block exponent as the smallest one under which the block
    maximum does not saturate, instead of floor(log2 amax) - 2."""
    x = _bf16_arr(x)
    rows, cols = x.shape
    out = np.empty_like(x)
    codes = np.empty((rows, cols // 2), np.uint8)
    scales = np.empty(scales_shape(fmt, rows, cols), np.uint8)
    ts = np.array([0.0 if tensor_scale is None else tensor_scale], np.float32)
    rc = lib().orc_qdq(fmt, _p(x), rows, cols, _p(out), _p(codes), _p(scales), _p(ts),
                       0 if tensor_scale is None else 1, 1 if mxfp4_noclip else 0)
    if rc != 0:
        raise ValueError("orc_qdq: bad format or shape")
    return {"out": out, "codes": codes, "scales": scales,
            "tensor_scale": np.float32(ts[0]) if fmt == FMT_NVFP4 else None}


def qdq_out(fmt: int, x, tensor_scale: float | None = None, mxfp4_noclip: bool = False) -> np.ndarray:
    """X_hat only; ``fmt == FMT_NONE`` is the identity (an unquantized operand)."""
    if fmt == FMT_NONE:
        return _bf16_arr(x)
    return qdq(fmt, x, tensor_scale, mxfp4_noclip)["out"]


def dequant(fmt: int, codes, scales, tensor_scale, rows: int, cols: int) -> np.ndarray:
    codes = np.ascontiguousarray(codes, np.uint8)
    scales = np.ascontiguousarray(scales, np.uint8)
    ts = np.array([1.0 if tensor_scale is None else tensor_scale], np.float32)
    out = np.empty((rows, cols), np.uint16)
    rc = lib().orc_dequant(fmt, _p(codes), _p(scales), _p(ts), rows, cols, _p(out))
    if rc != 0:
        raise ValueError("orc_dequant: bad format or shape")
    return out


# ---- matmuls on (already fake-quantized) BF16 operands, FP64 accumulation ----------------------

def matmul_fwd(xh, wh) -> np.ndarray:
    xh, wh = _bf16_arr(xh), _bf16_arr(wh)
    M, K = xh.shape
    N, K2 = wh.shape
    assert K == K2
    y = np.empty((M, N), np.float32)
    lib().orc_matmul_fwd(_p(xh), _p(wh), M, N, K, _p(y))
    return y


def matmul_dgrad(dy, wh) -> np.ndarray:
    dy, wh = _bf16_arr(dy), _bf16_arr(wh)
    M, N = dy.shape
    N2, K = wh.shape
    assert N == N2
    dx = np.empty((M, K), np.float32)
    lib().orc_matmul_dgrad(_p(dy), _p(wh), M, N, K, _p(dx))
    return dx


def matmul_wgrad(dy, xh, n_idx=None) -> np.ndarray:
    dy, xh = _bf16_arr(dy), _bf16_arr(xh)
    M, N = dy.shape
    M2, K = xh.shape
    assert M == M2
    idx = None if n_idx is None else np.ascontiguousarray(n_idx, np.int64)
    n_rows = N if idx is None else idx.size
    dw = np.empty((n_rows, K), np.float32)
    lib().orc_matmul_wgrad(_p(dy), _p(xh), M, N, K, _p(idx), n_rows, _p(dw))
    return dw


# ---- the quantization-aware layer (Eq. fakequant) and its STE backward (Eq. ste) ---------------

def fq_linear_fwd(x, w, wq_fmt: int, aq_fmt: int, w_tscale=None, a_tscale=None, mxfp4_noclip=False) -> np.ndarray:
    """Y = QDQ_a(X) . QDQ_w(W)^T with X [M,K], W [N,K]; returns float32 [M,N]."""
    return matmul_fwd(qdq_out(aq_fmt, x, a_tscale, mxfp4_noclip), qdq_out(wq_fmt, w, w_tscale, mxfp4_noclip))


def fq_linear_bwd(dy, x, w, wq_fmt: int, aq_fmt: int, w_tscale=None, a_tscale=None, n_idx=None,
                  mxfp4_noclip=False):
    """(dX, dW): dX = dY . QDQ_w(W), dW = dY^T . QDQ_a(X). The quantizers are treated as the
    identity in the backward pass; dY itself is never quantized."""
    dx = matmul_dgrad(dy, qdq_out(wq_fmt, w, w_tscale, mxfp4_noclip))
    dw = matmul_wgrad(dy, qdq_out(aq_fmt, x, a_tscale, mxfp4_noclip), n_idx)
    return dx, dw


# ---- engine-native packing (the export / weight-synchronisation step) -------------------------------

def pack_gguf_q4k(codes: np.ndarray, scales: np.ndarray) -> np.ndarray:
    """144-byte llama.cpp Q4_K records from the quantizer's outputs: for each super-block the 16
    metadata bytes {fp16 d, fp16 dmin, 12 packed 6-bit bytes} followed by its 128 code bytes.
    codes [rows, cols/2] uint8, scales [rows, cols/256, 16] uint8 -> [rows, cols/256, 144] uint8."""
    rows, nsb, _ = scales.shape
    rec = np.empty((rows, nsb, 144), np.uint8)
    for r in range(rows):
        for s in range(nsb):
            rec[r, s, :16] = scales[r, s]
            rec[r, s, 16:] = codes[r, s * 128:(s + 1) * 128]
    return rec


def swizzle_block_scales(scales: np.ndarray) -> np.ndarray:
    """FP4 block scales [rows, nblk] in the tiled layout block-scaled tensor-core GEMMs read: padded
    with zeros to multiples of 128 rows and 4 scale columns; tiles stored row-major, 512 bytes each;
    inside a tile, byte (r, c) sits at (r mod 32)*16 + (r div 32)*4 + c. Written element by element."""
    rows, nblk = scales.shape
    row_tiles, col_tiles = -(-rows // 128), -(-nblk // 4)
    out = np.zeros(row_tiles * col_tiles * 512, np.uint8)
    for r in range(rows):
        for c in range(nblk):
            tile = (r // 128) * col_tiles + c // 4
            ri = r % 128
            out[tile * 512 + (ri % 32) * 16 + (ri // 32) * 4 + c % 4] = scales[r, c]
    return out


# ---- LoRA merge ahead of the quantizer (Eq. qad-lora) -----------------------------------------------

def lora_merge(w, b, a, scale: float = 1.0) -> np.ndarray:
    """bf16(W + scale * B A): FP32 accumulation over the rank in order, one fused multiply-add per step."""
    w, b, a = _bf16_arr(w), _bf16_arr(b), _bf16_arr(a)
    rows, cols = w.shape
    rank = a.shape[0]
    assert b.shape == (rows, rank) and a.shape == (rank, cols)
    out = np.empty_like(w)
    lib().orc_lora_merge(_p(w), _p(b), _p(a), rows, cols, rank, float(scale), _p(out))
    return out


def qdq_lora(fmt: int, w, b, a, scale: float = 1.0, tensor_scale: float | None = None):
    """Q^-1(Q(W + scale * B A)): the quantizer applied to the merged weight."""
    return qdq(fmt, lora_merge(w, b, a, scale), tensor_scale)
