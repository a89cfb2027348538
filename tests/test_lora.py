"""LoRA merge ahead of the quantizer (Eq. qad-lora): W_hat = Q^-1(Q(W + s B A)). Oracle pins on CPU;
the CUDA path (merge fused into the quantizer kernels, merged tensor never materialised) bit-exact on GPU."""
import numpy as np
import pytest
import torch

import oracle
from oracle import FMT_MXFP4, FMT_NVFP4, FMT_Q4_K
from paper_2609_39223_b200 import api, synth
from util import bits_to_f32, f32_to_bits, torch_to_bits


def _case(rows, cols, rank, seed):
    rng = np.random.default_rng(seed)
    w = f32_to_bits(rng.normal(0, 0.02, (rows, cols)))
    b = f32_to_bits(rng.normal(0, 0.05, (rows, rank)))
    a = f32_to_bits(rng.normal(0, 0.05, (rank, cols)))
    return w, b, a


def test_oracle_merge_is_w_plus_scaled_ba_rounded_to_bf16():
    w, b, a = _case(24, 64, 8, 0)
    m = bits_to_f32(oracle.lora_merge(w, b, a, 2.0)).astype(np.float64)
    exact = bits_to_f32(w).astype(np.float64) + 2.0 * bits_to_f32(b).astype(np.float64) @ bits_to_f32(a).astype(np.float64)
    ulp = np.exp2(np.floor(np.log2(np.maximum(np.abs(exact), 2.0 ** -126))) - 7)
    # one BF16 rounding of an FP32 accumulation: half a BF16 ulp plus the (tiny) FP32 accumulation error
    assert np.all(np.abs(m - exact) <= 0.5 * ulp + 8 * np.abs(exact) * 2.0 ** -23 + 1e-12)
    np.testing.assert_array_equal(oracle.lora_merge(w, b[:, :0], a[:0], 1.0), w)                  # rank 0: nothing to merge
    np.testing.assert_array_equal(oracle.lora_merge(w, np.zeros_like(b), a, 1.0), w)              # B = 0: same
    # small integers: every product and sum is exact, so the merge equals the integer arithmetic
    wi = f32_to_bits(np.arange(12, dtype=np.float32).reshape(3, 4)); bi = f32_to_bits(np.array([[1, 2], [0, 1], [3, 0]], np.float32))
    ai = f32_to_bits(np.array([[1, 0, 2, 1], [0, 1, 1, 3]], np.float32))
    want = np.arange(12).reshape(3, 4) + np.array([[1, 2], [0, 1], [3, 0]]) @ np.array([[1, 0, 2, 1], [0, 1, 1, 3]])
    np.testing.assert_array_equal(bits_to_f32(oracle.lora_merge(wi, bi, ai, 1.0)), want.astype(np.float32))


def test_oracle_quantizes_the_merged_weight_not_the_base():
    w, b, a = _case(8, 256, 4, 1)
    r = oracle.qdq_lora(FMT_MXFP4, w, b, a, 4.0)
    np.testing.assert_array_equal(r["out"], oracle.qdq(FMT_MXFP4, oracle.lora_merge(w, b, a, 4.0))["out"])
    assert np.any(r["out"] != oracle.qdq(FMT_MXFP4, w)["out"])


@pytest.mark.gpu
@pytest.mark.parametrize("fmt", [api.FMT_NVFP4, api.FMT_MXFP4, api.FMT_Q4_K])
def test_gpu_fused_merge_on_wide_range_bit_patterns(fmt):
    """Base weight and factors drawn as raw BF16 bit patterns over forty binades, signs and zeros mixed in:
    the merge's FP32 accumulation order and its single BF16 rounding must agree bit for bit whatever cancels."""
    rng = np.random.default_rng(123)
    rows, cols, rank = 96, 1024, 12
    def pat(shape, lo, hi):
        n = int(np.prod(shape))
        bits = (rng.integers(0, 2, n) << 15) | (rng.integers(lo, hi, n) << 7) | rng.integers(0, 128, n)
        bits[rng.random(n) < 0.05] &= 0x8000
        return bits.astype(np.uint16).reshape(shape)
    w, b, a = pat((rows, cols), 100, 140), pat((rows, rank), 110, 130), pat((rank, cols), 110, 130)
    to_t = lambda x: torch.from_numpy(x.view(np.int16).copy()).view(torch.bfloat16).cuda()
    for scale in (1.0, -0.37, 1024.0):
        g = api.qf_qdq_lora(fmt, to_t(w), to_t(b), to_t(a), scale)
        o = oracle.qdq_lora(fmt, w, b, a, scale)
        np.testing.assert_array_equal(torch_to_bits(g["out"]), o["out"])
        np.testing.assert_array_equal(g["codes"].cpu().numpy(), o["codes"])
        np.testing.assert_array_equal(g["scales"].cpu().numpy(), o["scales"])


@pytest.mark.gpu
@pytest.mark.parametrize("fmt", [api.FMT_NVFP4, api.FMT_MXFP4, api.FMT_Q4_K])
@pytest.mark.parametrize("rows,cols,rank,scale", [(1, 256, 1, 1.0), (37, 768, 16, 2.0), (300, 1024, 64, 0.5), (64, 512, 0, 1.0)])
def test_gpu_fused_merge_and_quantize_is_bit_exact(fmt, rows, cols, rank, scale):
    w, b, a = _case(rows, cols, max(rank, 1), rows + rank)
    b, a = b[:, :rank].copy(), a[:rank].copy()
    to_t = lambda x, shape: torch.from_numpy(x.view(np.int16).copy()).view(torch.bfloat16).reshape(shape).cuda()
    g = api.qf_qdq_lora(fmt, to_t(w, (rows, cols)), to_t(b, (rows, rank)), to_t(a, (rank, cols)), scale)
    o = oracle.qdq_lora(fmt, w, b, a, scale)
    np.testing.assert_array_equal(torch_to_bits(g["out"]), o["out"])
    np.testing.assert_array_equal(g["codes"].cpu().numpy(), o["codes"])
    np.testing.assert_array_equal(g["scales"].cpu().numpy(), o["scales"])
    if fmt == api.FMT_NVFP4:
        assert np.float32(g["tensor_scale"].item()) == np.float32(o["tensor_scale"])


@pytest.mark.gpu
def test_gpu_lora_layer_forward_through_the_unquantized_weight_slot():
    """The LoRA-QAD student forward: quantize the merged weight, then run the layer on it."""
    M, N, K, rank = 256, 264, 512, 8
    w, b, a = _case(N, K, rank, 5)
    x = synth.randn_bf16((M, K), 1.0, 6)
    to_t = lambda arr, shape: torch.from_numpy(arr.view(np.int16).copy()).view(torch.bfloat16).reshape(shape).cuda()
    w_hat = api.qf_qdq_lora(api.FMT_MXFP4, to_t(w, (N, K)), to_t(b, (N, rank)), to_t(a, (rank, K)), 2.0)["out"]
    y = api.qf_fq_linear_fwd(x.cuda(), w_hat, api.FMT_NONE, api.FMT_MXFP4, y_dtype=torch.float32)
    ref = oracle.matmul_fwd(oracle.qdq(FMT_MXFP4, torch_to_bits(x))["out"], oracle.qdq_lora(FMT_MXFP4, w, b, a, 2.0)["out"])
    err = np.abs(y.cpu().numpy() - ref).max()
    assert err <= 1e-2 * np.sqrt(np.mean(ref.astype(np.float64) ** 2))
