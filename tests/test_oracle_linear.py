"""Pins for the oracle's quantization-aware layer (Eq. fakequant) and STE backward (Eq. ste,
Eq. activation-ste): reduction to a library matmul when nothing is quantized, one-hot inputs that
tie the matmul to the already-pinned quantizers, and the adjoint identity that ties the backward
to the forward. Finite differences are useless through a quantizer and are not used."""
import numpy as np
import pytest
import torch

import oracle
from oracle import FMT_MXFP4, FMT_NONE, FMT_NVFP4, FMT_Q4_K
from util import bits_to_f32, f32_to_bits


def _case(M, N, K, seed):
    rng = np.random.default_rng(seed)
    x = f32_to_bits(rng.normal(0, 1, (M, K)))
    w = f32_to_bits(rng.normal(0, 0.02, (N, K)))
    dy = f32_to_bits(rng.normal(0, 1e-3, (M, N)))
    return x, w, dy


def test_unquantized_layer_is_a_textbook_matmul():
    x, w, dy = _case(24, 40, 96, 0)
    X, W, DY = (torch.from_numpy(bits_to_f32(a)).double() for a in (x, w, dy))
    y = oracle.fq_linear_fwd(x, w, FMT_NONE, FMT_NONE)
    dx, dw = oracle.fq_linear_bwd(dy, x, w, FMT_NONE, FMT_NONE)
    np.testing.assert_array_equal(y, (X @ W.T).float().numpy())
    np.testing.assert_array_equal(dx, (DY @ W).float().numpy())
    np.testing.assert_array_equal(dw, (DY.T @ X).float().numpy())


@pytest.mark.parametrize("fmt,K", [(FMT_NVFP4, 64), (FMT_MXFP4, 64), (FMT_Q4_K, 256)])
def test_one_hot_activations_read_out_the_quantized_weight(fmt, K):
    # rows of the identity are on every format's grid, so Y = W_hat^T restricted to those rows
    _, w, _ = _case(1, 16, K, 1)
    eye = f32_to_bits(np.eye(K, dtype=np.float32))
    aq = FMT_NONE if fmt == FMT_Q4_K else fmt
    y = oracle.fq_linear_fwd(eye, w, fmt, aq)
    w_hat = bits_to_f32(oracle.qdq(fmt, w)["out"])
    np.testing.assert_array_equal(y, w_hat.T)


@pytest.mark.parametrize("wq,aq,K", [(FMT_MXFP4, FMT_MXFP4, 128), (FMT_NVFP4, FMT_NONE, 64), (FMT_Q4_K, FMT_NONE, 256),
                                     (FMT_NVFP4, FMT_NVFP4, 64)])
def test_backward_is_the_adjoint_of_the_forward(wq, aq, K):
    M, N = 12, 20
    x, w, dy = _case(M, N, K, 2)
    DY = bits_to_f32(dy).astype(np.float64)
    dx, dw = oracle.fq_linear_bwd(dy, x, w, wq, aq)
    rng = np.random.default_rng(3)
    # <dY, U W_hat^T> = <dX, U> for any U; take U already on the BF16 grid and skip its quantizer
    u = f32_to_bits(rng.normal(0, 1, (M, K)))
    w_hat = oracle.qdq_out(wq, w)
    lhs = np.sum(DY * oracle.matmul_fwd(u, w_hat).astype(np.float64))
    rhs = np.sum(dx.astype(np.float64) * bits_to_f32(u))
    assert abs(lhs - rhs) <= 1e-5 * max(abs(lhs), 1e-12)
    # <dY, X_hat V^T> = <dW, V>
    v = f32_to_bits(rng.normal(0, 0.02, (N, K)))
    x_hat = oracle.qdq_out(aq, x)
    lhs = np.sum(DY * oracle.matmul_fwd(x_hat, v).astype(np.float64))
    rhs = np.sum(dw.astype(np.float64) * bits_to_f32(v))
    assert abs(lhs - rhs) <= 1e-5 * max(abs(lhs), 1e-12)


def test_wgrad_row_subset_equals_full():
    x, w, dy = _case(16, 24, 64, 4)
    full = oracle.matmul_wgrad(dy, x)
    idx = np.array([3, 0, 23, 7])
    np.testing.assert_array_equal(oracle.matmul_wgrad(dy, x, idx), full[idx])


def test_forward_uses_quantized_not_latent_operands():
    x, w, _ = _case(8, 8, 64, 5)
    y_q = oracle.fq_linear_fwd(x, w, FMT_MXFP4, FMT_MXFP4)
    y_manual = oracle.matmul_fwd(oracle.qdq(FMT_MXFP4, x)["out"], oracle.qdq(FMT_MXFP4, w)["out"])
    np.testing.assert_array_equal(y_q, y_manual)
    assert np.abs(y_q - oracle.fq_linear_fwd(x, w, FMT_NONE, FMT_NONE)).max() > 0
