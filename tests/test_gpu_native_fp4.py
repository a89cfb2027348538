"""The equivalence the fake-quantized layer rests on, checked on the hardware that has FP4 tensor
cores: the BF16 matmul of dequantized operands (the training path, Eq. fakequant) against the
block-scaled FP4 tensor-core product taken directly on the emitted codes and scales (the deployment
path). References are FP64 products of the dequantization equations applied to the oracle's codes
and scales."""
import ml_dtypes
import numpy as np
import pytest
import torch

import oracle
from paper_2609_39223_b200 import api, synth
from util import E2M1_VALUES, torch_to_bits, unpack_nibbles

pytestmark = pytest.mark.gpu
SHAPES = [(128, 128, 256), (200, 264, 768), (333, 520, 1024), (1, 8, 32), (130, 136, 288), (256, 256, 4096)]


def _case(M, N, K):
    """Operands whose blocks differ in magnitude by up to 2^6 (so a misplaced block scale shows), plus
    a few outlier channels as in the layer tests."""
    c = synth.linear_case(M, N, K, seed=M + K, outlier_channels=4)
    g = torch.Generator().manual_seed(K)
    sx = torch.exp2(torch.randint(-3, 4, (M, K // 32), generator=g).float()).repeat_interleave(32, 1)
    sw = torch.exp2(torch.randint(-3, 4, (N, K // 32), generator=g).float()).repeat_interleave(32, 1)
    return (c.X.float() * sx).bfloat16(), (c.W.float() * sw).bfloat16()


def _dequant_exact(fmt, r):
    """Eq. mxfp4-dequant / the block level of Eq. nvfp4-dequant in FP64, with no rounding."""
    v = E2M1_VALUES[unpack_nibbles(r["codes"])]
    if fmt == api.FMT_MXFP4:
        return v * np.exp2(r["scales"].astype(np.float64) - 127).repeat(32, axis=1)
    return v * r["scales"].view(ml_dtypes.float8_e4m3fn).astype(np.float64).repeat(16, axis=1)


def _rms(a):
    return float(np.sqrt(np.mean(np.square(a))))


@pytest.mark.parametrize("noclip", [False, True])
@pytest.mark.parametrize("M,N,K", SHAPES)
def test_mxfp4_native_product_equals_the_fake_quantized_matmul(M, N, K, noclip):
    X, W = _case(M, N, K)
    xb, wb = torch_to_bits(X), torch_to_bits(W)
    f = api.MXFP4_NO_CLIP if noclip else 0
    gx, gw = api.qf_qdq(api.FMT_MXFP4, X.cuda(), flags=f), api.qf_qdq(api.FMT_MXFP4, W.cuda(), flags=f)
    ws = api.workspace(api.OP_QDQ, M, 0, K)
    y_native = api.qf_fp4_matmul_native(api.FMT_MXFP4, gx, gw, K, ws=ws).double().cpu().numpy()
    assert api.qf_read_status(ws) == 0
    y_fake = api.qf_fq_linear_fwd(X.cuda(), W.cuda(), api.FMT_MXFP4, api.FMT_MXFP4, y_dtype=torch.float32, flags=f).double().cpu().numpy()
    ox, ow = oracle.qdq(api.FMT_MXFP4, xb, mxfp4_noclip=noclip), oracle.qdq(api.FMT_MXFP4, wb, mxfp4_noclip=noclip)
    ref = _dequant_exact(api.FMT_MXFP4, ox) @ _dequant_exact(api.FMT_MXFP4, ow).T
    # the same sum the oracle's layer computes (its BF16 operands hold 2^p * C exactly)
    np.testing.assert_array_equal(ref.astype(np.float32), oracle.fq_linear_fwd(xb, wb, api.FMT_MXFP4, api.FMT_MXFP4, mxfp4_noclip=noclip))
    tol = 1e-5 * _rms(ref)                    # FP32 accumulation of exact products on both sides
    assert np.abs(y_native - ref).max() <= tol
    assert np.abs(y_fake - ref).max() <= tol
    assert np.abs(y_native - y_fake).max() <= tol


@pytest.mark.parametrize("M,N,K", SHAPES)
def test_nvfp4_native_product_differs_from_the_fake_quantized_matmul_only_by_bf16_rounding(M, N, K):
    X, W = _case(M, N, K)
    xb, wb = torch_to_bits(X), torch_to_bits(W)
    gx, gw = api.qf_qdq(api.FMT_NVFP4, X.cuda()), api.qf_qdq(api.FMT_NVFP4, W.cuda())
    ws = api.workspace(api.OP_QDQ, M, 0, K)
    y_native = api.qf_fp4_matmul_native(api.FMT_NVFP4, gx, gw, K, ws=ws).double().cpu().numpy()
    assert api.qf_read_status(ws) == 0
    ox, ow = oracle.qdq(api.FMT_NVFP4, xb), oracle.qdq(api.FMT_NVFP4, wb)
    ex, ew = _dequant_exact(api.FMT_NVFP4, ox), _dequant_exact(api.FMT_NVFP4, ow)
    ts = float(ox["tensor_scale"]) * float(ow["tensor_scale"])
    ref = (ex @ ew.T) * ts
    assert np.abs(y_native - ref).max() <= 1e-4 * _rms(ref)
    # The training path rounds every dequantized value to BF16 (8 significant bits: relative error <= 2^-8 per
    # operand), the native product does not: term by term the two differ by at most (2^-7 + 2^-16) |term|.
    y_fake = api.qf_fq_linear_fwd(X.cuda(), W.cuda(), api.FMT_NVFP4, api.FMT_NVFP4, y_dtype=torch.float32).double().cpu().numpy()
    bound = (np.abs(ex) @ np.abs(ew).T) * ts * (2.0 ** -7 + 2.0 ** -16) + 1e-4 * _rms(ref)
    assert np.all(np.abs(y_fake - y_native) <= bound)
    assert np.abs(y_fake - y_native).max() > 0 or K <= 32


@pytest.mark.parametrize("fmt", [api.FMT_MXFP4, api.FMT_NVFP4])
@pytest.mark.parametrize("M,N,K", [(200, 264, 768), (130, 136, 288), (1, 8, 32), (256, 256, 1024)])
def test_tensor_cores_read_the_tiled_scale_layout_as_packed(fmt, M, N, K):
    """The tiled block-scale layout written by qf_pack goes to the tensor cores tile by tile, unchanged:
    the product must be the one obtained from the row-major scales, bit for bit. This is the hardware's
    reading of the layout, not a formula of ours."""
    X, W = _case(M, N, K)
    gx, gw = api.qf_qdq(fmt, X.cuda()), api.qf_qdq(fmt, W.cuda())
    y_rows = api.qf_fp4_matmul_native(fmt, gx, gw, K)
    tx = dict(gx, scales=api.qf_pack(api.LAYOUT_FP4_SWIZZLED_SCALES, fmt, None, gx["scales"], M, K))
    tw = dict(gw, scales=api.qf_pack(api.LAYOUT_FP4_SWIZZLED_SCALES, fmt, None, gw["scales"], N, K))
    ws = api.workspace(api.OP_QDQ, M, 0, K)
    y_tiled = api.qf_fp4_matmul_native(fmt, tx, tw, K, flags=api.SCALES_TILED, ws=ws)
    assert api.qf_read_status(ws) == 0
    assert torch.equal(y_rows, y_tiled)


def test_native_product_argument_checks_and_empty_shapes():
    X, W = _case(128, 128, 256)
    gx, gw = api.qf_qdq(api.FMT_MXFP4, X.cuda()), api.qf_qdq(api.FMT_MXFP4, W.cuda())
    with pytest.raises(api.QfError) as e:
        api.qf_fp4_matmul_native(api.FMT_Q4_K, gx, gw, 256)
    assert e.value.code == 4
    with pytest.raises(api.QfError) as e:
        api.qf_fp4_matmul_native(api.FMT_MXFP4, gx, gw, 48)
    assert e.value.code == 2
    y0 = api.qf_fp4_matmul_native(api.FMT_MXFP4, gx, gw, 0)                    # empty contraction: zeros
    assert y0.shape == (128, 128) and not y0.any()
    empty = {"codes": torch.empty((0, 128), dtype=torch.uint8, device="cuda"), "scales": torch.empty((0, 8), dtype=torch.uint8, device="cuda")}
    assert api.qf_fp4_matmul_native(api.FMT_MXFP4, empty, gw, 256).shape == (0, 128)
