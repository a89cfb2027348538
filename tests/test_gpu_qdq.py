"""GPU parity: the CUDA quantize-dequantize kernels against the CPU oracle, bit for bit, through
the C ABI. Codes, scales, tensor scale and dequantized BF16 values must all be identical."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_39223_b200 import api, synth
from util import bits_to_f32, bits_to_torch, f32_to_bits, torch_to_bits

pytestmark = pytest.mark.gpu
FMTS = [(api.FMT_NVFP4, "nvfp4"), (api.FMT_MXFP4, "mxfp4"), (api.FMT_Q4_K, "q4_k")]


def _compare(fmt, xbits, tensor_scale=None, noclip=False):
    x = bits_to_torch(xbits, "cuda")
    ts = None if tensor_scale is None else torch.tensor([tensor_scale], dtype=torch.float32, device="cuda")
    g = api.qf_qdq(fmt, x, tensor_scale=ts, flags=api.MXFP4_NO_CLIP if noclip else 0)
    torch.cuda.synchronize()
    o = oracle.qdq(fmt, xbits, tensor_scale, mxfp4_noclip=noclip)
    np.testing.assert_array_equal(torch_to_bits(g["out"]), o["out"])
    np.testing.assert_array_equal(g["codes"].cpu().numpy(), o["codes"])
    np.testing.assert_array_equal(g["scales"].cpu().numpy(), o["scales"])
    if fmt == api.FMT_NVFP4:
        assert np.float32(g["tensor_scale"].item()).tobytes() == np.float32(o["tensor_scale"]).tobytes()
    # the inverse half alone reproduces the same tensor from the emitted codes and metadata
    d = api.qf_dequant(fmt, g["codes"], g["scales"], g["tensor_scale"], *xbits.shape)
    np.testing.assert_array_equal(torch_to_bits(d), o["out"])
    return g, o


def test_hardware_conversions_match_oracle_encoders():
    rng = np.random.default_rng(0)
    mids = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 6.0, 0.5, 1, 1.5, 2, 3, 4], np.float32)
    e4 = np.array([oracle.e4m3_value(c) for c in range(0x7F)], np.float32)
    e4mid = (e4[:-1] + e4[1:]) / 2
    v = np.concatenate([rng.uniform(-8, 8, 200000), rng.normal(0, 1, 100000), np.exp(rng.uniform(np.log(1e-5), np.log(600), 100000)),
                        mids, e4, e4mid, np.array([0.0, 1e-30, 1e9, 448, 449, 464, 465, 480, 2.0 ** -10, 2.0 ** -9])]).astype(np.float32)
    v = np.concatenate([v, -v, np.nextafter(v, np.float32(np.inf)), np.nextafter(v, np.float32(-np.inf))])
    e2m1, e4m3 = api.qf_selftest_cvt(torch.from_numpy(v).cuda())
    want2 = np.array([oracle.e2m1_encode(x) for x in v], np.uint8)
    want4 = np.array([oracle.e4m3_encode(abs(x)) for x in v], np.uint8)
    np.testing.assert_array_equal(e2m1.cpu().numpy(), want2)
    np.testing.assert_array_equal(e4m3.cpu().numpy(), want4)


def test_reciprocal_based_division_is_the_ieee_quotient():
    """The NVFP4 / Q4_K kernels divide through one exactly rounded reciprocal per block plus two fused
    residual corrections; that must give the IEEE quotient bit for bit wherever it is used."""
    rng = np.random.default_rng(11)
    all_bf16 = (np.arange(0, 0x7F80, dtype=np.uint32) << 16).view(np.float32)          # every finite non-negative BF16
    sb = np.array([oracle.e4m3_value(c) for c in range(1, 0x7F)], np.float32)
    s_t = np.concatenate([np.float32(2.0) ** np.arange(-40, 20, 7), rng.uniform(1e-7, 1e-2, 24).astype(np.float32)])
    ys = (s_t[:, None] * sb[None, :]).astype(np.float32).ravel()                       # NVFP4 divisors S = s_t * s_b
    ys = ys[(ys >= 2.0 ** -60) & (ys <= 2.0 ** 60)]
    xs = np.concatenate([all_bf16, rng.normal(0, 1, 20000).astype(np.float32)])        # plus FP32 numerators as in Q4_K
    assert api.qf_selftest_div(torch.from_numpy(xs).cuda(), torch.from_numpy(ys).cuda()) == 0
    ys2 = np.exp(rng.uniform(np.log(1e-9), np.log(1e3), 4000)).astype(np.float32)      # Q4_K style divisors
    ys2 = np.concatenate([ys2, np.array([15.0, 63.0], np.float32)])
    xs2 = np.concatenate([rng.normal(0, 1, 60000) * np.exp(rng.uniform(-12, 8, 60000)), np.arange(0, 16.5, 0.5)]).astype(np.float32)
    assert api.qf_selftest_div(torch.from_numpy(xs2).cuda(), torch.from_numpy(ys2).cuda()) == 0


@pytest.mark.parametrize("fmt,name", FMTS)
@pytest.mark.parametrize("shape", [(1, 256), (3, 512), (37, 768), (129, 2304), (5, 8192)])
def test_random_weights_small_and_ragged(fmt, name, shape):
    w = synth.weight_with_outliers(*shape, seed=shape[0])
    _compare(fmt, torch_to_bits(w))


@pytest.mark.parametrize("fmt,name", FMTS)
def test_wide_dynamic_range_blocks(fmt, name):
    rng = np.random.default_rng(5)
    rows, cols = 64, 1024
    x = rng.normal(0, 1, (rows, cols)) * np.exp2(rng.integers(-30, 30, (rows, cols // 16))).repeat(16, axis=1)
    x[rng.random((rows, cols)) < 0.05] = 0.0
    x[:, 256:512] = 0.0                                   # whole zero blocks / super-blocks
    x[3, 512:544] = -0.0
    _compare(fmt, f32_to_bits(x))


def _random_bit_patterns(rng, rows, cols, group, top=220):
    """Raw BF16 bit patterns: every `group` elements share an exponent centre drawn from the whole range in use
    (biased exponent 0 = subnormals up to 220 = 2^93; beyond that differences of two values can overflow FP32,
    which the formats' arithmetic is not defined for), individual exponents scatter around it by a per-group
    spread of 0 to 40 binades, mantissas and signs are uniform, and a tenth of the groups get zeros mixed in."""
    ng = rows * cols // group
    centre = rng.integers(0, top + 1, ng)
    spread = rng.choice([0, 1, 3, 8, 20, 40], ng)
    e = centre[:, None] + np.rint(rng.normal(0, 1, (ng, group)) * spread[:, None]).astype(np.int64)
    e = np.clip(e, 0, top)
    bits = (rng.integers(0, 2, (ng, group)) << 15) | (e << 7) | rng.integers(0, 128, (ng, group))
    zero = (rng.random((ng, 1)) < 0.1) & (rng.random((ng, group)) < 0.5)
    bits[zero] &= 0x8000                                   # +0 and -0
    return bits.astype(np.uint16).reshape(rows, cols)


@pytest.mark.parametrize("fmt,name", FMTS)
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_random_bit_patterns_over_the_whole_exponent_range(fmt, name, seed):
    rng = np.random.default_rng(1000 + seed)
    group = [16, 32, 256, 4096][seed % 4] if fmt != api.FMT_Q4_K else [32, 256, 2048][seed % 3]
    x = _random_bit_patterns(rng, 128, 4096, group)
    _compare(fmt, x)
    if fmt == api.FMT_NVFP4:
        for ts in (2.0 ** -40, 3.7e-9, 1.0, 2.0 ** 20):
            _compare(fmt, x, tensor_scale=ts)
    if fmt == api.FMT_MXFP4:
        _compare(fmt, x, noclip=True)
    if fmt != api.FMT_Q4_K:
        # the two FP4 formats never subtract two inputs, so every finite BF16 value is fair game
        _compare(fmt, _random_bit_patterns(rng, 64, 4096, group, top=254))


@pytest.mark.parametrize("fmt,name", FMTS)
def test_dequantizer_alone_on_arbitrary_codes_and_metadata(fmt, name):
    """Q^-1 on its own (the path a checkpoint reader takes): every code byte, every valid scale byte, arbitrary
    finite FP16 super-block factors and 6-bit fields, not only combinations the quantizer would emit."""
    rng = np.random.default_rng(31)
    rows, cols = 64, 2048
    codes = rng.integers(0, 256, (rows, cols // 2), dtype=np.uint8)
    if fmt == api.FMT_NVFP4:
        scales = rng.integers(0, 0x7F, (rows, cols // 16), dtype=np.uint8)           # E4M3 codes 0x00..0x7E
    elif fmt == api.FMT_MXFP4:
        scales = rng.integers(0, 255, (rows, cols // 32), dtype=np.uint8)            # E8M0 codes 0..254
    else:
        scales = rng.integers(0, 256, (rows, cols // 256, 16), dtype=np.uint8)
        half = rng.integers(0, 0x7C00, (rows, cols // 256, 2)).astype(np.uint16)     # finite non-negative FP16 d, dmin
        scales[..., 0:4] = half.view(np.uint8).reshape(rows, cols // 256, 4)
    for ts in ((3.1e-5, 1.0, 2.0 ** 30) if fmt == api.FMT_NVFP4 else (None,)):
        t = None if ts is None else torch.tensor([ts], dtype=torch.float32, device="cuda")
        d = api.qf_dequant(fmt, torch.from_numpy(codes).cuda(), torch.from_numpy(scales).cuda(), t, rows, cols)
        np.testing.assert_array_equal(torch_to_bits(d), oracle.dequant(fmt, codes, scales, ts, rows, cols))


def test_amax_over_odd_lengths_and_negative_maxima():
    """max|x| over tensors whose length is not a multiple of the 8-element load width, with the maximum placed in the
    ragged tail, at the front, and carried by a negative value; and over several tensors at once."""
    rng = np.random.default_rng(8)
    for n in (1, 7, 8, 9, 1023, 4097, 70001, 1 << 20 | 5):
        x = synth.randn_bf16((n,), 1.0, n, device="cuda")
        for pos, val in ((n - 1, -37.5), (0, 41.0), (int(rng.integers(0, n)), -53.0)):
            x[pos] = val
            assert api.qf_amax(x).item() == abs(val)
    parts = [synth.randn_bf16((m,), 1.0, 3 * m, device="cuda") for m in (5, 4096, 33, 100003)]
    parts[2][17] = -99.0
    state = torch.zeros(1, dtype=torch.float32, device="cuda")
    scale = api.qf_nvfp4_tensor_scale(parts, state)
    assert state.item() == 99.0 and np.float32(scale.item()) == np.float32(99.0) / np.float32(2688.0)


@pytest.mark.parametrize("shape", [(64, 512), (129, 2304), (1024, 8192)])
def test_nvfp4_speculative_tensor_scale_hit_and_miss(shape):
    """QF_TENSOR_SCALE_SPECULATIVE: whatever the guess, the outputs and the returned scale are those of deriving
    the scale from the tensor; a wrong guess is corrected by the second pass, a right one leaves the first pass's
    results in place (the output buffers are poisoned before each call to prove who wrote them)."""
    xb = torch_to_bits(synth.weight_with_outliers(*shape, seed=shape[0]))
    x = bits_to_torch(xb, "cuda")
    o = oracle.qdq(api.FMT_NVFP4, xb)
    out = torch.empty_like(x); codes = torch.empty((shape[0], shape[1] // 2), dtype=torch.uint8, device="cuda")
    scales = torch.empty((shape[0], shape[1] // 16), dtype=torch.uint8, device="cuda")
    exact = float(o["tensor_scale"])
    for guess in (1.0, 0.0, -3.0, float("nan"), exact * 2, exact, exact):            # misses, then two hits in a row
        ts = torch.tensor([guess], dtype=torch.float32, device="cuda")
        out.fill_(-7.0); codes.fill_(0xEE); scales.fill_(0xEE)
        api.qf_qdq(api.FMT_NVFP4, x, tensor_scale=ts, out=out, codes=codes, scales=scales, flags=api.TENSOR_SCALE_SPECULATIVE)
        torch.cuda.synchronize()
        assert np.float32(ts.item()).tobytes() == np.float32(exact).tobytes()
        np.testing.assert_array_equal(torch_to_bits(out), o["out"])
        np.testing.assert_array_equal(codes.cpu().numpy(), o["codes"])
        np.testing.assert_array_equal(scales.cpu().numpy(), o["scales"])
    # in place (out = in) the guess is not used: the first pass would overwrite what the second needs
    ts = torch.tensor([exact * 2], dtype=torch.float32, device="cuda")
    xin = x.clone()
    api.qf_qdq(api.FMT_NVFP4, xin, tensor_scale=ts, out=xin, want_codes=False, want_scales=False, flags=api.TENSOR_SCALE_SPECULATIVE)
    np.testing.assert_array_equal(torch_to_bits(xin), o["out"])
    assert np.float32(ts.item()) == np.float32(exact)
    # an all-zero tensor derives the scale 1.0
    z = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
    ts = torch.tensor([1.0], dtype=torch.float32, device="cuda")
    r = api.qf_qdq(api.FMT_NVFP4, z, tensor_scale=ts, flags=api.TENSOR_SCALE_SPECULATIVE)
    assert ts.item() == 1.0 and not r["out"].any()


def test_nvfp4_exact_ties_and_given_scale():
    # with s_t = 2^-10 and a block maximum of 2.625 the block scale is 448 and S = 7/16, so these
    # inputs sit exactly on the rounding midpoints 0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5 (times S)
    ties = np.array([0.109375, 0.328125, 0.546875, 0.765625, 1.09375, 1.53125, 2.1875], np.float32)
    x = np.zeros((4, 64), np.float32)
    x[0, :7] = ties; x[0, 15] = 2.625
    x[1, :7] = -ties; x[1, 15] = -2.625
    x[2, 16:23] = ties; x[2, 31] = 2.625; x[2, 0] = 1e-6      # first block underflows to scale 0
    x[3, :] = 2.625
    g, o = _compare(api.FMT_NVFP4, f32_to_bits(x), tensor_scale=2.0 ** -10)
    assert list(bits_to_f32(o["out"])[0, :7] / 0.4375) == [0, 1, 1, 2, 2, 4, 4]
    _compare(api.FMT_NVFP4, f32_to_bits(x))               # derived scale: the same 2^-10
    _compare(api.FMT_NVFP4, f32_to_bits(x), tensor_scale=3.1e-4)   # a tied / running scale that clips blocks


def test_nvfp4_degenerate_tensors():
    _compare(api.FMT_NVFP4, np.zeros((2, 64), np.uint16))
    _compare(api.FMT_NVFP4, f32_to_bits(np.full((2, 64), 0.3125)))
    x = np.full((2, 64), 1e-4, np.float32); x[0, 0] = 3e4
    _compare(api.FMT_NVFP4, f32_to_bits(x))
    sub = np.full((2, 64), 2.0 ** -130, np.float32)       # BF16 subnormals everywhere
    _compare(api.FMT_NVFP4, f32_to_bits(sub))


def test_mxfp4_ties_clipping_subnormals_extremes():
    x = np.zeros((4, 128), np.float32)
    x[0, :8] = [7, 5, 2.5, 3.5, 0.25, 0.75, 1.25, 1.75]
    x[0, 32:40] = [-7, -5, -2.5, -3.5, -0.25, -0.75, -1.25, -1.75]
    x[0, 64:66] = [3.90625, 1]
    x[1, :32] = 2.0 ** -133
    x[1, 32:64] = np.linspace(1, 127, 32) * 2.0 ** -133
    x[1, 64] = 3.0e38; x[1, 65] = 1e30
    x[1, 96] = 2.0 ** -126; x[1, 97] = 1.5 * 2.0 ** -126
    x[2, :] = 0.02001953125
    x[3, 5] = -0.0
    _compare(api.FMT_MXFP4, f32_to_bits(x))


@pytest.mark.parametrize("noclip", [False, True])
def test_mxfp4_every_bf16_value_as_block_maximum(noclip):
    """Both scale rules, with each of the 32640 finite positive BF16 values in turn as a block's
    maximum (the rule is a function of that value alone); the other elements are fractions of it."""
    amax = np.arange(1, 0x7F80, dtype=np.uint16)
    rng = np.random.default_rng(41)
    frac = rng.uniform(-1, 1, (amax.size, 32)).astype(np.float32)
    frac[:, 7] = 1.0
    x = f32_to_bits(frac * bits_to_f32(amax)[:, None])
    x[:, 7] = amax                                                     # exact, whatever the product rounded to
    pad = (-amax.size) % 8
    x = np.concatenate([x, np.zeros((pad, 32), np.uint16)]).reshape(-1, 256)
    g, o = _compare(api.FMT_MXFP4, x, noclip=noclip)
    if noclip:
        p0 = oracle.qdq(api.FMT_MXFP4, x)["scales"].astype(int)
        assert set(np.unique(o["scales"].astype(int) - p0)) == {0, 1}


def test_mxfp4_noclip_random_ragged_and_worked_blocks():
    for shape, seed in [((37, 768), 5), ((129, 2304), 6), ((3, 64), 7)]:
        _compare(api.FMT_MXFP4, torch_to_bits(synth.randn_bf16(shape, 1.0, seed)), noclip=True)
    x = np.zeros((2, 128), np.float32)
    x[0, :8] = [7, 5, 2.5, 3.5, 0.25, 0.75, 1.25, 1.75]
    x[0, 32:35] = [6, 0.25, -1.75]
    x[0, 64:68] = [6.03125, -6.03125, 1, 0.5]
    x[1, :32] = 2.0 ** -133
    x[1, 64] = 2.9e38
    x[1, 96] = 6 * 2.0 ** -127
    g, o = _compare(api.FMT_MXFP4, f32_to_bits(x), noclip=True)
    assert list(bits_to_f32(torch_to_bits(g["out"]))[0, :8]) == [8, 4, 2, 4, 0, 1, 1, 2]
    # the flag leaves the other formats alone
    xb = torch_to_bits(synth.randn_bf16((16, 512), 0.05, 9))
    _compare(api.FMT_NVFP4, xb, noclip=True)
    _compare(api.FMT_Q4_K, xb, noclip=True)


def test_q4k_worked_and_degenerate():
    x = np.zeros((3, 512), np.float32)
    x[0, 0:32] = 0.5; x[0, 32:64] = -0.5
    for b in range(8):
        x[1, b * 32:(b + 1) * 32] = (b + 1) / 8 * (-1 + 0.125 * (np.arange(32) % 16))
    x[2, :256] = 0.75
    x[2, 256:] = -np.abs(np.random.default_rng(1).normal(0, 1, 256))
    g, o = _compare(api.FMT_Q4_K, f32_to_bits(x))
    tiny = np.full((1, 256), 2.0 ** -40, np.float32)      # d underflows FP16 -> everything collapses to -em
    _compare(api.FMT_Q4_K, f32_to_bits(tiny))


def test_q4k_large_tensor_with_a_ragged_last_tile():
    """Tensors of 2^25 elements and more take the Q4_K kernel that stages input and output through shared memory with
    bulk asynchronous copies, 256 sub-blocks per tile. 4099 x 8448 has 1082136 sub-blocks: a last tile of 24. All
    outputs, the codes-and-metadata-only form, and in place, bit for bit against the oracle."""
    rows, cols = 4099, 8448
    assert (rows * cols // 32) % 256 == 24 and rows * cols >= 2 ** 25
    xb = torch_to_bits(synth.weight_with_outliers(rows, cols, seed=41))
    g, o = _compare(api.FMT_Q4_K, xb)
    x = bits_to_torch(xb, "cuda")
    only = api.qf_qdq(api.FMT_Q4_K, x, want_out=False)
    assert only["out"] is None and torch.equal(only["codes"], g["codes"]) and torch.equal(only["scales"], g["scales"])
    inplace = api.qf_qdq(api.FMT_Q4_K, x, out=x)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(torch_to_bits(x), o["out"])
    assert torch.equal(inplace["codes"], g["codes"])


@pytest.mark.parametrize("fmt,name", FMTS)
def test_two_runs_are_bitwise_identical(fmt, name):
    x = synth.weight_with_outliers(256, 4096, seed=9, device="cuda")
    a = api.qf_qdq(fmt, x)
    b = api.qf_qdq(fmt, x)
    for k in ("out", "codes", "scales"):
        assert torch.equal(a[k], b[k])


@pytest.mark.parametrize("fmt,name", FMTS)
def test_in_place(fmt, name):
    """out = in: every thread has read all it needs of its blocks before it writes them."""
    xb = torch_to_bits(synth.weight_with_outliers(257, 2304 if fmt != api.FMT_Q4_K else 2048, seed=12))
    o = oracle.qdq(fmt, xb)
    x = bits_to_torch(xb, "cuda")
    g = api.qf_qdq(fmt, x, out=x)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(torch_to_bits(x), o["out"])
    np.testing.assert_array_equal(g["codes"].cpu().numpy(), o["codes"])
    np.testing.assert_array_equal(g["scales"].cpu().numpy(), o["scales"])


def test_optional_outputs_and_empty_tensor():
    x = synth.weight_with_outliers(16, 512, seed=2, device="cuda")
    full = api.qf_qdq(api.FMT_MXFP4, x)
    only_out = api.qf_qdq(api.FMT_MXFP4, x, want_codes=False, want_scales=False)
    only_codes = api.qf_qdq(api.FMT_MXFP4, x, want_out=False)
    assert only_out["codes"] is None and torch.equal(only_out["out"], full["out"])
    assert only_codes["out"] is None and torch.equal(only_codes["codes"], full["codes"])
    e = api.qf_qdq(api.FMT_NVFP4, torch.empty((0, 64), dtype=torch.bfloat16, device="cuda"))
    assert e["tensor_scale"].item() == 1.0
    assert api.qf_amax(x).item() == x.abs().max().item()


def test_full_size_nvfp4_weight_2048():
    w = synth.nvfp4_weight_2048()
    _compare(api.FMT_NVFP4, torch_to_bits(w))


@pytest.mark.parametrize("name", ["k_proj", "down_proj"])
def test_full_size_q4k_decoder_matrices(name):
    # one narrow and one wide matrix of the 32-layer dense decoder, complete and bit-exact
    w = synth.dense_decoder_weight(3, name)
    _compare(api.FMT_Q4_K, torch_to_bits(w))


@pytest.mark.parametrize("name", ["q_proj", "v_proj", "o_proj", "gate_proj", "up_proj"])
def test_full_size_q4k_decoder_matrices_row_slices(name):
    """The other five linear weights of a decoder layer at full size (per-layer seed): the GPU quantizes the whole
    matrix, the oracle the first, a middle and the last 48 rows (rows are independent in Q4_K)."""
    w = synth.dense_decoder_weight(17, name, device="cuda")
    g = api.qf_qdq(api.FMT_Q4_K, w)
    rows = w.shape[0]
    pick = np.concatenate([np.arange(48), rows // 2 + np.arange(48), rows - 48 + np.arange(48)])
    sel = torch.from_numpy(pick).cuda()
    o = oracle.qdq(api.FMT_Q4_K, torch_to_bits(w[sel]))
    np.testing.assert_array_equal(torch_to_bits(g["out"][sel]), o["out"])
    np.testing.assert_array_equal(g["codes"][sel].cpu().numpy(), o["codes"])
    np.testing.assert_array_equal(g["scales"][sel].cpu().numpy(), o["scales"])
    # nothing left unwritten: every row of the dequantized matrix is within one quantization step of its input
    err = (g["out"].float() - w.float()).abs_().amax(dim=1)
    assert float(err.max()) <= 0.02 * 6 / 15 and float(err.min()) > 0


def test_full_size_mxfp4_activation():
    x = synth.activations_with_outlier_channels(8192, 4096, seed=0)
    _compare(api.FMT_MXFP4, torch_to_bits(x))


@pytest.mark.parametrize("fmt,name", FMTS)
def test_more_than_2_to_the_31_elements(fmt, name):
    """A tensor whose element count does not fit in 32 bits (36864 x 65536 = 2.4e9): every index in the
    kernels must be 64-bit. Rows are independent given the tensor scale, so sampled rows from the start,
    the middle, the 2^31-element boundary and the end are compared with the oracle run on those rows alone."""
    rows, cols = 36864, 65536
    assert rows * cols > 2 ** 31
    x = synth.randn_bf16((rows, cols), 0.02, 17, device="cuda")
    x[rows - 1, cols - 1] = 3.0                                  # the tensor maximum sits in the very last element
    g = api.qf_qdq(fmt, x)
    torch.cuda.synchronize()
    ts = None
    if fmt == api.FMT_NVFP4:
        ts = float(g["tensor_scale"].item())
        assert np.float32(ts) == np.float32(3.0) / np.float32(2688.0)
    boundary = 2 ** 31 // cols
    sample = [0, 1, rows // 3, boundary - 1, boundary, boundary + 1, rows - 2, rows - 1]
    xb = torch_to_bits(x[sample].cpu())
    o = oracle.qdq(fmt, xb, ts)
    np.testing.assert_array_equal(torch_to_bits(g["out"][sample].cpu()), o["out"])
    np.testing.assert_array_equal(g["codes"][sample].cpu().numpy(), o["codes"])
    np.testing.assert_array_equal(g["scales"][sample].cpu().numpy(), o["scales"])
    # nothing was left unwritten anywhere: the dequantized tensor is within one grid step of the input in every row
    err = (g["out"].float() - x.float()).abs_().amax(dim=1)
    assert float(err.max()) <= 0.5 and float(err.min()) > 0
    del g, x


def _guarded(nbytes, dtype, shape):
    """A tensor carved out of the middle of a larger byte buffer whose margins are filled with a canary."""
    pad = 1 << 16
    raw = torch.full((nbytes + 2 * pad,), 0xA5, dtype=torch.uint8, device="cuda")
    view = raw[pad:pad + nbytes].view(dtype).view(shape)
    return raw, view, pad


@pytest.mark.parametrize("fmt,name", FMTS)
def test_large_ragged_tensor_stays_inside_its_buffers(fmt, name):
    """A tensor large enough that the capped grid loops several times with a ragged last iteration:
    outputs must be bit-exact and nothing may be written outside the output buffers."""
    rows, cols = 9001, 4352
    w = synth.randn_bf16((rows, cols), 0.02, 17, device="cuda")
    n = rows * cols
    raw_o, out, pad = _guarded(n * 2, torch.bfloat16, (rows, cols))
    raw_c, codes, _ = _guarded(n // 2, torch.uint8, (rows, cols // 2))
    sshape = api.scales_shape(fmt, rows, cols)
    raw_s, scales, _ = _guarded(int(np.prod(sshape)), torch.uint8, sshape)
    g = api.qf_qdq(fmt, w, out=out, codes=codes, scales=scales)          # NVFP4: derived scale (amax pass + reverse walk)
    torch.cuda.synchronize()
    for raw in (raw_o, raw_c, raw_s):
        assert bool((raw[:pad] == 0xA5).all()) and bool((raw[-pad:] == 0xA5).all())
    o = oracle.qdq(fmt, torch_to_bits(w))
    np.testing.assert_array_equal(torch_to_bits(out), o["out"])
    np.testing.assert_array_equal(codes.cpu().numpy(), o["codes"])
    np.testing.assert_array_equal(scales.cpu().numpy(), o["scales"])
    if fmt == api.FMT_NVFP4:
        out.zero_()
        api.qf_qdq(fmt, w, out=out, codes=codes, scales=scales, tensor_scale=g["tensor_scale"])   # forward walk
        torch.cuda.synchronize()
        for raw in (raw_o, raw_c, raw_s):
            assert bool((raw[:pad] == 0xA5).all()) and bool((raw[-pad:] == 0xA5).all())
        np.testing.assert_array_equal(torch_to_bits(out), o["out"])


def test_conversion_free_mxfp4_rounding_matches_the_conversion_route_exhaustively():
    assert api.qf_selftest_mxfp4_bf16() == 0


def test_tied_tensor_scale_over_fused_projections_and_running_activation_maximum():
    # one weight scale for q/k/v computed over their concatenation: each quantizes as a slice of the concatenation would
    q = synth.randn_bf16((64, 256), 0.02, 1); k = synth.randn_bf16((16, 256), 0.05, 2); v = synth.randn_bf16((16, 256), 0.01, 3)
    state = torch.zeros(1, device="cuda")
    scale = api.qf_nvfp4_tensor_scale([q.cuda(), k.cuda(), v.cuda()], state)
    cat = torch.cat([q, k, v])
    whole = oracle.qdq(api.FMT_NVFP4, torch_to_bits(cat))
    assert np.float32(scale.item()) == whole["tensor_scale"] and state.item() == cat.abs().max().item()
    parts = [api.qf_qdq(api.FMT_NVFP4, t.cuda(), tensor_scale=scale) for t in (q, k, v)]
    np.testing.assert_array_equal(np.concatenate([torch_to_bits(p["out"]) for p in parts]), whole["out"])
    np.testing.assert_array_equal(np.concatenate([p["codes"].cpu().numpy() for p in parts]), whole["codes"])
    # running maximum of an activation across steps
    state.zero_()
    seen = 0.0
    for step, std in enumerate((1.0, 3.0, 0.5)):
        x = synth.randn_bf16((128, 256), std, 10 + step, device="cuda")
        s = api.qf_nvfp4_tensor_scale([x], state, running=True)
        seen = max(seen, x.abs().max().item())
        assert state.item() == seen and np.float32(s.item()) == np.float32(seen) / np.float32(2688.0)
    zero = api.qf_nvfp4_tensor_scale([torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")], torch.zeros(1, device="cuda"))
    assert zero.item() == 1.0
    # the steps a row-sharded weight takes: maximum of each shard without a scale, the maxima combined (here by hand, across
    # ranks by a MAX all-reduce), and the combined state turned into the scale by a call that is given no tensor at all
    a_state, b_state = torch.zeros(1, device="cuda"), torch.zeros(1, device="cuda")
    assert api.qf_nvfp4_tensor_scale([cat[:40].cuda()], a_state, want_scale=False) is None
    api.qf_nvfp4_tensor_scale([cat[40:].cuda()], b_state, want_scale=False)
    combined = torch.maximum(a_state, b_state)
    shared = api.qf_nvfp4_tensor_scale([], combined, running=True)
    assert np.float32(shared.item()) == whole["tensor_scale"]
