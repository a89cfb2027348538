"""Property tests for the oracle's quantizers on inputs drawn by hypothesis: arbitrary finite BF16
bit patterns arranged in blocks, not only Gaussian data. Each property follows from the formats'
definitions (Eq. nvfp4-dequant, Eq. mxfp4-dequant, Eq. q4k-dequant and the value grid of
Eq. e2m1-values) and involves nothing but the oracle's outputs and plain arithmetic on them."""
import ml_dtypes
import numpy as np
from hypothesis import given, settings, strategies as st

import oracle
from oracle import FMT_MXFP4, FMT_NVFP4, FMT_Q4_K
from test_oracle_qdq import _q4k_codes, _q4k_meta
from util import E2M1_VALUES, bits_to_f32, unpack_nibbles

# exponent fields 40..200 keep every intermediate far from FP32 overflow and underflow
_bits = st.builds(lambda s, e, m: (s << 15) | (e << 7) | m, st.integers(0, 1), st.integers(40, 200), st.integers(0, 127))
_zero_or_bits = st.one_of(st.sampled_from([0, 0x8000]), _bits, _bits, _bits)


def _tensor(data, rows, cols):
    flat = data.draw(st.lists(_zero_or_bits, min_size=rows * cols, max_size=rows * cols))
    return np.array(flat, dtype=np.uint16).reshape(rows, cols)


@settings(max_examples=40, deadline=None, derandomize=True)
@given(st.data())
def test_mxfp4_properties(data):
    x = _tensor(data, 2, 64)
    r = oracle.qdq(FMT_MXFP4, x)
    xf, out = bits_to_f32(x).astype(np.float64), bits_to_f32(r["out"]).astype(np.float64)
    p = r["scales"].astype(np.int64) - 127
    step = np.exp2(p.astype(np.float64)).repeat(32, axis=1)
    codes = unpack_nibbles(r["codes"])
    np.testing.assert_array_equal(out, step * E2M1_VALUES[codes])                     # Eq. mxfp4-dequant, exactly
    amax = np.abs(xf).reshape(2, 2, 32).max(-1)
    nz = amax > 0
    assert np.all((amax[nz] >= 4 * np.exp2(p[nz])) & (amax[nz] < 8 * np.exp2(p[nz])))  # p = floor(log2 amax) - 2
    # inside the grid's range the error is at most half the local spacing (<= 1 * 2^p); beyond 6 * 2^p it saturates
    inside = np.abs(xf) <= 6 * step
    assert np.all(np.abs(out - xf)[inside] <= step[inside])
    assert np.all(np.abs(out[~inside]) == 6 * step[~inside])
    # sign symmetry, idempotence, scaling by a power of two
    np.testing.assert_array_equal(oracle.qdq(FMT_MXFP4, x ^ 0x8000)["out"], r["out"] ^ np.where(nz.repeat(32, axis=1), 0x8000, 0).astype(np.uint16))
    np.testing.assert_array_equal(oracle.qdq(FMT_MXFP4, r["out"])["out"], r["out"])
    x8 = ((x.astype(np.int64) + (3 << 7)) & 0xFFFF).astype(np.uint16)
    x8[(x & 0x7FFF) == 0] = x[(x & 0x7FFF) == 0]
    r8 = oracle.qdq(FMT_MXFP4, x8)
    np.testing.assert_array_equal(r8["codes"], r["codes"])
    np.testing.assert_array_equal((r8["scales"].astype(int) - r["scales"].astype(int))[nz], 3)


@settings(max_examples=40, deadline=None, derandomize=True)
@given(st.data())
def test_nvfp4_properties(data):
    x = _tensor(data, 2, 64)
    r = oracle.qdq(FMT_NVFP4, x)
    xf = bits_to_f32(x).astype(np.float64)
    ts = np.float32(r["tensor_scale"])
    amax_t = np.abs(xf).max()
    assert ts == (np.float32(amax_t) / np.float32(2688.0) if amax_t > 0 else np.float32(1.0))
    # with the derived tensor scale no block scale exceeds the E4M3 maximum, and the block holding the tensor maximum gets it
    assert int(r["scales"].max()) <= 0x7E
    if amax_t > 0:
        assert int(r["scales"].max()) == 0x7E
    # idempotent with the tensor scale held fixed; sign symmetric
    again = oracle.qdq(FMT_NVFP4, r["out"], float(ts))
    np.testing.assert_array_equal(again["out"], r["out"])
    neg = oracle.qdq(FMT_NVFP4, x ^ 0x8000)
    np.testing.assert_array_equal(neg["scales"], r["scales"])
    live = (r["scales"] > 0).repeat(8, axis=1)                     # a block whose scale rounds to zero emits code 0 throughout
    np.testing.assert_array_equal(neg["codes"][live], r["codes"][live] ^ 0x88)
    assert not r["codes"][~live].any() and not neg["codes"][~live].any()
    # every output is a grid point times the block's scale, rounded once to BF16
    codes = unpack_nibbles(r["codes"])
    sb = r["scales"].view(ml_dtypes.float8_e4m3fn).astype(np.float32).repeat(16, axis=1)
    want = ((sb * E2M1_VALUES[codes].astype(np.float32)) * ts).astype(ml_dtypes.bfloat16)
    np.testing.assert_array_equal(r["out"], want.view(np.uint16))


_q4k_bits = st.builds(lambda s, e, m: (s << 15) | (e << 7) | m, st.integers(0, 1), st.integers(105, 132), st.integers(0, 127))


@settings(max_examples=30, deadline=None, derandomize=True)
@given(st.data())
def test_q4k_properties(data):
    flat = data.draw(st.lists(st.one_of(st.sampled_from([0, 0x8000]), _q4k_bits, _q4k_bits, _q4k_bits), min_size=512, max_size=512))
    x = np.array(flat, dtype=np.uint16).reshape(1, 512)
    if data.draw(st.booleans()):
        x[0, :32] &= 0x7FFF                                      # one sub-block without negative values
    r = oracle.qdq(FMT_Q4_K, x)
    xf, out = bits_to_f32(x), bits_to_f32(r["out"])
    d, dmin, s6, m6 = _q4k_meta(r["scales"])
    codes = _q4k_codes(r["codes"], 1, 512)
    assert np.all(d >= 0) and np.all(dmin >= 0) and np.all(np.isfinite(d)) and np.all(np.isfinite(dmin))
    assert codes.min() >= 0 and codes.max() <= 15 and s6.min() >= 0 and s6.max() <= 63 and m6.min() >= 0 and m6.max() <= 63
    # Eq. q4k-dequant from the emitted fields, one FP32 rounding of es * C - em, then BF16
    es = (d[..., None] * s6.astype(np.float32)).reshape(1, 16).repeat(32, axis=1)
    em = (dmin[..., None] * m6.astype(np.float32)).reshape(1, 16).repeat(32, axis=1)
    want = (es.astype(np.float64) * codes - em.astype(np.float64)).astype(np.float32).astype(ml_dtypes.bfloat16)
    np.testing.assert_array_equal(r["out"], want.view(np.uint16))
    # the quantizer is monotone inside a sub-block, and a sub-block with no negative value has no offset
    for b in range(16):
        seg = slice(b * 32, (b + 1) * 32)
        order = np.argsort(xf[0, seg], kind="stable")
        assert np.all(np.diff(out[0, seg][order]) >= 0)
        assert np.all(np.diff(codes[0, seg][order]) >= 0)
        if xf[0, seg].min() >= 0:
            assert m6.reshape(16)[b] == 0 and out[0, seg].min() >= 0
    # the largest sub-block step and offset of a super-block use the top of their 6-bit ranges
    for s in range(2):
        if d[0, s] > 0:
            assert s6[0, s].max() == 63
        if dmin[0, s] > 0:
            assert m6[0, s].max() == 63
