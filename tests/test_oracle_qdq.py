"""Pins for the oracle's three quantize-dequantize routines. Nothing here calls the CUDA path.

Each format is checked against (a) hand-worked blocks stored under tests/golden, (b) an independent
route through library casts (ml_dtypes for the 4- and 8-bit floats, gguf for MXFP4 scales and the
Q4_K record reader), (c) the dequantization equation applied to the emitted codes and metadata,
(d) invariants the formats imply (sign symmetry, power-of-two equivariance, idempotence, error
bounds), and (e) brute-force nearest-grid search on the emitted scales."""
from pathlib import Path

import ml_dtypes
import numpy as np
import pytest

import oracle
from oracle import FMT_MXFP4, FMT_NVFP4, FMT_Q4_K
from util import E2M1_VALUES, bits_to_f32, f32_to_bits, unpack_nibbles

GOLDEN = Path(__file__).parent / "golden"
E4M3 = np.arange(0, 0x7F, dtype=np.uint8).view(ml_dtypes.float8_e4m3fn).astype(np.float32)


def _rows(path):
    for line in (GOLDEN / path).read_text().splitlines():
        if line.strip() and not line.startswith("#"):
            yield [f.split() for f in line.split("|")]


def _weights(rows, cols, seed, std=0.02, outliers=True):
    rng = np.random.default_rng(seed)
    w = rng.normal(0, std, (rows, cols)).astype(np.float32)
    if outliers:
        idx = rng.choice(w.size, max(1, w.size // 1000), replace=False)
        w.reshape(-1)[idx] *= 20
    return f32_to_bits(w)


# ------------------------------------------------------------------------------------------
# NVFP4
# ------------------------------------------------------------------------------------------

def test_nvfp4_worked_blocks():
    for ts, sb, xs, want in _rows("nvfp4_worked.txt"):
        x = np.zeros((1, 16), np.float32)
        x[0, :len(xs)] = [float(v) for v in xs]
        r = oracle.qdq(FMT_NVFP4, f32_to_bits(x), tensor_scale=float(ts[0]))
        assert oracle.e4m3_value(int(r["scales"][0, 0])) == float(sb[0])
        got = bits_to_f32(r["out"])[0, :len(want)]
        w = np.array([float(v) for v in want], np.float32)
        np.testing.assert_array_equal(got, w)
        np.testing.assert_array_equal(np.signbit(got), np.signbit(w))


def test_nvfp4_tensor_scale_is_amax_over_6x448():
    x = np.zeros((2, 32), np.float32)
    x[1, 5] = -2.625
    r = oracle.qdq(FMT_NVFP4, f32_to_bits(x))
    assert r["tensor_scale"] == np.float32(2.0 ** -10)
    x[1, 5] = 0.400390625
    r = oracle.qdq(FMT_NVFP4, f32_to_bits(x))
    assert r["tensor_scale"] == np.float32(0.400390625) / np.float32(2688.0)
    assert oracle.e4m3_value(int(r["scales"][1, 0])) == 448.0     # q = 448.00003 clamps to 448


def test_nvfp4_all_zero_tensor():
    r = oracle.qdq(FMT_NVFP4, np.zeros((3, 64), np.uint16))
    assert r["tensor_scale"] == 1.0
    assert not r["codes"].any() and not r["scales"].any() and not r["out"].any()


def _nvfp4_via_library_casts(xbits, s_t):
    """Same format, different route: ml_dtypes does the E4M3 and E2M1 rounding, numpy the rest."""
    x = bits_to_f32(xbits)
    rows, cols = x.shape
    xb = x.reshape(rows, cols // 16, 16)
    amax_b = np.abs(xb).max(-1)
    q = amax_b / (np.float32(6.0) * np.float32(s_t))
    sb8 = np.minimum(q, np.float32(448)).astype(ml_dtypes.float8_e4m3fn)
    sb = sb8.astype(np.float32)
    S = np.float32(s_t) * sb
    with np.errstate(divide="ignore", invalid="ignore"):
        v = xb / S[..., None]
    c = np.clip(v, -6, 6).astype(ml_dtypes.float4_e2m1fn).astype(np.float32)
    c = np.where(S[..., None] == 0, np.float32(0), c)
    out = ((sb[..., None] * c) * np.float32(s_t)).astype(np.float32)
    return f32_to_bits(out.reshape(rows, cols)), sb8.view(np.uint8)


@pytest.mark.parametrize("seed", [0, 1])
def test_nvfp4_matches_library_cast_route(seed):
    xb = _weights(64, 512, seed)
    r = oracle.qdq(FMT_NVFP4, xb)
    out, sc = _nvfp4_via_library_casts(xb, r["tensor_scale"])
    np.testing.assert_array_equal(r["scales"], sc)
    np.testing.assert_array_equal(r["out"], out)


def test_nvfp4_output_is_dequant_equation_of_codes_and_scales():
    xb = _weights(32, 256, 5)
    r = oracle.qdq(FMT_NVFP4, xb)
    codes = unpack_nibbles(r["codes"])
    sb = E4M3[r["scales"]].astype(np.float64)
    exact = np.float64(r["tensor_scale"]) * np.repeat(sb, 16, axis=1) * E2M1_VALUES[codes].astype(np.float64)
    got = bits_to_f32(r["out"]).astype(np.float64)
    ulp = np.exp2(np.floor(np.log2(np.maximum(np.abs(exact), 2.0 ** -126))) - 7)     # BF16 spacing at |exact|
    # Eq. nvfp4-dequant rounded to BF16; the FP32 intermediate may move an exact tie by 2^-24 relative
    assert np.all(np.abs(got - exact) <= 0.5 * ulp + np.abs(exact) * 2.0 ** -24)
    np.testing.assert_array_equal(oracle.dequant(FMT_NVFP4, r["codes"], r["scales"], r["tensor_scale"], 32, 256), r["out"])
    # 4.50 bits per weight: 16 codes x 4 bits + one 8-bit scale per 16 weights
    assert (r["codes"].size * 8 + r["scales"].size * 8) / xb.size == 4.5


def test_nvfp4_codes_are_nearest_grid_points_brute_force():
    xb = _weights(8, 128, 7)
    r = oracle.qdq(FMT_NVFP4, xb)
    x = bits_to_f32(xb).astype(np.float64)
    S = (np.float32(r["tensor_scale"]) * E4M3[r["scales"]]).astype(np.float64)       # one FP32 product
    S = np.repeat(S, 16, axis=1)
    codes = unpack_nibbles(r["codes"])
    grid = np.array([0, .5, 1, 1.5, 2, 3, 4, 6], np.float64)
    v = (bits_to_f32(xb) / S.astype(np.float32)).astype(np.float64)                  # the FP32 quotient
    d = np.abs(np.abs(v)[..., None] - grid)
    chosen = np.take_along_axis(d, (codes & 7)[..., None].astype(np.int64), -1)[..., 0]
    assert np.all(chosen == d.min(-1))
    assert np.all((codes >> 3) == np.signbit(x))
    # the block maximum lands on +-6 or +-4 (E4M3 rounding moves the scale by at most 1/16)
    top = np.abs(E2M1_VALUES[codes]).reshape(8, -1, 16).max(-1)
    assert np.all(top[np.abs(x).reshape(8, -1, 16).max(-1) > 0] >= 4)


def test_nvfp4_sign_symmetry_and_pow2_equivariance():
    xb = _weights(16, 256, 9)
    r = oracle.qdq(FMT_NVFP4, xb)
    rn = oracle.qdq(FMT_NVFP4, xb ^ 0x8000)
    np.testing.assert_array_equal(rn["out"], r["out"] ^ 0x8000)
    np.testing.assert_array_equal(rn["scales"], r["scales"])
    np.testing.assert_array_equal(rn["codes"], r["codes"] ^ 0x88)
    x8 = f32_to_bits(bits_to_f32(xb) * 8)
    r8 = oracle.qdq(FMT_NVFP4, x8)
    assert r8["tensor_scale"] == r["tensor_scale"] * 8
    np.testing.assert_array_equal(r8["codes"], r["codes"])
    np.testing.assert_array_equal(r8["scales"], r["scales"])
    np.testing.assert_array_equal(bits_to_f32(r8["out"]), bits_to_f32(r["out"]) * 8)


def test_nvfp4_idempotent_with_tensor_scale_held_fixed():
    xb = _weights(32, 512, 11)
    r = oracle.qdq(FMT_NVFP4, xb)
    r2 = oracle.qdq(FMT_NVFP4, r["out"], tensor_scale=float(r["tensor_scale"]))
    np.testing.assert_array_equal(r2["out"], r["out"])


def test_nvfp4_constant_tensor_and_underflowing_blocks():
    c = np.full((4, 64), 0.3125, np.float32)
    r = oracle.qdq(FMT_NVFP4, f32_to_bits(c))
    assert np.all(E4M3[r["scales"]] == 448) and np.all((unpack_nibbles(r["codes"]) & 7) == 7)
    np.testing.assert_array_equal(bits_to_f32(r["out"]), c)
    # one huge outlier pushes every other block scale to zero -> those blocks dequantize to +0
    x = np.full((2, 64), 1e-4, np.float32)
    x[0, 0] = 3e4
    r = oracle.qdq(FMT_NVFP4, f32_to_bits(x))
    assert r["scales"][1].max() == 0 and not r["out"][1].any() and not r["codes"][1].any()
    assert bits_to_f32(r["out"])[0, 0] == bits_to_f32(f32_to_bits(np.float32(3e4)))


# ------------------------------------------------------------------------------------------
# MXFP4
# ------------------------------------------------------------------------------------------

def test_mxfp4_worked_blocks():
    for p, xs, want in _rows("mxfp4_worked.txt"):
        x = np.zeros((1, 32), np.float32)
        x[0, :len(xs)] = [float(v) for v in xs]
        r = oracle.qdq(FMT_MXFP4, f32_to_bits(x))
        assert int(r["scales"][0, 0]) - 127 == int(p[0])
        np.testing.assert_array_equal(bits_to_f32(r["out"])[0, :len(want)], np.array([float(v) for v in want], np.float32))


def test_mxfp4_scales_are_powers_of_two_and_match_gguf():
    from gguf import GGMLQuantizationType as T, quants
    rng = np.random.default_rng(3)
    x = bits_to_f32(f32_to_bits(rng.normal(0, 1, (16, 256)) * np.exp(rng.uniform(-8, 8, (16, 1)))))
    r = oracle.qdq(FMT_MXFP4, f32_to_bits(x))
    g = quants.quantize(x, T.MXFP4).reshape(16, 8, 17)
    np.testing.assert_array_equal(r["scales"], g[..., 0])                        # same E8M0 exponent byte
    gd = quants.dequantize(g.reshape(16, -1), T.MXFP4)
    ours = bits_to_f32(r["out"])
    # gguf breaks element ties differently; everywhere else the two agree exactly
    v = np.abs(x.reshape(16, 8, 32) * np.exp2(127.0 - r["scales"].astype(np.float64))[..., None]).reshape(16, 256)
    tie = np.isin(v, [0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0])
    np.testing.assert_array_equal(ours[~tie], gd[~tie])
    # 4.25 bits per weight
    assert (r["codes"].size * 8 + r["scales"].size * 8) / x.size == 4.25


def test_mxfp4_output_is_dequant_equation_exactly():
    xb = _weights(16, 256, 21, std=1.0)
    r = oracle.qdq(FMT_MXFP4, xb)
    codes = unpack_nibbles(r["codes"])
    want = np.exp2(r["scales"].astype(np.float64) - 127).repeat(32, axis=1) * E2M1_VALUES[codes]
    np.testing.assert_array_equal(bits_to_f32(r["out"]).astype(np.float64), want)   # Eq. mxfp4-dequant, no rounding
    np.testing.assert_array_equal(oracle.dequant(FMT_MXFP4, r["codes"], r["scales"], None, 16, 256), r["out"])
    # brute force: nearest grid point to x / 2^p, and clipping only inside (6, 8)
    v = bits_to_f32(xb).astype(np.float64) / np.exp2(r["scales"].astype(np.float64) - 127).repeat(32, axis=1)
    grid = np.array([0, .5, 1, 1.5, 2, 3, 4, 6], np.float64)
    d = np.abs(np.abs(v)[..., None] - grid)
    assert np.all(np.take_along_axis(d, (codes & 7)[..., None].astype(np.int64), -1)[..., 0] == d.min(-1))
    assert np.abs(v).max() < 8 and np.all(np.abs(v).reshape(16, -1, 32).max(-1) >= 4)


def test_mxfp4_full_idempotence_sign_symmetry_equivariance():
    xb = _weights(32, 512, 23, std=1.0)
    r = oracle.qdq(FMT_MXFP4, xb)
    r2 = oracle.qdq(FMT_MXFP4, r["out"])
    for k in ("out", "codes", "scales"):
        np.testing.assert_array_equal(r2[k], r[k])
    rn = oracle.qdq(FMT_MXFP4, xb ^ 0x8000)
    np.testing.assert_array_equal(rn["out"], r["out"] ^ 0x8000)
    r16 = oracle.qdq(FMT_MXFP4, f32_to_bits(bits_to_f32(xb) * 2.0 ** -5))
    np.testing.assert_array_equal(r16["codes"], r["codes"])
    np.testing.assert_array_equal(r16["scales"].astype(int), r["scales"].astype(int) - 5)


def test_mxfp4_zero_block_subnormals_and_extremes():
    x = np.zeros((1, 128), np.float32)
    x[0, 32:64] = 2.0 ** -133                     # smallest BF16 subnormal
    x[0, 64] = 3.0e38                             # near the top of the BF16 range
    x[0, 96] = -0.0
    xb = f32_to_bits(x)
    r = oracle.qdq(FMT_MXFP4, xb)
    assert list(r["scales"][0]) == [0, 0, 127 + 125, 0]
    out = bits_to_f32(r["out"])[0]
    assert not r["out"][0, :64].any()             # zero block and sub-grid block -> +0
    assert out[64] == 1.5 * 2.0 ** 127            # 3e38 = 1.76 * 2^127 -> v = 7.05 clips to 6 * 2^125
    assert r["out"][0, 96] == 0                   # -0 in an all-zero block comes back as +0
    assert 0xFF not in r["scales"]


def test_mxfp4_noclip_worked_blocks():
    for p, xs, want in _rows("mxfp4_noclip_worked.txt"):
        x = np.zeros((1, 32), np.float32)
        x[0, :len(xs)] = [float(v) for v in xs]
        r = oracle.qdq(FMT_MXFP4, f32_to_bits(x), mxfp4_noclip=True)
        assert int(r["scales"][0, 0]) - 127 == int(p[0])
        np.testing.assert_array_equal(bits_to_f32(r["out"])[0, :len(want)], np.array([float(v) for v in want], np.float32))


def test_mxfp4_noclip_rule_is_minimal_exponent_without_saturation():
    rng = np.random.default_rng(29)
    x = bits_to_f32(f32_to_bits(rng.normal(0, 1, (32, 512)) * np.exp(rng.uniform(-8, 8, (32, 1)))))
    xb = f32_to_bits(x)
    r0 = oracle.qdq(FMT_MXFP4, xb)
    r1 = oracle.qdq(FMT_MXFP4, xb, mxfp4_noclip=True)
    p0 = r0["scales"].astype(np.int64) - 127
    p1 = r1["scales"].astype(np.int64) - 127
    amax = np.abs(x.astype(np.float64)).reshape(32, -1, 32).max(-1)
    # one step up exactly where the floor rule would saturate the block maximum
    np.testing.assert_array_equal(p1 - p0, (amax > 6 * np.exp2(p0)).astype(np.int64))
    assert 0 < (p1 != p0).mean() < 1
    assert np.all(amax <= 6 * np.exp2(p1)) and np.all(amax > 6 * np.exp2(p1 - 1))      # smallest such exponent
    # dequantization equation, and nearest grid point with nothing outside the grid's range
    codes = unpack_nibbles(r1["codes"])
    want = np.exp2(p1.astype(np.float64)).repeat(32, axis=1) * E2M1_VALUES[codes]
    np.testing.assert_array_equal(bits_to_f32(r1["out"]).astype(np.float64), want)
    np.testing.assert_array_equal(oracle.dequant(FMT_MXFP4, r1["codes"], r1["scales"], None, 32, 512), r1["out"])
    v = x.astype(np.float64) / np.exp2(p1.astype(np.float64)).repeat(32, axis=1)
    grid = np.array([0, .5, 1, 1.5, 2, 3, 4, 6], np.float64)
    d = np.abs(np.abs(v)[..., None] - grid)
    assert np.all(np.take_along_axis(d, (codes & 7)[..., None].astype(np.int64), -1)[..., 0] == d.min(-1))
    assert np.abs(v).max() <= 6
    assert np.all(np.abs(x - bits_to_f32(r1["out"])) <= np.exp2(p1.astype(np.float64)).repeat(32, axis=1))
    # blocks the floor rule does not saturate are left as they were
    same = (p1 == p0).repeat(32, axis=1)
    np.testing.assert_array_equal(r1["out"][same], r0["out"][same])
    np.testing.assert_array_equal(r1["codes"][same[:, ::2]], r0["codes"][same[:, ::2]])
    # idempotent in value (a block whose maximum rounds to 3 * 2^p re-encodes one exponent lower)
    np.testing.assert_array_equal(oracle.qdq(FMT_MXFP4, r1["out"], mxfp4_noclip=True)["out"], r1["out"])
    np.testing.assert_array_equal(oracle.qdq(FMT_MXFP4, xb ^ 0x8000, mxfp4_noclip=True)["out"], r1["out"] ^ 0x8000)


def test_mxfp4_noclip_extremes():
    x = np.zeros((1, 160), np.float32)
    x[0, 32:64] = 2.0 ** -133                     # smallest BF16 subnormal: the exponent clamps at -127
    x[0, 64] = 2.9e38                             # 3.41 * 2^126 -> 3 * 2^126, finite
    x[0, 96] = 6 * 2.0 ** -127                    # exactly 6 * 2^-127: lowest exponent, top code
    x[0, 128] = -0.0
    r = oracle.qdq(FMT_MXFP4, f32_to_bits(x), mxfp4_noclip=True)
    assert list(r["scales"][0]) == [0, 0, 127 + 126, 0, 0]
    out = bits_to_f32(r["out"])[0]
    assert not r["out"][0, :64].any()
    assert out[64] == 3 * 2.0 ** 126
    assert out[96] == np.float32(6 * 2.0 ** -127)
    assert r["out"][0, 128] == 0


# ------------------------------------------------------------------------------------------
# Q4_K
# ------------------------------------------------------------------------------------------

def _q4k_meta(scales):
    """Unpack [rows, nsb, 16] metadata bytes with numpy (independent of the oracle's C unpacker)."""
    d = scales[..., 0:2].copy().view(np.float16)[..., 0].astype(np.float32)
    dmin = scales[..., 2:4].copy().view(np.float16)[..., 0].astype(np.float32)
    pk = scales[..., 4:].astype(np.int32)
    s6 = np.concatenate([pk[..., 0:4] & 63, (pk[..., 8:12] & 15) | ((pk[..., 0:4] >> 6) << 4)], -1)
    m6 = np.concatenate([pk[..., 4:8] & 63, (pk[..., 8:12] >> 4) | ((pk[..., 4:8] >> 6) << 4)], -1)
    return d, dmin, s6, m6


def _q4k_codes(codes, rows, cols):
    q = codes.reshape(rows, cols // 256, 4, 32)
    return np.stack([q & 15, q >> 4], axis=3).reshape(rows, cols)       # chunk j: l -> low, l+32 -> high


def test_q4k_worked_constant_subblocks():
    x = np.zeros((1, 256), np.float32)
    x[0, 0:32] = 0.5
    x[0, 32:64] = -0.5
    r = oracle.qdq(FMT_Q4_K, f32_to_bits(x))
    d, dmin, s6, m6 = _q4k_meta(r["scales"])
    codes = _q4k_codes(r["codes"], 1, 256)
    out = bits_to_f32(r["out"])
    for b, s, m, c, xh in _rows("q4k_worked.txt"):
        b = int(b[0])
        assert s6[0, 0, b] == int(s[0]) and m6[0, 0, b] == int(m[0])
        assert np.all(codes[0, b * 32:(b + 1) * 32] == int(c[0]))
        assert np.all(out[0, b * 32:(b + 1) * 32] == float(xh[0]))


def test_q4k_worked_ramp_superblock():
    """A whole super-block with eight different sub-block ranges, worked by hand in the golden file."""
    x = np.zeros((1, 256), np.float32)
    for b in range(8):
        x[0, b * 32:(b + 1) * 32] = (b + 1) / 8 * (-1 + 0.125 * (np.arange(32) % 16))
    xb = f32_to_bits(x)
    np.testing.assert_array_equal(bits_to_f32(xb), x)                # the inputs are BF16 numbers
    r = oracle.qdq(FMT_Q4_K, xb)
    (dh, dminh, s6w, m6w, x0, err), = list(_rows("q4k_worked_ramp.txt"))
    raw = r["scales"][0, 0]
    assert int(raw[0]) | int(raw[1]) << 8 == int(dh[0], 16)
    assert int(raw[2]) | int(raw[3]) << 8 == int(dminh[0], 16)
    d, dmin, s6, m6 = _q4k_meta(r["scales"])
    assert list(s6[0, 0]) == [int(v) for v in s6w] and list(m6[0, 0]) == [int(v) for v in m6w]
    codes = _q4k_codes(r["codes"], 1, 256)[0]
    np.testing.assert_array_equal(codes[224:], np.tile(np.arange(16), 2))
    out = bits_to_f32(r["out"])[0]
    np.testing.assert_array_equal(out[224:], x[0, 224:])
    assert codes[0] == 0 and out[0] == float(x0[0])
    assert np.abs(out - x[0]).max() == float(err[0])


def test_q4k_record_reads_back_through_gguf():
    from gguf import GGMLQuantizationType as T, quants
    rows, cols = 8, 1024
    xb = _weights(rows, cols, 31, outliers=False)
    r = oracle.qdq(FMT_Q4_K, xb)
    # 144-byte engine record = {d, dmin, 12 packed bytes} + 128 code bytes  => 4.5 bits per weight
    rec = np.concatenate([r["scales"].reshape(rows, cols // 256, 16), r["codes"].reshape(rows, cols // 256, 128)], -1)
    assert rec.shape[-1] == 144 and rec.shape[-1] * 8 / 256 == 4.5
    g = quants.dequantize(rec.reshape(rows, -1), T.Q4_K)                # float32, Eq. q4k-dequant
    np.testing.assert_array_equal(f32_to_bits(g), r["out"])
    np.testing.assert_array_equal(oracle.dequant(FMT_Q4_K, r["codes"], r["scales"], None, rows, cols), r["out"])


def test_q4k_metadata_rule_and_error_bound():
    rows, cols = 8, 512
    xb = _weights(rows, cols, 33, outliers=True)
    x = bits_to_f32(xb)
    r = oracle.qdq(FMT_Q4_K, xb)
    d, dmin, s6, m6 = _q4k_meta(r["scales"])
    xs = x.reshape(rows, cols // 256, 8, 32)
    lo = np.minimum(xs.min(-1), 0)
    hi = xs.max(-1)
    sc = ((hi - lo) / np.float32(15)).astype(np.float32)
    off = -lo
    np.testing.assert_array_equal(d, (sc.max(-1) / np.float32(63)).astype(np.float16).astype(np.float32))
    np.testing.assert_array_equal(dmin, (off.max(-1) / np.float32(63)).astype(np.float16).astype(np.float32))
    assert s6.max() == 63 or np.all(d == 0)
    assert np.all(np.abs(s6 * d[..., None] - sc) <= d[..., None] / 2 * 1.0001)       # 6-bit rounding of sc/d
    assert np.all(np.abs(m6 * dmin[..., None] - off) <= dmin[..., None] / 2 * 1.0001)
    es = (d[..., None] * s6).astype(np.float64)[..., None]
    em = (dmin[..., None] * m6).astype(np.float64)[..., None]
    codes = _q4k_codes(r["codes"], rows, cols).reshape(xs.shape).astype(np.float64)
    # brute force: the code is the nearest of the 16 levels
    lv = es * np.arange(16) - em
    t = ((xs + em.astype(np.float32)) / es.astype(np.float32)).astype(np.float64)   # the FP32 quotient
    dist = np.abs(np.clip(t, 0, 15)[..., None] - np.arange(16))
    assert np.all(np.take_along_axis(dist, codes[..., None].astype(np.int64), -1)[..., 0] == dist.min(-1))
    # error bound inside the representable range
    xh = bits_to_f32(r["out"]).reshape(xs.shape).astype(np.float64)
    inside = (xs >= -em) & (xs <= 15 * es - em)
    bound = es / 2 * 1.001 + np.abs(xh) * 2.0 ** -8
    assert np.all(np.abs(xs - xh)[inside] <= np.broadcast_to(bound, xs.shape)[inside])


def test_q4k_degenerate_blocks():
    r = oracle.qdq(FMT_Q4_K, np.zeros((2, 256), np.uint16))
    assert not r["out"].any() and not r["codes"].any() and not r["scales"].any()
    x = np.full((1, 256), 0.75, np.float32)               # all-positive: offset 0, top code everywhere
    r = oracle.qdq(FMT_Q4_K, f32_to_bits(x))
    d, dmin, s6, m6 = _q4k_meta(r["scales"])
    assert dmin[0, 0] == 0 and np.all(m6 == 0) and np.all(s6 == 63)
    assert np.all(_q4k_codes(r["codes"], 1, 256) == 15)
    np.testing.assert_array_equal(bits_to_f32(r["out"]), x)
