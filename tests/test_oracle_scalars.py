"""Pins for the oracle's scalar number formats (E2M1, E4M3, BF16, FP16) against things other than
the oracle itself: the paper's E2M1 value set, a hand-written threshold table, and the
independent ``ml_dtypes`` / numpy / torch casts."""
from pathlib import Path

import ml_dtypes
import numpy as np
import pytest
import torch

import oracle
from util import bits_to_f32, f32_to_bits

GOLDEN = Path(__file__).parent / "golden"


def _ulp_neighbours(v):
    v = np.float32(v)
    return np.nextafter(v, np.float32(-np.inf)), v, np.nextafter(v, np.float32(np.inf))


def test_e2m1_value_set_matches_paper():
    # Eq. e2m1-values: {0, +-0.5, +-1, +-1.5, +-2, +-3, +-4, +-6}
    mags = [oracle.e2m1_value(c) for c in range(8)]
    assert mags == [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]
    for c in range(8):
        assert oracle.e2m1_value(c | 8) == -mags[c]
    assert len({oracle.e2m1_value(c) for c in range(16)}) == 15     # +0 and -0 compare equal


def test_e2m1_threshold_table():
    for line in (GOLDEN / "e2m1_thresholds.txt").read_text().splitlines():
        if not line.strip() or line.startswith("#"):
            continue
        a, want = map(float, line.split())
        for sign in (1.0, -1.0):
            c = oracle.e2m1_encode(sign * a)
            assert abs(oracle.e2m1_value(c)) == want, (a, c)
            assert (c >> 3) == (1 if sign < 0 else 0)       # sign kept even when rounding to zero


def test_e2m1_one_ulp_around_every_midpoint():
    mids = [(0.25, 0.0, 0.5), (0.75, 0.5, 1.0), (1.25, 1.0, 1.5), (1.75, 1.5, 2.0),
            (2.5, 2.0, 3.0), (3.5, 3.0, 4.0), (5.0, 4.0, 6.0)]
    for mid, lo, hi in mids:
        below, _, above = _ulp_neighbours(mid)
        assert oracle.e2m1_value(oracle.e2m1_encode(below)) == lo
        assert oracle.e2m1_value(oracle.e2m1_encode(above)) == hi
        assert oracle.e2m1_encode(mid) % 2 == 0                 # the tie goes to the even code


def test_e2m1_saturates_at_6_however_large_the_value():
    # Eq. e2m1-values: 6 is the largest magnitude of the grid, so everything beyond it lands there, including
    # values so large that their distances to all grid points coincide in double precision
    for v in (6.0, 6.5, 8.0, 1e9, 2.0 ** 53, 2.0 ** 54 + 2.0 ** 31, 1e20, 3.7e25, 3.0e38, float(np.finfo(np.float32).max)):
        assert oracle.e2m1_encode(v) == 7 and oracle.e2m1_encode(-v) == 15, v
    x = np.zeros((1, 32), np.float32); x[0, 0] = 1.6557448e28; x[0, 1] = -1.0154977e27; x[0, 2] = 448 * 5.5
    r = oracle.qdq(oracle.FMT_NVFP4, f32_to_bits(x), 1.0)          # a supplied tensor scale far too small: block scale 448
    assert r["scales"][0, 0] == 0x7E
    assert list(bits_to_f32(r["out"])[0, :3]) == [2688.0, -2688.0, 2688.0]


def test_e2m1_matches_ml_dtypes_cast():
    rng = np.random.default_rng(0)
    v = np.concatenate([
        rng.uniform(-8, 8, 50000), rng.normal(0, 1, 50000), rng.normal(0, 1e-3, 1000),
        np.array([0.0, -0.0, 0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 6.0, 6.5, 1e9, 1e-30]),
    ]).astype(np.float32)
    v = np.concatenate([v, -v, np.nextafter(v, np.float32(np.inf)), np.nextafter(v, np.float32(-np.inf))])
    want = np.clip(v, -6, 6).astype(ml_dtypes.float4_e2m1fn)
    got = np.array([oracle.e2m1_value(oracle.e2m1_encode(x)) for x in v], np.float32)
    np.testing.assert_array_equal(got, want.astype(np.float32))
    # sign of zero
    np.testing.assert_array_equal(np.signbit(got), np.signbit(v))


def test_e4m3_decode_all_codes_matches_ml_dtypes():
    codes = np.arange(0, 0x7F, dtype=np.uint8)
    want = codes.view(ml_dtypes.float8_e4m3fn).astype(np.float32)
    got = np.array([oracle.e4m3_value(int(c)) for c in codes], np.float32)
    np.testing.assert_array_equal(got, want)
    assert got.max() == 448.0 and got[1] == 2.0 ** -9


def test_e4m3_encode_hand_values():
    assert oracle.e4m3_value(oracle.e4m3_encode(51.333)) == 52.0
    assert oracle.e4m3_value(oracle.e4m3_encode(448.00003)) == 448.0
    assert oracle.e4m3_value(oracle.e4m3_encode(1e9)) == 448.0          # saturates, never NaN
    assert oracle.e4m3_value(oracle.e4m3_encode(0.0029)) == 2.0 ** -9
    assert oracle.e4m3_encode(2.0 ** -10) == 0                          # tie with zero -> even code 0
    assert oracle.e4m3_encode(float(np.nextafter(np.float32(2.0 ** -10), np.float32(1)))) == 1
    assert oracle.e4m3_encode(3 * 2.0 ** -10) == 2                      # tie between codes 1 and 2
    assert oracle.e4m3_encode(0.0) == 0


def test_e4m3_encode_matches_ml_dtypes_cast():
    rng = np.random.default_rng(1)
    q = np.concatenate([
        rng.uniform(0, 460, 20000), np.exp(rng.uniform(np.log(1e-4), np.log(500), 20000)),
    ]).astype(np.float32)
    # every midpoint between neighbouring codes, and one ulp either side
    vals = np.arange(0, 0x7F, dtype=np.uint8).view(ml_dtypes.float8_e4m3fn).astype(np.float32)
    mids = (vals[:-1] + vals[1:]) / 2
    q = np.concatenate([q, mids, np.nextafter(mids, np.float32(0)), np.nextafter(mids, np.float32(1e9)), vals])
    want = np.minimum(q, np.float32(448)).astype(ml_dtypes.float8_e4m3fn).view(np.uint8)
    got = np.array([oracle.e4m3_encode(x) for x in q], np.uint8)
    np.testing.assert_array_equal(got, want)


def test_bf16_round_matches_torch_and_ml_dtypes():
    rng = np.random.default_rng(2)
    f = np.concatenate([rng.normal(0, 1, 20000), rng.normal(0, 1e-38, 2000),
                        np.array([1.00390625, 1.01171875, 0.0, -0.0, 3.3895e38])]).astype(np.float32)
    want_t = torch.from_numpy(f).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    want_m = f.astype(ml_dtypes.bfloat16).view(np.uint16)
    got = np.array([oracle.bf16_round(x) for x in f], np.uint16)
    np.testing.assert_array_equal(got, want_t)
    np.testing.assert_array_equal(got, want_m)


def test_fp16_round_matches_numpy_and_saturates():
    rng = np.random.default_rng(3)
    f = np.concatenate([rng.normal(0, 1e-3, 20000), rng.normal(0, 1e-6, 5000), rng.uniform(0, 65504, 2000),
                        np.array([0.0, 6.1e-5, 5.96e-8, 2.98e-8, 2.9e-8, 65504.0])]).astype(np.float32)
    want = f.astype(np.float16).view(np.uint16)
    got = np.array([oracle.fp16_round_sat(x) for x in f], np.uint16)
    np.testing.assert_array_equal(got, want)
    assert oracle.fp16_value(oracle.fp16_round_sat(1e9)) == 65504.0
    assert oracle.fp16_value(oracle.fp16_round_sat(-1e9)) == -65504.0
    for h in (0x0001, 0x03FF, 0x0400, 0x3C00, 0x7BFF):
        assert oracle.fp16_value(h) == float(np.array([h], np.uint16).view(np.float16)[0])
