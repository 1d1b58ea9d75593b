"""Pins of the oracle's generator and codec against what is fixed outside the oracle."""
import itertools
from fractions import Fraction

import ml_dtypes
import numpy as np
import pytest

from conftest import golden_path
from oracle import fp8, philox

ML = {fp8.E4M3: ml_dtypes.float8_e4m3fn, fp8.E5M2: ml_dtypes.float8_e5m2}


def _kat():
    rows = []
    for line in open(golden_path("philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        c, k, o = [[int(w, 16) for w in part.split()] for part in line.split("|")]
        rows.append((c, k, o))
    return rows


def test_philox_known_answers():
    rows = _kat()
    assert len(rows) == 3
    for c, k, o in rows:
        out = philox.philox4x32_10(c[0], c[1], c[2], c[3], k[0], k[1])
        assert [int(w) for w in out] == o


def test_philox_word_order_and_key_matter():
    # a transposed counter/key or a swapped word would collide with another vector
    a = philox.philox4x32_10(1, 2, 3, 4, 5, 6)
    b = philox.philox4x32_10(2, 1, 3, 4, 5, 6)
    c = philox.philox4x32_10(1, 2, 3, 4, 6, 5)
    assert [int(w) for w in a] != [int(w) for w in b]
    assert [int(w) for w in a] != [int(w) for w in c]


def test_element_words_layout_independent():
    seed, tid, stream, draw = 0x1234567890ABCDEF, 7, 2, 5
    n = 1003
    full = philox.tensor_words(seed, tid, stream, draw, n)
    idx = np.array([0, 1, 2, 3, 4, 5, 17, 1000, 1002], dtype=np.uint64)
    assert np.array_equal(philox.element_words(seed, tid, stream, draw, idx), full[idx.astype(int)])
    assert np.array_equal(philox.element_words(seed, tid, stream, draw, np.arange(n)), full)
    # element e uses word e&3 of the block whose counter is (e>>2, 0, draw, tid<<8|stream)
    blk = philox.philox4x32_10(250, 0, draw, (tid << 8) | stream, seed & 0xFFFFFFFF, seed >> 32)
    assert int(full[1002]) == int(blk[2])
    # every field of the key changes the words
    for other in [philox.tensor_words(seed + 1, tid, stream, draw, 8),
                  philox.tensor_words(seed, tid + 1, stream, draw, 8),
                  philox.tensor_words(seed, tid, stream + 1, draw, 8),
                  philox.tensor_words(seed, tid, stream, draw + 1, 8),
                  philox.tensor_words(seed + (1 << 32), tid, stream, draw, 8)]:
        assert not np.array_equal(other, full[:8])


def test_element_words_high_index():
    e = np.array([(1 << 34) + 5], dtype=np.uint64)
    w = philox.element_words(3, 1, 0, 0, e)
    q = int(e[0]) >> 2
    blk = philox.philox4x32_10(q & 0xFFFFFFFF, q >> 32, 0, (1 << 8) | 0, 3, 0)
    assert int(w[0]) == int(blk[1])


@pytest.mark.parametrize("fmt", [fp8.E4M3, fp8.E5M2])
def test_decode_table_matches_independent_bitcast(fmt):
    codes = np.arange(256, dtype=np.uint8)
    ref = codes.view(ML[fmt]).astype(np.float64)
    mine = fp8.decode(codes, fmt)
    assert np.array_equal(np.isnan(ref), np.isnan(mine))
    ok = ~np.isnan(ref)
    assert np.array_equal(ref[ok], mine[ok])
    assert np.array_equal(np.signbit(ref[ok]), np.signbit(mine[ok]))


@pytest.mark.parametrize("fmt", [fp8.E4M3, fp8.E5M2])
def test_all_codes_round_trip(fmt):
    codes = np.arange(256, dtype=np.uint8)
    val = fp8.decode(codes, fmt)
    finite = np.isfinite(val)
    assert finite.sum() == (254 if fmt == fp8.E4M3 else 248)
    v32 = val[finite].astype(np.float32)
    back, n_sat, n_nf = fp8.encode(v32, fmt, fp8.RN)
    assert np.array_equal(back, codes[finite]) and n_sat == 0 and n_nf == 0
    for word in (0, 1, 0x7FFFFFFF, 0xFFFFFFFF):
        back, _, _ = fp8.encode(v32, fmt, fp8.SR, np.full(v32.shape, word, dtype=np.uint32))
        assert np.array_equal(back, codes[finite])        # representable values never move
    # every NaN maps to the one NaN code 0x7F, whatever its sign bit
    nan32 = np.array([0x7FC00000, 0xFFC00000], dtype=np.uint32).view(np.float32)
    back, _, n_nf = fp8.encode(nan32, fmt, fp8.RN)
    assert list(back) == [0x7F, 0x7F] and n_nf == 2


@pytest.mark.parametrize("fmt", [fp8.E4M3, fp8.E5M2])
def test_round_nearest_matches_independent_cast(fmt):
    F = fp8.FORMATS[fmt]
    rng = np.random.default_rng(1)
    pos = fp8.decode(np.arange(128, dtype=np.uint8), fmt)
    pos = np.sort(pos[np.isfinite(pos)])
    mids = (pos[:-1] + pos[1:]) / 2                       # every tie between adjacent codes
    near = np.concatenate([np.nextafter(mids.astype(np.float32), np.float32(0)),
                           np.nextafter(mids.astype(np.float32), np.float32(np.inf))]).astype(np.float64)
    rand = rng.standard_normal(40000) * np.exp(rng.uniform(-12, 6, 40000) if fmt == fp8.E4M3
                                               else rng.uniform(-20, 10, 40000))
    tiny = np.array([0.0, 2.0 ** -30, 2.0 ** -10, 2.0 ** -9 * 0.5, 2.0 ** -17, 2.0 ** -16 * 0.5])
    vals = np.concatenate([pos, mids, near, rand, tiny])
    vals = np.concatenate([vals, -vals]).astype(np.float32)
    vals = vals[np.abs(vals) <= F.fmax]
    mine, n_sat, _ = fp8.encode(vals, fmt, fp8.RN)
    ref = vals.astype(ML[fmt]).view(np.uint8)
    assert n_sat == 0
    assert np.array_equal(mine, ref)


@pytest.mark.parametrize("fmt", [fp8.E4M3, fp8.E5M2])
def test_saturation_and_nonfinite(fmt):
    F = fp8.FORMATS[fmt]
    top = 0x7E if fmt == fp8.E4M3 else 0x7B
    v = np.array([F.fmax, -F.fmax, F.fmax * 1.01, -1e30, np.inf, -np.inf], dtype=np.float32)
    for mode, words in ((fp8.RN, None), (fp8.SR, np.zeros(6, np.uint32))):
        codes, n_sat, n_nf = fp8.encode(v, fmt, mode, words)
        assert list(codes) == [top, top | 0x80, top, top | 0x80, top, top | 0x80]
        assert n_sat == 2 and n_nf == 2
    # just below the top: the upper neighbour is fmax itself, never beyond
    below = np.nextafter(np.float32(F.fmax), np.float32(0))
    codes, n_sat, _ = fp8.encode(np.array([below], np.float32), fmt, fp8.SR, np.array([0], np.uint32))
    assert codes[0] == top and n_sat == 0
    # the sign of zero and of values that round to zero is kept
    z = np.array([0.0, -0.0, 1e-30, -1e-30], dtype=np.float32)
    codes, _, _ = fp8.encode(z, fmt, fp8.SR, np.full(4, 0xFFFFFFFF, np.uint32))
    assert list(codes) == [0x00, 0x80, 0x00, 0x80]


@pytest.mark.parametrize("fmt", [fp8.E4M3, fp8.E5M2])
def test_stochastic_rounding_threshold_brute_force(fmt):
    rng = np.random.default_rng(2)
    v = (rng.standard_normal(2000) * np.exp(rng.uniform(-8, 4, 2000))).astype(np.float32)
    v = v[np.abs(v) < fp8.FORMATS[fmt].fmax]
    lo, hi, P = fp8.neighbours(v, fmt)
    sgn = np.where(np.signbit(v), -1.0, 1.0)
    for name, word in (("zero", np.zeros_like(P)), ("Pm1", P - 1), ("P", P), ("max", np.full_like(P, 2.0 ** 32 - 1))):
        usable = (word >= 0) & (word < 2.0 ** 32)
        codes, _, _ = fp8.encode(v[usable], fmt, fp8.SR, word[usable].astype(np.uint32))
        got = fp8.decode(codes, fmt)
        up = word[usable] < P[usable]
        want = sgn[usable] * np.where(up, hi[usable], lo[usable])
        assert np.array_equal(got, want), name
    # lo and hi are adjacent codes (or equal-value fixed points) that bracket |v|
    a = np.abs(v.astype(np.float64))
    assert np.all(lo <= a) and np.all(a < hi)
    pos = fp8.decode(np.arange(128, dtype=np.uint8), fmt)
    pos = np.sort(pos[np.isfinite(pos)])
    assert np.all(np.searchsorted(pos, hi) - np.searchsorted(pos, lo) == 1)


@pytest.mark.parametrize("fmt", [fp8.E4M3, fp8.E5M2])
def test_stochastic_rounding_expectation_is_exact(fmt):
    """E[SR(v)] = lo (1 - P/2^32) + hi P/2^32 = v, exhaustively over every FP32 mantissa pattern
    below the kept bits in one binade (2^20 patterns for E4M3, 2^21 for E5M2), in exact integer
    arithmetic."""
    F = fp8.FORMATS[fmt]
    drop = 23 - F.mbits
    kept = 5 % (1 << F.mbits)
    mant = (kept << drop) | np.arange(1 << drop, dtype=np.uint32)
    bits = (np.uint32(127 + 1) << np.uint32(23)) | mant          # values in [2, 4)
    v = bits.view(np.float32)
    lo, hi, P = fp8.neighbours(v, fmt)
    ulp32 = 2.0 ** (1 - 23)                                       # FP32 ulp in this binade
    vi = (v.astype(np.float64) / ulp32).astype(np.int64)          # exact integers
    loi = (lo / ulp32).astype(np.int64)
    hii = (hi / ulp32).astype(np.int64)
    Pi = P.astype(np.int64)
    # lo*(2^32-P) + hi*P == v*2^32 exactly
    lhs = loi * ((1 << 32) - Pi) + hii * Pi
    assert np.array_equal(lhs, vi << 32)
    assert np.array_equal(Pi, (mant.astype(np.int64) & ((1 << drop) - 1)) << (32 - drop))
    # a few cases with rationals, subnormal target range included
    for x in [0.3, 1.7, 2.0 ** -8 * 1.3, 2.0 ** -15 * 1.1, 100.3, -5.77]:
        x32 = np.float32(x)
        lo1, hi1, P1 = fp8.neighbours(np.array([x32]), fmt)
        e = Fraction(float(lo1[0])) * (1 - Fraction(int(P1[0]), 1 << 32)) + Fraction(float(hi1[0])) * Fraction(int(P1[0]), 1 << 32)
        assert abs(e - abs(Fraction(float(x32)))) <= Fraction(float(hi1[0] - lo1[0])) / (1 << 32)


def test_stochastic_rounding_empirical_mean():
    # independent of `neighbours`: average many draws of one value
    v = np.full(200000, 0.3, dtype=np.float32)
    words = philox.tensor_words(11, 1, 1, 0, v.size)
    codes, _, _ = fp8.encode(v, fp8.E4M3, fp8.SR, words)
    got = fp8.decode(codes, fp8.E4M3)
    assert set(np.unique(got)) == {0.28125, 0.3125}
    se = np.std(got) / np.sqrt(v.size)
    assert abs(np.mean(got) - float(np.float32(0.3))) < 4 * se


def test_scale_from_amax():
    s, inv = fp8.scale_from_amax(np.float32(3.5), fp8.E4M3)
    assert s == np.float32(448.0) / np.float32(3.5) and inv == np.float32(1.0) / s
    for bad in (0.0, np.inf, np.nan, 1e-42):
        s, inv = fp8.scale_from_amax(np.float32(bad), fp8.E5M2)
        assert s == 1.0 and inv == 1.0
