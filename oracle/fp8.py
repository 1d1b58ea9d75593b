"""Software FP8 codec (E4M3, E5M2), round-to-nearest-even and stochastic rounding.

Formats: the paper trains with E4M3 in the forward and E5M2 for gradients (Appendix
"Experimental setup", FP8 recipe); bit-level conventions are the OCP FP8 ones.  The stochastic
rounding law is the paper's: a value bracketed by two representable numbers goes up or down at
random with a zero-mean error (Section "Same rounding distribution, opposite outcomes");
values at the top of the range round to nearest and are counted (Appendix "The forks").

Test infrastructure: see the package docstring.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

E4M3 = 0
E5M2 = 1
RN = 0
SR = 1


@dataclass(frozen=True)
class Format:
    name: str
    ebits: int
    mbits: int
    bias: int
    fmax: float
    emin: int          # exponent of the smallest normal
    has_inf: bool


FORMATS = {
    E4M3: Format("e4m3", 4, 3, 7, 448.0, -6, False),
    E5M2: Format("e5m2", 5, 2, 15, 57344.0, -14, True),
}


def decode_table(fmt: int) -> np.ndarray:
    """float64 value of each of the 256 codes, written out from the bit fields.

    E4M3: no infinity; exponent field 15 with mantissa 7 is NaN, every other pattern is finite
    (max 1.75 * 2^8 = 448).  E5M2: exponent field 31 is inf (mantissa 0) or NaN.
    """
    F = FORMATS[fmt]
    out = np.empty(256, dtype=np.float64)
    for code in range(256):
        sign = -1.0 if code & 0x80 else 1.0
        efield = (code >> F.mbits) & ((1 << F.ebits) - 1)
        mant = code & ((1 << F.mbits) - 1)
        if fmt == E4M3 and efield == 15 and mant == 7:
            val = np.nan
        elif fmt == E5M2 and efield == 31:
            val = np.inf if mant == 0 else np.nan
        elif efield == 0:
            val = mant * 2.0 ** (F.emin - F.mbits)
        else:
            val = (1.0 + mant / (1 << F.mbits)) * 2.0 ** (efield - F.bias)
        out[code] = sign * val if not np.isnan(val) else np.nan
    return out


_DECODE = {E4M3: decode_table(E4M3), E5M2: decode_table(E5M2)}


def decode(codes, fmt: int) -> np.ndarray:
    """Exact float64 value of uint8 codes."""
    return _DECODE[fmt][np.asarray(codes, dtype=np.uint8)]


def _positive_finite(fmt: int):
    """(values, codes) of the non-negative finite codes, ascending."""
    tab = _DECODE[fmt][:128]
    ok = np.isfinite(tab)
    codes = np.nonzero(ok)[0].astype(np.uint8)
    return tab[ok], codes


def encode(v32, fmt: int, mode: int = RN, words=None):
    """Round FP32 values to FP8 codes.

    Steps for a finite value v with magnitude a below the largest finite number fmax:
    e = max(floor(log2 a), emin), ulp = 2^(e - mbits), t = a / ulp (exact), n = floor(t),
    f = t - n.  Nearest: up iff f > 1/2 or (f == 1/2 and n odd).  Stochastic: P = floor(f 2^32),
    up iff U < P with U the element's 32-bit random word, so P(up) = f and the mean is v.
    The result magnitude is (n + up) * ulp; the sign bit of v is kept even when that is zero.
    a >= fmax gives +-fmax (counted as saturated when a > fmax); NaN gives the NaN code
    0x7F whatever its sign bit (IEEE 754 leaves the sign of a NaN produced by the scaling multiply
    unspecified); infinities saturate and are counted as non-finite.

    Returns (codes uint8, n_saturated, n_nonfinite).
    """
    F = FORMATS[fmt]
    v32 = np.asarray(v32, dtype=np.float32)
    shape = v32.shape
    v = v32.astype(np.float64).ravel()
    sign = np.signbit(v32).ravel()
    a = np.abs(v)
    isnan = np.isnan(a)
    isinf = np.isinf(a)
    top = (a >= F.fmax) & ~isnan
    n_sat = int(np.count_nonzero((a > F.fmax) & ~isnan & ~isinf))
    n_nonfinite = int(np.count_nonzero(isnan | isinf))

    safe = np.where(isnan | top | (a == 0.0), 1.0, a)
    _, ex = np.frexp(safe)                 # safe = m * 2^ex with m in [0.5, 1)
    e = np.maximum(ex - 1, F.emin)         # floor(log2 a), clamped to the subnormal binade
    ulp = np.ldexp(1.0, e - F.mbits)
    t = safe / ulp
    n = np.floor(t)
    f = t - n
    if mode == RN:
        up = (f > 0.5) | ((f == 0.5) & (np.mod(n, 2.0) == 1.0))
    else:
        if words is None:
            raise ValueError("stochastic rounding needs the random words")
        U = np.asarray(words, dtype=np.uint32).ravel().astype(np.float64)
        P = np.floor(f * 4294967296.0)
        up = U < P
    mag = (n + up.astype(np.float64)) * ulp
    mag = np.where(a == 0.0, 0.0, mag)
    mag = np.where(top, F.fmax, mag)

    vals, poscodes = _positive_finite(fmt)
    idx = np.searchsorted(vals, np.where(isnan, 0.0, mag))
    idx = np.clip(idx, 0, len(vals) - 1)
    if not np.array_equal(vals[idx][~isnan], mag[~isnan]):
        raise AssertionError("rounded magnitude is not representable")
    codes = poscodes[idx].astype(np.uint8)
    codes = codes | (sign.astype(np.uint8) << np.uint8(7))
    codes = np.where(isnan, np.uint8(0x7F), codes)       # one NaN code, whatever the NaN's sign bit
    return codes.reshape(shape).astype(np.uint8), n_sat, n_nonfinite


def neighbours(v32, fmt: int):
    """The bracketing representable magnitudes (lo, hi) of |v| and the up-probability numerator
    P (of 2^32), for finite |v| < fmax.  Used by the closed-form expectation pin."""
    F = FORMATS[fmt]
    a = np.abs(np.asarray(v32, dtype=np.float32).astype(np.float64))
    safe = np.where(a == 0.0, 1.0, a)
    _, ex = np.frexp(safe)
    e = np.maximum(ex - 1, F.emin)
    ulp = np.ldexp(1.0, e - F.mbits)
    t = safe / ulp
    n = np.floor(t)
    f = t - n
    lo = np.where(a == 0.0, 0.0, n * ulp)
    hi = np.where(a == 0.0, 0.0, (n + 1.0) * ulp)
    P = np.where(a == 0.0, 0.0, np.floor(f * 4294967296.0))
    return lo, hi, P


def scale_from_amax(amax, fmt: int):
    """Per-group scale: scale = fl32(fmax / amax), inv_scale = fl32(1 / scale); margin 0.
    amax of zero, a non-finite amax, or a quotient that overflows FP32 gives scale 1.  (One scale for the whole tensor:
    Appendix "The same dependence in a normalization backward".)"""
    F = FORMATS[fmt]
    amax = np.asarray(amax, dtype=np.float32)
    bad = ~np.isfinite(amax) | (amax == 0)
    with np.errstate(divide="ignore", invalid="ignore", over="ignore"):
        scale = (np.float32(F.fmax) / np.where(bad, np.float32(1), amax)).astype(np.float32)
    scale = np.where(bad | ~np.isfinite(scale), np.float32(1.0), scale).astype(np.float32)
    inv = (np.float32(1.0) / scale).astype(np.float32)
    return scale, inv
