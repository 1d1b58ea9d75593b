"""The linear layer after the store: incoming gradient, weight gradient, input gradient.

y = u_q W in the paper's orientation; here W is stored [O, C] (y = u_q W^T), so the weight
gradient is dW[O, C] = dY^T X with X the copy of u the weight use reads (Eq. norm-uses:
dW = u_q^T dy; reading the original adds -r^T dy).  du = dY W passes through the rounding
unchanged (Appendix "The normalization store").

Test infrastructure: see the package docstring.
"""
from __future__ import annotations

import numpy as np

from . import fp8


def bf16_round(a) -> np.ndarray:
    """Round to the nearest bf16 value, ties to even; float64 in, float64 out.  This is the
    operand rounding of a BF16 tensor-core contraction, applied here so that the comparison
    measures accumulation and not the operand format."""
    a32 = np.asarray(a, dtype=np.float64).astype(np.float32)
    b = a32.view(np.uint32).astype(np.uint64)
    lsb = (b >> np.uint64(16)) & np.uint64(1)
    b = (b + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    return b.astype(np.uint32).view(np.float32).reshape(a32.shape).astype(np.float64)


def incoming_gradient(dY, fmt: int = fp8.E5M2):
    """The gradient the uses actually receive: dY rounded to nearest onto the gradient format at
    a per-tensor scale from its own amax (FP8 recipe: E5M2 for gradients, margin 0).
    Returns dict(codes, scale, inv_scale, amax, value) with value = decode(codes) * inv_scale."""
    dY32 = np.asarray(dY, dtype=np.float32)
    amax = np.float32(np.max(np.abs(dY32))) if dY32.size else np.float32(0)
    scale, inv = fp8.scale_from_amax(amax, fmt)
    v = (dY32 * np.float32(scale)).astype(np.float32)
    codes, n_sat, n_nf = fp8.encode(v, fmt, fp8.RN)
    value = fp8.decode(codes, fmt) * float(inv)
    return dict(codes=codes, scale=np.float32(scale), inv_scale=np.float32(inv), amax=amax,
                value=value, n_saturated=n_sat, n_nonfinite=n_nf)


def wgrad(dY_value, x_copy, rows=None, cols=None) -> np.ndarray:
    """dW[O, C] = dY^T X in float64 (sum over tokens).  `rows`/`cols` select a sub-block of the
    output (index arrays into O and C) without changing any entry's value."""
    dYv = np.asarray(dY_value, dtype=np.float64)
    X = np.asarray(x_copy, dtype=np.float64)
    if rows is not None:
        dYv = dYv[:, rows]
    if cols is not None:
        X = X[:, cols]
    return dYv.T @ X


def dgrad(dY_value, W) -> np.ndarray:
    """du[T, C] = dY W in float64 (W stored [O, C])."""
    return np.asarray(dY_value, dtype=np.float64) @ np.asarray(W, dtype=np.float64)
