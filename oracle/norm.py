"""Normalisation store: forward, the three reads of the saved tensor, backward.

Follows Section "The original matches the reference at only one use" (Eq. norm-uses) and
Appendix "The normalization store": z, u = gamma o z (+ beta), u_q = round(u), y = u_q W; the
backward passes du through the rounding unchanged and returns dgamma = sum_tokens z_g o du and
the input gradient from unrounded values; z_g follows the policy table (z, u_q/gamma,
u_f/gamma).

float64 throughout, except `store_value_fp32`, which pins the *value being rounded* to a fixed
chain of FP32 operations so that codes are reproducible bit for bit.

Test infrastructure: see the package docstring.
"""
from __future__ import annotations

import numpy as np

from . import fp8, philox

RMS = 0
LAYER = 1

READ_ORIGINAL = 0   # U
READ_FORWARD = 1    # R
READ_FRESH = 2      # N


def forward(x, gamma, beta, kind: int, eps: float):
    """Row statistics and the normalised tensors in float64.

    RMSNorm: ms = mean_j x_j^2, rstd = 1/sqrt(ms + eps), z = x rstd, u = gamma o z.
    LayerNorm: mu = mean x, var = mean (x - mu)^2 (biased), rstd = 1/sqrt(var + eps),
    z = (x - mu) rstd, u = gamma o z + beta.
    Returns dict(z, u, rstd, mean).
    """
    x = np.asarray(x, dtype=np.float64)
    gamma = np.asarray(gamma, dtype=np.float64)
    if kind == RMS:
        ms = np.mean(x * x, axis=1)
        rstd = 1.0 / np.sqrt(ms + eps)
        mean = np.zeros_like(rstd)
        z = x * rstd[:, None]
        u = gamma[None, :] * z
    else:
        mean = np.mean(x, axis=1)
        xc = x - mean[:, None]
        var = np.mean(xc * xc, axis=1)
        rstd = 1.0 / np.sqrt(var + eps)
        z = xc * rstd[:, None]
        u = gamma[None, :] * z + np.asarray(beta, dtype=np.float64)[None, :]
    return dict(z=z, u=u, rstd=rstd, mean=mean)


def store_value_fp32(x, gamma, beta, kind: int, rstd32, mean32, scale32=None):
    """The FP32 value handed to the rounding, one IEEE single operation per step, no FMA:
    RMS   v = fl(fl(fl(x * rstd) * gamma) * scale)
    LN    v = fl(fl(fl(fl(fl(x - mu) * rstd) * gamma) + beta) * scale)
    from the *saved* FP32 statistics.  With scale32=None the chain stops before the scaling
    (that value's largest magnitude is the amax the scale is derived from).
    """
    x32 = np.asarray(x, dtype=np.float32)
    g32 = np.asarray(gamma, dtype=np.float32)[None, :]
    r32 = np.asarray(rstd32, dtype=np.float32)[:, None]
    if kind == RMS:
        v = (x32 * r32).astype(np.float32)
        v = (v * g32).astype(np.float32)
    else:
        m32 = np.asarray(mean32, dtype=np.float32)[:, None]
        b32 = np.asarray(beta, dtype=np.float32)[None, :]
        v = (x32 - m32).astype(np.float32)
        v = (v * r32).astype(np.float32)
        v = (v * g32).astype(np.float32)
        v = (v + b32).astype(np.float32)
    if scale32 is not None:
        v = (v * np.float32(scale32)).astype(np.float32)
    return v


def store_codes(v32, fmt: int, mode: int, seed: int, tensor_id: int, stream: int, draw: int,
                elem=None):
    """Codes of the scaled FP32 values `v32` under the given rounding law and key.  `elem`
    gives the row-major logical indices of the entries (default: the whole tensor in order), so
    a sub-block gets exactly the words it has inside the full tensor."""
    v32 = np.asarray(v32, dtype=np.float32)
    if mode == fp8.SR:
        if elem is None:
            words = philox.tensor_words(seed, tensor_id, stream, draw, v32.size).reshape(v32.shape)
        else:
            words = philox.element_words(seed, tensor_id, stream, draw, elem)
    else:
        words = None
    return fp8.encode(v32, fmt, mode, words)


def read_value(codes, fmt: int, inv_scale32) -> np.ndarray:
    """Value a use reads from stored codes: decode(code) * inv_scale, float64."""
    return fp8.decode(codes, fmt) * float(np.float32(inv_scale32))


def backward(x, gamma, beta, kind: int, eps: float, du, gain_copy=None, dx_copy=None):
    """Gradients of the normalisation with the incoming gradient `du` passed through the
    rounding unchanged.

    gain_copy / dx_copy: the copy of u (float64, [T, C]) that the gain use / input-gradient use
    reads, or None for the original.  A copy is turned back into z as (copy - beta) / gamma
    (plain division; "for nonzero gamma").
    dgamma = sum_t z_g o du; dbeta = sum_t du (reads no saved tensor);
    dz = gamma o du; RMS: dx = rstd (dz - z mean_j(dz o z));
    LN: dx = rstd (dz - mean_j dz - z mean_j(dz o z)).
    Returns dict(dgamma, dbeta, dx).
    """
    fw = forward(x, gamma, beta, kind, eps)
    gamma = np.asarray(gamma, dtype=np.float64)
    b = np.zeros_like(gamma) if beta is None else np.asarray(beta, dtype=np.float64)
    du = np.asarray(du, dtype=np.float64)
    z = fw["z"]
    z_g = z if gain_copy is None else (np.asarray(gain_copy, np.float64) - b[None, :]) / gamma[None, :]
    z_x = z if dx_copy is None else (np.asarray(dx_copy, np.float64) - b[None, :]) / gamma[None, :]
    dgamma = np.sum(z_g * du, axis=0)
    dbeta = np.sum(du, axis=0)
    dz = gamma[None, :] * du
    rstd = fw["rstd"][:, None]
    proj = np.mean(dz * z_x, axis=1, keepdims=True)
    if kind == RMS:
        dx = rstd * (dz - z_x * proj)
    else:
        dx = rstd * (dz - np.mean(dz, axis=1, keepdims=True) - z_x * proj)
    return dict(dgamma=dgamma, dbeta=dbeta, dx=dx)


def dgamma_from_copy(copy, gamma, beta, du) -> np.ndarray:
    """The gain gradient alone, reading a copy of u: sum_t ((copy - beta) / gamma) o du."""
    gamma = np.asarray(gamma, dtype=np.float64)
    b = np.zeros_like(gamma) if beta is None else np.asarray(beta, dtype=np.float64)
    z_g = (np.asarray(copy, dtype=np.float64) - b[None, :]) / gamma[None, :]
    return np.sum(z_g * np.asarray(du, dtype=np.float64), axis=0)
