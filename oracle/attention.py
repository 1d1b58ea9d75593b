"""Causal softmax attention: forward statistics and the backward whose correction term D reads
a copy of the saved output.

Section "Same rounding distribution, opposite outcomes": P = softmax(S), O = P V;
dV = P^T dO, dP = dO V^T, dS = P o (dP - D), D = rowsum(P o dP) = rowsum(dO o O); reading a copy
O + E adds rowsum(dO o E) (Eq. dterm).  dQ = c dS K, dK = c dS^T Q with c the softmax scale.
The FP8-operand mode follows the emulated backward of Appendix "The forks": dO cast to E5M2,
P recomputed from the dequantised Q and K, dV = P_q^T dO with P_q rounded at a forward scale,
dP = dO V^T, D from the assigned output copy, dS = P o (dP - D), dS cast to E5M2 at a supplied
scale before the last two products.  Its quantisation points and the P / dS scales are this
build's reading of that prose: parity unpinned.

All functions work on one (batch, head) slice: q, k, v, dO are [S, d] arrays.
Test infrastructure: see the package docstring.
"""
from __future__ import annotations

import numpy as np

from . import fp8


def probabilities(q, k, c: float, causal: bool = True):
    """S = c Q K^T (keys j > i masked when causal), P = softmax(S) row by row,
    LSE_i = log sum_j exp(S_ij).  float64.  Returns (P, LSE)."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    s = c * (q @ k.T)
    if causal:
        n, m = s.shape
        mask = np.arange(m)[None, :] > np.arange(n)[:, None]
        s = np.where(mask, -np.inf, s)
    mx = np.max(s, axis=1, keepdims=True)
    e = np.exp(s - mx)
    den = np.sum(e, axis=1, keepdims=True)
    p = e / den                      # the softmax itself; exact when every score is equal
    lse = mx[:, 0] + np.log(den[:, 0])
    return p, lse


def quantise_rn(a, fmt: int, scale=None):
    """Nearest rounding of one slice at a per-slice scale (from its own amax unless given).
    Returns (value float64, codes, scale32, inv_scale32)."""
    a32 = np.asarray(a, dtype=np.float32)
    if scale is None:
        amax = np.float32(np.max(np.abs(a32))) if a32.size else np.float32(0)
        scale, inv = fp8.scale_from_amax(amax, fmt)
    else:
        scale = np.float32(scale)
        inv = np.float32(np.float32(1.0) / scale)
    codes, _, _ = fp8.encode((a32 * np.float32(scale)).astype(np.float32), fmt, fp8.RN)
    return fp8.decode(codes, fmt) * float(inv), codes, np.float32(scale), np.float32(inv)


def forward_output(q, k, v, c: float, causal: bool = True):
    """O = P V in float64 from the operands exactly as the backward will see them, with P
    unrounded, and the LSE.  Returns (O, LSE)."""
    p, lse = probabilities(q, k, c, causal)
    return p @ np.asarray(v, dtype=np.float64), lse


def backward(q, k, v, dO, c: float, o_copy, causal: bool = True, fp8_operands: bool = False,
             scale_p: float = 256.0, scale_ds=None, operand_round=None):
    """Attention backward for one slice with D = rowsum(dO o o_copy).

    BF16-operand mode (fp8_operands False): every product in float64 on the given operands.
    `operand_round` (e.g. rounding to bf16), when given, is applied to the two computed operands
    of the last three products -- P before dV = P^T dO, dS before dQ = c dS K and dK = c dS^T Q --
    as a tensor-core contraction in that operand type does; None keeps them unrounded.
    FP8-operand mode: q, k, v must already be the dequantised E4M3 operands and dO the
    dequantised E5M2 gradient; P_q = RN_E4M3(P scale_p) / scale_p feeds dV, and
    dS_q = RN_E5M2(dS scale_ds) / scale_ds feeds dQ and dK.
    Returns dict(dq, dk, dv, D, dS).
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    dO = np.asarray(dO, dtype=np.float64)
    p, _ = probabilities(q, k, c, causal)
    D = np.sum(dO * np.asarray(o_copy, dtype=np.float64), axis=1)
    dP = dO @ v.T
    dS = p * (dP - D[:, None])
    if fp8_operands:
        p_dv, _, _, _ = quantise_rn(p, fp8.E4M3, scale=scale_p)
        if scale_ds is None:
            raise ValueError("the FP8-operand mode needs the caller's dS scale")
        dS_mm, _, _, _ = quantise_rn(dS, fp8.E5M2, scale=scale_ds)
    elif operand_round is not None:
        p_dv, dS_mm = operand_round(p), operand_round(dS)
    else:
        p_dv, dS_mm = p, dS
    dv = p_dv.T @ dO
    dq = c * (dS_mm @ k)
    dk = c * (dS_mm.T @ q)
    return dict(dq=dq, dk=dk, dv=dv, D=D, dS=dS)


def d_from_probabilities(q, k, v, dO, c: float, causal: bool = True):
    """The control of Eq. dterm: D = rowsum(P o dP), reading no copy of O."""
    p, _ = probabilities(q, k, c, causal)
    dP = np.asarray(dO, dtype=np.float64) @ np.asarray(v, dtype=np.float64).T
    return np.sum(p * dP, axis=1)
