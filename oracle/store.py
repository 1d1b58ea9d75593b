"""The paper's own normalisation store: a b-bit uniform grid per token, and its reads.

Appendix "The normalization store": z, u = gamma o z (+ beta), and for each token a b-bit grid
of step s = max_j |u_j| / (2^(b-1) - 1); u_q = s floor(u / s + xi) with an independent uniform xi
per entry, so that u_q averages to u without clipping; the new rounding u_f = u + r_f uses a
separate generator stream; y = u_q W.  The backward passes du = dy W^T through the rounding and
returns dW = u_W^T dy and dgamma = sum_tokens z_g o du with (z_g, u_W) from the table "Store
policies": gain use z | u_q / gamma | u_f / gamma; weight use u | u_q | u_f | u_q + (u_f - u)
(the last is the table's U/R+eps).  Reference: gain use reads z, weight use reads u_q.

Readings taken where the text leaves the arithmetic open (both sides of the parity tests use them):
  * the step is the FP32 quotient s = fl32(amax / M), M = 2^(b-1) - 1 (s = 1 for an all-zero token);
  * the position on the grid is the FP32 quotient t = fl32(u32 / s) of the FP32 chain value u32;
  * floor(t + xi) is taken in threshold form, the same law with the generator's 32-bit word W in
    place of xi: n0 = floor(t), f = fl32(t - n0), P = floor(f 2^32), n = n0 + [W < P], so that
    P(n = n0 + 1) = f up to 2^-32 and every code is a pure function of (value, word);
  * with a bias beta (LayerNorm) a copy is turned back into z as (copy - beta) / gamma.
The entry at a token's maximum has t = fl32(amax / s), which can exceed M by one rounding; it then
rounds up to M + 1 with probability about 1e-7.  Codes are kept as small integers, not clipped.

Test infrastructure: see the package docstring.
"""
from __future__ import annotations

import numpy as np

from . import fp8, linear, mc, norm, philox

TENSOR_U = 1
READ_U, READ_R, READ_N, READ_R_EPS = 0, 1, 2, 3


def levels(bits: int) -> int:
    """M = 2^(b-1) - 1: the grid has the codes -M .. M."""
    if not 2 <= bits <= 7:
        raise ValueError("store width must be 2..7 bits")
    return (1 << (bits - 1)) - 1


def steps(u32, bits: int) -> np.ndarray:
    """Per-token step s[T] = fl32(max_j |u_j| / M); 1 for a token that is all zero."""
    u32 = np.asarray(u32, dtype=np.float32)
    amax = np.max(np.abs(u32), axis=1).astype(np.float32)
    s = (amax / np.float32(levels(bits))).astype(np.float32)
    return np.where(amax > 0, s, np.float32(1.0)).astype(np.float32)


def position(u32, s32):
    """t = fl32(u / s), n0 = floor(t), f = fl32(t - n0), P = min(floor(f 2^32), 2^32 - 1): a 32-bit
    threshold (f can round to 1 when t is a hair below an integer; P then saturates)."""
    u32 = np.asarray(u32, dtype=np.float32)
    t = (u32 / np.asarray(s32, dtype=np.float32)[:, None]).astype(np.float32)
    n0 = np.floor(t).astype(np.float32)
    f = (t - n0).astype(np.float32)
    P = np.minimum(np.floor(f.astype(np.float64) * 4294967296.0), 4294967295.0).astype(np.uint64)
    return t, n0.astype(np.int64), f, P


def codes_from_words(u32, s32, words) -> np.ndarray:
    """n = n0 + [W < P] for generator words W (same shape as u32).  int64 codes."""
    _, n0, _, P = position(u32, s32)
    return n0 + (np.asarray(words, dtype=np.uint64) < P).astype(np.int64)


def store_codes(u32, s32, seed: int, stream: int, draw: int, elem=None) -> np.ndarray:
    """Codes of the store under the generator key (seed, TENSOR_U, stream, draw).  `elem` gives the
    row-major logical indices of the entries (default: the whole tensor in order)."""
    u32 = np.asarray(u32, dtype=np.float32)
    if elem is None:
        words = philox.tensor_words(seed, TENSOR_U, stream, draw, u32.size).reshape(u32.shape)
    else:
        words = philox.element_words(seed, TENSOR_U, stream, draw, elem)
    return codes_from_words(u32, s32, words)


def value(codes, s32) -> np.ndarray:
    """u_q = s n in float64 (exact: a 24-bit step times a small integer)."""
    return np.asarray(codes, dtype=np.float64) * np.asarray(s32, dtype=np.float32).astype(np.float64)[:, None]


def expected_value(u32, s32) -> np.ndarray:
    """E[u_q] over the generator word, in closed form: s (n0 + P / 2^32)."""
    _, n0, _, P = position(u32, s32)
    return (n0.astype(np.float64) + P.astype(np.float64) / 4294967296.0) * \
        np.asarray(s32, dtype=np.float32).astype(np.float64)[:, None]


def variance(u32, s32) -> np.ndarray:
    """Var[u_q] = s^2 p (1 - p), p = P / 2^32."""
    _, _, _, P = position(u32, s32)
    p = P.astype(np.float64) / 4294967296.0
    return (np.asarray(s32, dtype=np.float32).astype(np.float64)[:, None] ** 2) * p * (1.0 - p)


def prepare(x, gamma, beta, W, dY, kind, eps, seed, bits, act_dtype="f32", grad_fmt=fp8.E5M2,
            rstd32=None, mean32=None, du=None):
    """Once per workload: the forward with its b-bit store (stream 0, draw 0), the incoming gradient
    and du.  `rstd32` / `mean32` / `du` may be supplied so that both sides of a parity test start
    from the same saved statistics and the same received gradient."""
    fw = norm.forward(x, gamma, beta, kind, eps)
    if rstd32 is None:
        rstd32 = fw["rstd"].astype(np.float32)
    if mean32 is None:
        mean32 = fw["mean"].astype(np.float32)
    u32 = norm.store_value_fp32(x, gamma, beta, kind, rstd32, mean32, None)
    s32 = steps(u32, bits)
    codes = store_codes(u32, s32, seed, philox.STREAM_FORWARD, 0)
    g = linear.incoming_gradient(dY, grad_fmt)
    if du is None:
        du = linear.dgrad(g["value"], W)
        du = linear.bf16_round(du) if act_dtype == "bf16" else du.astype(np.float32).astype(np.float64)
    return dict(fw=fw, rstd32=rstd32, mean32=mean32, u32=u32, s32=s32, codes=codes, bits=bits, dy=g,
                du=np.asarray(du, dtype=np.float64))


def copy_for(prep, read: int, seed: int, stream: int, draw: int, cols=None) -> np.ndarray:
    """The value a use reads, float64 [T, len(cols)]: u (READ_U), u_q (READ_R), u_f (READ_N) or
    u_q + (u_f - u) (READ_R_EPS); fresh roundings come from (stream, draw)."""
    u32, s32 = prep["u32"], prep["s32"]
    T, C = u32.shape
    if cols is None:
        cols = np.arange(C)
    cols = np.asarray(cols, dtype=np.int64)
    u = u32[:, cols].astype(np.float64)
    if read == READ_U:
        return u
    uq = value(prep["codes"][:, cols], s32)
    if read == READ_R:
        return uq
    elem = np.arange(T, dtype=np.uint64)[:, None] * np.uint64(C) + cols.astype(np.uint64)[None, :]
    uf = value(store_codes(u32[:, cols], s32, seed, stream, draw, elem), s32)
    if read == READ_N:
        return uf
    if read == READ_R_EPS:
        return uq + (uf - u)
    raise ValueError("unknown read")


def gain_use(x, gamma, beta, kind, eps, prep, read: int, K: int, seed: int, stream=philox.STREAM_GAIN):
    """dgamma under one read at the gain use (U, R or N), against the reference (read U).
    Returns dict(ref, mean, m2, stats)."""
    ref = norm.backward(x, gamma, beta, kind, eps, prep["du"])["dgamma"]
    if read == READ_U:
        return dict(ref=ref, mean=ref, m2=None, stats=mc.statistics(ref, None, 1, ref, False))
    if read == READ_R:
        g = norm.dgamma_from_copy(copy_for(prep, READ_R, seed, stream, 0), gamma, beta, prep["du"])
        return dict(ref=ref, mean=g, m2=None, stats=mc.statistics(g, None, 1, ref, False))
    if read != READ_N:
        raise ValueError("the gain use reads U, R or N")
    acc = mc.Welford(ref.shape)
    for k in range(K):
        acc.add(norm.dgamma_from_copy(copy_for(prep, READ_N, seed, stream, k), gamma, beta, prep["du"]))
    return dict(ref=ref, mean=acc.mean, m2=acc.m2, stats=mc.statistics(acc.mean, acc.m2, K, ref, True))


def wgrad_use(prep, read: int, K: int, seed: int, rows=None, cols=None, stream=philox.STREAM_WGRAD):
    """dW = dY^T X under one read at the weight use (U, R, N or R+eps), against the reference (read
    R), optionally on the output sub-block rows x cols.  Returns dict(ref, mean, m2, stats)."""
    dyv = prep["dy"]["value"]
    ref = linear.wgrad(dyv, copy_for(prep, READ_R, seed, stream, 0, cols), rows, None)
    if read == READ_R:
        return dict(ref=ref, mean=ref, m2=None, stats=mc.statistics(ref, None, 1, ref, False))
    if read == READ_U:
        g = linear.wgrad(dyv, copy_for(prep, READ_U, seed, stream, 0, cols), rows, None)
        return dict(ref=ref, mean=g, m2=None, stats=mc.statistics(g, None, 1, ref, False))
    acc = mc.Welford(ref.shape)
    for k in range(K):
        acc.add(linear.wgrad(dyv, copy_for(prep, read, seed, stream, k, cols), rows, None))
    return dict(ref=ref, mean=acc.mean, m2=acc.m2, stats=mc.statistics(acc.mean, acc.m2, K, ref, True))
