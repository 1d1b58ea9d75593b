"""Philox4x32-10 counter-based generator (Salmon et al., SC'11) and the per-element keying.

The paper asks only for a counter-based generator keyed on the rounding seed and a stream, with
a separate stream for a new rounding (Appendix "The forks", Appendix "The normalization
store").  The keying used here is (seed, tensor, use/stream, draw, element).

Test infrastructure: see the package docstring.
"""
from __future__ import annotations

import numpy as np

M0 = np.uint64(0xD2511F53)
M1 = np.uint64(0xCD9E8D57)
W0 = np.uint64(0x9E3779B9)
W1 = np.uint64(0xBB67AE85)
MASK = np.uint64(0xFFFFFFFF)
SH = np.uint64(32)

# streams (the "use" field of the key)
STREAM_FORWARD = 0      # the forward's own rounding, draw 0
STREAM_GAIN = 1         # fresh rounding read by the gain use
STREAM_WGRAD = 2        # fresh rounding read by the weight-gradient use
STREAM_DX = 3           # fresh rounding read by the input-gradient use
STREAM_ATTN_D = 4       # fresh rounding read by attention's correction term D
STREAM_SHARED = 255     # one fresh draw handed to several uses (the paper's N/N)


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Ten rounds of Philox-4x32.  All arguments broadcastable uint32-valued arrays (any int
    dtype); returns four uint32 arrays.

    One round: (hi0, lo0) = M0 * c0, (hi1, lo1) = M1 * c2 as 32x32->64 products; the new counter
    is (hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0); the key is bumped by the Weyl constants between
    rounds.
    """
    c0 = np.asarray(c0).astype(np.uint64) & MASK
    c1 = np.asarray(c1).astype(np.uint64) & MASK
    c2 = np.asarray(c2).astype(np.uint64) & MASK
    c3 = np.asarray(c3).astype(np.uint64) & MASK
    k0 = np.asarray(k0).astype(np.uint64) & MASK
    k1 = np.asarray(k1).astype(np.uint64) & MASK
    for r in range(10):
        p0 = M0 * c0
        p1 = M1 * c2
        hi0, lo0 = p0 >> SH, p0 & MASK
        hi1, lo1 = p1 >> SH, p1 & MASK
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
        if r < 9:
            k0 = (k0 + W0) & MASK
            k1 = (k1 + W1) & MASK
    return (c0.astype(np.uint32), c1.astype(np.uint32), c2.astype(np.uint32), c3.astype(np.uint32))


def element_words(seed: int, tensor_id: int, stream: int, draw: int, elem) -> np.ndarray:
    """The 32-bit random word of each element.

    Element with row-major logical index e of tensor `tensor_id` uses word (e & 3) of
    philox(counter = (lo32(e >> 2), hi32(e >> 2), draw, (tensor_id << 8) | stream),
           key = (lo32(seed), hi32(seed))).
    The word depends on nothing else, so any sub-block of a tensor can be regenerated alone.
    """
    e = np.asarray(elem, dtype=np.uint64)
    q = e >> np.uint64(2)
    c0 = q & MASK
    c1 = q >> SH
    c2 = np.uint64(draw & 0xFFFFFFFF)
    c3 = np.uint64(((tensor_id << 8) | (stream & 0xFF)) & 0xFFFFFFFF)
    k0 = np.uint64(seed & 0xFFFFFFFF)
    k1 = np.uint64((seed >> 32) & 0xFFFFFFFF)
    w = philox4x32_10(c0, c1, c2, c3, k0, k1)
    lane = (e & np.uint64(3)).astype(np.int64)
    out = np.where(lane == 0, w[0], np.where(lane == 1, w[1], np.where(lane == 2, w[2], w[3])))
    return out.astype(np.uint32)


def tensor_words(seed: int, tensor_id: int, stream: int, draw: int, n: int) -> np.ndarray:
    """Words of elements 0..n-1 of a tensor, in order: the same values as `element_words` on
    arange(n), with each Philox block evaluated once for its four elements."""
    nq = (n + 3) // 4
    q = np.arange(nq, dtype=np.uint64)
    w = philox4x32_10(q & MASK, q >> SH, np.uint64(draw & 0xFFFFFFFF),
                      np.uint64(((tensor_id << 8) | (stream & 0xFF)) & 0xFFFFFFFF),
                      np.uint64(seed & 0xFFFFFFFF), np.uint64((seed >> 32) & 0xFFFFFFFF))
    return np.stack(w, axis=1).reshape(-1)[:n].astype(np.uint32)
