"""Rounded attention probabilities as the saved tensor: one row, two uses.

Appendix "Theory" (Theorem "No shared substitute serves both uses of attention probabilities";
"The errors of four policies, predicted and enumerated exactly"; "One new rounding suffices at the
softmax's backward").  One row of attention has probabilities p = softmax(s) and values V (rows
v_j).  The forward rounds p to p_q = p + r and outputs o = V^T p_q.  With the loss
L = (1/2) ||o||^2 the row's incoming gradient is h = o and dp = V h = G p_q, G = V V^T.  The
reference computes dV = p_q h^T and ds = J(p) dp, J(x) = diag(x) - x x^T.  A policy reads a vector
p_hat at the gradient of V and a matrix J_hat at the softmax's backward; its errors are
Delta_V = (p_hat - p_q) h^T and Delta_s = (J_hat - J(p)) dp.

Everything here is exact: rationals (fractions.Fraction), every rounding outcome enumerated with its
probability, each backward formed from its operands and not from the closed forms.  The closed
forms of the paper's table are separate functions, used by the tests as pins.

Test infrastructure: see the package docstring.
"""
from __future__ import annotations

import itertools
from fractions import Fraction as Fr

# ----------------------------------------------------------------------------- tiny exact linear algebra


def vec(xs):
    return [Fr(x) for x in xs]


def matvec(M, x):
    return [sum(a * b for a, b in zip(row, x)) for row in M]


def outer(x, y):
    return [[a * b for b in y] for a in x]


def transpose(M):
    return [list(c) for c in zip(*M)]


def J(x):
    """diag(x) - x x^T."""
    n = len(x)
    return [[(x[i] if i == j else Fr(0)) - x[i] * x[j] for j in range(n)] for i in range(n)]


def K_op(a):
    """diag(a (1^T a)) - a a^T: the one-copy operator, built from products of different entries."""
    n, tot = len(a), sum(a)
    return [[(a[i] * tot if i == j else Fr(0)) - a[i] * a[j] for j in range(n)] for i in range(n)]


def J2(a, b):
    """diag((a + b) / 2) - (a b^T + b a^T) / 2: the two-copy operator."""
    n = len(a)
    return [[((a[i] + b[i]) / 2 if i == j else Fr(0)) - (a[i] * b[j] + b[i] * a[j]) / 2 for j in range(n)]
            for i in range(n)]


def msub(A, B):
    return [[a - b for a, b in zip(ra, rb)] for ra, rb in zip(A, B)]


# ----------------------------------------------------------------------------- cells and rounding laws

CELL_A = dict(p=vec([Fr(2, 5), Fr(1, 4), Fr(1, 5), Fr(3, 20)]),
              V=[vec(r) for r in ([1, 0, 2], [0, 1, -1], [2, -1, 1], [3, 1, 0])], grid=Fr(1, 8))
CELL_B = dict(p=vec([Fr(1, 2), Fr(3, 10), Fr(1, 5)]),
              V=[vec(r) for r in ([1, 1], [2, -1], [0, 3])], grid=Fr(1, 6))


def law_stochastic(p, grid):
    """Per entry the outcomes (error, probability) of stochastic rounding to a grid of the given
    spacing: the two neighbouring grid points with probabilities that make the error zero on average;
    an entry on the grid is never rounded."""
    out = []
    for x in p:
        lo = (x / grid).__floor__() * grid
        f = (x - lo) / grid
        out.append([(Fr(0), Fr(1))] if f == 0 else [(lo - x, 1 - f), (lo + grid - x, f)])
    return out


def law_symmetric(p, eps):
    """r_j = +-eps, each sign with probability one half (third moments zero)."""
    return [[(-Fr(eps), Fr(1, 2)), (Fr(eps), Fr(1, 2))] for _ in p]


def outcomes(law):
    """Every joint outcome (error vector, probability) of independent entries."""
    for combo in itertools.product(*law):
        prob = Fr(1)
        for _, q in combo:
            prob *= q
        yield [e for e, _ in combo], prob


def moments(law):
    """Per entry (variance, third moment) of the error."""
    s2 = [sum(q * e * e for e, q in ent) for ent in law]
    m3 = [sum(q * e ** 3 for e, q in ent) for ent in law]
    return s2, m3


# ----------------------------------------------------------------------------- policies

# what the softmax's backward reads / what the gradient of V reads; "q" the forward's rounding,
# "f" and "b" new roundings, "u" the original
POLICIES = {
    "U/R": ("J(u)", "q"), "R/R": ("J(q)", "q"), "U/U": ("J(u)", "u"), "N/N": ("J(f)", "f"), "R/U": ("J(q)", "u"),
    # operators of the section "One new rounding suffices at the softmax's backward", each with p_q at dV
    "K(f)/R": ("K(f)", "q"), "J2(f,b)/R": ("J2(f,b)", "q"), "J2(q,b)/R": ("J2(q,b)", "q"),
}


def average_errors(cell, law, policy, per_draw=False):
    """E[Delta_s | F] (n-vector) and E[Delta_V | F] (n x d) of one policy, by enumeration over the
    forward's rounding and over as many new roundings as the policy uses.  With per_draw also returns
    whether each error is zero in every outcome."""
    p, V = cell["p"], cell["V"]
    n, d = len(p), len(V[0])
    Vt = transpose(V)
    Jp = J(p)
    j_read, v_read = POLICIES[policy]
    needs_f = "f" in j_read or v_read == "f"
    needs_b = "b" in j_read
    Es = [Fr(0)] * n
    EV = [[Fr(0)] * d for _ in range(n)]
    zero_s = zero_V = True
    one = [([Fr(0)] * n, Fr(1))]
    for r, pr in outcomes(law):
        pq = [a + b for a, b in zip(p, r)]
        h = matvec(Vt, pq)                       # o = V^T p_q, and h = o under L = ||o||^2 / 2
        dp = matvec(V, h)
        for rf, pf_ in (outcomes(law) if needs_f else one):
            pf = [a + b for a, b in zip(p, rf)]
            for rb, pb_ in (outcomes(law) if needs_b else one):
                pb = [a + b for a, b in zip(p, rb)]
                w = pr * pf_ * pb_
                Jhat = {"J(u)": lambda: Jp, "J(q)": lambda: J(pq), "J(f)": lambda: J(pf), "K(f)": lambda: K_op(pf),
                        "J2(f,b)": lambda: J2(pf, pb), "J2(q,b)": lambda: J2(pq, pb)}[j_read]()
                phat = {"q": pq, "u": p, "f": pf}[v_read]
                ds = matvec(msub(Jhat, Jp), dp)
                dV = outer([a - b for a, b in zip(phat, pq)], h)
                zero_s &= all(x == 0 for x in ds)
                zero_V &= all(x == 0 for row in dV for x in row)
                Es = [a + w * b for a, b in zip(Es, ds)]
                EV = [[a + w * b for a, b in zip(ra, rb_)] for ra, rb_ in zip(EV, dV)]
    return (Es, EV, zero_s, zero_V) if per_draw else (Es, EV)


# ----------------------------------------------------------------------------- the paper's closed forms


def closed_forms(cell, law):
    """delta of the replayed rounding, -Sigma_r G p of a plugged-in new rounding, the half-replayed
    J2 error, and the rows -sigma_j^2 v_j^T at the gradient of V."""
    p, V = cell["p"], cell["V"]
    n = len(p)
    G = [[sum(a * b for a, b in zip(V[i], V[j])) for j in range(n)] for i in range(n)]
    g = [G[i][i] for i in range(n)]
    s2, m3 = moments(law)
    tau = sum(gk * sk for gk, sk in zip(g, s2))
    Gp = matvec(G, p)
    SGp = [s2[i] * Gp[i] for i in range(n)]
    delta = [g[i] * s2[i] - tau * p[i] - 2 * SGp[i] - g[i] * m3[i] for i in range(n)]
    half = [(g[i] * s2[i] - tau * p[i] - SGp[i]) / 2 for i in range(n)]
    dV = [[-s2[j] * x for x in V[j]] for j in range(n)]
    return dict(delta=delta, minus_SGp=[-x for x in SGp], half_replay=half, dV_rows=dV)


# ----------------------------------------------------------------------------- Monte-Carlo form (float64)
#
# The same quantities for many rows at once, over seeded draws instead of every outcome: the form
# the GPU path evaluates.  p[R, n] rows of probabilities, V[n, d] shared values.  Per draw k the
# forward's rounding comes from generator stream 0, the new roundings a and b from streams 1 and 2
# (tensor id TENSOR_P, element = row * n + entry, draw = k).  Laws: LAW_GRID, stochastic rounding to
# a uniform grid of spacing `param` in threshold form (t = fl32(p / param), up iff W < floor(frac(t)
# 2^32)); LAW_SIGN, r = +param when the top bit of W is set, else -param.

import numpy as np  # noqa: E402

from . import philox  # noqa: E402

TENSOR_P = 4
LAW_GRID, LAW_SIGN = 0, 1
OPERATORS = ("J(q)", "J(f)", "K(f)", "J2(f,b)", "J2(q,b)")        # read at the softmax's backward
V_READS = ("u", "f")                                               # read at the gradient of V (p_q is exact)


def rounded(p32, law: int, param: float, seed: int, stream: int, draw: int, first_row: int = 0) -> np.ndarray:
    """One rounding of every entry of p32[R, n] (float64 result).  The rows are rows first_row ..
    first_row + R - 1 of the whole tensor: an entry's word is keyed by its index there."""
    p32 = np.asarray(p32, dtype=np.float32)
    if first_row == 0:
        w = philox.tensor_words(seed, TENSOR_P, stream, draw, p32.size).reshape(p32.shape)
    else:
        idx = np.arange(first_row * p32.shape[1], (first_row + p32.shape[0]) * p32.shape[1], dtype=np.uint64)
        w = philox.element_words(seed, TENSOR_P, stream, draw, idx).reshape(p32.shape)
    if law == LAW_SIGN:
        return p32.astype(np.float64) + np.where((w >> np.uint64(31)) & np.uint64(1), param, -param)
    g = np.float32(param)
    t = (p32 / g).astype(np.float32)
    n0 = np.floor(t).astype(np.float32)
    f = (t - n0).astype(np.float32)
    P = np.minimum(np.floor(f.astype(np.float64) * 4294967296.0), 4294967295.0).astype(np.uint64)
    return (n0.astype(np.float64) + (w < P)) * float(g)


def apply_J(x, dp):
    return x * dp - x * np.sum(x * dp, axis=1, keepdims=True)


def apply_K(a, dp):
    return a * np.sum(a, axis=1, keepdims=True) * dp - a * np.sum(a * dp, axis=1, keepdims=True)


def apply_J2(a, b, dp):
    return 0.5 * (a + b) * dp - 0.5 * (a * np.sum(b * dp, axis=1, keepdims=True) + b * np.sum(a * dp, axis=1, keepdims=True))


def mc_sums(p32, V, law: int, param: float, seed: int, K: int, draw0: int = 0, first_row: int = 0):
    """Sums over draws draw0 .. draw0 + K - 1 of the errors Delta_s (per operator of OPERATORS,
    [5, R, n]) and Delta_V (per read of V_READS, [2, R, n, d]), and of the squares of Delta_s.
    first_row: where these rows sit in the whole tensor (rows are independent but for their keys)."""
    p = np.asarray(p32, dtype=np.float32).astype(np.float64)
    V = np.asarray(V, dtype=np.float64)
    R, n = p.shape
    ds = np.zeros((len(OPERATORS), R, n))
    ds2 = np.zeros_like(ds)
    dV = np.zeros((len(V_READS), R, n, V.shape[1]))
    for k in range(draw0, draw0 + K):
        pq = rounded(p32, law, param, seed, 0, k, first_row)
        pf = rounded(p32, law, param, seed, 1, k, first_row)
        pb = rounded(p32, law, param, seed, 2, k, first_row)
        h = pq @ V                                  # o = V^T p_q row by row; h = o
        dp = h @ V.T
        ref = apply_J(p, dp)
        errs = (apply_J(pq, dp), apply_J(pf, dp), apply_K(pf, dp), apply_J2(pf, pb, dp), apply_J2(pq, pb, dp))
        for i, e in enumerate(errs):
            ds[i] += e - ref
            ds2[i] += (e - ref) ** 2
        dV[0] += (p - pq)[:, :, None] * h[:, None, :]
        dV[1] += (pf - pq)[:, :, None] * h[:, None, :]
    return ds, ds2, dV


def closed_forms_rows(p32, V, law: int, param: float):
    """The paper's closed forms row by row (float64): delta, -Sigma_r G p, the half-replayed J2 error
    and the rows -sigma_j^2 v_j^T, from the law's exact per-entry variance and third moment."""
    p32 = np.asarray(p32, dtype=np.float32)
    p = p32.astype(np.float64)
    V = np.asarray(V, dtype=np.float64)
    if law == LAW_SIGN:
        s2, m3 = np.full_like(p, param * param), np.zeros_like(p)
    else:
        g = np.float32(param)
        t = (p32 / g).astype(np.float32)
        n0 = np.floor(t).astype(np.float32)
        f = (t - n0).astype(np.float32)
        pu = np.minimum(np.floor(f.astype(np.float64) * 4294967296.0), 4294967295.0) / 4294967296.0
        lo = n0.astype(np.float64) * float(g)
        mean = lo + pu * float(g)                   # the law's own mean (p up to the FP32 quotient's rounding)
        e_lo, e_hi = lo - mean, lo + float(g) - mean
        s2 = (1 - pu) * e_lo ** 2 + pu * e_hi ** 2
        m3 = (1 - pu) * e_lo ** 3 + pu * e_hi ** 3
    G = V @ V.T
    gd = np.diag(G)[None, :]
    Gp = p @ G
    tau = np.sum(gd * s2, axis=1, keepdims=True)
    delta = gd * s2 - tau * p - 2 * s2 * Gp - gd * m3
    half = 0.5 * (gd * s2 - tau * p - s2 * Gp)
    dV_rows = -s2[:, :, None] * V[None, :, :]
    return dict(delta=delta, minus_SGp=-s2 * Gp, half_replay=half, dV_rows=dV_rows, s2=s2)
