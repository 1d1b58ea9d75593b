"""Monte-Carlo reduction over K fresh draws, the statistics and the per-use verdict.

Per-use requirement (Section "Each use has a checkable requirement"): a use reads the value its
forward operation used, or a substitute whose gradient, averaged over the substitute's own draw
with the forward and the incoming gradient held fixed, equals the reference gradient.
Statistics: z = |m| / se with the standard error taken over trials (Appendix "Checkpointing");
R = ||m||^2 / sum_j se_j^2, near one at zero mean (Appendix "The normalization store").

The verdict thresholds are this build's reading (the paper registers a separate rule per test):
parity unpinned.

Test infrastructure: see the package docstring.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

HOLDS = 0
FAILS = 1
UNDECIDED = 2

REL_TOL_DETERMINISTIC = 1e-4
QPRIME_HOLD, R_HOLD = 2.0, 3.0
QPRIME_FAIL, R_FAIL = 4.0, 6.0


class Welford:
    """Streaming per-element mean and sum of squared deviations in float64."""

    def __init__(self, shape):
        self.n = 0
        self.mean = np.zeros(shape, dtype=np.float64)
        self.m2 = np.zeros(shape, dtype=np.float64)

    def add(self, g):
        g = np.asarray(g, dtype=np.float64)
        self.n += 1
        d = g - self.mean
        self.mean += d / self.n
        self.m2 += d * (g - self.mean)

    def merge(self, other: "Welford"):
        """Combine two disjoint draw ranges (Chan et al.)."""
        if other.n == 0:
            return
        if self.n == 0:
            self.n, self.mean, self.m2 = other.n, other.mean.copy(), other.m2.copy()
            return
        n = self.n + other.n
        d = other.mean - self.mean
        self.m2 = self.m2 + other.m2 + d * d * (self.n * other.n / n)
        self.mean = self.mean + d * (other.n / n)
        self.n = n


@dataclass
class UseStats:
    K: int
    n_elements: int
    rel_l2_mean_err: float
    R: float
    Qprime: float
    mean_z: float
    rms_z: float
    max_abs_z: float
    frac_abs_z_gt3: float
    verdict: int


def statistics(mean, m2, K: int, g_ref, fresh: bool) -> UseStats:
    """Reduce per-element (mean, M2 = sum_k (g_k - mean)^2) against the reference gradient.

    s^2 = M2 / (K - 1); se^2 = s^2 / K; z_j = (m_j - g*_j) / se_j; where se_j = 0 (every draw gave
    the same value: the read is deterministic at that element) z_j = 0 if |m_j - g*_j| is within
    the deterministic tolerance of |g*_j| and +-inf otherwise; R = sum_j (m_j - g*_j)^2 / sum_j se_j^2;
    Q' = mean_j z_j^2 (K - 3) / (K - 1)  (about one at zero bias: E t^2 of a t_{K-1} is
    (K-1)/(K-3)); rel = ||m - g*||_2 / ||g*||_2.
    A deterministic read (original or forward's rounding) has K_eff = 1 and only `rel`.
    """
    mean = np.asarray(mean, dtype=np.float64).ravel()
    g_ref = np.asarray(g_ref, dtype=np.float64).ravel()
    err = mean - g_ref
    num = float(np.sqrt(np.sum(err * err)))
    den = float(np.sqrt(np.sum(g_ref * g_ref)))
    rel = 0.0 if num == 0.0 else (num / den if den > 0 else float("inf"))
    n = mean.size
    if not fresh:
        v = HOLDS if rel <= REL_TOL_DETERMINISTIC else FAILS
        return UseStats(1, n, rel, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0, v)
    m2 = np.asarray(m2, dtype=np.float64).ravel()
    se2 = m2 / (K - 1) / K
    se = np.sqrt(se2)
    with np.errstate(divide="ignore", invalid="ignore"):
        # an element whose draws all coincide is read deterministically: it is judged by the
        # deterministic rule (z = 0 within REL_TOL_DETERMINISTIC of the reference, else +-inf)
        flat = np.where(np.abs(err) <= REL_TOL_DETERMINISTIC * np.abs(g_ref), 0.0, np.sign(err) * np.inf)
        z = np.where(se == 0.0, flat, err / se)
    sum_se2 = float(np.sum(se2))
    sum_err2 = float(np.sum(err * err))
    R = 0.0 if sum_err2 == 0.0 else (sum_err2 / sum_se2 if sum_se2 > 0 else float("inf"))
    q = float(np.mean(z * z)) * (K - 3) / (K - 1)
    st = UseStats(K, n, rel, R, q, float(np.mean(z)), float(np.sqrt(np.mean(z * z))),
                  float(np.max(np.abs(z))), float(np.mean(np.abs(z) > 3.0)), UNDECIDED)
    st.verdict = verdict_fresh(q, R)
    return st


def verdict_fresh(qprime: float, R: float) -> int:
    """Three-valued verdict for a fresh read: HOLDS if Q' <= 2 and R <= 3; FAILS if Q' >= 4 or
    R >= 6; otherwise UNDECIDED."""
    if qprime >= QPRIME_FAIL or R >= R_FAIL:
        return FAILS
    if qprime <= QPRIME_HOLD and R <= R_HOLD:
        return HOLDS
    return UNDECIDED


def shifted_sums_to_moments(S1, S2, K: int, g_ref):
    """(mean, M2) from the shifted sums S1 = sum_k (g_k - g*), S2 = sum_k (g_k - g*)^2:
    mean = g* + S1 / K, M2 = S2 - S1^2 / K.  (The accumulation form of the fused GPU epilogue;
    here only to state the identity that the tests pin against Welford and two-pass.)"""
    S1 = np.asarray(S1, dtype=np.float64)
    S2 = np.asarray(S2, dtype=np.float64)
    mean = np.asarray(g_ref, dtype=np.float64) + S1 / K
    return mean, S2 - S1 * S1 / K
