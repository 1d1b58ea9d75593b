"""Log-softmax backward with a +-eps error injected into its saved output.

Appendix "Log-softmax": the operator's backward takes the incoming gradient h and the saved
output S and returns h - exp(S) (1^T h).  The saved output is S = l + r with l the exact output
and r_j = +-eps independently with equal probability; under reuse the backward reads this S, under
an independent copy it reads l + r' with r' drawn anew.  With p = exp(l), g the returned gradient
and g* what the operator returns from l with the same h, the statistic averages (g_j - g*_j) / p_j
over rows and classes.  Two losses: the negative log-likelihood with a fixed target, h = -e_y; and
the constructed loss (1/2) ||S - l||^2 with l held constant, h = r.  Predictions: under the
likelihood each entry's error over p_j is e^{r_j} - 1, mean cosh(eps) - 1 for either copy; under
the constructed loss it is -(e^{r_j} - 1) sum_k r_k, mean -eps sinh(eps) under reuse and zero for
the independent copy; dividing the reconstruction exp(S) by cosh(eps) removes the likelihood's mean
error and leaves the constructed loss's effect of reuse scaled by 1 / cosh(eps).

Readings: r_j = +eps when the top bit of the element's generator word is set, -eps otherwise; the
consumed error comes from stream 0 and the independent copy from stream 1 of the same key, the
trial index is the draw; element index = row * classes + class.

Test infrastructure: see the package docstring.
"""
from __future__ import annotations

import numpy as np

from . import philox

TENSOR_S = 3
STATS = ("likelihood_reuse", "likelihood_independent", "constructed_reuse", "constructed_independent",
         "likelihood_reuse_calibrated", "constructed_reuse_calibrated")


def log_softmax(x):
    x = np.asarray(x, dtype=np.float64)
    m = np.max(x, axis=1, keepdims=True)
    return x - m - np.log(np.sum(np.exp(x - m), axis=1, keepdims=True))


def backward(h, S, scale: float = 1.0):
    """The operator's backward from a saved output S: h - exp(S) / scale * (1^T h), row by row."""
    h = np.asarray(h, dtype=np.float64)
    return h - np.exp(np.asarray(S, dtype=np.float64)) / scale * np.sum(h, axis=1, keepdims=True)


def errors(rows: int, classes: int, seed: int, stream: int, trial: int, eps: float) -> np.ndarray:
    """r[rows, classes]: +eps where the top bit of the element's word is set, else -eps."""
    w = philox.tensor_words(seed, TENSOR_S, stream, trial, rows * classes).reshape(rows, classes)
    return np.where((w >> np.uint64(31)) & np.uint64(1), eps, -eps).astype(np.float64)


def trial_statistics(logits, target, eps: float, seed: int, trial: int) -> np.ndarray:
    """The six per-trial statistics (mean over rows and classes of (g - g*) / p), in the order of
    STATS, each formed from the operator's backward, not from the closed forms."""
    l = log_softmax(logits)
    R, n = l.shape
    p = np.exp(l)
    r = errors(R, n, seed, philox.STREAM_FORWARD, trial, eps)
    r2 = errors(R, n, seed, philox.STREAM_GAIN, trial, eps)
    h_lik = np.zeros((R, n))
    h_lik[np.arange(R), np.asarray(target)] = -1.0
    c = np.cosh(eps)
    out = []
    for h, S, scale in ((h_lik, l + r, 1.0), (h_lik, l + r2, 1.0), (r, l + r, 1.0), (r, l + r2, 1.0),
                        (h_lik, l + r, c), (r, l + r, c)):
        g, g_star = backward(h, S, scale), backward(h, l)
        out.append(np.mean((g - g_star) / p))
    return np.array(out)


def summarise(per_trial):
    """mean, standard error over trials and z = |mean| / se for each column of per_trial [trials, k]."""
    v = np.asarray(per_trial, dtype=np.float64)
    n = v.shape[0]
    mean = v.mean(axis=0)
    se = v.std(axis=0, ddof=1) / np.sqrt(n)
    with np.errstate(divide="ignore", invalid="ignore"):
        z = np.where(se > 0, np.abs(mean) / se, np.where(mean == 0, 0.0, np.inf))
    return mean, se, z


def run(logits, target, eps: float, seed: int, trials: int):
    """All trials: per-trial statistics [trials, 6] plus the two paired contrasts reuse - independent
    (likelihood, constructed) as columns 6 and 7, and their summary."""
    v = np.stack([trial_statistics(logits, target, eps, seed, t) for t in range(trials)])
    v = np.concatenate([v, (v[:, 0] - v[:, 1])[:, None], (v[:, 2] - v[:, 3])[:, None]], axis=1)
    return v, summarise(v)


def predicted(eps: float) -> np.ndarray:
    """The registered constants, in the order of run()'s columns."""
    c, s = np.cosh(eps), np.sinh(eps)
    return np.array([c - 1, c - 1, -eps * s, 0.0, 0.0, -eps * s / c, 0.0, -eps * s])
