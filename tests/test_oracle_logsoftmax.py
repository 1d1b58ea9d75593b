"""Pins of the log-softmax test (Appendix "Log-softmax"): the per-entry errors of the operator's
backward against the stated formulas, the exact constants cosh(eps) - 1 and -eps sinh(eps) by
enumeration over every sign pattern, and the registered statements at the paper's sizes."""
import itertools

import numpy as np
import pytest

from oracle import logsoftmax as ls


def test_backward_is_the_softmax_jacobian_transpose():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((3, 5))
    h = rng.standard_normal((3, 5))
    l = ls.log_softmax(x)
    g = ls.backward(h, l)
    # finite differences of sum(h * log_softmax(x)) with h held constant
    for i in range(3):
        for j in range(5):
            d = np.zeros_like(x); d[i, j] = 1e-6
            fd = (np.sum(h * ls.log_softmax(x + d)) - np.sum(h * ls.log_softmax(x - d))) / 2e-6
            assert abs(fd - g[i, j]) < 1e-8
    assert np.allclose(np.sum(np.exp(l), axis=1), 1.0)


@pytest.mark.parametrize("eps", [0.1, 0.5])
def test_exact_constants_by_enumeration(eps):
    """Every sign pattern of a 3-class row (and of an independent copy): the averages of the per-entry
    errors over p_j are cosh(eps) - 1 under the likelihood (either copy), -eps sinh(eps) under the
    constructed loss with reuse, zero with an independent copy, and the calibrated variants."""
    l = ls.log_softmax(np.array([[0.3, -1.2, 0.8]]))
    p = np.exp(l)
    h_lik = np.array([[0.0, -1.0, 0.0]])
    c = np.cosh(eps)
    acc = np.zeros(6)
    pats = [np.array([s]) * eps for s in itertools.product((-1.0, 1.0), repeat=3)]
    for r in pats:
        for r2 in pats:
            for i, (h, S, sc) in enumerate(((h_lik, l + r, 1.0), (h_lik, l + r2, 1.0), (r, l + r, 1.0), (r, l + r2, 1.0),
                                            (h_lik, l + r, c), (r, l + r, c))):
                acc[i] += np.mean((ls.backward(h, S, sc) - ls.backward(h, l)) / p)
    acc /= len(pats) ** 2
    assert np.allclose(acc, ls.predicted(eps)[:6], rtol=0, atol=1e-14)
    # the entry formulas themselves
    r = pats[5]
    assert np.allclose((ls.backward(h_lik, l + r) - ls.backward(h_lik, l)) / p, np.exp(r) - 1)
    assert np.allclose((ls.backward(r, l + r) - ls.backward(r, l)) / p, -(np.exp(r) - 1) * np.sum(r))
    # the constants are not their leading terms (the second configuration's statements)
    assert abs((c - 1) / (eps * eps / 2) - 1) > (0.01 if eps == 0.5 else 0.0005)
    assert abs((-eps * np.sinh(eps)) / (-eps * eps) - 1) > (0.02 if eps == 0.5 else 0.001)


def test_errors_are_signs_of_the_keyed_generator():
    r = ls.errors(4, 8, 7, 0, 3, 0.25)
    assert set(np.unique(r)) == {-0.25, 0.25}
    assert np.array_equal(r, ls.errors(4, 8, 7, 0, 3, 0.25))
    assert not np.array_equal(r, ls.errors(4, 8, 7, 1, 3, 0.25)) and not np.array_equal(r, ls.errors(4, 8, 7, 0, 4, 0.25))
    big = ls.errors(64, 128, 1, 0, 0, 1.0)
    assert abs(big.mean()) < 4 / np.sqrt(big.size)


@pytest.mark.parametrize("eps,trials", [(0.1, 1024), (0.5, 512)])
def test_registered_statements_at_the_papers_sizes(eps, trials):
    """128 classes, 64 rows (the paper ran 4096 trials; fewer here keep the test short, the rules
    are the paper's): LS1 reuse changes nothing under the likelihood, LS2 the mean error is
    cosh(eps) - 1, LS3 reuse shifts the constructed loss's error by -eps sinh(eps), LS4 the independent
    copy's mean error is zero there, LS5a / LS5b the division by cosh(eps)."""
    rng = np.random.default_rng(1926)
    logits = rng.standard_normal((64, 128))
    target = rng.integers(0, 128, 64)
    v, (mean, se, z) = ls.run(logits, target, eps, 1926, trials)
    pred = ls.predicted(eps)
    effect = abs(pred[2])
    assert abs(mean[6]) + 1.96 * se[6] < 0.05 * effect                      # LS1 / LS1'
    assert abs(mean[0] / pred[0] - 1) < 0.02 and z[0] > 5                   # LS2
    assert abs(mean[2] / pred[2] - 1) < 0.05 and z[2] > 5                   # LS3
    assert abs(mean[3]) + 1.96 * se[3] < 0.10 * pred[0] or z[3] < 3         # LS4 / LS4' (an equivalence test)
    assert abs(mean[4]) + 1.96 * se[4] < 0.05 * pred[0]                     # LS5a
    assert abs(mean[5] / pred[2] - 1 / np.cosh(eps)) < 0.05                 # LS5b: the coupling stays, scaled
    # under the likelihood the per-trial statistic is the mean of e^{r_j} - 1 exactly (LS6's identity)
    r = ls.errors(64, 128, 1926, 0, 0, eps)
    assert abs(v[0, 0] - np.mean(np.exp(r) - 1)) < 1e-13
