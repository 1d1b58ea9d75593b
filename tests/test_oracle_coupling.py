"""Pins of the averages over the forward's rounding: the mean-error / coupling split, the paired
statistic T with its control, and the estimator X, against their closed forms under stochastic
rounding, and the exact zero of T under round-to-nearest."""
import numpy as np
import pytest

from oracle import coupling, fp8, norm
from paper_2609_39813_b200 import workloads


@pytest.fixture(scope="module")
def res():
    inp = workloads.config2(T=96, C=64, O=48, K=4, seed=5)
    prep = coupling.prepare(inp.x, inp.gamma, None, inp.W, norm.RMS, inp.eps)
    # two independent halves: their difference measures the sampling error of the averages
    a, b = coupling.run(prep, inp.seed, 300), coupling.run(prep, inp.seed + 1, 300)
    out = {k: (np.concatenate([a[k], b[k]]) if k in ("T", "control") else 0.5 * (a[k] + b[k])) for k in a}
    noise = {k: np.linalg.norm(a[k] - b[k]) / 2 for k in a if k not in ("T", "control")}
    return inp, prep, out, coupling.closed_forms(prep), noise


def test_gain_error_is_all_coupling(res):
    inp, prep, out, cf, noise = res
    # the rounding is right on average, so the mean part vanishes (to sampling error) and the whole
    # error is coupling, at its closed form
    assert np.linalg.norm(out["gain_mean_part"]) < 3 * noise["gain_mean_part"] + 1e-12
    assert np.linalg.norm(out["gain_coupling"] - cf["gain"]) < 3 * noise["gain_coupling"]
    assert np.linalg.norm(out["gain_coupling"] - cf["gain"]) < 0.25 * np.linalg.norm(cf["gain"])
    assert np.all(cf["gain"] > 0)
    # the total resolves it without the split's noise
    assert np.linalg.norm(out["gain_total"] - cf["gain"]) < 3 * noise["gain_total"]
    # a fresh read has no coupling: no error on average
    assert np.linalg.norm(out["gain_fresh"]) < 3 * noise["gain_fresh"]


def test_paired_statistic_and_control(res):
    inp, prep, out, cf, noise = res
    T, ctl = out["T"], out["control"]
    se = T.std(ddof=1) / np.sqrt(T.size)
    assert abs(T.mean() - cf["T"]) < 5 * se and T.mean() / se > 10           # resolved, at the closed form
    assert abs(ctl.mean()) < 5 * ctl.std(ddof=1) / np.sqrt(ctl.size)          # the independent copy: zero
    # T's mean is the difference between the consumed copy's and the independent copy's error:
    # sum_c gamma_c E[gain error]_c = E<r, du>
    assert abs(np.sum(prep["gamma"] * cf["gain"]) - cf["T"]) < 1e-9 * cf["T"]


def test_x_estimates_the_weight_use_error(res):
    inp, prep, out, cf, noise = res
    assert np.linalg.norm(out["X"] - cf["X"]) < 3 * noise["X"]
    assert np.linalg.norm(out["X"] - cf["X"]) < 0.1 * np.linalg.norm(cf["X"])
    # the direct average of -dy^T r agrees too, with far more noise: that is what X is for
    assert np.linalg.norm(out["wgrad_error"] - cf["wgrad_error"]) < 3 * noise["wgrad_error"]
    assert noise["X"] < 0.2 * noise["wgrad_error"]
    assert np.allclose(cf["X"], cf["wgrad_error"].T)


def test_round_to_nearest_gives_identical_forwards():
    inp = workloads.config2(T=32, C=32, O=16, K=4, seed=6)
    prep = coupling.prepare(inp.x, inp.gamma, None, inp.W, norm.RMS, inp.eps)
    out = coupling.run(prep, inp.seed, 3, mode=fp8.RN)
    assert np.all(out["T"] == 0.0) and not out["X"].any()
    # the gain error under round-to-nearest is one fixed number per column: all "mean part"
    assert np.allclose(out["gain_coupling"], 0.0, atol=1e-12 * np.max(np.abs(out["gain_total"])))


def test_split_is_an_identity_and_layernorm_bias():
    inp = workloads.config4(T=40, C=32, O=24, K=4, seed=7)
    prep = coupling.prepare(inp.x, inp.gamma, inp.beta, inp.W, norm.LAYER, inp.eps)
    out = coupling.run(prep, inp.seed, 5)
    assert np.allclose(out["gain_total"], out["gain_mean_part"] + out["gain_coupling"])
