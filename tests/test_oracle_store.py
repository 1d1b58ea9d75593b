"""Pins of the oracle's b-bit per-token store (Appendix "The normalization store"): the grid, the
rounding law against the paper's formula in exact rational arithmetic, its exact expectation, the
identities of Eq. norm-uses carried over, the closed-form variance and the table of expected
verdicts (U/R exact at both uses; N and U/R+eps right on average where the paper says so)."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import linear, mc, norm, philox, store
from paper_2609_39813_b200 import workloads


@pytest.fixture(scope="module", params=[6, 5], ids=["6bit", "5bit"])
def cfg(request):
    inp = workloads.config1()
    prep = store.prepare(inp.x, inp.gamma, None, inp.W, inp.dY, norm.RMS, inp.eps, inp.seed, request.param)
    return inp, prep


def test_grid_step_and_code_range(cfg):
    inp, prep = cfg
    M = store.levels(prep["bits"])
    assert M == (31 if prep["bits"] == 6 else 15)
    amax = np.max(np.abs(prep["u32"]), axis=1)
    assert np.array_equal(prep["s32"], (amax / np.float32(M)).astype(np.float32))
    codes = prep["codes"]
    assert codes.min() >= -M - 1 and codes.max() <= M + 1
    # the entry that sets the token's step sits at +-M (up to the one-rounding slack of the quotient)
    j = np.argmax(np.abs(prep["u32"]), axis=1)
    top = codes[np.arange(inp.T), j]
    assert np.all(np.abs(np.abs(top) - M) <= 1) and np.mean(np.abs(top) == M) > 0.9
    # an all-zero token: step 1, codes 0
    z = np.zeros((1, 8), np.float32)
    assert store.steps(z, 6)[0] == 1.0 and not store.codes_from_words(z, store.steps(z, 6), np.zeros((1, 8), np.uint64)).any()


def test_rounding_law_is_the_papers_formula_in_exact_arithmetic(cfg):
    """n = floor(u/s + xi) with xi = 1 - (W + 1) / 2^32 in rationals, for the generator's own words:
    the threshold form is the paper's formula under that reading of the uniform."""
    inp, prep = cfg
    u32, s32 = prep["u32"][:3], prep["s32"][:3]
    words = philox.tensor_words(inp.seed, store.TENSOR_U, 0, 0, u32.size).reshape(u32.shape)
    got = store.codes_from_words(u32, s32, words)
    t, n0, f, P = store.position(u32, s32)
    for r in range(u32.shape[0]):
        for c in range(u32.shape[1]):
            tt = Fraction(float(t[r, c]))                       # the FP32 quotient, exactly
            xi = 1 - Fraction(int(words[r, c]) + 1, 1 << 32)
            want = (tt + xi).__floor__()
            assert got[r, c] == want, (r, c)
            assert Fraction(float(f[r, c])) == tt - tt.__floor__() or abs(float(f[r, c]) - float(tt - tt.__floor__())) < 2.0 ** -24
    # decision at the threshold itself
    one = np.array([[0.3, -0.3, 1.75]], np.float32)
    s1 = np.array([0.5], np.float32)
    _, n0, _, P = store.position(one, s1)
    for j in range(3):
        p = int(P[0, j])
        for w, up in ((0, p > 0), (p - 1, True), (p, False), ((1 << 32) - 1, False)):
            if w < 0:
                continue
            n = store.codes_from_words(one, s1, np.full((1, 3), w, np.uint64))[0, j]
            assert n == n0[0, j] + int(up)


def test_store_is_right_on_average_without_clipping(cfg):
    """E[u_q] = s (n0 + P / 2^32) equals u up to the rounding of the FP32 quotient (well below one
    part in 10^6 of the step), and values on the grid never move."""
    inp, prep = cfg
    e = store.expected_value(prep["u32"], prep["s32"])
    assert np.max(np.abs(e - prep["u32"]) / prep["s32"][:, None]) < 2.0 ** -18
    # exact rationals on the first row
    t, n0, f, P = store.position(prep["u32"][:1], prep["s32"][:1])
    s = Fraction(float(prep["s32"][0]))
    for c in range(prep["u32"].shape[1]):
        E = s * (int(n0[0, c]) + Fraction(int(P[0, c]), 1 << 32))
        assert abs(E - s * Fraction(float(t[0, c]))) <= s * Fraction(1, 1 << 23)
    on_grid = (np.arange(-4, 5, dtype=np.float32) * np.float32(0.25))[None, :]
    sg = np.array([0.25], np.float32)
    for w in (0, 12345, (1 << 32) - 1):
        assert np.array_equal(store.codes_from_words(on_grid, sg, np.full(on_grid.shape, w, np.uint64))[0], np.arange(-4, 5))


def test_read_error_identities_carry_over(cfg):
    """dW(U) - dW(R) = -r^T dy and dgamma(R) - dgamma(U) = sum_t (r / gamma) o du with r = u_q - u;
    the gain use reading the original has exactly zero error."""
    inp, prep = cfg
    r = store.value(prep["codes"], prep["s32"]) - prep["u32"].astype(np.float64)
    dy = prep["dy"]["value"]
    wu = store.wgrad_use(prep, store.READ_U, 1, inp.seed)
    assert np.allclose(wu["mean"] - wu["ref"], -(dy.T @ r), rtol=1e-10, atol=1e-12)
    gr = store.gain_use(inp.x, inp.gamma, None, norm.RMS, inp.eps, prep, store.READ_R, 1, inp.seed)
    # (against the float64 u = gamma o z that the reference's z comes from)
    r64 = store.value(prep["codes"], prep["s32"]) - inp.gamma.astype(np.float64)[None, :] * prep["fw"]["z"]
    assert np.allclose(gr["mean"] - gr["ref"], np.sum(r64 / inp.gamma[None, :] * prep["du"], axis=0), rtol=1e-9, atol=1e-12)
    gu = store.gain_use(inp.x, inp.gamma, None, norm.RMS, inp.eps, prep, store.READ_U, 1, inp.seed)
    assert gu["stats"].rel_l2_mean_err == 0.0
    # the rounding error is the size a b-bit grid gives: rms r about step / sqrt(12) .. step / 2
    rms = np.sqrt(np.mean(r * r, axis=1)) / prep["s32"]
    assert np.all(rms > 0.2) and np.all(rms < 0.5)


def test_expected_verdicts_of_the_policy_table(cfg):
    inp, prep = cfg
    K = 96
    gain = {p: store.gain_use(inp.x, inp.gamma, None, norm.RMS, inp.eps, prep, p, K, inp.seed)["stats"].verdict
            for p in (store.READ_U, store.READ_R, store.READ_N)}
    assert gain == {store.READ_U: mc.HOLDS, store.READ_R: mc.FAILS, store.READ_N: mc.HOLDS}
    res = {p: store.wgrad_use(prep, p, K, inp.seed) for p in (store.READ_U, store.READ_R, store.READ_N, store.READ_R_EPS)}
    assert {p: r["stats"].verdict for p, r in res.items()} == \
        {store.READ_U: mc.FAILS, store.READ_R: mc.HOLDS, store.READ_N: mc.FAILS, store.READ_R_EPS: mc.HOLDS}
    assert res[store.READ_R]["stats"].rel_l2_mean_err == 0.0
    # U/R+eps is right on average with the variance of a fresh rounding; N's mean sits at U's value
    var = (prep["dy"]["value"] ** 2).T @ store.variance(prep["u32"], prep["s32"])
    for p in (store.READ_N, store.READ_R_EPS):
        ratio = (res[p]["m2"] / (K - 1)) / var
        assert abs(np.mean(ratio) - 1) < 0.02 and np.all(np.abs(ratio - 1) < 7 * np.sqrt(2.0 / (K - 1)))
    zN = (res[store.READ_N]["mean"] - res[store.READ_U]["mean"]) / np.sqrt(var / K)
    zE = (res[store.READ_R_EPS]["mean"] - res[store.READ_R]["ref"]) / np.sqrt(var / K)
    for z in (zN, zE):
        assert np.max(np.abs(z)) < 5.5 and abs(np.mean(z * z) - 1) < 0.1
    # mutation: swapping the reads of the two uses breaks the table (the weight use reading the
    # original fails, the gain use reading the rounded copy fails)
    assert res[store.READ_U]["stats"].verdict == mc.FAILS and gain[store.READ_R] == mc.FAILS


def test_sub_blocks_agree_with_the_full_tensor(cfg):
    inp, prep = cfg
    rows, cols = np.array([1, 17, 90]), np.array([0, 5, 64, 127])
    full = store.wgrad_use(prep, store.READ_R_EPS, 5, inp.seed)
    sub = store.wgrad_use(prep, store.READ_R_EPS, 5, inp.seed, rows, cols)
    assert np.allclose(sub["mean"], full["mean"][np.ix_(rows, cols)], rtol=1e-12, atol=1e-12)
    assert np.allclose(sub["m2"], full["m2"][np.ix_(rows, cols)], rtol=1e-9, atol=1e-14)


def test_layernorm_bias_is_removed_before_the_gain(cfg):
    inp4 = workloads.config4(T=48, C=64, O=32, K=4)
    prep = store.prepare(inp4.x, inp4.gamma, inp4.beta, inp4.W, inp4.dY, norm.LAYER, inp4.eps, inp4.seed, 6)
    u64 = inp4.gamma.astype(np.float64)[None, :] * prep["fw"]["z"] + inp4.beta.astype(np.float64)[None, :]
    r = store.value(prep["codes"], prep["s32"]) - u64
    g = store.gain_use(inp4.x, inp4.gamma, inp4.beta, norm.LAYER, inp4.eps, prep, store.READ_R, 1, inp4.seed)
    assert np.allclose(g["mean"] - g["ref"], np.sum(r / inp4.gamma[None, :] * prep["du"], axis=0), rtol=1e-9, atol=1e-12)
