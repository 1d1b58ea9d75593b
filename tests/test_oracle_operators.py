"""Pins of the oracle's operators: finite differences, the paper's identities and its worked
attention row."""
import numpy as np
import pytest

from conftest import golden_path
from oracle import attention, check, fp8, linear, mc, norm, philox
from paper_2609_39813_b200 import workloads


def _fd(f, a, h=1e-6):
    """Central finite differences of a scalar function of array a (float64)."""
    g = np.zeros_like(a)
    it = np.nditer(a, flags=["multi_index"])
    for _ in it:
        i = it.multi_index
        ap, am = a.copy(), a.copy()
        ap[i] += h
        am[i] -= h
        g[i] = (f(ap) - f(am)) / (2 * h)
    return g


@pytest.mark.parametrize("kind,eps", [(norm.RMS, 1e-6), (norm.LAYER, 1e-5), (norm.RMS, 0.3)])
def test_norm_backward_matches_finite_differences(kind, eps):
    rng = np.random.default_rng(0)
    T, C = 3, 5
    x = rng.standard_normal((T, C))
    gamma = 1 + 0.3 * rng.standard_normal(C)
    beta = 0.2 * rng.standard_normal(C) if kind == norm.LAYER else None
    du = rng.standard_normal((T, C))
    loss_x = lambda xx: float(np.sum(norm.forward(xx, gamma, beta, kind, eps)["u"] * du))
    loss_g = lambda gg: float(np.sum(norm.forward(x, gg, beta, kind, eps)["u"] * du))
    out = norm.backward(x, gamma, beta, kind, eps, du)
    assert np.allclose(out["dx"], _fd(loss_x, x), rtol=1e-7, atol=1e-8)
    assert np.allclose(out["dgamma"], _fd(loss_g, gamma), rtol=1e-7, atol=1e-8)
    if kind == norm.LAYER:
        loss_b = lambda bb: float(np.sum(norm.forward(x, gamma, bb, kind, eps)["u"] * du))
        assert np.allclose(out["dbeta"], _fd(loss_b, beta), rtol=1e-7, atol=1e-8)


def test_norm_forward_against_textbook():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((4, 8))
    g = rng.standard_normal(8)
    b = rng.standard_normal(8)
    fw = norm.forward(x, g, None, norm.RMS, 1e-6)
    assert np.allclose(fw["u"], g * x / np.sqrt((x ** 2).mean(1, keepdims=True) + 1e-6))
    fw = norm.forward(x, g, b, norm.LAYER, 1e-5)
    assert np.allclose(fw["u"], g * (x - x.mean(1, keepdims=True)) / np.sqrt(x.var(1, keepdims=True) + 1e-5) + b)


def test_store_value_chain_is_fp32_and_close_to_float64():
    inp = workloads.config1()
    prep = check.prepare_norm_linear(inp.x, inp.gamma, None, inp.W, inp.dY, norm.RMS, inp.eps, inp.seed)
    assert prep["v32"].dtype == np.float32 and prep["u32"].dtype == np.float32
    assert np.allclose(prep["u32"], prep["fw"]["u"], rtol=3e-7, atol=0)
    assert prep["scale"] == np.float32(448.0) / prep["amax"]
    # the store's rounding error is at the size E4M3 gives (a few percent), not zero, not huge
    r = norm.read_value(prep["codes"], fp8.E4M3, prep["inv_scale"]) - prep["fw"]["u"]
    rel = np.sqrt(np.mean(r ** 2) / np.mean(prep["fw"]["u"] ** 2))
    assert 0.01 < rel < 0.1


@pytest.fixture(scope="module")
def cfg1():
    inp = workloads.config1()
    prep = check.prepare_norm_linear(inp.x, inp.gamma, None, inp.W, inp.dY, norm.RMS, inp.eps, inp.seed)
    return inp, prep


def test_read_error_identities(cfg1):
    """Eq. norm-uses: the original at the weight use adds -r^T dy; the rounded value at the gain
    use adds sum_tokens (r/gamma) o du; the original at the gain use has exactly zero error."""
    inp, prep = cfg1
    u = prep["fw"]["u"]
    uq = norm.read_value(prep["codes"], fp8.E4M3, prep["inv_scale"])
    r = uq - u
    dy = prep["dy"]["value"]
    dW_R = linear.wgrad(dy, uq)
    dW_U = linear.wgrad(dy, u)
    assert np.allclose(dW_U - dW_R, -(dy.T @ r), rtol=0, atol=1e-10)           # dW is [O, C]
    g_U = check.gain_use(inp.x, inp.gamma, None, norm.RMS, inp.eps, prep, check.U, 1, inp.seed)
    g_R = check.gain_use(inp.x, inp.gamma, None, norm.RMS, inp.eps, prep, check.R, 1, inp.seed)
    add = np.sum((r / inp.gamma.astype(np.float64)[None, :]) * prep["du"], axis=0)
    assert np.allclose(g_R["mean"] - g_U["mean"], add, rtol=0, atol=1e-10)
    assert g_U["stats"].rel_l2_mean_err == 0.0
    # dgamma from the copy u itself is the reference (the reconstruction is exact for the original)
    assert np.allclose(norm.dgamma_from_copy(u, inp.gamma, None, prep["du"]), g_U["ref"], atol=1e-10)


def test_wgrad_is_plain_matmul_and_subblocks_agree(cfg1):
    inp, prep = cfg1
    dy = fp8.decode(prep["dy"]["codes"], fp8.E5M2) * float(prep["dy"]["inv_scale"])
    uq = fp8.decode(prep["codes"], fp8.E4M3) * float(prep["inv_scale"])
    full = np.einsum("to,tc->oc", dy, uq)
    assert np.allclose(linear.wgrad(prep["dy"]["value"], uq), full, rtol=1e-12, atol=1e-12)
    rows = np.array([3, 77, 100])
    cols = np.array([0, 5, 127])
    sub = check.wgrad_use(prep, check.N, 4, inp.seed, rows, cols)
    fullN = check.wgrad_use(prep, check.N, 4, inp.seed)
    assert np.allclose(sub["mean"], fullN["mean"][np.ix_(rows, cols)], rtol=1e-12, atol=1e-12)
    assert np.allclose(sub["m2"], fullN["m2"][np.ix_(rows, cols)], rtol=1e-9, atol=1e-12)


def test_incoming_gradient_is_nearest_e5m2(cfg1):
    inp, prep = cfg1
    g = prep["dy"]
    assert g["scale"] == np.float32(57344.0) / np.max(np.abs(inp.dY))
    err = g["value"] - inp.dY
    assert np.max(np.abs(err) / np.abs(inp.dY)) <= 2.0 ** -3 + 1e-6        # half an ulp of 2 mantissa bits
    assert g["n_saturated"] == 0


def test_dgrad_shape_and_value(cfg1):
    inp, prep = cfg1
    assert prep["du"].shape == inp.x.shape
    assert np.allclose(prep["du"], (prep["dy"]["value"] @ inp.W.astype(np.float64)).astype(np.float32))


def test_fresh_read_mean_and_variance_closed_form(cfg1):
    """Policy N at the gain use: E[g_N] = g_U and Var = sum_t (du/gamma)^2 (v-lo)(hi-v)/scale^2;
    the sample variance over K draws matches it within sampling error."""
    inp, prep = cfg1
    K = 256
    res = check.gain_use(inp.x, inp.gamma, None, norm.RMS, inp.eps, prep, check.N, K, inp.seed)
    lo, hi, _ = fp8.neighbours(prep["v32"], fp8.E4M3)
    a = np.abs(prep["v32"].astype(np.float64))
    var_el = (a - lo) * (hi - a) * float(prep["inv_scale"]) ** 2
    var_cf = np.sum((prep["du"] / inp.gamma.astype(np.float64)[None, :]) ** 2 * var_el, axis=0)
    ratio = (res["m2"] / (K - 1)) / var_cf
    assert abs(np.mean(ratio) - 1) < 4 * np.sqrt(2.0 / (K - 1)) / np.sqrt(inp.C)
    assert np.all(np.abs(ratio - 1) < 6 * np.sqrt(2.0 / (K - 1)))
    # the mean is the value obtained by reading the FP32 chain value itself (up to 2^-32 ulp)
    g_chain = norm.dgamma_from_copy(prep["u32"].astype(np.float64), inp.gamma, None, prep["du"])
    z = (res["mean"] - g_chain) / np.sqrt(var_cf / K)
    assert np.max(np.abs(z)) < 5 and abs(np.mean(z * z) - 1) < 0.5


def test_expected_verdicts_and_mutation(cfg1):
    """Gain use: U holds exactly, R fails, N holds on average.  Weight use: U fails, R holds
    exactly, N fails (its mean tends to U's value).  Swapping the reads at the two uses flips
    the table."""
    inp, prep = cfg1
    args = (inp.x, inp.gamma, None, norm.RMS, inp.eps, prep)
    gain = {p: check.gain_use(*args, p, inp.K, inp.seed)["stats"] for p in (check.U, check.R, check.N)}
    wg = {p: check.wgrad_use(prep, p, 64, inp.seed)["stats"] for p in (check.U, check.R, check.N)}
    assert [gain[p].verdict for p in (check.U, check.R, check.N)] == [mc.HOLDS, mc.FAILS, mc.HOLDS]
    assert [wg[p].verdict for p in (check.U, check.R, check.N)] == [mc.FAILS, mc.HOLDS, mc.FAILS]
    assert gain[check.U].rel_l2_mean_err == 0 and wg[check.R].rel_l2_mean_err == 0
    assert 0.005 < gain[check.R].rel_l2_mean_err < 0.2 and 0.005 < wg[check.U].rel_l2_mean_err < 0.2
    assert wg[check.N].R > 10 and gain[check.N].R < 2
    # mutation: a checker whose reference reads were swapped (gain R, weight U) would certify the
    # opposite cells; emulate by judging each policy against the swapped reference
    uq = norm.read_value(prep["codes"], fp8.E4M3, prep["inv_scale"])
    swapped_gain_ref = norm.dgamma_from_copy(uq, inp.gamma, None, prep["du"])
    st = mc.statistics(check.gain_use(*args, check.U, 1, inp.seed)["mean"], None, 1, swapped_gain_ref, False)
    assert st.verdict == mc.FAILS


def test_shared_stream_reproduces_one_draw_for_both_uses(cfg1):
    inp, prep = cfg1
    a, ca = check.fresh_copy(prep, inp.seed, philox.STREAM_SHARED, 3)
    b, cb = check.fresh_copy(prep, inp.seed, philox.STREAM_SHARED, 3)
    c, cc = check.fresh_copy(prep, inp.seed, philox.STREAM_GAIN, 3)
    assert np.array_equal(ca, cb) and not np.array_equal(ca, cc)


# ---------------------------------------------------------------------------- Monte Carlo


def test_welford_two_pass_shifted_sums_and_merge():
    rng = np.random.default_rng(3)
    K, n = 37, 50
    g = 5.0 + 0.01 * rng.standard_normal((K, n))
    ref = g.mean(0) + 1e-3 * rng.standard_normal(n)
    w = mc.Welford((n,))
    for k in range(K):
        w.add(g[k])
    mean2 = g.mean(0)
    m2_2 = ((g - mean2) ** 2).sum(0)
    assert np.allclose(w.mean, mean2, rtol=1e-14) and np.allclose(w.m2, m2_2, rtol=1e-10)
    S1 = (g - ref).sum(0)
    S2 = ((g - ref) ** 2).sum(0)
    m3, m2_3 = mc.shifted_sums_to_moments(S1, S2, K, ref)
    assert np.allclose(m3, mean2, rtol=1e-14) and np.allclose(m2_3, m2_2, rtol=1e-8)
    a, b = mc.Welford((n,)), mc.Welford((n,))
    for k in range(K):
        (a if k < 20 else b).add(g[k])
    a.merge(b)
    assert a.n == K and np.allclose(a.mean, mean2, rtol=1e-14) and np.allclose(a.m2, m2_2, rtol=1e-10)


def test_statistics_on_known_distributions():
    rng = np.random.default_rng(4)
    K, n = 64, 4000
    g = rng.standard_normal((K, n))
    zero = mc.statistics(g.mean(0), ((g - g.mean(0)) ** 2).sum(0), K, np.zeros(n), True)
    assert abs(zero.R - 1) < 0.15 and abs(zero.Qprime - 1) < 0.15 and zero.verdict == mc.HOLDS
    # a bias of one standard deviation per draw: R ~ 1 + K
    biased = mc.statistics(g.mean(0) + 1.0, ((g - g.mean(0)) ** 2).sum(0), K, np.zeros(n), True)
    assert abs(biased.R / (1 + K) - 1) < 0.15 and biased.verdict == mc.FAILS
    # z = |m| / se with se over trials, one element by hand
    one = mc.statistics(np.array([2.0]), np.array([12.0]), 4, np.array([1.0]), True)
    assert np.isclose(one.max_abs_z, 1.0 / np.sqrt(12.0 / 3 / 4))
    exact = mc.statistics(np.zeros(3), np.zeros(3), 8, np.zeros(3), True)
    assert exact.R == 0 and exact.Qprime == 0 and exact.verdict == mc.HOLDS
    assert mc.verdict_fresh(3.0, 1.0) == mc.UNDECIDED and mc.verdict_fresh(1.0, 7.0) == mc.FAILS


# ------------------------------------------------------------------------------ attention


def _tiny_attention(seed=5, S=6, d=4):
    rng = np.random.default_rng(seed)
    return [rng.standard_normal((S, d)) for _ in range(4)]


@pytest.mark.parametrize("causal", [True, False])
def test_attention_backward_matches_finite_differences(causal):
    q, k, v, G = _tiny_attention()
    c = 0.37
    O, _ = attention.forward_output(q, k, v, c, causal)
    out = attention.backward(q, k, v, G, c, O, causal)
    loss = lambda qq, kk, vv: float(np.sum(attention.forward_output(qq, kk, vv, c, causal)[0] * G))
    assert np.allclose(out["dq"], _fd(lambda a: loss(a, k, v), q), rtol=1e-6, atol=1e-8)
    assert np.allclose(out["dk"], _fd(lambda a: loss(q, a, v), k), rtol=1e-6, atol=1e-8)
    assert np.allclose(out["dv"], _fd(lambda a: loss(q, k, a), v), rtol=1e-6, atol=1e-8)


def test_attention_d_identities():
    q, k, v, dO = _tiny_attention(6, 9, 5)
    c = 0.5
    O, _ = attention.forward_output(q, k, v, c)
    ref = attention.backward(q, k, v, dO, c, O)
    assert np.allclose(ref["D"], attention.d_from_probabilities(q, k, v, dO, c), rtol=0, atol=1e-12)
    E = 0.1 * np.random.default_rng(7).standard_normal(O.shape)
    pol = attention.backward(q, k, v, dO, c, O + E)
    dD = np.sum(dO * E, axis=1)
    assert np.allclose(pol["D"] - ref["D"], dD, atol=1e-13)                     # Eq. dterm
    assert np.array_equal(pol["dv"], ref["dv"])                                 # dV never reads O
    P, _ = attention.probabilities(q, k, c)
    assert np.allclose(pol["dq"] - ref["dq"], -c * (dD[:, None] * (P @ k)), atol=1e-13)
    assert np.allclose(pol["dk"] - ref["dk"], -c * (P.T @ (dD[:, None] * q)), atol=1e-13)


def _row_case(x, h, fp8_operands):
    S, d = 64, 8
    q = np.zeros((S, d)); q[:, 1] = 1.0
    k = np.zeros((S, d)); k[:, 0] = 1.0
    v = np.zeros((S, d)); v[:, 0] = np.where(np.arange(S) % 2 == 0, 1.0, 1.5)
    dO = np.zeros((S, d)); dO[63, 0] = h
    c = 1.0 / 8.0
    O, _ = attention.forward_output(q, k, v, c)
    assert O[63, 0] == 1.25
    Osaved = O.copy(); Osaved[63, 0] = x
    out = attention.backward(q, k, v, dO, c, Osaved, True, fp8_operands, scale_p=256.0, scale_ds=1024.0)
    return out["dq"][63, 0], c


@pytest.mark.parametrize("fp8_operands", [False, True])
def test_attention_row_case_of_the_paper(fp8_operands):
    a, s = 0.25, 1.25
    cells = [l.split() for l in open(golden_path("attention_row_cells.txt")) if l[0] in "+-"]
    assert len(cells) == 4
    means = [0.0, 0.0]
    for sig, tau, t_dev, t_fixed in cells:
        sig, tau, t_dev, t_fixed = float(sig), float(tau), float(t_dev), float(t_fixed)
        for col, (h, want) in enumerate(((sig * a, t_dev), (a, t_fixed))):
            dq_sh, c = _row_case(s + sig * a, h, fp8_operands)
            dq_in, _ = _row_case(s + tau * a, h, fp8_operands)
            assert dq_sh == c * h * (s - (s + sig * a))             # closed form, exact
            T = (dq_in - dq_sh) / c
            assert T == want == h * (sig - tau) * a                 # zero deviation
            means[col] += T / 4
    assert means == [a * a, 0.0]


def test_attention_fp8_mode_quantisation_points():
    q, k, v, dO = _tiny_attention(8, 16, 8)
    c = 0.35
    O, _ = attention.forward_output(q, k, v, c)
    exact = attention.backward(q, k, v, dO, c, O)
    amax_ds = np.max(np.abs(exact["dS"]))
    a = attention.backward(q, k, v, dO, c, O, True, True, 256.0, 57344.0 / amax_ds)
    # the roundings perturb but do not change the gradients' scale; D itself is untouched
    assert np.array_equal(a["D"], exact["D"])
    for n in ("dq", "dk", "dv"):
        rel = np.linalg.norm(a[n] - exact[n]) / np.linalg.norm(exact[n])
        assert 1e-4 < rel < 0.2, (n, rel)


def test_attention_check_expected_verdicts():
    inp = workloads.config3(B=1, H=2, S=48, D=16, K=48, seed=9)
    q, k, v, dO = inp.q[0, 1], inp.k[0, 1], inp.v[0, 1], inp.dO[0, 1]
    prep = check.prepare_attention_slice(q, k, v, dO, inp.softmax_scale, inp.seed, 1)
    res = {p: check.attention_d_use(q, k, v, dO, inp.softmax_scale, prep, p, inp.K, inp.seed)
           for p in (check.U, check.R, check.N)}
    for name in ("D", "dq", "dk"):
        assert [res[p][name]["stats"].verdict for p in (check.U, check.R, check.N)] == \
            [mc.HOLDS, mc.FAILS, mc.HOLDS], name
        assert res[check.U][name]["stats"].rel_l2_mean_err == 0
    for p in (check.U, check.R, check.N):
        assert res[p]["dv"]["stats"].verdict == mc.HOLDS
        assert np.array_equal(res[p]["dv"]["mean"], res[check.U]["dv"]["ref"])
    # the slice's words are those of the full tensor at the slice's offset
    w_full = philox.tensor_words(inp.seed, check.TENSOR_O, 0, 0, 2 * 48 * 16)
    assert np.array_equal(philox.element_words(inp.seed, check.TENSOR_O, 0, 0, prep["elem"]).ravel(),
                          w_full[48 * 16:])


def test_attention_operand_rounding_option():
    """Rounding P and dS to bf16 before their products (what a BF16 tensor-core contraction does)
    moves the gradients by about 2^-9, leaves D untouched, and is the identity when the rounding
    is the identity."""
    q, k, v, dO = _tiny_attention(11, 40, 8)
    c = 0.3
    O, _ = attention.forward_output(q, k, v, c)
    exact = attention.backward(q, k, v, dO, c, O)
    same = attention.backward(q, k, v, dO, c, O, operand_round=lambda a: a)
    rounded = attention.backward(q, k, v, dO, c, O, operand_round=linear.bf16_round)
    for n in ("dq", "dk", "dv"):
        assert np.array_equal(same[n], exact[n])
        rel = np.linalg.norm(rounded[n] - exact[n]) / np.linalg.norm(exact[n])
        assert 1e-5 < rel < 4e-3, (n, rel)
    assert np.array_equal(rounded["D"], exact["D"])


def test_bf16_round_against_an_independent_cast():
    """linear.bf16_round (the operand rounding of the U read) against ml_dtypes' bfloat16 cast:
    random values over many binades, every tie between neighbouring bf16 values in a binade, zeros,
    subnormals of float32, and values that round up into the next binade."""
    ml_dtypes = pytest.importorskip("ml_dtypes")
    rng = np.random.default_rng(12)
    a = (rng.standard_normal(200000) * np.exp(rng.uniform(-60, 60, 200000))).astype(np.float32)
    # exact ties: a bf16 value plus half its spacing (representable in float32), both parities
    base = np.arange(0x3F80, 0x4000, dtype=np.uint32) << np.uint32(16)
    ties = (base | np.uint32(0x8000)).view(np.float32)
    special = np.array([0.0, -0.0, 1e-40, -1e-45, 1.0, -1.0, np.float32(1.99609375), np.float32(1.998046875),
                        3.3e38, -3.3e38], dtype=np.float32)
    for v in (a, ties, -ties, special):
        want = v.astype(ml_dtypes.bfloat16).astype(np.float32)
        got = linear.bf16_round(v.astype(np.float64)).astype(np.float32)
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    # float64 inputs are first brought to float32 (the operands are float32 tensors)
    assert linear.bf16_round(np.float64(1.0) + 2.0 ** -30) == 1.0


def test_fresh_read_variance_closed_form_weight_use_and_d(cfg1):
    """The closed-form variances of the other two uses under a fresh read: weight use
    Var dW[o, c] = sum_t dY[t, o]^2 sigma^2[t, c]; attention's D: Var D[i] = sum_d dO[i, d]^2 sigma^2[i, d],
    with sigma^2 = (v - lo)(hi - v) / scale^2 the variance of one stochastic rounding.  Sample variances
    over K draws match within sampling error, and the means are the values read from the unrounded
    tensor."""
    inp, prep = cfg1
    K = 192
    res = check.wgrad_use(prep, check.N, K, inp.seed)
    lo, hi, _ = fp8.neighbours(prep["v32"], fp8.E4M3)
    a = np.abs(prep["v32"].astype(np.float64))
    var_el = (a - lo) * (hi - a) * float(prep["inv_scale"]) ** 2
    dy = prep["dy"]["value"]
    var_cf = (dy * dy).T @ var_el
    ratio = (res["m2"] / (K - 1)) / var_cf
    assert abs(np.mean(ratio) - 1) < 4 * np.sqrt(2.0 / (K - 1)) / np.sqrt(ratio.size)
    assert np.all(np.abs(ratio - 1) < 7 * np.sqrt(2.0 / (K - 1)))
    # the mean tends to the value of the chain's own FP32 u (the original), not to the reference
    g_u = linear.wgrad(dy, prep["u32"].astype(np.float64))
    z = (res["mean"] - g_u) / np.sqrt(var_cf / K)
    assert np.max(np.abs(z)) < 5.5 and abs(np.mean(z * z) - 1) < 0.1
    # ---- attention's D use
    ai = workloads.config3(B=1, H=1, S=96, D=64, K=K, seed=5)
    q, k, v, dO = ai.q[0, 0], ai.k[0, 0], ai.v[0, 0], ai.dO[0, 0]
    ap = check.prepare_attention_slice(q, k, v, dO, ai.softmax_scale, ai.seed, 0, True)
    rd = check.attention_d_use(q, k, v, dO, ai.softmax_scale, ap, check.N, K, ai.seed, outputs=("D",))["D"]
    lo, hi, _ = fp8.neighbours(ap["v32"], fp8.E4M3)
    a = np.abs(ap["v32"].astype(np.float64))
    var_o = (a - lo) * (hi - a) * float(ap["inv_scale"]) ** 2
    var_d = np.sum(dO.astype(np.float64) ** 2 * var_o, axis=1)
    ratio = (rd["m2"] / (K - 1)) / var_d
    assert abs(np.mean(ratio) - 1) < 4 * np.sqrt(2.0 / (K - 1)) / np.sqrt(ratio.size)
    assert np.all(np.abs(ratio - 1) < 6 * np.sqrt(2.0 / (K - 1)))
    z = (rd["mean"] - rd["ref"]) / np.sqrt(var_d / K)
    assert np.max(np.abs(z)) < 5 and abs(np.mean(z * z) - 1) < 0.5


def test_elements_without_variance_are_judged_as_deterministic_reads():
    """Where every draw of an element gave the same value, z is 0 if the error is within the
    deterministic tolerance of the reference and infinite otherwise; the other elements keep z = err/se."""
    K = 8
    ref = np.array([1.0, 1.0, 1.0, 0.0, 2.0])
    mean = np.array([1.0 + 5e-8, 1.0 + 1e-3, 1.2, 0.0, 2.0])
    m2 = np.array([0.0, 0.0, 0.7, 0.0, 0.0])
    st = mc.statistics(mean, m2, K, ref, True)
    assert np.isinf(st.max_abs_z) and np.isinf(st.Qprime) and st.verdict == mc.FAILS
    st = mc.statistics(np.array([1.0 + 5e-8, 1.2, 0.0]), np.array([0.0, 0.7, 0.0]), K, np.array([1.0, 1.0, 0.0]), True)
    se = np.sqrt(0.7 / (K - 1) / K)
    assert st.max_abs_z == pytest.approx(0.2 / se) and st.mean_z == pytest.approx(0.2 / se / 3)
    assert st.frac_abs_z_gt3 == 0.0 if 0.2 / se <= 3 else st.frac_abs_z_gt3 == pytest.approx(1 / 3)
