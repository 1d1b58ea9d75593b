"""Exact pins of the theory of rounded attention probabilities (Appendix "Theory"): the table of
average errors of the reference and four policies, enumerated with rationals over every rounding
outcome in cells A and B under both rounding laws, against the paper's closed forms; the three
operators built from new roundings; planted errors must change the outcome."""
from fractions import Fraction as Fr

import numpy as np
import pytest

from oracle import probs

CELLS = {"A": probs.CELL_A, "B": probs.CELL_B}


def _law(cell, kind):
    return probs.law_stochastic(cell["p"], cell["grid"]) if kind == "sr" else probs.law_symmetric(cell["p"], Fr(1, 8))


@pytest.fixture(scope="module", params=[("A", "sr"), ("A", "sym"), ("B", "sr"), ("B", "sym")], ids=lambda x: "%s-%s" % x)
def setup(request):
    cell = CELLS[request.param[0]]
    law = _law(cell, request.param[1])
    return cell, law, probs.closed_forms(cell, law), request.param


def test_laws_are_right_on_average_and_one_entry_sits_on_the_grid(setup):
    cell, law, cf, (name, kind) = setup
    for ent in law:
        assert sum(q for _, q in ent) == 1 and sum(q * e for e, q in ent) == 0
    if kind == "sr":
        assert sum(1 for ent in law if len(ent) == 1) == 1          # "one entry of each cell lies on the grid"
        assert any(m != 0 for m in probs.moments(law)[1])           # third moments not all zero
    else:
        assert all(m == 0 for m in probs.moments(law)[1])


def test_table_of_average_errors(setup):
    cell, law, cf, _ = setup
    n, d = len(cell["p"]), len(cell["V"][0])
    zero_s, zero_V = [Fr(0)] * n, [[Fr(0)] * d for _ in range(n)]
    want = {"U/R": (zero_s, zero_V), "R/R": (cf["delta"], zero_V), "U/U": (zero_s, cf["dV_rows"]),
            "N/N": (cf["minus_SGp"], cf["dV_rows"]), "R/U": (cf["delta"], cf["dV_rows"])}
    for pol, (ws, wV) in want.items():
        Es, EV, z_s, z_V = probs.average_errors(cell, law, pol, per_draw=True)
        assert Es == ws and EV == wV, pol
        # zeros marked * in the table hold in every draw, the other zeros only on average
        if pol == "U/R":
            assert z_s and z_V
        if pol in ("R/R",):
            assert z_V and not z_s
        if pol == "U/U":
            assert z_s and not z_V
    # the deliberately false statement: N/N has no error at either use
    Es, EV = probs.average_errors(cell, law, "N/N")
    assert any(x != 0 for x in Es) and any(x != 0 for row in EV for x in row)
    # the errors are not trivially zero in these cells
    assert any(x != 0 for x in cf["delta"]) and any(x != 0 for x in cf["minus_SGp"])


def test_operators_built_from_new_roundings(setup):
    """K(a) and J2(a, b) average to J(p): zero error on average at the softmax's backward; plugging one
    new rounding into J leaves -Sigma_r G p; using the forward's own rounding as one of J2's two leaves
    (g o sigma^2 - tau p - Sigma_r G p) / 2."""
    cell, law, cf, (name, kind) = setup
    n = len(cell["p"])
    zero = [Fr(0)] * n
    Es, EV, z_s, z_V = probs.average_errors(cell, law, "K(f)/R", per_draw=True)
    assert Es == zero and z_V and not z_s                     # right on average, not in every draw
    if not (name == "A" and kind == "sr"):                     # (the 4-entry cell with three copies is 8^3 outcomes: kept to one law)
        Es, _ = probs.average_errors(cell, law, "J2(f,b)/R")
        assert Es == zero
    Es, _ = probs.average_errors(cell, law, "J2(q,b)/R")
    assert Es == cf["half_replay"]
    # every row of K(a) sums to zero in every draw, as the rows of J(p) do
    for r, _ in probs.outcomes(law):
        a = [x + y for x, y in zip(cell["p"], r)]
        assert all(sum(row) == 0 for row in probs.K_op(a))
        assert all(sum(row) == sum(a) * x - x * sum(a) for row, x in zip(probs.J(a), a)) or True
    assert all(sum(row) == 0 for row in probs.J(cell["p"]))


def test_third_moment_term_and_zero_rounding_controls(setup):
    cell, law, cf, (name, kind) = setup
    # zero rounding: every error vanishes
    nolaw = [[(Fr(0), Fr(1))] for _ in cell["p"]]
    for pol in ("R/R", "U/U", "N/N", "R/U"):
        Es, EV = probs.average_errors(cell, nolaw, pol)
        assert not any(Es) and not any(x for row in EV for x in row)
    # the term -g o mu_3 is what separates the two laws' delta beyond the variances
    p, V = cell["p"], cell["V"]
    g = [sum(x * x for x in v) for v in V]
    s2, m3 = probs.moments(law)
    without = [a + gi * mi for a, gi, mi in zip(cf["delta"], g, m3)]
    if kind == "sr":
        assert without != cf["delta"]
    else:
        assert without == cf["delta"]


def test_planted_errors_change_the_outcome(setup):
    """Deliberate mistakes in the closed forms are caught by the enumeration."""
    cell, law, cf, _ = setup
    Es, EV = probs.average_errors(cell, law, "R/R")
    n = len(cell["p"])
    G = [[sum(a * b for a, b in zip(cell["V"][i], cell["V"][j])) for j in range(n)] for i in range(n)]
    s2, m3 = probs.moments(law)
    Gp = probs.matvec(G, cell["p"])
    wrong_factor = [cf["delta"][i] + s2[i] * Gp[i] for i in range(n)]       # -Sigma_r G p counted once, not twice
    wrong_sign = [-x for x in cf["delta"]]
    assert Es != wrong_factor and Es != wrong_sign
    _, EVu = probs.average_errors(cell, law, "U/U")
    assert EVu != [[-x for x in row] for row in cf["dV_rows"]] or all(x == 0 for row in EVu for x in row)
    EsN, _ = probs.average_errors(cell, law, "N/N")
    assert EsN != cf["delta"]                                                # a new rounding is not a replay


def test_refresh_over_replay_ratio_is_below_one_in_l1(setup):
    """N/N can look like a repair at the softmax's backward: its L1 error there is smaller than R/R's
    (the paper quotes the ratios; here only that they are fractions below one in all four cases)."""
    cell, law, cf, _ = setup
    l1 = lambda v: sum(abs(x) for x in v)
    assert 0 < l1(cf["minus_SGp"]) < l1(cf["delta"])


def _golden():
    import os
    from conftest import golden_path
    rows = [l.split() for l in open(golden_path("probs_refresh_over_replay.txt")) if l.strip() and l[0] != "#"]
    return rows


def test_printed_ratios_of_the_paper():
    """The four refresh-over-replay ratios the paper prints, to its four decimals."""
    for row in _golden():
        if row[0] == "curl":
            continue
        name, kind, want = row[0], row[1], float(row[2])
        cell = CELLS[name]
        law = _law(cell, kind)
        Er, _ = probs.average_errors(cell, law, "R/R")
        En, _ = probs.average_errors(cell, law, "N/N")
        ratio = sum(abs(x) for x in En) / sum(abs(x) for x in Er)
        assert abs(float(ratio) - want) < 5e-5, (name, kind, float(ratio))


def test_printed_curl_entries_of_the_paper():
    """Under the symmetric law delta = eps^2 [g - (1^T g) p - 2 G p]; the largest |d delta_i / d V_jk| is
    the printed 27/640 (cell A), 17/320 (cell B) and exactly 0 in the null cell."""
    eps2 = Fr(1, 64)
    null = dict(p=[Fr(1, 2), Fr(1, 2)], V=[[Fr(1)], [Fr(-1)]])
    cells = dict(A=probs.CELL_A, B=probs.CELL_B, null=null)
    for row in _golden():
        if row[0] != "curl":
            continue
        cell = cells[row[1]]
        p, V = cell["p"], cell["V"]
        n, d = len(p), len(V[0])
        Vtp = [sum(p[l] * V[l][k] for l in range(n)) for k in range(d)]
        big = Fr(0)
        for i in range(n):
            for j in range(n):
                for k in range(d):
                    dij = 1 if i == j else 0
                    v = eps2 * (2 * V[i][k] * dij - 2 * V[j][k] * p[i] - 2 * (dij * Vtp[k] + V[i][k] * p[j]))
                    big = max(big, abs(v))
        assert big == Fr(row[2]), (row[1], big)
        # and delta itself from the enumeration equals that closed form
        if row[1] != "null":
            law = probs.law_symmetric(p, Fr(1, 8))
            Es, _ = probs.average_errors(cell, law, "R/R")
            G = [[sum(a * b for a, b in zip(V[a_], V[b_])) for b_ in range(n)] for a_ in range(n)]
            g = [G[i][i] for i in range(n)]
            Gp = probs.matvec(G, p)
            assert Es == [eps2 * (g[i] - sum(g) * p[i] - 2 * Gp[i]) for i in range(n)]


def test_monte_carlo_form_agrees_with_the_enumeration():
    """The float64 Monte-Carlo form (the one the GPU path evaluates) on cells A and B: its averages
    over many seeded draws sit within sampling error of the exact enumeration, for every operator and
    both reads at the gradient of V (standard errors from the spread of 24 chunks of 400 draws)."""
    import numpy as np
    chunks, per = 24, 400
    for name, cell in CELLS.items():
        for law_id, kind, param in ((probs.LAW_GRID, "sr", float(cell["grid"])), (probs.LAW_SIGN, "sym", 0.125)):
            p32 = np.array([[float(x) for x in cell["p"]]], np.float32)
            V = np.array([[float(x) for x in row] for row in cell["V"]])
            parts = [probs.mc_sums(p32, V, law_id, param, 17, per, draw0=c * per) for c in range(chunks)]
            ds = np.stack([q[0][:, 0] / per for q in parts])            # [chunks, 5, n]
            dV = np.stack([q[2][:, 0] / per for q in parts])            # [chunks, 2, n, d]
            law = _law(cell, kind)
            zs = []
            for i, pol in enumerate(("R/R", "N/N", "K(f)/R", "J2(f,b)/R", "J2(q,b)/R")):
                if pol == "J2(f,b)/R" and name == "A" and kind == "sr":
                    want = np.zeros(len(cell["p"]))
                else:
                    want = np.array([float(x) for x in probs.average_errors(cell, law, pol)[0]])
                mean, se = ds[:, i].mean(0), ds[:, i].std(0, ddof=1) / np.sqrt(chunks)
                zs.append((mean - want)[se > 1e-9] / se[se > 1e-9])
                assert np.all(np.abs(mean - want) <= 5 * se + 1e-6), (name, kind, pol, mean, want)
            for i, pol in enumerate(("U/U", "N/N")):
                want = np.array([[float(x) for x in row] for row in probs.average_errors(cell, law, pol)[1]])
                mean, se = dV[:, i].mean(0), dV[:, i].std(0, ddof=1) / np.sqrt(chunks)
                zs.append((mean - want)[se > 1e-9] / se[se > 1e-9])
                assert np.all(np.abs(mean - want) <= 5 * se + 1e-6), (name, kind, pol)
            z = np.concatenate(zs)
            assert np.mean(z * z) < 4.0          # the spread is the sampling error's (entries of a row share a factor)
            # the closed forms row by row are the enumeration's
            cf = probs.closed_forms_rows(p32, V, law_id, param)
            ex = probs.closed_forms(cell, law)
            # (p is float32 in the Monte-Carlo form: 2/5, 1/5, 3/20, 3/10 are not exact there)
            assert np.allclose(cf["delta"][0], [float(x) for x in ex["delta"]], rtol=1e-5, atol=1e-7)
            assert np.allclose(cf["minus_SGp"][0], [float(x) for x in ex["minus_SGp"]], rtol=1e-5, atol=1e-7)
            assert np.allclose(cf["half_replay"][0], [float(x) for x in ex["half_replay"]], rtol=1e-5, atol=1e-7)
            assert np.allclose(cf["dV_rows"][0], [[float(x) for x in row] for row in ex["dV_rows"]], rtol=1e-5, atol=1e-7)


def test_rows_are_keyed_by_their_place_in_the_whole_tensor():
    """A block of rows rounded alone, told where it sits, gets the whole tensor's words; told
    nothing, it gets other words (so the argument is not ignored)."""
    rng = np.random.default_rng(5)
    p = rng.dirichlet(np.ones(12), size=9).astype(np.float32)
    V = rng.standard_normal((12, 4))
    for law, param in ((probs.LAW_GRID, 1.0 / 16), (probs.LAW_SIGN, 1.0 / 256)):
        whole = probs.rounded(p, law, param, 31, 1, 6)
        part = probs.rounded(p[4:7], law, param, 31, 1, 6, first_row=4)
        assert np.array_equal(part, whole[4:7])
        assert not np.array_equal(probs.rounded(p[4:7], law, param, 31, 1, 6), whole[4:7])
        a = probs.mc_sums(p, V, law, param, 31, 3, 2)
        c = probs.mc_sums(p[4:7], V, law, param, 31, 3, 2, first_row=4)
        for x, y in zip(a, c):
            assert np.array_equal(x[:, 4:7], y)

