"""Rounded attention probabilities on the GPU (bsp_probs_mc) against the oracle's Monte-Carlo form
draw for draw, and against the paper's closed forms (the table of average errors and the operators
built from new roundings) within sampling error."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import probs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_39813_b200 import binding
    binding.lib()
    return binding


def _rows(R, n, d, seed):
    rng = np.random.default_rng(seed)
    s = rng.standard_normal((R, n)) * 1.5
    p = np.exp(s - s.max(1, keepdims=True))
    p = (p / p.sum(1, keepdims=True)).astype(np.float32)
    V = (rng.standard_normal((n, d)) / np.sqrt(d)).astype(np.float32)
    return p, V


def _run(b, p, V, law, param, seed, draw0, K):
    R, n = p.shape
    d = V.shape[1]
    ds = torch.zeros(5 * R * n, device="cuda")
    sq = torch.zeros(5 * R * n, device="cuda")
    dV = torch.zeros(2 * R * n * d, device="cuda")
    b.bsp_probs_mc(torch.from_numpy(p).cuda(), torch.from_numpy(V).cuda(), R, n, d, law, param, seed, probs.TENSOR_P,
                   draw0, K, ds, sq, dV)
    torch.cuda.synchronize()
    return (ds.cpu().numpy().reshape(5, R, n).astype(np.float64), sq.cpu().numpy().reshape(5, R, n).astype(np.float64),
            dV.cpu().numpy().reshape(2, R, n, d).astype(np.float64))


@pytest.mark.parametrize("R,n,d,law,param", [(7, 4, 3, 0, 0.125), (5, 3, 2, 1, 0.125), (33, 48, 16, 0, 1.0 / 64),
                                            (9, 200, 64, 1, 1.0 / 512), (3, 256, 64, 0, 1.0 / 256),
                                            # 128 x 64 takes the kernel of its own (eight draws at a time: K = 9 leaves one over)
                                            (11, 128, 64, 0, 1.0 / 64), (6, 128, 64, 1, 1.0 / 512),
                                            (600, 128, 64, 0, 1.0 / 64)])       # more blocks than the GPU holds at once
def test_sums_match_the_oracle_draw_for_draw(b, R, n, d, law, param):
    p, V = _rows(R, n, d, 5 + n)
    K, draw0 = 9, 3
    ds, sq, dV = _run(b, p, V, law, param, 41, draw0, K)
    want_ds, want_sq, want_dV = probs.mc_sums(p, V, law, param, 41, K, draw0)
    # FP32 sums of K errors: relative to the size of the largest error of the operator / read
    for i in range(5):
        scale = np.max(np.abs(want_ds[i])) + 1e-30
        assert np.max(np.abs(ds[i] - want_ds[i])) <= 2e-5 * scale, (i, np.max(np.abs(ds[i] - want_ds[i])) / scale)
        assert np.max(np.abs(sq[i] - want_sq[i])) <= 1e-4 * (np.max(np.abs(want_sq[i])) + 1e-30)
    for i in range(2):
        scale = np.max(np.abs(want_dV[i])) + 1e-30
        assert np.max(np.abs(dV[i] - want_dV[i])) <= 2e-5 * scale


def test_bench_size_on_sampled_rows(b):
    """The size `bench.py` times (16384 rows of 128 probabilities, d = 64, grid 1/64, 256 draws; rows
    drawn by the same recipe): blocks of rows from the start, the middle and the end of the tensor
    against the oracle on those rows alone, keyed by their place in the whole tensor."""
    R, n, d, K = 16384, 128, 64, 256
    rng = np.random.default_rng(3003)
    sc = rng.standard_normal((R, n)) * 1.5
    p = np.exp(sc - sc.max(1, keepdims=True))
    p = (p / p.sum(1, keepdims=True)).astype(np.float32)
    V = (rng.standard_normal((n, d)) / np.sqrt(d)).astype(np.float32)
    ds = torch.zeros(5 * R * n, device="cuda")
    sq = torch.zeros(5 * R * n, device="cuda")
    dV = torch.zeros(2 * R * n * d, device="cuda")
    b.bsp_probs_mc(torch.from_numpy(p).cuda(), torch.from_numpy(V).cuda(), R, n, d, 0, 1.0 / 64, 3003, probs.TENSOR_P, 0, K,
                   ds, sq, dV)
    torch.cuda.synchronize()
    ds, sq, dV = ds.view(5, R, n), sq.view(5, R, n), dV.view(2, R, n, d)
    for r0, m in ((0, 3), (8191, 3), (R - 2, 2)):
        want_ds, want_sq, want_dV = probs.mc_sums(p[r0:r0 + m], V, 0, 1.0 / 64, 3003, K, 0, first_row=r0)
        got_ds = ds[:, r0:r0 + m].cpu().numpy().astype(np.float64)
        got_sq = sq[:, r0:r0 + m].cpu().numpy().astype(np.float64)
        got_dV = dV[:, r0:r0 + m].cpu().numpy().astype(np.float64)
        for i in range(5):
            # FP32 sums of 256 errors
            assert np.max(np.abs(got_ds[i] - want_ds[i])) <= 1e-4 * (np.max(np.abs(want_ds[i])) + 1e-30), (r0, i)
            assert np.max(np.abs(got_sq[i] - want_sq[i])) <= 3e-4 * (np.max(np.abs(want_sq[i])) + 1e-30), (r0, i)
        for i in range(2):
            assert np.max(np.abs(got_dV[i] - want_dV[i])) <= 1e-4 * (np.max(np.abs(want_dV[i])) + 1e-30), (r0, i)


def test_cells_of_the_paper_on_the_gpu(b):
    """Cells A and B as rows of the kernel: the averages over 40 000 draws against the exact
    enumeration (every operator, both reads), within five standard errors."""
    K = 40000
    for name, cell in (("A", probs.CELL_A), ("B", probs.CELL_B)):
        p = np.array([[float(x) for x in cell["p"]]], np.float32)
        V = np.array([[float(x) for x in row] for row in cell["V"]], np.float32)
        for law_id, kind, param in ((0, "sr", float(cell["grid"])), (1, "sym", 0.125)):
            law = probs.law_stochastic(cell["p"], cell["grid"]) if kind == "sr" else probs.law_symmetric(cell["p"], 0.125)
            ds, sq, dV = _run(b, p, V, law_id, param, 99, 0, K)
            mean = ds[:, 0] / K
            se = np.sqrt(np.maximum(sq[:, 0] / K - mean ** 2, 0) / K)
            for i, pol in enumerate(("R/R", "N/N", "K(f)/R", "J2(f,b)/R", "J2(q,b)/R")):
                if pol == "J2(f,b)/R" and name == "A" and kind == "sr":
                    want = np.zeros(len(cell["p"]))
                else:
                    want = np.array([float(x) for x in probs.average_errors(cell, law, pol)[0]])
                assert np.all(np.abs(mean[i] - want) <= 5 * se[i] + 2e-5), (name, kind, pol, mean[i], want)
            for i, pol in enumerate(("U/U", "N/N")):
                want = np.array([[float(x) for x in row] for row in probs.average_errors(cell, law, pol)[1]])
                # |Delta_V| <= step * |h|: a bound on the standard error of its mean
                bound = 5 * 2 * param * np.max(np.abs(V).sum(0)) / np.sqrt(K)
                assert np.max(np.abs(dV[i, 0] / K - want)) <= bound, (name, kind, pol)
                assert np.max(np.abs(dV[i, 0] / K - want)) < 0.35 * np.max(np.abs(want)) or np.max(np.abs(want)) == 0


def test_closed_forms_on_attention_sized_rows(b):
    """2048 rows of 64 probabilities with 64-wide values, a grid of 1/64: R/R's error at the softmax's
    backward is delta, a plugged-in new rounding leaves -Sigma_r G p, K(a) and J2(a, b) are right on
    average, the half-replayed J2 leaves half of it; both reads at the gradient of V leave -sigma_j^2 v_j^T."""
    R, n, d, K = 2048, 64, 64, 512
    p, V = _rows(R, n, d, 3)
    law, param = 0, 1.0 / 64
    ds, sq, dV = _run(b, p, V, law, param, 7, 0, K)
    cf = probs.closed_forms_rows(p, V, law, param)
    want = [cf["delta"], cf["minus_SGp"], np.zeros_like(cf["delta"]), np.zeros_like(cf["delta"]), cf["half_replay"]]
    for i in range(5):
        mean = ds[i] / K
        se2 = np.maximum(sq[i] / K - mean ** 2, 0) / K
        # the paper's detection statistic on the deviation from the closed form: the squared norm of the
        # mean deviation over the summed squared standard errors is about one when the closed form is
        # right (entry-wise z-scores are no use here: an entry far below the grid step moves in a handful
        # of the draws, and its sample standard error is then unreliable)
        R_dev = np.sum((mean - want[i]) ** 2) / np.sum(se2)
        assert 0.85 < R_dev < 1.2, (i, R_dev)
        # while R/R's error itself is resolved (the others are too small for 512 draws), and the two
        # operators that are right on average show nothing
        R_err = np.sum(mean ** 2) / np.sum(se2)
        if i == 0:
            assert R_err > 1.5, (i, R_err)
        if i in (2, 3):
            assert R_err < 1.2, (i, R_err)
    for i in range(2):
        got = dV[i] / K
        # entry by entry 512 draws do not resolve -sigma_j^2 v_j^T; pooled they do: project each row of
        # the mean error on its v_j and regress the coefficients on -sigma_j^2 over all rows and entries
        vv = np.sum(V.astype(np.float64) ** 2, axis=1)[None, :]
        coef = np.sum(got * V.astype(np.float64)[None, :, :], axis=2) / vv
        slope = np.sum(coef * (-cf["s2"])) / np.sum(cf["s2"] ** 2)
        assert abs(slope - 1) < 0.1, (i, slope)
