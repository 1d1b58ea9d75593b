"""The log-softmax +-eps test on the GPU (Appendix "Log-softmax") against the oracle trial by trial,
and its registered statements at the paper's sizes (128 classes, 64 rows, 4096 trials)."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import logsoftmax as ls

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_39813_b200 import binding
    binding.lib()
    return binding


def _inputs(rows, classes, seed):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((rows, classes)).astype(np.float32), rng.integers(0, classes, rows).astype(np.int32)


@pytest.mark.parametrize("rows,classes,eps", [(64, 128, 0.1), (5, 36, 0.5), (3, 1028, 0.25)])
def test_per_trial_statistics_match_the_oracle(b, rows, classes, eps):
    logits, target = _inputs(rows, classes, 11)
    trials = 48
    pt = torch.zeros(trials * 6, device="cuda")
    ws = b.workspace(b.bsp_lsm_check_workspace_bytes(rows, classes, trials))
    stats = b.bsp_lsm_check(torch.from_numpy(logits).cuda(), torch.from_numpy(target).cuda(), rows, classes, eps, trials,
                            77, ls.TENSOR_S, pt, ws)
    want, (mean, se, z) = ls.run(logits, target, eps, 77, trials)
    got = pt.cpu().numpy().reshape(trials, 6)
    # FP32 evaluation of the operator: each entry's error over p_j carries about 1e-6 of rounding
    scale = np.maximum(np.abs(want[:, :6]), eps * eps)
    assert np.max(np.abs(got - want[:, :6]) / scale) <= 2e-4
    for c in range(8):
        assert abs(stats[c].mean - mean[c]) <= 2e-4 * max(abs(mean[c]), eps * eps)
        assert abs(stats[c].se - se[c]) <= 1e-3 * se[c] + 1e-9
    # determinism
    pt2 = torch.zeros_like(pt)
    b.bsp_lsm_check(torch.from_numpy(logits).cuda(), torch.from_numpy(target).cuda(), rows, classes, eps, trials, 77,
                    ls.TENSOR_S, pt2, ws)
    assert torch.equal(pt, pt2)


@pytest.mark.parametrize("eps", [0.1, 0.5])
def test_registered_statements(b, eps):
    rows, classes, trials = 64, 128, 4096
    logits, target = _inputs(rows, classes, 1926)
    ws = b.workspace(b.bsp_lsm_check_workspace_bytes(rows, classes, trials))
    s = b.bsp_lsm_check(torch.from_numpy(logits).cuda(), torch.from_numpy(target).cuda(), rows, classes, eps, trials,
                        1926, ls.TENSOR_S, None, ws)
    pred = ls.predicted(eps)
    effect = abs(pred[2])
    assert abs(s[6].mean) + 1.96 * s[6].se < 0.05 * effect                      # LS1: reuse changes nothing under the likelihood
    assert abs(s[0].mean / pred[0] - 1) < 0.01 and s[0].z > 5                   # LS2: mean error cosh(eps) - 1
    assert abs(s[1].mean / pred[1] - 1) < 0.01 and s[1].z > 5                   #      for either copy
    assert abs(s[2].mean / pred[2] - 1) < 0.05 and s[2].z > 5                   # LS3: reuse shifts by -eps sinh(eps)
    assert abs(s[7].mean / pred[7] - 1) < 0.05 and s[7].z > 5
    assert abs(s[3].mean) + 1.96 * s[3].se < 0.10 * pred[0]                     # LS4': the independent copy's mean error is zero
    assert abs(s[4].mean) + 1.96 * s[4].se < 0.05 * pred[0]                     # LS5a: the division removes the likelihood's error
    assert abs(s[5].mean / pred[2] - 1 / np.cosh(eps)) < 0.05                   # LS5b: the coupling stays, scaled by 1 / cosh
    if eps == 0.5:                                                               # the constants, not their leading terms
        assert abs(s[0].mean / (eps * eps / 2) - 1) >= 0.01 and abs(s[2].mean / (-eps * eps) - 1) >= 0.02


def test_vocabulary_sized_rows_on_sampled_trials(b):
    """The size `bench.py` times beside the paper's (256 rows of 8192 classes, 256 trials, eps 0.1,
    seeded inputs of the same law): sampled trials against the oracle's per-trial statistics, and the
    summary against the oracle's summary of the GPU's own per-trial values."""
    rows, classes, trials, eps = 256, 8192, 256, 0.1
    rng = np.random.default_rng(1926)
    logits = rng.standard_normal((rows, classes)).astype(np.float32)
    target = rng.integers(0, classes, rows).astype(np.int32)
    pt = torch.zeros(trials * 6, device="cuda")
    ws = b.workspace(b.bsp_lsm_check_workspace_bytes(rows, classes, trials))
    stats = b.bsp_lsm_check(torch.from_numpy(logits).cuda(), torch.from_numpy(target).cuda(), rows, classes, eps, trials,
                            1926, ls.TENSOR_S, pt, ws)
    got = pt.cpu().numpy().reshape(trials, 6).astype(np.float64)
    for t in (0, 1, 100, 255):
        want = ls.trial_statistics(logits, target, eps, 1926, t)
        scale = np.maximum(np.abs(want), eps * eps)
        assert np.max(np.abs(got[t] - want) / scale) <= 2e-4, (t, got[t], want)
    full = np.concatenate([got, (got[:, 0] - got[:, 1])[:, None], (got[:, 2] - got[:, 3])[:, None]], axis=1)
    mean, se, z = ls.summarise(full)
    for c in range(8):
        assert abs(stats[c].mean - mean[c]) <= 1e-5 * max(abs(mean[c]), eps * eps)
        assert abs(stats[c].se - se[c]) <= 1e-3 * se[c] + 1e-12


def test_argument_errors(b):
    x, y = torch.zeros(8 * 6, device="cuda"), torch.zeros(8, dtype=torch.int32, device="cuda")
    ws = b.workspace(4096)
    with pytest.raises(b.BspError):
        b.bsp_lsm_check(x, y, 8, 6, 0.1, 16, 0, 3, None, ws)              # classes not a multiple of 4
    with pytest.raises(b.BspError):
        b.bsp_lsm_check(x, y, 6, 8, 0.1, 1, 0, 3, None, ws)               # fewer than two trials
    with pytest.raises(b.BspError):
        b.bsp_lsm_check(x, y, 6, 8, 0.1, 1 << 20, 0, 3, None, ws)         # workspace too small
