"""Averages over the forward's rounding on the GPU (bsp_coupling_check) against the oracle on the
same draws: the paired statistic T and its control pair by pair, the gain-use error with its split
into mean part and coupling, the fresh read, and the estimator X; then the closed forms."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import coupling, fp8, norm
from paper_2609_39813_b200 import workloads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_39813_b200 import binding
    binding.lib()
    return binding


from gpu_util import down, rel_l2, up  # noqa: E402


def _run(b, inp, pairs, mode=1):
    kind = b.RMSNORM if inp.norm == "rms" else b.LAYERNORM
    x, gamma, W = up(inp.x, inp.dtype), up(inp.gamma), up(inp.W, inp.dtype)
    beta = up(inp.beta) if inp.beta is not None else None
    d = b.CouplingDesc()
    d.norm_kind, d.dtype = kind, b.BF16 if inp.dtype == "bf16" else b.F32
    d.T, d.C, d.O = inp.T, inp.C, inp.O
    d.x, d.gamma, d.beta, d.W = b.ptr(x), b.ptr(gamma), b.ptr(beta), b.ptr(W)
    d.eps, d.store_fmt, d.forward_mode, d.seed, d.tensor_id = inp.eps, fp8.E4M3, mode, inp.seed, coupling.TENSOR_U
    ws = b.workspace(b.bsp_coupling_check_workspace_bytes(d, pairs))
    diag = b.new_diag()
    T, ctl = b.bsp_coupling_check(d, pairs, ws, diag)
    assert b.read_diag(diag)["status"] == 0
    lay = b.bsp_coupling_layout(d, pairs)
    C, O = inp.C, inp.O
    out = dict(T=np.array(T), control=np.array(ctl),
               gain_total=down(b.ws_view(ws, lay.gain_total, C)).astype(np.float64),
               gain_mean_part=down(b.ws_view(ws, lay.gain_mean_part, C)).astype(np.float64),
               gain_fresh=down(b.ws_view(ws, lay.gain_fresh, C)).astype(np.float64),
               X=down(b.ws_view(ws, lay.X, C * O)).reshape(C, O).astype(np.float64),
               X_sq=down(b.ws_view(ws, lay.X_sq, C * O)).reshape(C, O).astype(np.float64))
    # the statistics the GPU saved, for the oracle's teacher forcing
    rstd = torch.zeros(inp.T, device="cuda"); mean = torch.zeros(inp.T, device="cuda"); amax = torch.zeros(1, device="cuda")
    b.bsp_norm_stats(kind, x, inp.T, inp.C, gamma, beta, inp.eps, rstd, mean, amax)
    return out, down(rstd), down(mean)


CASES = {
    "rms_bf16_ragged": lambda: workloads.config2(T=200, C=128, O=96, K=4, seed=21),
    "layernorm_f32": lambda: workloads.config4(T=160, C=96, O=64, K=4, seed=22),
}


@pytest.mark.parametrize("name", list(CASES))
def test_against_the_oracle_on_the_same_draws(b, name):
    inp = CASES[name]()
    if inp.dtype == "f32":          # W reaches the tensor cores as bf16: give both sides that W
        inp.W = workloads.to_bf16_grid(inp.W)
    pairs = 5
    got, rstd, mean = _run(b, inp, pairs)
    kind = norm.RMS if inp.norm == "rms" else norm.LAYER
    prep = coupling.prepare(inp.x, inp.gamma, inp.beta, inp.W, kind, inp.eps, rstd32=rstd,
                            mean32=mean if kind == norm.LAYER else None)
    want = coupling.run(prep, inp.seed, pairs)
    assert np.allclose(got["T"], want["T"], rtol=2e-4, atol=1e-6 * np.max(np.abs(want["T"])))
    assert np.allclose(got["control"], want["control"], rtol=0, atol=2e-4 * np.max(np.abs(want["control"])) + 1e-6 * np.sqrt(np.mean(want["T"] ** 2)) * 100)
    assert rel_l2(got["gain_total"], want["gain_total"]) <= 2e-4
    assert rel_l2(got["gain_fresh"], want["gain_fresh"]) <= 2e-4
    assert np.linalg.norm(got["gain_mean_part"] - want["gain_mean_part"]) <= 2e-4 * np.linalg.norm(want["gain_total"])
    assert rel_l2(got["X"], want["X"]) <= 2e-3


def test_at_the_390m_shape(b):
    """Config 2's tensors (T = 4096, C = 1024, O = 4096, bf16, outlier channels), two pairs of forwards:
    the contractions at the size the benchmark times them, against the oracle on the same draws."""
    inp = workloads.config2()
    pairs = 2
    got, rstd, _ = _run(b, inp, pairs)
    prep = coupling.prepare(inp.x, inp.gamma, None, inp.W, norm.RMS, inp.eps, rstd32=rstd)
    want = coupling.run(prep, inp.seed, pairs)
    assert np.allclose(got["T"], want["T"], rtol=5e-4)
    assert np.max(np.abs(got["control"] - want["control"])) <= 5e-4 * np.max(np.abs(want["T"]))
    assert rel_l2(got["gain_total"], want["gain_total"]) <= 5e-4
    assert rel_l2(got["gain_fresh"], want["gain_fresh"]) <= 5e-4
    assert rel_l2(got["X"], want["X"]) <= 2e-3


def test_closed_forms_and_round_to_nearest(b):
    inp = workloads.config2(T=256, C=128, O=128, K=4, seed=23)
    pairs = 200
    got, rstd, _ = _run(b, inp, pairs)
    prep = coupling.prepare(inp.x, inp.gamma, None, inp.W, norm.RMS, inp.eps, rstd32=rstd)
    cf = coupling.closed_forms(prep)
    T, ctl = got["T"], got["control"]
    se = T.std(ddof=1) / np.sqrt(pairs)
    assert abs(T.mean() - cf["T"]) < 5 * se and T.mean() / se > 10
    assert abs(ctl.mean()) < 5 * ctl.std(ddof=1) / np.sqrt(pairs)
    # X against -diag(sum_t sigma^2) W^T: close to it, and the deviation is no more than sampling error
    # (the paper's statistic R on the deviation; the outlier channels of this workload carry most of
    # the variance, so R itself scatters more than 16384 entries would suggest), while X is resolved
    se2 = np.maximum(got["X_sq"] - got["X"] ** 2, 0) / pairs
    assert rel_l2(got["X"], cf["X"]) < 0.05
    assert np.sum((got["X"] - cf["X"]) ** 2) / np.sum(se2) < 2.0
    assert np.sum(got["X"] ** 2) / np.sum(se2) > 100.0
    # the gain error is all coupling; a fresh read shows none
    # (400 forwards leave about 15 % of sampling noise on these column sums; the tight comparison is
    # the one against the oracle on the same draws above)
    assert np.linalg.norm(got["gain_total"] - cf["gain"]) < 0.3 * np.linalg.norm(cf["gain"])
    assert np.linalg.norm(got["gain_total"] - got["gain_mean_part"] - cf["gain"]) < 0.4 * np.linalg.norm(cf["gain"])
    assert np.linalg.norm(got["gain_fresh"]) < 0.4 * np.linalg.norm(cf["gain"])
    assert np.sum(got["gain_total"] * cf["gain"]) / (np.linalg.norm(got["gain_total"]) * np.linalg.norm(cf["gain"])) > 0.95
    # round-to-nearest: identical forwards, T and X exactly zero
    rn, _, _ = _run(b, inp, 3, mode=0)
    assert not rn["T"].any() and not rn["X"].any()
