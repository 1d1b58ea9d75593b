"""The draw-sharded fresh reads on one GPU: the ranks' shares are evaluated one after the other
through the draw-range entry points (no kernel waits on another), their sums are added as the
all-reduce would add them, and the statistics must be those of the single call of bsp_mc_check with
the same K.  The collective itself is covered on CPU (tests/test_sharded_draws_gloo.py)."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from paper_2609_39813_b200 import workloads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_39813_b200 import binding
    binding.lib()
    return binding


@pytest.mark.parametrize("name,world", [("cfg1", 2), ("cfg2_small", 3), ("cfg4_small", 2)])
def test_sharded_draws_match_the_single_call(b, name, world):
    from paper_2609_39813_b200.harness import NormLinearGpu
    from paper_2609_39813_b200.sharded import ShardedFreshReads
    inp = {"cfg1": lambda: workloads.config1(K=10),
           "cfg2_small": lambda: workloads.config2(T=300, C=256, O=192, K=11),
           "cfg4_small": lambda: workloads.config4(T=200, C=320, O=128, K=8)}[name]()
    K = inp.K
    g = NormLinearGpu(inp)
    ranks = [ShardedFreshReads(g, K, r, world, draw_buffer_draws=3) for r in range(world)]
    assert sum(r.nd for r in ranks) == K
    for r in ranks:
        r.prepare()
        r.local_sums()
    torch.cuda.synchronize()
    # what the all-reduce does: every rank ends up with the sum over ranks
    first = ranks[0]
    for name_ in ("S1g", "S2g", "S1w", "S2w"):
        total = sum(getattr(r, name_) for r in ranks)
        getattr(first, name_).copy_(total)
    rg, rw = first.statistics()
    # the single call
    d = g.desc(policy_mask=0b100100)                           # N at both uses
    ws = b.workspace(b.bsp_mc_check_workspace_bytes(d, K))
    diag = b.new_diag()
    res = [r for r in b.bsp_mc_check(d, K, ws, diag) if r.output_id != b.OUT_DBETA]
    assert b.read_diag(diag)["status"] == 0 and b.read_diag(g.diag)["status"] == 0 and len(res) == 2
    for got, want in ((rg, res[0]), (rw, res[1])):
        assert got.verdict == want.verdict
        for f in ("rel_l2_mean_err", "R", "Qprime"):
            a, w = getattr(got, f), getattr(want, f)
            assert a == pytest.approx(w, rel=2e-4, abs=1e-9), (f, a, w)
    # one rank alone takes all the draws and gives the same sums as the shares added up
    alone = ShardedFreshReads(g, K, 0, 1, draw_buffer_draws=4)
    alone.prepare()
    alone.local_sums()
    torch.cuda.synchronize()
    for name_ in ("S1g", "S2g", "S1w", "S2w"):
        a, w = getattr(first, name_).cpu().numpy().astype(np.float64), getattr(alone, name_).cpu().numpy().astype(np.float64)
        assert np.linalg.norm(a - w) <= 1e-5 * (np.linalg.norm(w) + 1e-30), name_
