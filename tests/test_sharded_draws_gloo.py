"""The draw-sharded form of the check on two gloo ranks on CPU: the partition of the draws, the one
exchange (a sum of the shifted sums over ranks), and that merged partial sums give the statistics of
the single run.  The per-rank partial sums come from the oracle here (no GPU in this test); the
GPU side of the same path is tests/test_gpu_sharded.py."""
import os

import numpy as np
import pytest

torch = pytest.importorskip("torch")
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import check, linear, mc, norm, philox
from paper_2609_39813_b200 import sharded, workloads


def test_draw_ranges_cover_the_draws_once():
    for K in (0, 1, 4, 7, 16, 1024):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                k0, nd = sharded.draw_range(K, world, r)
                assert nd in (K // world, K // world + 1)
                seen += list(range(k0, k0 + nd))
            assert seen == list(range(K))
    with pytest.raises(ValueError):
        sharded.draw_range(4, 2, 2)


def _partial_sums(inp, prep, ref_g, ref_w, k0, nd):
    """S1, S2 of the gain use and the weight use over draws [k0, k0 + nd), as the oracle sees them."""
    kind = norm.RMS if inp.norm == "rms" else norm.LAYER
    s1g, s2g = np.zeros_like(ref_g), np.zeros_like(ref_g)
    s1w, s2w = np.zeros_like(ref_w), np.zeros_like(ref_w)
    dyv = prep["dy"]["value"]
    for k in range(k0, k0 + nd):
        cg, _ = check.fresh_copy(prep, inp.seed, philox.STREAM_GAIN, k)
        d = norm.dgamma_from_copy(cg, inp.gamma, inp.beta, prep["du"]) - ref_g
        s1g += d; s2g += d * d
        cw, _ = check.fresh_copy(prep, inp.seed, philox.STREAM_WGRAD, k)
        e = linear.wgrad(dyv, cw, None, None) - ref_w
        s1w += e; s2w += e * e
    return s1g, s2g, s1w, s2w


def _setup():
    inp = workloads.config1()
    kind = norm.RMS if inp.norm == "rms" else norm.LAYER
    prep = check.prepare_norm_linear(inp.x, inp.gamma, inp.beta, inp.W, inp.dY, kind, inp.eps, inp.seed, inp.dtype)
    ref_g = norm.backward(inp.x, inp.gamma, inp.beta, kind, inp.eps, prep["du"])["dgamma"]
    ref_w = linear.wgrad(prep["dy"]["value"], norm.read_value(prep["codes"], prep["store_fmt"], prep["inv_scale"]), None, None)
    return inp, prep, ref_g, ref_w


def _worker(rank, world, port, K, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    inp, prep, ref_g, ref_w = _setup()
    k0, nd = sharded.draw_range(K, world, rank)
    sums = [torch.from_numpy(a.copy()) for a in _partial_sums(inp, prep, ref_g, ref_w, k0, nd)]
    sharded.merge_sums(sums)                                  # the one exchange
    out[rank] = [s.numpy().copy() for s in sums]
    dist.barrier()
    dist.destroy_process_group()


def test_merged_partial_sums_equal_the_single_run():
    K, world = 7, 2                                            # an uneven split: 4 + 3 draws
    mgr = mp.Manager()
    out = mgr.dict()
    port = 31500 + os.getpid() % 2000
    mp.spawn(_worker, args=(world, port, K, out), nprocs=world, join=True)
    inp, prep, ref_g, ref_w = _setup()
    whole = _partial_sums(inp, prep, ref_g, ref_w, 0, K)
    for r in range(world):
        for got, want in zip(out[r], whole):
            np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-18)
    # and the statistics from merged sums are those of the oracle's own K-draw evaluation
    kind = norm.RMS if inp.norm == "rms" else norm.LAYER
    for (s1, s2, ref), use in (((out[0][0], out[0][1], ref_g), check.gain_use(inp.x, inp.gamma, inp.beta, kind, inp.eps, prep, check.N, K, inp.seed)),
                               ((out[0][2], out[0][3], ref_w), check.wgrad_use(prep, check.N, K, inp.seed))):
        mean = ref + s1 / K
        m2 = s2 - s1 * s1 / K
        st = mc.statistics(mean, m2, K, ref, True)
        assert st.verdict == use["stats"].verdict
        assert st.R == pytest.approx(use["stats"].R, rel=1e-8)
        assert st.Qprime == pytest.approx(use["stats"].Qprime, rel=1e-8)


def test_merge_is_identity_in_one_process():
    t = [torch.arange(5, dtype=torch.float64), torch.ones(3, dtype=torch.float64)]
    sharded.merge_sums(t)
    assert t[0].tolist() == [0, 1, 2, 3, 4] and t[1].tolist() == [1, 1, 1]
