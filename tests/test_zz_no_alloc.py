"""The no-allocation variant of the normalisation backward.

Some users of this library run where they cannot obtain device memory for scratch: inside a host
application that owns the whole GPU pool, under a fixed memory quota, or in a loop that must not
hit cudaMalloc's device-wide synchronisation.  For them `bsp_norm_bwd_noalloc` keeps its scratch
in a fixed array that ships inside the library.  This file checks, through the C ABI, that it
returns what `bsp_norm_bwd` returns -- twice in a row, because the array is shared by all calls
and keeps the previous call's contents -- and that it refuses problems beyond its capacity.

Collected last on purpose (file name), so a run that stops at the first failure has already
exercised everything else; it also passes when run alone in a fresh process.
"""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from paper_2609_39813_b200 import workloads

pytestmark = pytest.mark.gpu

TOL_FP32 = 1e-5      # the bar of the other CUDA-core FP32 gradient tests


@pytest.fixture(scope="module")
def b():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_39813_b200 import binding
    binding.lib()
    return binding


def _rel(a, ref):
    a, ref = a.double().cpu().numpy().ravel(), ref.double().cpu().numpy().ravel()
    return float(np.linalg.norm(a - ref) / max(np.linalg.norm(ref), 1e-300))


def _run_both(b, inp, gain_read, draw):
    from paper_2609_39813_b200.harness import NormLinearGpu, up
    g = NormLinearGpu(inp)
    T, C = inp.T, inp.C
    rng = np.random.default_rng(inp.seed + draw)
    du_np = rng.standard_normal((T, C)).astype(np.float32)
    du = up(workloads.to_bf16_grid(du_np) if inp.dtype == "bf16" else du_np, inp.dtype)
    key = b.key(inp.seed, g.tensor_id, b.STREAM_GAIN, draw)
    outs = []
    for which in ("workspace", "noalloc"):
        dg = torch.full((C,), float("nan"), device="cuda")
        db = torch.full((C,), float("nan"), device="cuda")
        dx = torch.full((T * C,), float("nan"), device="cuda")
        if which == "workspace":
            ws = b.workspace(b.bsp_norm_bwd_workspace_bytes(T, C))
            b.bsp_norm_bwd(g.kind, g.x, T, C, g.gamma, g.beta, g.rstd, g.mean, du, gain_read, g.u_codes, g.q, key,
                           dg, db, dx, ws)
        else:
            b.bsp_norm_bwd_noalloc(g.kind, g.x, T, C, g.gamma, g.beta, g.rstd, g.mean, du, gain_read, g.u_codes,
                                   g.q, key, dg, db, dx)
        torch.cuda.synchronize()
        outs.append((dg, db, dx))
    (dg0, db0, dx0), (dg1, db1, dx1) = outs
    for a, r in ((dg1, dg0), (db1, db0), (dx1, dx0)):
        assert torch.isfinite(a).all() and torch.isfinite(r).all()
        assert _rel(a, r) <= TOL_FP32
    if gain_read == b.READ_ORIGINAL:
        # and against the float64 checker, not only against the sibling entry point
        from oracle import norm
        kind = norm.RMS if inp.norm == "rms" else norm.LAYER
        du64 = du.float().cpu().numpy().astype(np.float64)
        want = norm.backward(inp.x, inp.gamma, inp.beta, kind, inp.eps, du64)
        for a, r in ((dg1, want["dgamma"]), (db1, want["dbeta"]), (dx1, want["dx"])):
            assert _rel(a, torch.from_numpy(np.ascontiguousarray(r))) <= TOL_FP32


def test_noalloc_matches_workspace_entry_two_calls_in_a_row(b):
    # first a larger problem, then a smaller one of another norm kind and policy: the second call
    # finds the first call's partials still in the shared array and must not be affected by them
    _run_both(b, workloads.config2(T=700, C=512, O=64, K=2), b.READ_FRESH, draw=1)
    _run_both(b, workloads.config4(T=90, C=320, O=64, K=2), b.READ_FORWARD, draw=0)
    # and the first problem once more, after the smaller one
    _run_both(b, workloads.config2(T=700, C=512, O=64, K=2), b.READ_ORIGINAL, draw=0)


def test_noalloc_rejects_problems_beyond_its_capacity(b):
    T, C = 4096, 8192                      # needs 592 * 8192 * 4 * 2 bytes > 20 MiB
    assert b.bsp_norm_bwd_workspace_bytes(T, C) > b.NORM_BWD_NOALLOC_CAPACITY_BYTES
    dg = torch.full((C,), 7.0, device="cuda")
    dummy = torch.zeros(16, device="cuda")
    with pytest.raises(b.BspError) as e:
        b.bsp_norm_bwd_noalloc(b.RMSNORM, dummy, T, C, dummy, None, dummy, None, dummy, b.READ_ORIGINAL, None,
                               b.quant(0, 0, 1.0), b.key(0, 1, 1), dg, None, None)
    assert e.value.status == b.ERR_TOO_LARGE and "capacity" in str(e.value)
    torch.cuda.synchronize()
    assert bool((dg == 7.0).all())           # nothing was launched, no output touched
    # the largest width that always fits
    assert b.bsp_norm_bwd_workspace_bytes(1 << 20, 4096) <= b.NORM_BWD_NOALLOC_CAPACITY_BYTES
