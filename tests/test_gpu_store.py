"""The paper's b-bit per-token normalisation store on the GPU against the oracle: codes and steps
bit-exact, the copies its uses read, the weight gradient from the split operand, and the whole
per-use check (the table "Store policies": U/R exact, N right on average at the gain use, U/R+eps
right on average at the weight use, U and N failing at the weight use)."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import mc, norm, philox, store
from paper_2609_39813_b200 import workloads

pytestmark = pytest.mark.gpu

TOL_FP32 = 1e-5
TOL_TC = 2e-3


@pytest.fixture(scope="module")
def b():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2609_39813_b200 import binding
    binding.lib()
    return binding


from gpu_util import NormLinearGpu, ceil16, down, rel_l2, up  # noqa: E402

CASES = {
    "cfg1_6bit": (lambda: workloads.config1(), 6),
    "cfg1_5bit": (lambda: workloads.config1(), 5),
    "cfg2_small_bf16_ragged": (lambda: workloads.config2(T=300, C=256, O=192, K=8), 6),
    "cfg4_small_layernorm": (lambda: workloads.config4(T=200, C=320, O=128, K=8), 5),
}


@pytest.fixture(scope="module", params=list(CASES), ids=list(CASES))
def case(request, b):
    make, bits = CASES[request.param]
    inp = make()
    g = NormLinearGpu(inp)
    kind = norm.RMS if inp.norm == "rms" else norm.LAYER
    prep = store.prepare(inp.x, inp.gamma, inp.beta, inp.W, inp.dY, kind, inp.eps, inp.seed, bits, inp.dtype,
                         rstd32=down(g.rstd), mean32=down(g.mean) if kind == norm.LAYER else None)
    codes = torch.zeros(inp.T * inp.C, dtype=torch.int8, device="cuda")
    steps = torch.zeros(inp.T, device="cuda")
    b.bsp_store_fwd(g.kind, g.x, inp.T, inp.C, g.gamma, g.beta, g.rstd, g.mean, bits,
                    b.key(inp.seed, store.TENSOR_U, b.STREAM_FORWARD, 0), codes, steps)
    return inp, g, kind, prep, bits, codes, steps


def test_store_codes_and_steps_bit_exact(b, case):
    inp, g, kind, prep, bits, codes, steps = case
    assert np.array_equal(down(steps), prep["s32"])
    assert np.array_equal(codes.cpu().numpy().reshape(inp.T, inp.C).astype(np.int64), prep["codes"])
    # a fresh rounding under another stream and draw is another, equally exact, set of codes
    c2 = torch.zeros_like(codes)
    b.bsp_store_fwd(g.kind, g.x, inp.T, inp.C, g.gamma, g.beta, g.rstd, g.mean, bits,
                    b.key(inp.seed, store.TENSOR_U, b.STREAM_WGRAD, 3), c2, steps)
    want = store.store_codes(prep["u32"], prep["s32"], inp.seed, philox.STREAM_WGRAD, 3)
    assert np.array_equal(c2.cpu().numpy().reshape(inp.T, inp.C).astype(np.int64), want)
    assert not np.array_equal(want, prep["codes"])


def test_store_forward_on_a_width_that_is_no_multiple_of_16(b):
    """C = 200: a row that does not fill whole groups of 16 columns."""
    inp = workloads.config2(T=37, C=200, O=16, K=4, seed=31)
    kind = norm.RMS
    fw = norm.forward(inp.x, inp.gamma, None, kind, inp.eps)
    x = up(inp.x, inp.dtype)
    gamma = up(inp.gamma)
    rstd = up(fw["rstd"].astype(np.float32))
    u32 = norm.store_value_fp32(inp.x, inp.gamma, None, kind, fw["rstd"].astype(np.float32), None, None)
    for bits in (6, 5):
        s32 = store.steps(u32, bits)
        codes = torch.zeros(inp.T * inp.C, dtype=torch.int8, device="cuda")
        steps = torch.zeros(inp.T, device="cuda")
        b.bsp_store_fwd(b.RMSNORM, x, inp.T, inp.C, gamma, None, rstd, None, bits, b.key(inp.seed, store.TENSOR_U, b.STREAM_FORWARD, 0),
                        codes, steps)
        assert np.array_equal(down(steps), s32)
        want = store.store_codes(u32, s32, inp.seed, philox.STREAM_FORWARD, 0)
        assert np.array_equal(codes.cpu().numpy().reshape(inp.T, inp.C).astype(np.int64), want)


@pytest.mark.parametrize("read", [0, 1, 2, 3])
def test_copies_and_weight_gradient(b, case, read):
    inp, g, kind, prep, bits, codes, steps = case
    T, C, O = inp.T, inp.C, inp.O
    ld_t = ceil16(T)
    key = b.key(inp.seed, store.TENSOR_U, b.STREAM_WGRAD, 2)
    copy = torch.zeros(T * C, device="cuda")
    split = torch.full((C * 2 * ld_t,), 7.0, dtype=torch.bfloat16, device="cuda")
    b.bsp_store_read(g.kind, g.x, T, C, g.gamma, g.beta, g.rstd, g.mean, codes, steps, read, key, copy, split, ld_t)
    want = store.copy_for(prep, read, inp.seed, philox.STREAM_WGRAD, 2)
    assert rel_l2(down(copy).reshape(T, C), want) <= 1e-6
    sp = down(split).reshape(C, 2 * ld_t).astype(np.float64)
    assert rel_l2((sp[:, :T] + sp[:, ld_t:ld_t + T]).T, want) <= 2.0 ** -15
    assert not sp[:, T:ld_t].any() and not sp[:, ld_t + T:].any()          # padding zeroed
    dW = torch.zeros(O * C, device="cuda")
    ws = b.workspace(b.bsp_store_wgrad_workspace_bytes(T, O))
    diag = b.new_diag()
    b.bsp_store_wgrad(T, O, C, g.dy_codes_t, g.q_dy, split, ld_t, dW, ws, diag)
    assert b.read_diag(diag)["status"] == 0
    ref = prep["dy"]["value"].T @ want
    dist = rel_l2(down(dW).reshape(O, C), ref)
    assert dist <= 1e-4, dist          # operands carried to 16 bits: far inside the 2e-3 bar of the contractions


def _desc(b, g, inp, bits, mask=0x7F):
    d = b.StoreDesc()
    d.norm_kind = g.kind
    d.dtype = b.BF16 if inp.dtype == "bf16" else b.F32
    d.T, d.C, d.O = inp.T, inp.C, inp.O
    d.x, d.gamma, d.beta, d.W, d.dY = b.ptr(g.x), b.ptr(g.gamma), b.ptr(g.beta), b.ptr(g.W), b.ptr(g.dY)
    d.eps, d.bits, d.grad_fmt = inp.eps, bits, inp.grad_fmt
    d.seed, d.tensor_id, d.policy_mask = inp.seed, store.TENSOR_U, mask
    return d


EXPECTED = [mc.HOLDS, mc.FAILS, mc.HOLDS, mc.FAILS, mc.HOLDS, mc.FAILS, mc.HOLDS]


def test_mc_check_store_verdicts_and_statistics(b, case):
    inp, g, kind, prep, bits, codes, steps = case
    K = 24
    d = _desc(b, g, inp, bits)
    ws = b.workspace(b.bsp_mc_check_store_workspace_bytes(d, K))
    diag = b.new_diag()
    res = b.bsp_mc_check_store(d, K, ws, diag)
    assert len(res) == 7 and b.read_diag(diag)["status"] == 0
    assert [(r.use_id, r.policy) for r in res] == [(b.STREAM_GAIN, p) for p in (0, 1, 2)] + [(b.STREAM_WGRAD, p) for p in (0, 1, 2, 3)]
    # the oracle on the du the GPU's helper made: it sits in the workspace after the two code tensors
    # of dY; simpler and independent of the layout: recompute it through the public helper
    du = torch.zeros(inp.T * inp.C, dtype=torch.bfloat16 if inp.dtype == "bf16" else torch.float32, device="cuda")
    wsd = b.workspace(b.bsp_linear_dgrad_workspace_bytes(inp.T, inp.O, inp.C))
    b.bsp_linear_dgrad(inp.T, inp.O, inp.C, g.dy_codes, g.q_dy, g.W, du, wsd)
    prep2 = dict(prep, du=down(du).reshape(inp.T, inp.C).astype(np.float64))
    want = [store.gain_use(inp.x, inp.gamma, inp.beta, kind, inp.eps, prep2, p, K, inp.seed)["stats"] for p in (0, 1, 2)]
    want += [store.wgrad_use(prep2, p, K, inp.seed)["stats"] for p in (0, 1, 2, 3)]
    for r, w, e in zip(res, want, EXPECTED):
        assert r.verdict == w.verdict == e, (r.as_dict(), w)
        assert r.K == w.K and r.n_elements == w.n_elements
        if r.policy in (0, 1):
            assert np.isclose(r.rel_l2_mean_err, w.rel_l2_mean_err, rtol=2e-3, atol=1e-9)
        else:
            for f in ("rel_l2_mean_err", "R", "Qprime", "rms_z"):
                assert np.isclose(getattr(r, f), getattr(w, f), rtol=5e-3, atol=1e-9), (r.as_dict(), w, f)
    assert res[0].rel_l2_mean_err == 0.0 and res[4].rel_l2_mean_err == 0.0
    res2 = b.bsp_mc_check_store(d, K, ws, diag)
    assert [bytes(r) for r in res] == [bytes(r) for r in res2]


def test_mc_check_store_at_the_390m_shape(b):
    """Config 2's shape (T = 4096, C = 1024, O = 4096, bf16) with the 6-bit store, K = 16: the
    verdict table, and the statistics of the U/R+eps read against the oracle on a column block."""
    inp = workloads.config2()
    g = NormLinearGpu(inp)
    K, bits = 16, 6
    d = _desc(b, g, inp, bits)
    ws = b.workspace(b.bsp_mc_check_store_workspace_bytes(d, K))
    diag = b.new_diag()
    res = b.bsp_mc_check_store(d, K, ws, diag)
    assert b.read_diag(diag)["status"] == 0
    assert [r.verdict for r in res] == EXPECTED
    assert res[0].rel_l2_mean_err == 0.0 and res[4].rel_l2_mean_err == 0.0
    # the size of the errors: a 6-bit grid per token is a few per cent of the gradient
    assert 0.005 < res[1].rel_l2_mean_err < 0.5 and 0.005 < res[3].rel_l2_mean_err < 0.5
    assert res[6].Qprime < 1.6 and res[6].R < 2.0 and res[5].R > 6.0
    # a column block of the weight use through the single entry points, against the oracle
    prep = store.prepare(inp.x, inp.gamma, None, inp.W, inp.dY, norm.RMS, inp.eps, inp.seed, bits, inp.dtype,
                         rstd32=down(g.rstd), du=np.zeros((inp.T, inp.C)))
    cols = np.sort(np.random.default_rng(3).choice(inp.C, 16, replace=False))
    T, C, O = inp.T, inp.C, inp.O
    codes = torch.zeros(T * C, dtype=torch.int8, device="cuda")
    steps = torch.zeros(T, device="cuda")
    b.bsp_store_fwd(g.kind, g.x, T, C, g.gamma, g.beta, g.rstd, g.mean, bits, b.key(inp.seed, store.TENSOR_U, 0, 0), codes, steps)
    assert np.array_equal(codes.cpu().numpy().reshape(T, C)[:, cols].astype(np.int64), prep["codes"][:, cols])
    split = torch.zeros(C * 2 * g.ld_t, dtype=torch.bfloat16, device="cuda")
    dW = torch.zeros(O * C, device="cuda")
    wsw = b.workspace(b.bsp_store_wgrad_workspace_bytes(T, O))
    b.bsp_store_read(g.kind, g.x, T, C, g.gamma, g.beta, g.rstd, g.mean, codes, steps, 3,
                     b.key(inp.seed, store.TENSOR_U, b.STREAM_WGRAD, 5), None, split, g.ld_t)
    b.bsp_store_wgrad(T, O, C, g.dy_codes_t, g.q_dy, split, g.ld_t, dW, wsw)
    want = prep["dy"]["value"].T @ store.copy_for(prep, 3, inp.seed, philox.STREAM_WGRAD, 5, cols)
    assert rel_l2(down(dW).reshape(O, C)[:, cols], want) <= 1e-4
