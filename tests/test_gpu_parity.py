"""Parity of the CUDA path (through the C ABI) against the CPU oracle.

Bars: bit-exact generator words and FP8 codes; <= 1e-5 relative L2 per tensor on CUDA-core FP32
gradients; <= 2e-3 relative L2 on tensor-core contractions; identical verdicts.
"""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import check, fp8, linear, mc, norm, philox
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


# ------------------------------------------------------------------------------ generator, codec


@pytest.mark.parametrize("n", [1, 3, 4, 1003, 1 << 16])
def test_philox_words_bit_exact(b, n):
    seed, tid, stream, draw = 0xDEADBEEF12345678, 77, 2, 9
    out = torch.zeros(ceil16(n), dtype=torch.int32, device="cuda")
    b.bsp_philox_fill(b.key(seed, tid, stream, draw), n, out)
    got = out.cpu().numpy().view(np.uint32)[:n]
    assert np.array_equal(got, philox.tensor_words(seed, tid, stream, draw, n))


def _special_values(fmt):
    F = fp8.FORMATS[fmt]
    rng = np.random.default_rng(5)
    pos = fp8.decode(np.arange(128, dtype=np.uint8), fmt)
    pos = np.sort(pos[np.isfinite(pos)])
    mids = ((pos[:-1] + pos[1:]) / 2).astype(np.float32)
    v = np.concatenate([
        pos.astype(np.float32), mids, np.nextafter(mids, np.float32(0)), np.nextafter(mids, np.float32(np.inf)),
        np.array([0.0, -0.0, 1e-45, -1e-45, 1e-40, 2.0 ** -30, F.fmax, F.fmax * 1.001, 1e30, -1e30, np.inf,
                  -np.inf, np.nan], dtype=np.float32),
        (rng.standard_normal(5000) * np.exp(rng.uniform(-25, 12, 5000))).astype(np.float32)])
    return np.concatenate([v, -v]).astype(np.float32)


@pytest.mark.parametrize("fmt", [fp8.E4M3, fp8.E5M2])
@pytest.mark.parametrize("mode", [fp8.RN, fp8.SR])
def test_round_special_values_bit_exact(b, fmt, mode):
    v = _special_values(fmt)
    n = v.size
    x = up(v)
    codes = torch.zeros(ceil16(n), dtype=torch.uint8, device="cuda")
    diag = b.new_diag()
    seed, tid, stream, draw = 42, 3, 1, 2
    b.bsp_round(x, n, b.quant(fmt, mode, 1.0), b.key(seed, tid, stream, draw), 0, codes, diag)
    words = philox.tensor_words(seed, tid, stream, draw, n)
    want, n_sat, n_nf = fp8.encode(v, fmt, mode, words)
    got = codes.cpu().numpy()[:n]
    assert np.array_equal(got, want)
    d = b.read_diag(diag)
    assert d["n_saturated"] == n_sat and d["n_nonfinite"] == n_nf and d["status"] == b.ERR_NONFINITE


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("n,offset", [(100003, 0), (4096, 64), (777, 5)])
def test_round_scaled_ragged_bit_exact(b, dtype, n, offset):
    rng = np.random.default_rng(n)
    v = rng.standard_normal(n).astype(np.float32) * 3
    if dtype == "bf16":
        v = workloads.to_bf16_grid(v)
    scale = np.float32(448.0) / np.max(np.abs(v))
    x = up(v, dtype)
    codes = torch.zeros(ceil16(n), dtype=torch.uint8, device="cuda")
    sdev = torch.tensor([scale], device="cuda")
    b.bsp_round(x, n, b.quant(fp8.E4M3, fp8.SR, 0.0, sdev), b.key(7, 1, 0, 0), offset, codes)
    words = philox.element_words(7, 1, 0, 0, np.arange(offset, offset + n))
    want, _, _ = fp8.encode((v * scale).astype(np.float32), fp8.E4M3, fp8.SR, words)
    assert np.array_equal(codes.cpu().numpy()[:n], want)


def test_amax_scale_and_grouped_round(b):
    rng = np.random.default_rng(8)
    G, S = 6, 2048
    v = (rng.standard_normal((G, S)) * rng.uniform(0.1, 10, (G, 1))).astype(np.float32)
    v[2] = 0.0
    x = up(v)
    amax = torch.zeros(G, device="cuda")
    scales = torch.zeros(G, device="cuda")
    b.bsp_amax(x, G, S, amax)
    b.bsp_scale_from_amax(amax, G, fp8.E4M3, scales)
    want_amax = np.max(np.abs(v), axis=1)
    want_scale, _ = fp8.scale_from_amax(want_amax, fp8.E4M3)
    assert np.array_equal(down(amax), want_amax) and np.array_equal(down(scales), want_scale)
    codes = torch.zeros(G * S, dtype=torch.uint8, device="cuda")
    b.bsp_round_grouped(x, G, S, fp8.E4M3, fp8.SR, scales, b.key(3, 2, 0, 0), codes)
    words = philox.tensor_words(3, 2, 0, 0, G * S).reshape(G, S)
    want, _, _ = fp8.encode((v * want_scale[:, None]).astype(np.float32), fp8.E4M3, fp8.SR, words)
    assert np.array_equal(codes.cpu().numpy().reshape(G, S), want)


@pytest.mark.parametrize("rows,cols", [(64, 128), (100, 48), (257, 320)])
def test_round_2d_transposed_copy(b, rows, cols):
    rng = np.random.default_rng(rows)
    v = workloads.to_bf16_grid(rng.standard_normal((rows, cols)).astype(np.float32))
    x = up(v, "bf16")
    ld = ceil16(rows)
    codes = torch.zeros(rows * cols, dtype=torch.uint8, device="cuda")
    codes_t = torch.full((cols * ld,), 0xAA, dtype=torch.uint8, device="cuda")
    b.bsp_round_2d(x, rows, cols, b.quant(fp8.E5M2, fp8.RN, 1000.0), b.key(0, 0, 0), codes, codes_t, ld)
    want, _, _ = fp8.encode((v * np.float32(1000.0)).astype(np.float32), fp8.E5M2, fp8.RN)
    assert np.array_equal(codes.cpu().numpy().reshape(rows, cols), want)
    got_t = codes_t.cpu().numpy().reshape(cols, ld)
    assert np.array_equal(got_t[:, :rows], want.T)
    assert np.all(got_t[:, rows:] == 0)                      # the padding up to ld_t is zeroed


# ------------------------------------------------------------------------------ normalisation


def _small_cases():
    return [workloads.config1(),
            workloads.config2(T=200, C=512, O=192, K=8),
            workloads.config4(T=150, C=320, O=128, K=8),
            # whole 512-column stages and T a multiple of four: the LayerNorm / FP32 form of the streamed
            # statistics and backward kernels (cfg2_small is their RMSNorm / bf16 form; cfg1 and
            # cfg4_small take the plain kernels)
            workloads.config4(T=156, C=512, O=128, K=8)]


@pytest.fixture(scope="module", params=[0, 1, 2, 3], ids=["cfg1", "cfg2_small", "cfg4_small", "cfg4_stream"])
def case(request, b):
    inp = _small_cases()[request.param]
    g = NormLinearGpu(inp)
    kind = norm.RMS if inp.norm == "rms" else norm.LAYER
    rstd32, mean32 = down(g.rstd), down(g.mean)
    prep = check.prepare_norm_linear(inp.x, inp.gamma, inp.beta, inp.W, inp.dY, kind, inp.eps, inp.seed,
                                     inp.dtype, rstd32=rstd32, mean32=mean32 if kind == norm.LAYER else None)
    return inp, g, kind, prep


def test_norm_statistics_and_store(b, case):
    inp, g, kind, prep = case
    fw = prep["fw"]
    assert np.max(np.abs(down(g.rstd) / fw["rstd"] - 1)) < 1e-6
    if kind == norm.LAYER:
        assert np.max(np.abs(down(g.mean) - fw["mean"])) < 1e-6 * max(1.0, np.max(np.abs(fw["mean"])))
    # amax, scale and every code are bit-exact given the saved statistics
    assert down(g.amax)[0] == prep["amax"]
    assert down(g.scale)[0] == prep["scale"]
    assert np.array_equal(down(g.u_f32).reshape(inp.T, inp.C), prep["u32"])
    codes = g.u_codes.cpu().numpy().reshape(inp.T, inp.C)
    assert np.array_equal(codes, prep["codes"])
    ct = g.u_codes_t.cpu().numpy().reshape(inp.C, g.ld_t)
    assert np.array_equal(ct[:, :inp.T], prep["codes"].T)
    ub = down(g.u_bf16_t).reshape(inp.C, g.ld_t)[:, :inp.T]
    assert np.array_equal(ub, linear.bf16_round(prep["u32"].astype(np.float64)).T.astype(np.float32))
    # the incoming gradient: amax, scale, E5M2 codes
    assert down(g.amax_dy)[0] == prep["dy"]["amax"] and down(g.scale_dy)[0] == prep["dy"]["scale"]
    assert np.array_equal(g.dy_codes.cpu().numpy().reshape(inp.T, inp.O), prep["dy"]["codes"])
    d = b.read_diag(g.diag)
    assert d["n_saturated"] == prep["n_saturated"] + prep["dy"]["n_saturated"]
    assert d["n_nonfinite"] == 0 and d["status"] == 0


def test_fresh_rounding_pass_bit_exact(b, case):
    inp, g, kind, prep = case
    fresh = torch.zeros(inp.T * inp.C, dtype=torch.uint8, device="cuda")
    q = b.quant(inp.store_fmt, b.ROUND_STOCHASTIC, 1.0, g.scale)
    for stream, draw in ((b.STREAM_WGRAD, 0), (b.STREAM_WGRAD, 5), (b.STREAM_GAIN, 1)):
        b.bsp_norm_fwd(g.kind, g.x, inp.T, inp.C, g.gamma, g.beta, g.rstd, g.mean, q,
                       b.key(inp.seed, g.tensor_id, stream, draw), fresh, None, g.ld_t)
        _, want = check.fresh_copy(prep, inp.seed, stream, draw)
        assert np.array_equal(fresh.cpu().numpy().reshape(inp.T, inp.C), want)


@pytest.mark.parametrize("policy", [0, 1, 2])
def test_norm_backward_three_reads(b, case, policy):
    inp, g, kind, prep = case
    T, C = inp.T, inp.C
    du = up(prep["du"].astype(np.float32), inp.dtype)
    dg = torch.zeros(C, device="cuda")
    db = torch.zeros(C, device="cuda")
    dx = torch.zeros(T * C, device="cuda")
    ws = b.workspace(b.bsp_norm_bwd_workspace_bytes(T, C))
    draw = 3
    b.bsp_norm_bwd(g.kind, g.x, T, C, g.gamma, g.beta, g.rstd, g.mean, du, policy, g.u_codes, g.q,
                   b.key(inp.seed, g.tensor_id, b.STREAM_GAIN, draw), dg, db, dx, ws)
    if policy == 0:
        copy = None
    elif policy == 1:
        copy = norm.read_value(prep["codes"], inp.store_fmt, prep["inv_scale"])
    else:
        copy, _ = check.fresh_copy(prep, inp.seed, philox.STREAM_GAIN, draw)
    want = norm.backward(inp.x, inp.gamma, inp.beta, kind, inp.eps, prep["du"], gain_copy=copy)
    assert rel_l2(down(dg), want["dgamma"]) <= TOL_FP32
    assert rel_l2(down(db), want["dbeta"]) <= TOL_FP32
    assert rel_l2(down(dx), want["dx"]) <= TOL_FP32


def test_gain_use_monte_carlo_sums(b, case):
    inp, g, kind, prep = case
    T, C, K = inp.T, inp.C, 12
    du = up(prep["du"].astype(np.float32), inp.dtype)
    ref64 = norm.backward(inp.x, inp.gamma, inp.beta, kind, inp.eps, prep["du"])["dgamma"]
    ref32 = ref64.astype(np.float32)
    S1 = torch.zeros(C, device="cuda")
    S2 = torch.zeros(C, device="cuda")
    ws = b.workspace(b.bsp_norm_gain_mc_workspace_bytes(T, C, K))
    q = b.quant(inp.store_fmt, b.ROUND_STOCHASTIC, 1.0, g.scale)
    k = b.key(inp.seed, g.tensor_id, b.STREAM_GAIN, 0)
    # two draw ranges merged by addition
    b.bsp_norm_gain_mc(g.kind, g.x, T, C, g.gamma, g.beta, g.rstd, g.mean, du, q, k, 0, 5, up(ref32), S1, S2, ws)
    b.bsp_norm_gain_mc(g.kind, g.x, T, C, g.gamma, g.beta, g.rstd, g.mean, du, q, k, 5, K - 5, up(ref32), S1, S2, ws)
    gk = np.stack([norm.dgamma_from_copy(check.fresh_copy(prep, inp.seed, philox.STREAM_GAIN, kk)[0],
                                         inp.gamma, inp.beta, prep["du"]) for kk in range(K)])
    d = gk - ref32.astype(np.float64)
    # per-draw gradients agree to FP32 accuracy; the sums inherit it relative to the gradient's size
    scale = np.linalg.norm(ref64)
    assert np.linalg.norm(down(S1) - d.sum(0)) <= TOL_FP32 * scale * K
    assert rel_l2(down(S2), (d * d).sum(0)) <= 1e-3
    mean_gpu, m2_gpu = mc.shifted_sums_to_moments(down(S1), down(S2), K, ref32)
    assert rel_l2(mean_gpu, gk.mean(0)) <= TOL_FP32


# ------------------------------------------------------------------------------ contractions


@pytest.mark.parametrize("policy", [1, 0, 2])
def test_weight_gradient_three_reads(b, case, policy):
    inp, g, kind, prep = case
    T, C, O = inp.T, inp.C, inp.O
    dW = torch.zeros(O * C, device="cuda")
    ws = b.workspace(b.bsp_linear_wgrad_workspace_bytes(T, O, C, policy))
    diag = b.new_diag()
    dyv = prep["dy"]["value"]
    if policy == 1:
        b.bsp_linear_wgrad(T, O, C, g.dy_codes_t, g.q_dy, policy, g.u_codes_t, g.q, g.ld_t, dW, ws=ws, diag=diag)
        want = linear.wgrad(dyv, norm.read_value(prep["codes"], inp.store_fmt, prep["inv_scale"]))
    elif policy == 0:
        b.bsp_linear_wgrad(T, O, C, g.dy_codes_t, g.q_dy, policy, g.u_bf16_t, g.q, g.ld_t, dW, ws=ws, diag=diag)
        want = linear.wgrad(dyv, linear.bf16_round(prep["u32"].astype(np.float64)))
    else:
        fresh_t = torch.zeros(C * g.ld_t, dtype=torch.uint8, device="cuda")
        q = b.quant(inp.store_fmt, b.ROUND_STOCHASTIC, 1.0, g.scale)
        b.bsp_norm_fwd(g.kind, g.x, T, C, g.gamma, g.beta, g.rstd, g.mean, q,
                       b.key(inp.seed, g.tensor_id, b.STREAM_WGRAD, 4), None, fresh_t, g.ld_t)
        b.bsp_linear_wgrad(T, O, C, g.dy_codes_t, g.q_dy, policy, fresh_t, q, g.ld_t, dW, ws=ws, diag=diag)
        want = linear.wgrad(dyv, check.fresh_copy(prep, inp.seed, philox.STREAM_WGRAD, 4)[0])
    assert b.read_diag(diag)["status"] == 0
    assert rel_l2(down(dW).reshape(O, C), want) <= TOL_TC


def test_weight_gradient_fused_monte_carlo_epilogue(b, case):
    inp, g, kind, prep = case
    T, C, O, K = inp.T, inp.C, inp.O, 6
    ref = linear.wgrad(prep["dy"]["value"], norm.read_value(prep["codes"], inp.store_fmt, prep["inv_scale"]))
    ref32 = ref.astype(np.float32)
    refd = up(ref32.ravel())
    S1 = torch.zeros(O * C, device="cuda")
    S2 = torch.zeros(O * C, device="cuda")
    fresh_t = torch.zeros(4 * C * g.ld_t, dtype=torch.uint8, device="cuda")
    q = b.quant(inp.store_fmt, b.ROUND_STOCHASTIC, 1.0, g.scale)
    key = b.key(inp.seed, g.tensor_id, b.STREAM_WGRAD, 0)
    diag = b.new_diag()
    acc = mc.Welford(ref.shape)
    want_codes = []
    for k in range(K):
        copy, codes = check.fresh_copy(prep, inp.seed, philox.STREAM_WGRAD, k)
        want_codes.append(codes)
        acc.add(linear.wgrad(prep["dy"]["value"], copy))
    # two chained draw ranges: 4 draws, then the remaining 2
    for k0, nd in ((0, 4), (4, K - 4)):
        b.bsp_norm_fwd_draws(g.kind, g.x, T, C, g.gamma, g.beta, g.rstd, g.mean, q, key, k0, nd, fresh_t, g.ld_t)
        got = fresh_t.cpu().numpy()[:nd * C * g.ld_t].reshape(nd, C, g.ld_t)
        for d in range(nd):
            assert np.array_equal(got[d, :, :T], want_codes[k0 + d].T)
        b.bsp_linear_wgrad_mc(T, O, C, g.dy_codes_t, g.q_dy, fresh_t, q, g.ld_t, nd, refd, S1, S2, diag)
    assert b.read_diag(diag)["status"] == 0
    mean_gpu, m2_gpu = mc.shifted_sums_to_moments(down(S1).reshape(O, C), down(S2).reshape(O, C), K, ref32)
    assert rel_l2(mean_gpu, acc.mean) <= TOL_TC
    assert rel_l2(m2_gpu, acc.m2) <= 1e-2
    # the single-draw form of bsp_linear_wgrad takes the same path and gives the same sums
    S1b = torch.zeros(O * C, device="cuda")
    S2b = torch.zeros(O * C, device="cuda")
    one = torch.zeros(C * g.ld_t, dtype=torch.uint8, device="cuda")
    for k in range(K):
        b.bsp_norm_fwd(g.kind, g.x, T, C, g.gamma, g.beta, g.rstd, g.mean, q,
                       b.key(inp.seed, g.tensor_id, b.STREAM_WGRAD, k), None, one, g.ld_t)
        b.bsp_linear_wgrad(T, O, C, g.dy_codes_t, g.q_dy, 2, one, q, g.ld_t, None, refd, S1b, S2b, ws=b.workspace(256))
    assert torch.equal(S1, S1b) and torch.equal(S2, S2b)


def test_input_gradient_helper(b, case):
    inp, g, kind, prep = case
    T, C, O = inp.T, inp.C, inp.O
    du = torch.zeros(T * C, dtype=torch.bfloat16 if inp.dtype == "bf16" else torch.float32, device="cuda")
    ws = b.workspace(b.bsp_linear_dgrad_workspace_bytes(T, O, C))
    b.bsp_linear_dgrad(T, O, C, g.dy_codes, g.q_dy, g.W, du, ws)
    want = linear.dgrad(prep["dy"]["value"], linear.bf16_round(inp.W))
    tol = TOL_TC if inp.dtype == "f32" else 4e-3       # a bf16 store alone costs 2^-9 per element
    assert rel_l2(down(du).reshape(T, C), want) <= tol


# ------------------------------------------------------------------------------ statistics, check


def test_mc_statistics_match_oracle(b):
    rng = np.random.default_rng(12)
    n, K = 50000, 24
    ref = rng.standard_normal(n).astype(np.float32)
    gk = ref[None, :].astype(np.float64) + 0.05 * rng.standard_normal((K, n)) + 0.03
    d = gk - ref.astype(np.float64)
    S1 = d.sum(0).astype(np.float32)
    S2 = (d * d).sum(0).astype(np.float32)
    ws = b.workspace(b.bsp_mc_stats_workspace_bytes(n))
    r = b.bsp_mc_stats(up(ref), up(S1), up(S2), n, K, 1, ws)
    mean, m2 = mc.shifted_sums_to_moments(S1, S2, K, ref)
    want = mc.statistics(mean, m2, K, ref, True)
    for name in ("rel_l2_mean_err", "R", "Qprime", "mean_z", "rms_z", "max_abs_z", "frac_abs_z_gt3"):
        # per-element arithmetic is FP32 on the GPU: agreement to 1e-4, far inside the verdict margins
        assert np.isclose(getattr(r, name), getattr(want, name), rtol=1e-4, atol=1e-9), name
    assert r.verdict == want.verdict == mc.FAILS and r.K == K and r.n_elements == n
    r0 = b.bsp_mc_stats(up(ref), up(ref), None, n, 1, 0, ws)
    assert r0.rel_l2_mean_err == 0.0 and r0.verdict == mc.HOLDS
    r1 = b.bsp_mc_stats(up(ref), up(ref * np.float32(1.01)), None, n, 1, 0, ws)
    assert np.isclose(r1.rel_l2_mean_err, 0.01, rtol=1e-4) and r1.verdict == mc.FAILS


@pytest.mark.parametrize("dx_read", [1, 2])
def test_input_gradient_reading_a_copy(b, case, dx_read):
    """dx with z read from the forward's codes (R) or from a fresh rounding under the input
    gradient's own generator stream (N); the gain use keeps reading the original."""
    inp, g, kind, prep = case
    T, C = inp.T, inp.C
    du = up(prep["du"].astype(np.float32), inp.dtype)
    dg, db, dx = torch.zeros(C, device="cuda"), torch.zeros(C, device="cuda"), torch.zeros(T * C, device="cuda")
    ws = b.workspace(b.bsp_norm_bwd_workspace_bytes(T, C))
    draw = 2
    b.bsp_norm_bwd(g.kind, g.x, T, C, g.gamma, g.beta, g.rstd, g.mean, du, 0, g.u_codes, g.q,
                   b.key(inp.seed, g.tensor_id, b.STREAM_GAIN, draw), dg, db, dx, ws, dx_read=dx_read)
    if dx_read == 1:
        copy = norm.read_value(prep["codes"], inp.store_fmt, prep["inv_scale"])
    else:
        copy, _ = check.fresh_copy(prep, inp.seed, philox.STREAM_DX, draw)
    want = norm.backward(inp.x, inp.gamma, inp.beta, kind, inp.eps, prep["du"], dx_copy=copy)
    assert rel_l2(down(dg), want["dgamma"]) <= TOL_FP32
    assert rel_l2(down(dx), want["dx"]) <= TOL_FP32
    # and it is a different tensor from the reference's input gradient
    ref = norm.backward(inp.x, inp.gamma, inp.beta, kind, inp.eps, prep["du"])
    assert rel_l2(down(dx), ref["dx"]) > 1e-4


def _oracle_table(inp, kind, prep, K):
    """Oracle statistics in the order the check returns them: gain U (dgamma, dbeta), R, N, weight U, R, N."""
    args = (inp.x, inp.gamma, inp.beta, kind, inp.eps, prep)
    out = []
    for p in (check.U, check.R, check.N):
        r = check.gain_use(*args, p, K, inp.seed)
        out.append(r["stats"])
        # dbeta reads no saved tensor: its value under every read is the reference's
        zero = np.zeros_like(r["dbeta"])
        out.append(mc.statistics(r["dbeta"], zero if p == check.N else None, K, r["dbeta"], p == check.N))
    for p in (check.U, check.R, check.N):
        out.append(check.wgrad_use(prep, p, K, inp.seed)["stats"])
    return out


def _gpu_du(b, g, desc, K, ws):
    lay = b.bsp_mc_check_layout(desc, K)
    dt = torch.bfloat16 if g.inp.dtype == "bf16" else torch.float32
    return lay, down(b.ws_view(ws, lay.du, g.T * g.C, dt)).reshape(g.T, g.C)


EXPECTED_NORM_LINEAR = [mc.HOLDS, mc.HOLDS, mc.FAILS, mc.HOLDS, mc.HOLDS, mc.HOLDS, mc.FAILS, mc.HOLDS, mc.FAILS]


def test_mc_check_small_configs_verdicts_and_statistics(b, case):
    inp, g, kind, _ = case
    K = min(inp.K, 32)
    desc = g.desc()
    ws = b.workspace(b.bsp_mc_check_workspace_bytes(desc, K))
    diag = b.new_diag()
    res = b.bsp_mc_check(desc, K, ws, diag)
    assert len(res) == 9 and b.read_diag(diag)["status"] == 0
    assert [(r.use_id, r.output_id, r.policy) for r in res] == \
        [(b.STREAM_GAIN, o, p) for p in (0, 1, 2) for o in (b.OUT_DGAMMA, b.OUT_DBETA)] + \
        [(b.STREAM_WGRAD, b.OUT_DW, p) for p in (0, 1, 2)]
    # the oracle takes the GPU's saved statistics and the incoming gradient du the GPU's helper made
    # (read back from the workspace), so both sides evaluate the uses on the same received gradient
    lay, du_gpu = _gpu_du(b, g, desc, K, ws)
    prep = check.prepare_norm_linear(inp.x, inp.gamma, inp.beta, inp.W, inp.dY, kind, inp.eps, inp.seed,
                                     inp.dtype, rstd32=down(g.rstd), mean32=down(g.mean) if kind == norm.LAYER else None,
                                     du=du_gpu)
    want = _oracle_table(inp, kind, prep, K)
    for r, w, e in zip(res, want, EXPECTED_NORM_LINEAR):
        assert r.verdict == w.verdict == e, (r.as_dict(), w)
        assert r.K == w.K and r.n_elements == w.n_elements
        if r.policy != b.READ_FRESH:
            assert np.isclose(r.rel_l2_mean_err, w.rel_l2_mean_err, rtol=2e-3, atol=1e-9)
        else:
            for f in ("rel_l2_mean_err", "R", "Qprime", "rms_z"):
                assert np.isclose(getattr(r, f), getattr(w, f), rtol=2e-3, atol=1e-9), (r.as_dict(), w, f)
    assert res[0].rel_l2_mean_err == 0.0 and res[7].rel_l2_mean_err == 0.0
    for i in (1, 3, 5):          # dbeta: exactly the reference under every read
        assert res[i].rel_l2_mean_err == 0.0 and res[i].R == 0.0 and res[i].max_abs_z == 0.0
    # per-element moments from the workspace: mean, variance and z of dgamma under the fresh read
    C = inp.C
    ref = b.ws_view(ws, lay.dgamma_ref, C)
    S1, S2 = b.ws_view(ws, lay.dgamma_S1, C), b.ws_view(ws, lay.dgamma_S2, C)
    mean, var, z = (torch.zeros(C, device="cuda") for _ in range(3))
    b.bsp_mc_moments(ref, S1, S2, C, K, mean, var, z)
    gain_n = check.gain_use(inp.x, inp.gamma, inp.beta, kind, inp.eps, prep, check.N, K, inp.seed)
    assert rel_l2(down(mean), gain_n["mean"]) <= TOL_FP32
    assert rel_l2(down(var), gain_n["m2"] / (K - 1)) <= 2e-3
    se = np.sqrt(gain_n["m2"] / (K - 1) / K)
    assert rel_l2(down(z), (gain_n["mean"] - gain_n["ref"]) / se) <= 2e-3
    # dbeta and dx of the reference are there too
    assert rel_l2(down(b.ws_view(ws, lay.dbeta_ref, C)), np.sum(du_gpu.astype(np.float64), axis=0)) <= TOL_FP32
    # determinism: a second call returns byte-identical results
    res2 = b.bsp_mc_check(desc, K, ws, diag)
    assert [bytes(r) for r in res] == [bytes(r) for r in res2]


def test_mc_check_draws_in_chunks(b, case):
    """A small code buffer makes the weight use take its K draws in several chunks (re-round launch +
    contraction launch per chunk, sums chained through memory, an odd tail): same per-element sums as
    the one-chunk run to FP32 accumulation order, same verdicts, and the oracle's statistics."""
    inp, g, kind, _ = case
    K = 11
    desc = g.desc(policy_mask=0x24)          # the two fresh reads
    ws = b.workspace(b.bsp_mc_check_workspace_bytes(desc, K))
    diag = b.new_diag()
    one = b.bsp_mc_check(desc, K, ws, diag)
    lay = b.bsp_mc_check_layout(desc, K)
    n = inp.O * inp.C
    s1_one, s2_one = down(b.ws_view(ws, lay.dW_S1, n)).copy(), down(b.ws_view(ws, lay.dW_S2, n)).copy()
    desc.draw_buffer_bytes = 3 * inp.C * g.ld_t + 7          # room for three draws: chunks 3, 3, 3, 2
    ws2 = b.workspace(b.bsp_mc_check_workspace_bytes(desc, K))
    assert ws2.numel() < ws.numel()
    side = torch.cuda.Stream()
    desc.side_stream = side.cuda_stream          # and the gain kernel beside the first contraction
    many = b.bsp_mc_check(desc, K, ws2, diag)
    assert b.read_diag(diag)["status"] == 0
    lay2 = b.bsp_mc_check_layout(desc, K)
    s1, s2 = down(b.ws_view(ws2, lay2.dW_S1, n)), down(b.ws_view(ws2, lay2.dW_S2, n))
    ref = down(b.ws_view(ws2, lay2.dW_ref, n))
    assert np.linalg.norm(s1 - s1_one) <= 1e-5 * K * np.linalg.norm(ref)
    assert rel_l2(s2, s2_one) <= 1e-4
    assert [r.verdict for r in many] == [r.verdict for r in one] == [mc.HOLDS, mc.HOLDS, mc.FAILS]
    for x, y in zip(many, one):
        assert np.isclose(x.R, y.R, rtol=1e-3, atol=1e-9) and np.isclose(x.Qprime, y.Qprime, rtol=1e-3, atol=1e-9)
    # against the oracle, element by element on the sums
    _, du_gpu = _gpu_du(b, g, desc, K, ws2)
    prep = check.prepare_norm_linear(inp.x, inp.gamma, inp.beta, inp.W, inp.dY, kind, inp.eps, inp.seed,
                                     inp.dtype, rstd32=down(g.rstd), mean32=down(g.mean) if kind == norm.LAYER else None,
                                     du=du_gpu)
    w = check.wgrad_use(prep, check.N, K, inp.seed)
    mean_gpu, m2_gpu = mc.shifted_sums_to_moments(s1.reshape(inp.O, inp.C), s2.reshape(inp.O, inp.C), K, ref.reshape(inp.O, inp.C))
    assert rel_l2(mean_gpu, w["mean"]) <= TOL_TC and rel_l2(m2_gpu, w["m2"]) <= 1e-2
    assert many[2].verdict == w["stats"].verdict and np.isclose(many[2].R, w["stats"].R, rtol=5e-3)


def test_verdict_rule_is_an_argument(b):
    """The thresholds are the caller's: the same sums read under a stricter and a looser rule."""
    rng = np.random.default_rng(5)
    n, K = 4096, 16
    ref = rng.standard_normal(n).astype(np.float32)
    d = rng.standard_normal((K, n)) * 0.1 + 0.05           # a bias of two standard errors per element
    S1, S2 = d.sum(0).astype(np.float32), (d * d).sum(0).astype(np.float32)
    ws = b.workspace(b.bsp_mc_stats_workspace_bytes(n))
    args = (up(ref), up(S1), up(S2), n, K, 1, ws)
    default = b.bsp_mc_stats(*args)
    assert default.verdict == mc.FAILS and 4.0 < default.Qprime < 8.0
    loose = b.bsp_mc_stats(*args, rule=b.rule(qprime_hold=10.0, r_hold=10.0, qprime_fail=20.0, r_fail=20.0))
    assert loose.verdict == mc.HOLDS and loose.Qprime == default.Qprime
    # "z < 2 and under x %": a magnitude bound on top of the statistics
    bounded = b.bsp_mc_stats(*args, rule=b.rule(qprime_hold=10.0, r_hold=10.0, qprime_fail=20.0, r_fail=20.0, rel_hold=1e-3))
    assert bounded.verdict == mc.UNDECIDED
    det = b.bsp_mc_stats(up(ref), up(ref * np.float32(1.001)), None, n, 1, 0, ws, rule=b.rule(rel_tol_deterministic=1e-2))
    assert det.verdict == mc.HOLDS
    with pytest.raises(b.BspError):
        b.bsp_mc_stats(*args, rule=b.rule(qprime_hold=5.0, qprime_fail=4.0))
    with pytest.raises(b.BspError):          # fresh statistics need K >= 4
        b.bsp_mc_stats(up(ref), up(S1), up(S2), n, 3, 1, ws)


def test_a_bounded_wait_that_runs_out(b):
    """A wait on a barrier that nothing completes gives up after its limit: the kernel returns, the
    status word says BSP_ERR_TIMEOUT, and the device goes on working (a contraction right after)."""
    diag = b.new_diag()
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    b.bsp_selftest_bounded_wait(1_000_000, diag)          # 1 ms
    t1.record()
    d = b.read_diag(diag)
    assert d["status"] == b.ERR_TIMEOUT
    assert 0.5 <= t0.elapsed_time(t1) < 200.0
    with pytest.raises(b.BspError):
        b.bsp_selftest_bounded_wait(0, diag)
    with pytest.raises(b.BspError):
        b.bsp_selftest_bounded_wait(10**9, diag)
    # the context is intact: a tensor-core product on the same device, against numpy
    rng = np.random.default_rng(0)
    A = workloads.to_bf16_grid(rng.standard_normal((128, 64)).astype(np.float32))
    Bm = workloads.to_bf16_grid(rng.standard_normal((128, 64)).astype(np.float32))
    Cd = torch.zeros(128 * 128, device="cuda")
    diag2 = b.new_diag()
    b.bsp_gemm(128, 128, 64, 2, up(A, "bf16"), 64, False, 0, up(Bm, "bf16"), 64, False, 0, 1.0, Cd, 128, diag2)
    assert b.read_diag(diag2)["status"] == 0
    assert rel_l2(down(Cd).reshape(128, 128), A.astype(np.float64) @ Bm.astype(np.float64).T) <= 1e-5


def test_edge_cases(b):
    # empty inputs are accepted and launch nothing
    z = torch.zeros(16, device="cuda")
    c = torch.zeros(16, dtype=torch.uint8, device="cuda")
    b.bsp_round(z, 0, b.quant(0, 0, 1.0), b.key(0, 0, 0), 0, c)
    b.bsp_philox_fill(b.key(0, 0, 0), 0, c)
    b.bsp_round_2d(z, 0, 16, b.quant(0, 0, 1.0), b.key(0, 0, 0), c, None, 0)
    # all-zero tensor: scale 1, codes 0, amax 0
    amax = torch.ones(1, device="cuda")
    s = torch.zeros(1, device="cuda")
    b.bsp_amax(z, 1, 16, amax)
    b.bsp_scale_from_amax(amax, 1, 0, s)
    assert down(amax)[0] == 0 and down(s)[0] == 1.0
    # a NaN in the input is counted, never trapped, and becomes the canonical NaN code
    v = np.zeros(32, dtype=np.float32)
    v[5] = np.nan
    diag = b.new_diag()
    codes = torch.zeros(32, dtype=torch.uint8, device="cuda")
    b.bsp_round(up(v), 32, b.quant(0, 0, 1.0), b.key(0, 0, 0), 0, codes, diag)
    d = b.read_diag(diag)
    assert d["n_nonfinite"] == 1 and d["status"] == b.ERR_NONFINITE and codes.cpu().numpy()[5] == 0x7F
