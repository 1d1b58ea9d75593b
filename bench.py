#!/usr/bin/env python
"""Benchmark of the per-use check (one JSON line on stdout).

A step is one pass of the whole hot path over one batch of synthetic input: statistics and
current-amax scale, forward store, incoming gradient to E5M2, du = dY W, then the six
(use, policy) evaluations of the check -- gain use {U, R, N x K}, weight use {U, R, N x K} --
i.e. one call of bsp_mc_check.  Workload at every N: config 5, RMSNorm -> Linear at the large-MLP
shape (T = 16384, C = 4096, O = 11008, bf16, K = 16 draws), the largest single-GPU configuration,
from the seeded host recipe; N GPUs run N independent replicas (the path has no exchange step:
weak scaling).  Configs 2, 3 (both operand modes) and 4 (K = 1024) ride along as sub-objects.

metric = per-use check elements/s: sum over use-evaluations of (saved-tensor elements x draws
consumed) divided by the time of the step.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With --gpus N > 1 and no launcher environment, bench.py starts its N ranks itself (one process per
GPU, rendezvous on 127.0.0.1); under torchrun it is one of the ranks.
"""
import argparse
import json
import os
import socket
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "per_use_check_elements_per_s"
UNIT = "elements/s"
WORKLOAD = "cfg5_rmsnorm_linear_large_mlp"
NOMINAL_HBM_GBS = 8000.0
NOMINAL_BF16_TFLOPS = 2250.0
NOMINAL_FP8_TFLOPS = 4500.0


def check_elements(T, C, K):
    """Saved-tensor elements x draws over the six use-evaluations (U, R: 1 draw; N: K draws)."""
    return T * C * (2 * (1 + 1 + K))


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"], samples=0)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        for l in self.lines:
            f = [x.strip() for x in l.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                smax.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return dict(sm_mhz=sm[len(sm) // 2] if sm else None, sm_max_mhz=max(smax) if smax else None,
                    reasons=sorted(reasons), samples=len(sm))


# ----------------------------------------------------------------------------------- replicas


def free_port():
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_replicas(n, argv):
    """Starts n copies of this script, one per GPU, with the launcher environment a rank expects
    (RANK, LOCAL_RANK, WORLD_SIZE, MASTER_ADDR, MASTER_PORT); rank 0 prints the line.  Returns the
    largest exit code."""
    port = free_port()
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + argv, env=env))
    return max(p.wait() for p in procs)


def replica_selftest(args):
    """The timing protocol of the replicas alone, on CPU with gloo (no CUDA): every rank reports a
    made-up step time, rank 0 prints the line built from the maximum.  Used by the CPU tests to cover
    the launch path of --gpus N."""
    import torch.distributed as dist
    from paper_2609_39813_b200.harness import max_over_ranks, replica_throughput
    world, rank = int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0"))
    if world > 1:
        dist.init_process_group("gloo", init_method="env://")
    ms = 10.0 * (rank + 1)
    ms_max = max_over_ranks(ms, device="cpu")
    if rank == 0:
        print(json.dumps(dict(selftest="replicas", n_gpus=world, ms_max=ms_max,
                              value=replica_throughput(1000, 1, world, ms_max))), flush=True)
    if world > 1:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------------- oracle arm


def oracle_sample(inp, rows, k_gain, k_wgrad):
    """The oracle as it stands on the first `rows` tokens of the workload: preparation, gain use
    {U, R, N x k_gain}, weight use {U, R, N x k_wgrad}.  Returns (seconds, check elements)."""
    from oracle import check, norm
    kind = norm.RMS if inp.norm == "rms" else norm.LAYER
    x, dY = inp.x[:rows], inp.dY[:rows]
    t0 = time.perf_counter()
    prep = check.prepare_norm_linear(x, inp.gamma, inp.beta, inp.W, dY, kind, inp.eps, inp.seed, inp.dtype)
    for p in (0, 1, 2):
        check.gain_use(x, inp.gamma, inp.beta, kind, inp.eps, prep, p, k_gain, inp.seed)
    for p in (0, 1, 2):
        check.wgrad_use(prep, p, k_wgrad, inp.seed)
    dt = time.perf_counter() - t0
    return dt, rows * inp.C * (2 + k_gain + 2 + k_wgrad)


def library_fp8_tflops(n=8192, reps=10):
    """TFLOP/s of the library FP8 GEMM (torch._scaled_mm) at n^3; None where it is not available.
    A measurement of the machine, not part of the path."""
    import torch
    try:
        a = torch.randn(n, n, device="cuda").to(torch.float8_e4m3fn)
        bt = torch.randn(n, n, device="cuda").to(torch.float8_e4m3fn).t()
        one = torch.ones((), device="cuda")
        for _ in range(3):
            torch._scaled_mm(a, bt, scale_a=one, scale_b=one, out_dtype=torch.bfloat16)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            torch._scaled_mm(a, bt, scale_a=one, scale_b=one, out_dtype=torch.bfloat16)
        e1.record()
        torch.cuda.synchronize()
        return 2.0 * n ** 3 * reps / (e0.elapsed_time(e1) * 1e-3) / 1e12
    except Exception:
        return None


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads") for i in threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else os.cpu_count()
    except Exception:
        return os.cpu_count()


def run_reference(args):
    """The oracle, as it stands, on the host cores: each step is the check on a token slice of
    config 5 (every column, every output row, all K = 16 draws of both uses)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2609_39813_b200 import workloads
    inp = workloads.config5()
    K = inp.K
    # calibrate on a small slice, then size each step so the whole run stays within ~2.5 minutes
    dt0, el0 = oracle_sample(inp, 32, K, K)
    budget = 150.0 / max(1, args.steps + args.warmup)
    rows = int(max(32, min(inp.T, 32 * budget / max(dt0, 1e-3))))
    rows = max(32, rows // 32 * 32)
    for _ in range(args.warmup):
        oracle_sample(inp, rows, K, K)
    total_t, total_el = 0.0, 0
    for _ in range(args.steps):
        dt, el = oracle_sample(inp, rows, K, K)
        total_t += dt
        total_el += el
    value = total_el / total_t
    sample = ("first %d of %d tokens, all %d columns and %d output rows, gain {U,R,N x%d} + weight {U,R,N x%d}, "
              "numpy float64" % (rows, inp.T, inp.C, inp.O, K, K))
    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps, warmup=args.warmup,
                ms_per_step=1e3 * total_t / max(1, args.steps), higher_is_better=True, scaling="weak",
                vs_baseline=None, dtype="f64", data="synthetic", impl="reference",
                config=dict(workload=WORKLOAD, T=inp.T, C=inp.C, O=inp.O, K=inp.K),
                cpu_baseline=dict(value=value, unit=UNIT, cores=blas_threads(), kind="oracle", sample=sample),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------- CUDA arm


def timed(torch, stream, fn, reps=5, warm=2):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    a, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(reps):
        fn()
    c.record(stream)
    torch.cuda.synchronize()
    return a.elapsed_time(c) / reps


def norm_linear_check(b, torch, inp, steps=3, side=None):
    """One normalisation -> linear configuration from the seeded host recipe: the whole check, timed."""
    from paper_2609_39813_b200.harness import NormLinearGpu
    g = NormLinearGpu(inp)
    d = g.desc()
    if side is not None:
        d.side_stream = side.cuda_stream
    ws = b.workspace(b.bsp_mc_check_workspace_bytes(d, inp.K))
    diag = b.new_diag()
    stream = torch.cuda.current_stream()
    res = b.bsp_mc_check(d, inp.K, ws, diag)
    ms = timed(torch, stream, lambda: b.bsp_mc_check(d, inp.K, ws, diag), reps=steps, warm=1)
    return dict(workload=inp.name, T=inp.T, C=inp.C, O=inp.O, K=inp.K, ms_per_check=ms,
                check_elements_per_s=check_elements(inp.T, inp.C, inp.K) / (ms * 1e-3),
                verdicts=[int(r.verdict) for r in res if r.output_id != b.OUT_DBETA],
                dbeta_verdicts=[int(r.verdict) for r in res if r.output_id == b.OUT_DBETA],
                data="seeded host recipe", diag_status=b.read_diag(diag)["status"])


def attention_section(b, peaks, steps=3):
    """Config 3 (causal attention backward, B=8 H=16 S=2048 d=64, K=32) from the seeded host recipe:
    the per-use check of the D use in both operand modes, timed as a whole, and its kernels alone."""
    import torch
    from paper_2609_39813_b200 import workloads
    from paper_2609_39813_b200.harness import up
    inp = workloads.config3()
    B, H, S, D, K = inp.B, inp.H, inp.S, inp.D, inp.K
    tensor_o = 2                                              # generator tensor id of the attention output store
    n = B * H * S * D
    q, k, v, dO = (up(a, "bf16").reshape(-1) for a in (inp.q, inp.k, inp.v, inp.dO))
    stream = torch.cuda.current_stream()
    diag = b.new_diag()
    elements = n * (1 + 1 + K)

    def check(fp8_operands):
        d = b.AttnDesc()
        d.B, d.H, d.S, d.Dh, d.causal, d.softmax_scale, d.dtype = B, H, S, D, 1, inp.softmax_scale, b.BF16
        d.q, d.k, d.v, d.dO = b.ptr(q), b.ptr(k), b.ptr(v), b.ptr(dO)
        d.store_fmt, d.forward_mode, d.seed, d.tensor_id, d.policy_mask = b.E4M3, b.ROUND_STOCHASTIC, inp.seed, tensor_o, 7
        d.fp8_operands, d.p_scale, d.ds_scale = fp8_operands, 256.0, 1024.0
        ws = b.workspace(b.bsp_mc_check_attn_workspace_bytes(d, K))
        res = b.bsp_mc_check_attn(d, K, ws, diag)
        ms = timed(torch, stream, lambda: b.bsp_mc_check_attn(d, K, ws, diag), reps=steps, warm=0)
        return dict(ms_per_check=ms, check_elements_per_s=elements / (ms * 1e-3), verdicts=[int(r.verdict) for r in res],
                    informational=[int(r.informational) for r in res])

    mode_b = check(0)
    mode_a = check(1)
    torch.cuda.empty_cache()
    # ---- the kernels alone
    c = inp.softmax_scale
    o = torch.zeros(n, device="cuda"); lse = torch.zeros(B * H * S, device="cuda")
    dq, dk, dv = (torch.zeros(n, device="cuda") for _ in range(3))
    dterm = torch.zeros(B * H * S, device="cuda")
    b.bsp_attn_fwd_stats(B, H, S, D, True, c, q, k, v, o, lse, diag)
    b.bsp_attn_dterm(B, H, S, D, dO, o, None, None, b.E4M3, b.READ_ORIGINAL, b.key(0, 2, 4), 0, 1, dterm)
    ms_dkv = timed(torch, stream, lambda: b.bsp_attn_bwd_dterm(B, H, S, D, True, c, q, k, v, dO, lse, dterm, None, dk, dv, diag))
    ms_dq = timed(torch, stream, lambda: b.bsp_attn_bwd_dterm(B, H, S, D, True, c, q, k, v, dO, lse, dterm, dq, None, None, diag))
    # the one-kernel form: S, dP and the exponentials once per score tile, dQ by reduce-adds (its clearing included)
    ms_one = timed(torch, stream, lambda: b.bsp_attn_bwd_dterm_fused(B, H, S, D, True, c, q, k, v, dO, lse, dterm, dq, dk, dv, diag))
    # the D pre-pass alone under its three reads (HBM-bound for U and R: dO read once, the copy of O
    # read once; the fresh read is bound by the generator: one word per element and draw)
    amax_o, scales_o = torch.zeros(B * H, device="cuda"), torch.zeros(B * H, device="cuda")
    codes_o = torch.zeros(n, dtype=torch.uint8, device="cuda")
    b.bsp_amax(o, B * H, S * D, amax_o)
    b.bsp_scale_from_amax(amax_o, B * H, b.E4M3, scales_o)
    b.bsp_round_grouped(o, B * H, S * D, b.E4M3, b.ROUND_STOCHASTIC, scales_o, b.key(inp.seed, tensor_o, 0, 0), codes_o)
    d_draws = torch.zeros(K * B * H * S, device="cuda")
    kd = b.key(inp.seed, tensor_o, b.STREAM_ATTN_D, 0)
    ms_du = timed(torch, stream, lambda: b.bsp_attn_dterm(B, H, S, D, dO, o, codes_o, scales_o, b.E4M3, b.READ_ORIGINAL, kd, 0, 1, dterm))
    ms_dr = timed(torch, stream, lambda: b.bsp_attn_dterm(B, H, S, D, dO, o, codes_o, scales_o, b.E4M3, b.READ_FORWARD, kd, 0, 1, dterm))
    ms_dn = timed(torch, stream, lambda: b.bsp_attn_dterm(B, H, S, D, dO, o, codes_o, scales_o, b.E4M3, b.READ_FRESH, kd, 0, K, d_draws))
    hbm = peaks["hbm_gbs"]
    dterm_rows = dict(
        read_U=dict(us=ms_du * 1e3, algorithmic_mb=n * 6 / 1e6, gb_per_s=n * 6 / ms_du / 1e6, frac_of_hbm=n * 6 / ms_du / 1e6 / hbm,
                    frac_of_nominal_hbm=n * 6 / ms_du / 1e6 / NOMINAL_HBM_GBS),
        read_R=dict(us=ms_dr * 1e3, algorithmic_mb=n * 3 / 1e6, gb_per_s=n * 3 / ms_dr / 1e6, frac_of_hbm=n * 3 / ms_dr / 1e6 / hbm,
                    frac_of_nominal_hbm=n * 3 / ms_dr / 1e6 / NOMINAL_HBM_GBS),
        read_N=dict(us=ms_dn * 1e3, draws=K, g_element_draws_per_s=n * K / ms_dn / 1e6))
    # the forward helper, and the FP8-operand mode of the backward
    ms_fwd = timed(torch, stream, lambda: b.bsp_attn_fwd_stats(B, H, S, D, True, c, q, k, v, o, lse, diag))
    hatq, amq, scq = torch.zeros(n, dtype=torch.bfloat16, device="cuda"), torch.zeros(B * H, device="cuda"), torch.zeros(B * H, device="cuda")
    ms_quant = timed(torch, stream, lambda: b.bsp_attn_quantize(q, B * H, S * D, b.E4M3, hatq, amq, scq))
    ops = {}
    for nm, src, fmt in (("q", q, b.E4M3), ("k", k, b.E4M3), ("v", v, b.E4M3), ("dO", dO, b.E5M2)):
        xq, am, sc = torch.zeros(n, dtype=torch.bfloat16, device="cuda"), torch.zeros(B * H, device="cuda"), torch.zeros(B * H, device="cuda")
        cd = torch.zeros(n, dtype=torch.uint8, device="cuda")
        b.bsp_attn_quantize(src, B * H, S * D, fmt, xq, am, sc, codes=cd)
        ops[nm] = (xq, sc, cd)
    f8 = b.attn_fp8(ops["q"][1], ops["k"][1], ops["v"][1], ops["dO"][1], 256.0, 1024.0,
                    ops["q"][2], ops["k"][2], ops["v"][2], ops["dO"][2])
    o8, lse8 = torch.zeros(n, device="cuda"), torch.zeros(B * H * S, device="cuda")
    b.bsp_attn_fwd_stats(B, H, S, D, True, c, ops["q"][0], ops["k"][0], ops["v"][0], o8, lse8, diag, fp8=f8)
    d8 = torch.zeros(B * H * S, device="cuda")
    ms_fp8 = timed(torch, stream, lambda: b.bsp_attn_bwd(B, H, S, D, True, c, 1, ops["q"][0], ops["k"][0], ops["v"][0], ops["dO"][0],
                                                          lse8, o8, None, None, b.E4M3, b.READ_ORIGINAL, kd, dq, dk, dv, d8, diag, fp8=f8))
    prod = 2.0 * B * H * S * S * D / 2                         # one causal S x S x d product over all heads
    tf_dkv, tf_dq = 4 * prod / (ms_dkv * 1e-3) / 1e12, 3 * prod / (ms_dq * 1e-3) / 1e12
    peak = peaks["bf16_tflops"]
    bwd = (ms_dkv + ms_dq) * 1e-3
    return dict(workload="cfg3_causal_attention_bwd", B=B, H=H, S=S, D=D, K=K, data="seeded host recipe",
                ms_per_check=mode_b["ms_per_check"], check_elements_per_s=mode_b["check_elements_per_s"],
                verdicts=mode_b["verdicts"], bf16_operands=mode_b, fp8_operands=mode_a,
                bwd_dkv_us=ms_dkv * 1e3, bwd_dq_us=ms_dq * 1e3, bwd_one_kernel_us=ms_one * 1e3,
                bwd_one_kernel_algorithmic_frac=5 * prod / (ms_one * 1e-3) / 1e12 / peak, dterm=dterm_rows,
                fwd_stats_us=ms_fwd * 1e3, quantize_one_tensor_us=ms_quant * 1e3,
                bwd_fp8_operands_us=ms_fp8 * 1e3,   # D pre-pass + dK/dV + dQ kernels, FP8-operand mode
                roofline=dict(bound="tensor", kernel="attn_kernel<dK/dV> + attn_kernel<dQ> (bf16 operands)",
                              achieved=(4 + 3) * prod / bwd / 1e12, peak=peak, unit="TFLOP/s",
                              frac=(4 + 3) * prod / bwd / 1e12 / peak, dkv_tflops=tf_dkv, dq_tflops=tf_dq,
                              # a backward needs 5 of those products; the two kernels form S and dP once each
                              algorithmic_tflops=5 * prod / bwd / 1e12, algorithmic_frac=5 * prod / bwd / 1e12 / peak,
                              peak_nominal=NOMINAL_BF16_TFLOPS, frac_of_nominal=(4 + 3) * prod / bwd / 1e12 / NOMINAL_BF16_TFLOPS,
                              note="achieved counts the 7 causal products of 2*S*S*d/2 flop per head that the two "
                                   "kernels compute, algorithmic_* the 5 a backward needs; measured: paced by the hand-overs between "
                                   "the MMA warp and the softmax warps, tensor pipe 39-48 % and exp2/convert unit 46-52 % busy"),
                diag_status=b.read_diag(diag)["status"])


def widened_section(b, torch):
    """The rows built after the core path, each timed as a whole through its own entry point on seeded
    inputs: the b-bit per-token store's check (config 2's shape, 6 bits, K = 16), the averages over the
    forward's rounding (config 2's shape, 8 pairs of forwards), rounded attention probabilities
    (16384 rows of 128 keys, d = 64, 256 draws) and the log-softmax case (64 x 128, 4096 trials)."""
    import numpy as np
    from paper_2609_39813_b200 import workloads
    from paper_2609_39813_b200.harness import NormLinearGpu, up
    stream = torch.cuda.current_stream()
    out = {}
    inp = workloads.config2()
    g = NormLinearGpu(inp)
    diag = b.new_diag()

    # f1: the paper's own store
    K, bits = 16, 6
    d = b.StoreDesc()
    d.norm_kind, d.dtype = g.kind, b.BF16
    d.T, d.C, d.O = inp.T, inp.C, inp.O
    d.x, d.gamma, d.beta, d.W, d.dY = b.ptr(g.x), b.ptr(g.gamma), b.ptr(g.beta), b.ptr(g.W), b.ptr(g.dY)
    d.eps, d.bits, d.grad_fmt = inp.eps, bits, inp.grad_fmt
    d.seed, d.tensor_id, d.policy_mask = inp.seed, 1, 0x7F
    ws = b.workspace(b.bsp_mc_check_store_workspace_bytes(d, K))
    res = b.bsp_mc_check_store(d, K, ws, diag)
    ms = timed(torch, stream, lambda: b.bsp_mc_check_store(d, K, ws, diag), reps=5, warm=1)
    el = inp.T * inp.C * ((1 + 1 + K) + (1 + 1 + K + K))
    out["store"] = dict(workload="cfg2 shape, %d-bit per-token store, K=%d" % (bits, K), ms_per_check=ms,
                        check_elements_per_s=el / (ms * 1e-3), verdicts=[int(r.verdict) for r in res],
                        rows="gain U,R,N then weight U,R,N,R+eps")
    del ws

    # f2: averages over the forward's rounding
    pairs = 8
    c = b.CouplingDesc()
    c.norm_kind, c.dtype = g.kind, b.BF16
    c.T, c.C, c.O = inp.T, inp.C, inp.O
    c.x, c.gamma, c.beta, c.W = b.ptr(g.x), b.ptr(g.gamma), b.ptr(g.beta), b.ptr(g.W)
    c.eps, c.store_fmt, c.forward_mode, c.seed, c.tensor_id = inp.eps, 0, 1, inp.seed, 1
    ws = b.workspace(b.bsp_coupling_check_workspace_bytes(c, pairs))
    Tst, ctl = b.bsp_coupling_check(c, pairs, ws, diag)
    ms = timed(torch, stream, lambda: b.bsp_coupling_check(c, pairs, ws, diag), reps=3, warm=1)
    out["coupling"] = dict(workload="cfg2 shape, E4M3 store, loss |y|^2/2, %d pairs of forwards" % pairs,
                           ms_per_check=ms, forwards_per_s=2 * pairs / (ms * 1e-3),
                           T_mean=float(np.mean(Tst)), control_mean=float(np.mean(ctl)))
    del ws

    # f3: rounded probabilities
    R, n, dd, draws = 16384, 128, 64, 256
    rng = np.random.default_rng(3003)
    sc = rng.standard_normal((R, n)) * 1.5
    p = np.exp(sc - sc.max(1, keepdims=True))
    p = (p / p.sum(1, keepdims=True)).astype(np.float32)
    V = (rng.standard_normal((n, dd)) / np.sqrt(dd)).astype(np.float32)
    pg, Vg = torch.from_numpy(p).cuda(), torch.from_numpy(V).cuda()
    ds = torch.zeros(5 * R * n, device="cuda")
    sq = torch.zeros(5 * R * n, device="cuda")
    dV = torch.zeros(2 * R * n * dd, device="cuda")
    fn = lambda: b.bsp_probs_mc(pg, Vg, R, n, dd, 0, 1.0 / 64, 3003, 4, 0, draws, ds, sq, dV)
    ms = timed(torch, stream, fn, reps=3, warm=1)
    out["probs"] = dict(workload="%d rows x %d keys, d=%d, grid 1/64, %d draws" % (R, n, dd, draws), ms=ms,
                        entry_draws_per_s=R * n * draws / (ms * 1e-3))
    del ds, sq, dV

    # f4: log-softmax
    rows, classes, trials, eps = 64, 128, 4096, 0.1
    rng = np.random.default_rng(1926)
    logits = torch.from_numpy(rng.standard_normal((rows, classes)).astype(np.float32)).cuda()
    target = torch.from_numpy(rng.integers(0, classes, rows).astype(np.int32)).cuda()
    ws = b.workspace(b.bsp_lsm_check_workspace_bytes(rows, classes, trials))
    st = b.bsp_lsm_check(logits, target, rows, classes, eps, trials, 1926, 3, None, ws)
    ms = timed(torch, stream, lambda: b.bsp_lsm_check(logits, target, rows, classes, eps, trials, 1926, 3, None, ws),
               reps=3, warm=1)
    out["logsoftmax"] = dict(workload="%d x %d, eps %.2f, %d trials" % (rows, classes, eps, trials), ms=ms,
                             entry_trials_per_s=rows * classes * trials / (ms * 1e-3),
                             mean_error_reuse=st[0].mean, predicted=float(np.cosh(eps) - 1),
                             coupling=st[2].mean, predicted_coupling=float(-eps * np.sinh(eps)))
    # the same operator at a vocabulary-sized row (the generator's rate shows only on a large case)
    rows, classes, trials = 256, 8192, 256
    logits = torch.from_numpy(rng.standard_normal((rows, classes)).astype(np.float32)).cuda()
    target = torch.from_numpy(rng.integers(0, classes, rows).astype(np.int32)).cuda()
    ws = b.workspace(b.bsp_lsm_check_workspace_bytes(rows, classes, trials))
    ms = timed(torch, stream, lambda: b.bsp_lsm_check(logits, target, rows, classes, eps, trials, 1926, 3, None, ws),
               reps=3, warm=1)
    out["logsoftmax_large"] = dict(workload="%d x %d, eps %.2f, %d trials" % (rows, classes, eps, trials), ms=ms,
                                   entry_trials_per_s=rows * classes * trials / (ms * 1e-3))
    out["diag_status"] = b.read_diag(diag)["status"]
    return out


def kernel_table(b, peaks, g):
    """The streaming kernels one by one on config 5's own tensors (T=16384, C=4096, O=11008, bf16):
    microseconds per launch and algorithmic GB/s (bytes the method must move / time) against the
    measured copy bandwidth and the nominal 8 TB/s; then the K-draw kernels and the contractions."""
    import torch
    inp = g.inp
    T, C, O = inp.T, inp.C, inp.O
    x, dY, gamma = g.x, g.dY, g.gamma
    du = torch.randn(T * C, device="cuda").bfloat16()       # any incoming gradient: only its bytes matter here
    rstd, mean = torch.zeros(T, device="cuda"), torch.zeros(T, device="cuda")
    amax, scale = torch.zeros(1, device="cuda"), torch.ones(1, device="cuda")
    codes = torch.zeros(T * C, dtype=torch.uint8, device="cuda")
    codes_t = torch.zeros(C * T, dtype=torch.uint8, device="cuda")
    dyc = torch.zeros(T * O, dtype=torch.uint8, device="cuda")
    dyc_t = torch.zeros(O * T, dtype=torch.uint8, device="cuda")
    dg, db, dx = torch.zeros(C, device="cuda"), torch.zeros(C, device="cuda"), torch.zeros(T * C, device="cuda")
    ws = b.workspace(b.bsp_norm_bwd_workspace_bytes(T, C))
    ref, S2 = torch.zeros(O * C, device="cuda"), torch.zeros(O * C, device="cuda")
    wss = b.workspace(b.bsp_mc_stats_workspace_bytes(O * C))
    stream = torch.cuda.current_stream()
    q = b.quant(b.E4M3, b.ROUND_STOCHASTIC, 1.0, scale)
    qrn = b.quant(b.E5M2, b.ROUND_NEAREST, 1.0, g.scale_dy)
    k = b.key(1, 1, 0)
    b.bsp_norm_stats(b.RMSNORM, x, T, C, gamma, None, 1e-6, rstd, mean, amax)
    b.bsp_scale_from_amax(amax, 1, b.E4M3, scale)
    rows = []

    def t(name, bound, fn, nbytes, reps=10):
        us = timed(torch, stream, fn, reps=reps, warm=3) * 1e3
        gbs = nbytes / us / 1e3
        rows.append(dict(kernel=name, bound=bound, us=us, algorithmic_mb=nbytes / 1e6, gb_per_s=gbs,
                         frac_of_hbm=gbs / peaks["hbm_gbs"], frac_of_nominal_hbm=gbs / NOMINAL_HBM_GBS))

    t("amax(dY)", "hbm", lambda: b.bsp_amax(dY, 1, T * O, amax), T * O * 2)
    t("round dY -> E5M2 nearest", "hbm", lambda: b.bsp_round(dY, T * O, qrn, k, 0, dyc), T * O * 3)
    t("round_2d dY -> E5M2 nearest, both layouts", "hbm", lambda: b.bsp_round_2d(dY, T, O, qrn, k, dyc, dyc_t, T), T * O * 4)
    t("norm_stats + amax(u)", "hbm", lambda: b.bsp_norm_stats(b.RMSNORM, x, T, C, gamma, None, 1e-6, rstd, mean, amax), T * C * 2)
    t("norm_fwd store, stochastic, codes", "alu", lambda: b.bsp_norm_fwd(b.RMSNORM, x, T, C, gamma, None, rstd, mean, q, k, codes, None, T), T * C * 3)
    t("norm_fwd store, stochastic, codes + transposed", "alu", lambda: b.bsp_norm_fwd(b.RMSNORM, x, T, C, gamma, None, rstd, mean, q, k, codes, codes_t, T), T * C * 4)
    t("norm_bwd read U: dgamma, dbeta, dx", "hbm", lambda: b.bsp_norm_bwd(b.RMSNORM, x, T, C, gamma, None, rstd, mean, du, 0, codes, q, k, dg, db, dx, ws), T * C * 8)
    t("norm_bwd read R: dgamma", "hbm", lambda: b.bsp_norm_bwd(b.RMSNORM, x, T, C, gamma, None, rstd, mean, du, 1, codes, q, k, dg, None, None, ws), T * C * 5)
    t("norm_bwd read N: dgamma, one fresh draw", "alu", lambda: b.bsp_norm_bwd(b.RMSNORM, x, T, C, gamma, None, rstd, mean, du, 2, codes, q, k, dg, None, None, ws), T * C * 4)
    t("mc_stats (45 M elements, fresh)", "hbm", lambda: b.bsp_mc_stats(ref, ref, S2, O * C, 16, 1, wss), O * C * 12)
    # ---- the K-draw kernels and the contractions at the same shape (K = 16 draws, as config 5)
    Kd = inp.K
    qf = b.quant(b.E4M3, b.ROUND_STOCHASTIC, 1.0, scale)
    fresh_t = torch.zeros(Kd * C * T, dtype=torch.uint8, device="cuda")
    S1 = torch.zeros(O * C, device="cuda")
    diag = b.new_diag()
    b.bsp_round_2d(dY, T, O, qrn, k, dyc, dyc_t, T)
    b.bsp_norm_fwd(b.RMSNORM, x, T, C, gamma, None, rstd, mean, q, k, codes, codes_t, T)
    g1, g2 = torch.zeros(C, device="cuda"), torch.zeros(C, device="cuda")
    wsg = b.workspace(b.bsp_norm_gain_mc_workspace_bytes(T, C, Kd))
    dW = torch.zeros(O * C, device="cuda")
    wsw = b.workspace(max(b.bsp_linear_wgrad_workspace_bytes(T, O, C, b.READ_FORWARD), 256))
    compute = []

    def tc(name, bound, fn, work, unit, peak, nominal=None, reps=5):
        us = timed(torch, stream, fn, reps=reps, warm=2) * 1e3
        rate = work / (us * 1e-6) / (1e9 if unit == "G element-draws/s" else 1e12)
        row = dict(kernel=name, bound=bound, us=us, achieved=rate, unit=unit, peak=peak, frac=rate / peak)
        if nominal:
            row["peak_nominal"], row["frac_of_nominal"] = nominal, rate / nominal
        compute.append(row)

    # The ceiling of the generator-bound kernels is measured, not assumed: the rate at which the
    # generator alone produces its words (bsp_philox_fill: one Philox4x32-10 block per four words,
    # written out), in words = element-draws per second.  The derived figure is kept beside it.
    alu_derived = 2650.0    # G element-draws/s: 37.2 T lane-instructions/s over ~14 per element-draw
    nwords = 1 << 28
    words = torch.empty(nwords, dtype=torch.int32, device="cuda")
    tc("generator words only (philox_fill)", "alu", lambda: b.bsp_philox_fill(b.key(1, 1, 3), nwords, words),
       float(nwords), "G element-draws/s", alu_derived)
    alu_peak = compute[-1]["achieved"]
    compute[-1]["note"] = "the measured ceiling used as `peak` by the two rows below; its own peak is the derived ALU figure"
    del words
    tc("fresh code matrices, 16 draws (reround_draws)", "alu",
       lambda: b.bsp_norm_fwd_draws(b.RMSNORM, x, T, C, gamma, None, rstd, mean, qf, b.key(1, 1, 2), 0, Kd, fresh_t, T),
       float(T) * C * Kd, "G element-draws/s", alu_peak)
    tc("gain use, 16 draws (gain_mc)", "alu",
       lambda: b.bsp_norm_gain_mc(b.RMSNORM, x, T, C, gamma, None, rstd, mean, du, qf, b.key(1, 1, 1), 0, Kd, dg, g1, g2, wsg, diag),
       float(T) * C * Kd, "G element-draws/s", alu_peak)
    tc("weight gradient, read R (gemm_tc fp8)", "tensor",
       lambda: b.bsp_linear_wgrad(T, O, C, dyc_t, qrn, b.READ_FORWARD, codes_t, qf, T, dW, ws=wsw, diag=diag),
       2.0 * T * O * C, "TFLOP/s", 2.0 * peaks["bf16_tflops"], NOMINAL_FP8_TFLOPS)
    # the two BF16 contractions of the path: the weight gradient reading the original u, and the
    # incoming-gradient helper du = dY W (decoded dY codes; a bf16 W is read in place)
    u_bf16_t = torch.zeros(C * T, dtype=torch.bfloat16, device="cuda")
    b.bsp_norm_fwd(b.RMSNORM, x, T, C, gamma, None, rstd, mean, q, k, codes, codes_t, T, None, u_bf16_t)
    wsu = b.workspace(max(b.bsp_linear_wgrad_workspace_bytes(T, O, C, b.READ_ORIGINAL), 256))
    tc("weight gradient, read U (decode + gemm_tc bf16)", "tensor",
       lambda: b.bsp_linear_wgrad(T, O, C, dyc_t, qrn, b.READ_ORIGINAL, u_bf16_t, qf, T, dW, ws=wsu, diag=diag),
       2.0 * T * O * C, "TFLOP/s", peaks["bf16_tflops"], NOMINAL_BF16_TFLOPS)
    du_out = torch.zeros(T * C, dtype=torch.bfloat16, device="cuda")
    wsd = b.workspace(b.bsp_linear_dgrad_workspace_bytes(T, O, C))
    tc("incoming gradient du = dY W (decode + gemm_tc bf16)", "tensor",
       lambda: b.bsp_linear_dgrad(T, O, C, dyc, qrn, g.W, du_out, wsd, diag),
       2.0 * T * O * C, "TFLOP/s", peaks["bf16_tflops"], NOMINAL_BF16_TFLOPS)
    del u_bf16_t, du_out, wsu, wsd
    tc("weight gradient, 16 fresh draws with sums (gemm_mc)", "tensor",
       lambda: b.bsp_linear_wgrad_mc(T, O, C, dyc_t, qrn, fresh_t, qf, T, Kd, ref, S1, S2, diag),
       2.0 * T * O * C * Kd, "TFLOP/s", 2.0 * peaks["bf16_tflops"], NOMINAL_FP8_TFLOPS, reps=3)
    # ---- the b-bit per-token store (6 bits) on the same tensors
    del fresh_t
    torch.cuda.empty_cache()
    bits = 6
    scodes = torch.zeros(T * C, dtype=torch.int8, device="cuda")
    ssteps = torch.zeros(T, device="cuda")
    split = torch.zeros(C * 2 * T, dtype=torch.bfloat16, device="cuda")
    tc("b-bit store forward, stochastic (store_fwd_kernel)", "alu",
       lambda: b.bsp_store_fwd(b.RMSNORM, x, T, C, gamma, None, rstd, mean, bits, b.key(1, 1, 0), scodes, ssteps),
       float(T) * C, "G element-draws/s", alu_peak, reps=10)
    compute[-1]["gb_per_s"] = T * C * 3 / compute[-1]["us"] / 1e3
    tc("b-bit store, copy for the weight use, read U/R+eps (store_operand_kernel)", "alu",
       lambda: b.bsp_store_read(b.RMSNORM, x, T, C, gamma, None, rstd, mean, scodes, ssteps, 3, b.key(1, 1, 2, 1), None, split, T),
       float(T) * C, "G element-draws/s", alu_peak, reps=10)
    compute[-1]["gb_per_s"] = T * C * 7 / compute[-1]["us"] / 1e3
    t("b-bit store, copy for the weight use, read R (store_operand_kernel)", "hbm",
      lambda: b.bsp_store_read(b.RMSNORM, x, T, C, gamma, None, rstd, mean, scodes, ssteps, 1, b.key(1, 1, 2, 1), None, split, T),
      T * C * 7)
    wst = b.workspace(max(b.bsp_store_wgrad_workspace_bytes(T, O), 256))
    tc("b-bit store weight gradient, hi+lo split operand (decode + gemm_tc bf16, contraction over 2T)", "tensor",
       lambda: b.bsp_store_wgrad(T, O, C, dyc_t, qrn, split, T, dW, wst, diag),
       2.0 * T * O * C, "TFLOP/s", peaks["bf16_tflops"], NOMINAL_BF16_TFLOPS)
    compute[-1]["note"] = "algorithmic flop 2 T O C; the kernel computes twice that (two bf16 terms per operand value)"
    return dict(shape=dict(T=T, C=C, O=O, dtype="bf16"), data="seeded host recipe (config 5)",
                hbm_peak_gbs=peaks["hbm_gbs"], hbm_nominal_gbs=NOMINAL_HBM_GBS, peak_source=peaks["source"],
                kernels=rows, compute_kernels=compute, diag_status=b.read_diag(diag)["status"])


def sharded_draws_line(args, b, torch, dist, world, rank):
    """The fresh reads of config 5 (gain use and weight use, K = 16) with the draws split over the ranks:
    every rank prepares the same workload, evaluates its share of the draws, one all-reduce adds the
    shifted sums, every rank finishes the statistics.  Total work is fixed: strong scaling."""
    from paper_2609_39813_b200 import workloads
    from paper_2609_39813_b200.harness import NormLinearGpu, max_over_ranks
    from paper_2609_39813_b200.sharded import ShardedFreshReads
    inp = workloads.config5()
    g = NormLinearGpu(inp)
    sh = ShardedFreshReads(g, inp.K, rank, world, draw_buffer_draws=16)
    sh.prepare()
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        res = sh.step()
    barrier()
    a, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(args.steps):
        res = sh.step()
    c.record(stream)
    barrier()
    ms = max_over_ranks(a.elapsed_time(c), device="cuda")
    if rank != 0:
        return
    elements = inp.T * inp.C * 2 * inp.K                      # the fresh reads of both uses
    print(json.dumps(dict(metric=METRIC, value=elements * args.steps / (ms * 1e-3), unit=UNIT, n_gpus=world,
                          steps=args.steps, warmup=max(args.warmup, 3), ms_per_step=ms / args.steps, higher_is_better=True,
                          scaling="strong", vs_baseline=None, dtype="f8e4m3/f8e5m2 operands, f32 accumulate",
                          data="synthetic",
                          config=dict(workload=WORKLOAD, T=inp.T, C=inp.C, O=inp.O, K=inp.K,
                                      policies="gain{N} x weight{N}", parallelism="draws/%d" % world,
                                      draws_per_rank=sh.nd, exchange="one all-reduce (sum) of S1, S2 per step: %d bytes"
                                      % (4 * 2 * (inp.C + inp.O * inp.C)),
                                      l2="working set larger than L2"),
                          verdicts=[int(r.verdict) for r in res], diag_status=b.read_diag(g.diag)["status"])), flush=True)


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2609_39813_b200 import binding as b
    from paper_2609_39813_b200 import workloads
    from paper_2609_39813_b200.harness import NormLinearGpu, max_over_ranks, replica_throughput

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    b.lib()
    peaks = read_peaks()

    if args.attention_only:
        if rank == 0:
            print(json.dumps(dict(attention=attention_section(b, peaks, steps=args.attention_steps))), flush=True)
        return
    if args.widened_only:
        if rank == 0:
            print(json.dumps(dict(widened=widened_section(b, torch))), flush=True)
        return
    if args.config2_only:
        if rank == 0:
            side2 = torch.cuda.Stream()
            print(json.dumps(dict(config2=norm_linear_check(b, torch, workloads.config2(), steps=args.steps, side=side2))),
                  flush=True)
        return
    if args.shard_draws:
        sharded_draws_line(args, b, torch, dist, world, rank)
        if world > 1:
            dist.destroy_process_group()
        return

    inp = workloads.config5()
    T, C, O, K = inp.T, inp.C, inp.O, inp.K
    g = NormLinearGpu(inp)
    if args.kernel_table:
        if rank == 0:
            print(json.dumps(dict(kernel_table=kernel_table(b, peaks, g))), flush=True)
        return
    # the preparation NormLinearGpu did (codes, statistics) is for the isolated kernel timing further
    # down; the step itself starts from x, gamma, W, dY
    side = torch.cuda.Stream()
    desc = g.desc()
    desc.side_stream = side.cuda_stream
    ws = b.workspace(b.bsp_mc_check_workspace_bytes(desc, K))
    diag = b.new_diag()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")   # > 126 MB of L2
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def step():
        return b.bsp_mc_check(desc, K, ws, diag)

    warmup = max(args.warmup, 3)
    for _ in range(warmup):
        res = step()
    verdicts = [int(r.verdict) for r in res if r.output_id != b.OUT_DBETA]

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.2)
    barrier()
    n0, d0 = b.bsp_launch_count(), b.bsp_d2h_byte_count()
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    for i in range(args.steps):
        flush.fill_(i & 0xFF)              # evict L2 between timed steps (not timed)
        starts[i].record(stream)
        step()
        ends[i].record(stream)
    barrier()
    launches = b.bsp_launch_count() - n0
    d2h = (b.bsp_d2h_byte_count() - d0) // max(1, args.steps)
    clocks = sampler.stop() if rank == 0 else None
    ms = sum(s.elapsed_time(e) for s, e in zip(starts, ends))
    ms_total = max_over_ranks(ms, device="cuda")
    elements = check_elements(T, C, K)
    value = replica_throughput(elements, args.steps, world, ms_total)

    # ---- end to end: host buffers in, host results out, through the same entry point
    host = dict(x=g.x.cpu().pin_memory(), gamma=g.gamma.cpu().pin_memory(), W=g.W.cpu().pin_memory(),
                dY=g.dY.cpu().pin_memory())
    h2d = sum(v.numel() * v.element_size() for v in host.values())
    e2e_steps = max(3, args.steps)        # the first step's upload is not hidden behind anything: it is in the timed region too
    # two sets of device input buffers: the inputs of step i + 1 cross PCIe on a copy stream while
    # step i computes (every step's copy is inside the timed region; a step starts only when its own
    # inputs have landed, and bsp_mc_check returns with the results on the host)
    alt = dict(x=torch.empty_like(g.x), gamma=torch.empty_like(g.gamma), W=torch.empty_like(g.W), dY=torch.empty_like(g.dY))
    desc2 = g.desc()
    desc2.side_stream = side.cuda_stream
    desc2.x, desc2.gamma, desc2.W, desc2.dY = b.ptr(alt["x"]), b.ptr(alt["gamma"]), b.ptr(alt["W"]), b.ptr(alt["dY"])
    sets = [(dict(x=g.x, gamma=g.gamma, W=g.W, dY=g.dY), desc), (alt, desc2)]
    copy_stream = torch.cuda.Stream()

    def upload(bufs):
        with torch.cuda.stream(copy_stream):
            for name in ("x", "gamma", "W", "dY"):
                bufs[name].copy_(host[name], non_blocking=True)
            ev = torch.cuda.Event()
            ev.record(copy_stream)
        return ev

    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    copy_stream.wait_event(e0)
    landed = upload(sets[0][0])
    for i in range(e2e_steps):
        bufs, ds = sets[i & 1]
        stream.wait_event(landed)
        if i + 1 < e2e_steps:
            landed = upload(sets[(i + 1) & 1][0])
        b.bsp_mc_check(ds, K, ws, diag)
    e1.record(stream)
    barrier()
    e2e_value = replica_throughput(elements, e2e_steps, world, max_over_ranks(e0.elapsed_time(e1), device="cuda"))
    del alt, host

    # ---- roofline of the dominant kernel: the FP8 weight-gradient contraction with the fused
    # shifted-sum epilogue, timed alone with CUDA events on the launching stream
    lay = b.bsp_mc_check_layout(desc, K)
    qf = b.quant(inp.store_fmt, b.ROUND_STOCHASTIC, 1.0, g.scale)
    fresh_t = torch.zeros(K * C * g.ld_t, dtype=torch.uint8, device="cuda")
    b.bsp_norm_fwd_draws(g.kind, g.x, T, C, g.gamma, g.beta, g.rstd, g.mean, qf,
                         b.key(inp.seed, g.tensor_id, b.STREAM_WGRAD, 0), 0, K, fresh_t, g.ld_t)
    ref = b.ws_view(ws, lay.dW_ref, O * C)
    S1 = torch.zeros(O * C, device="cuda")
    S2 = torch.zeros(O * C, device="cuda")
    reps = 5
    for _ in range(2):
        b.bsp_linear_wgrad_mc(T, O, C, g.dy_codes_t, g.q_dy, fresh_t, qf, g.ld_t, K, ref, S1, S2, diag)
    torch.cuda.synchronize()
    r0 = [torch.cuda.Event(enable_timing=True) for _ in range(reps)]
    r1 = [torch.cuda.Event(enable_timing=True) for _ in range(reps)]
    for i in range(reps):
        flush.fill_(i)
        r0[i].record(stream)
        b.bsp_linear_wgrad_mc(T, O, C, g.dy_codes_t, g.q_dy, fresh_t, qf, g.ld_t, K, ref, S1, S2, diag)
        r1[i].record(stream)
    torch.cuda.synchronize()
    gemm_ms = sum(a.elapsed_time(c) for a, c in zip(r0, r1)) / reps
    flops = 2.0 * T * O * C * K               # one launch contracts all K draws
    achieved = flops / (gemm_ms * 1e-3) / 1e12
    peak = 2.0 * peaks["bf16_tflops"]        # FP8 dense = 2 x the measured BF16 burst figure
    # DRAM bytes of one launch of this kernel at this shape: dram__bytes_read.sum + dram__bytes_write.sum
    # of one ncu capture of this command (profiles/gemm_mc_kernel_cfg5.md); null for any other shape
    traffic = GEMM_MC_TRAFFIC.get((T, C, O, K))
    roofline = dict(bound="tensor", kernel="gemm_mc_kernel (FP8 weight gradient over K draws, TMEM-resident sums)",
                    achieved=achieved, peak=peak, unit="TFLOP/s", frac=achieved / peak, traffic=traffic,
                    traffic_unit="bytes per launch (ncu dram read + write, one capture)",
                    algorithmic_bytes=float(K * C * g.ld_t + O * g.ld_t + 5 * 4 * O * C),
                    us_per_launch=gemm_ms * 1e3, draws_per_launch=K,
                    share_of_step=gemm_ms / (ms_total / args.steps),
                    peak_source="2 x bf16_tflops (%s)" % peaks["source"],
                    peak_sustained=2.0 * peaks["bf16_tflops_sustained"],
                    frac_of_sustained=achieved / (2.0 * peaks["bf16_tflops_sustained"]),
                    peak_nominal=NOMINAL_FP8_TFLOPS, frac_of_nominal=achieved / NOMINAL_FP8_TFLOPS)
    # Context beside that denominator: what the vendor library's own FP8 contraction reaches on this
    # GPU in this run (8192^3, E4M3 x E4M3, a short burst), measured the way the BF16 figure was.
    lib_fp8 = library_fp8_tflops() if rank == 0 else None
    if lib_fp8:
        roofline["library_fp8_tflops_this_run"] = lib_fp8
        roofline["frac_of_library_fp8"] = achieved / lib_fp8
    dstat = b.read_diag(diag)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        # a bounded sample of the same workload: a token slice (every column, every output row, all K
        # draws of both uses), ten to thirty seconds of host work
        rows = 384
        dt, el = oracle_sample(inp, rows, K, K)
        cpu_baseline = dict(value=el / dt, unit=UNIT, cores=blas_threads(), kind="oracle",
                            sample="first %d of %d tokens, all columns and output rows, gain {U,R,N x%d} + weight "
                                   "{U,R,N x%d}, %.1f s" % (rows, T, K, K, dt))

    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=warmup,
                ms_per_step=ms_total / args.steps, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="f8e4m3/f8e5m2 operands, f32 accumulate", data="synthetic",
                config=dict(workload=WORKLOAD, T=T, C=C, O=O, K=K, policies="gain{U,R,N} x weight{U,R,N}",
                            inputs="seeded host recipe (numpy PCG64, data seed 1005)",
                            l2="inputs larger than L2, and L2 flushed between timed steps (256 MiB write, outside "
                               "the timed spans)", replicas=world),
                clocks=clocks,
                e2e=dict(value=e2e_value, unit=UNIT, h2d_bytes_per_step=h2d, d2h_bytes_per_step=int(d2h), steps=e2e_steps),
                gpu_launches=int(launches), roofline=roofline, cpu_baseline=cpu_baseline,
                verdicts=verdicts, diag_status=dstat["status"])
    if not args.no_extras and world == 1:
        del ws, flush, fresh_t, S1, S2, g
        torch.cuda.empty_cache()
        line["config2"] = norm_linear_check(b, torch, workloads.config2(), steps=10, side=side)
        line["config4"] = norm_linear_check(b, torch, workloads.config4(), steps=2, side=side)
        torch.cuda.empty_cache()
        line["attention"] = attention_section(b, peaks, steps=args.attention_steps)
        torch.cuda.empty_cache()
        line["widened"] = widened_section(b, torch)
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# DRAM traffic of one gemm_mc_kernel launch by (T, C, O, K), bytes: dram__bytes_read.sum +
# dram__bytes_write.sum of one ncu capture of `python bench.py --steps 1 --warmup 3 --no-extras
# --no-cpu-baseline` (profiles/gemm_mc_kernel_cfg5.md)
GEMM_MC_TRAFFIC = {(16384, 4096, 11008, 16): 8934639360.0 + 362149120.0}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the sub-objects for configs 2, 3 and 4")
    ap.add_argument("--attention-only", action="store_true", help="run only the config-3 attention section")
    ap.add_argument("--attention-steps", type=int, default=3)
    ap.add_argument("--shard-draws", action="store_true",
                    help="instead of replicas: the K draws of the fresh reads split over the ranks, one all-reduce of "
                         "the shifted sums per step (strong scaling)")
    ap.add_argument("--config2-only", action="store_true",
                    help="run only the check of config 2 (the small case: 0.6 GB on the device), --steps times")
    ap.add_argument("--widened-only", action="store_true",
                    help="run only the b-bit store, coupling, rounded-probabilities and log-softmax checks")
    ap.add_argument("--kernel-table", action="store_true",
                    help="time the kernels one by one on config 5's tensors and print their GB/s and TFLOP/s")
    ap.add_argument("--selftest-replicas", action="store_true", help=argparse.SUPPRESS)
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        # not under a launcher: start the ranks here
        sys.exit(spawn_replicas(args.gpus, sys.argv[1:]))
    if args.selftest_replicas:
        replica_selftest(args)
    elif args.impl == "reference":
        if args.steps == 30 and args.warmup == 3:
            args.steps, args.warmup = 3, 1
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
