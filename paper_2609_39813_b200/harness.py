"""Host-side helpers shared by the tests, the smoke entry and the benchmark: upload the seeded
numpy inputs and drive the once-per-workload preparation through the C-ABI entry points.  No
arithmetic of the method lives here."""
import numpy as np
import torch

from . import binding as b
from . import workloads


def up(a, dtype="f32"):
    """numpy float32 array -> CUDA tensor of the storage dtype (bf16 values must be on the grid)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    if dtype == "bf16":
        bits = workloads.bf16_bits(a)
        return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    return torch.from_numpy(a).cuda()


def down(t):
    if t.dtype == torch.bfloat16:
        return t.float().cpu().numpy()
    return t.cpu().numpy()


def rel_l2(a, ref):
    a = np.asarray(a, dtype=np.float64).ravel()
    ref = np.asarray(ref, dtype=np.float64).ravel()
    den = np.linalg.norm(ref)
    return float(np.linalg.norm(a - ref) / den) if den > 0 else float(np.linalg.norm(a - ref))


def ceil16(n):
    return (n + 15) // 16 * 16


class NormLinearGpu:
    """Device-side state of one normalisation -> linear workload, built through the C ABI."""

    def __init__(self, inp, tensor_id=1, forward_mode=b.ROUND_STOCHASTIC):
        self.inp = inp
        self.kind = b.RMSNORM if inp.norm == "rms" else b.LAYERNORM
        T, C, O = inp.T, inp.C, inp.O
        self.T, self.C, self.O, self.ld_t = T, C, O, ceil16(T)
        self.tensor_id = tensor_id
        dev = "cuda"
        self.x = up(inp.x, inp.dtype)
        self.gamma = up(inp.gamma)
        self.beta = up(inp.beta) if inp.beta is not None else None
        self.W = up(inp.W, inp.dtype)
        self.dY = up(inp.dY, inp.dtype)
        self.rstd = torch.empty(T, device=dev)
        self.mean = torch.zeros(T, device=dev)
        self.amax = torch.zeros(1, device=dev)
        self.scale = torch.zeros(1, device=dev)
        self.diag = b.new_diag()
        b.bsp_norm_stats(self.kind, self.x, T, C, self.gamma, self.beta, inp.eps, self.rstd, self.mean,
                         self.amax, self.diag)
        b.bsp_scale_from_amax(self.amax, 1, inp.store_fmt, self.scale)
        self.q = b.quant(inp.store_fmt, forward_mode, 1.0, self.scale)
        self.u_codes = torch.empty(T * C, dtype=torch.uint8, device=dev)
        self.u_codes_t = torch.zeros(C * self.ld_t, dtype=torch.uint8, device=dev)
        self.u_f32 = torch.empty(T * C, device=dev)
        self.u_bf16_t = torch.zeros(C * self.ld_t, dtype=torch.bfloat16, device=dev)
        b.bsp_norm_fwd(self.kind, self.x, T, C, self.gamma, self.beta, self.rstd, self.mean, self.q,
                       b.key(inp.seed, tensor_id, b.STREAM_FORWARD, 0), self.u_codes, self.u_codes_t,
                       self.ld_t, self.u_f32, self.u_bf16_t, self.diag)
        # incoming gradient
        self.amax_dy = torch.zeros(1, device=dev)
        self.scale_dy = torch.zeros(1, device=dev)
        b.bsp_amax(self.dY, 1, T * O, self.amax_dy, self.diag)
        b.bsp_scale_from_amax(self.amax_dy, 1, inp.grad_fmt, self.scale_dy)
        self.q_dy = b.quant(inp.grad_fmt, b.ROUND_NEAREST, 1.0, self.scale_dy)
        self.dy_codes = torch.empty(T * O, dtype=torch.uint8, device=dev)
        self.dy_codes_t = torch.zeros(O * self.ld_t, dtype=torch.uint8, device=dev)
        b.bsp_round_2d(self.dY, T, O, self.q_dy, b.key(0, 0, 0), self.dy_codes, self.dy_codes_t, self.ld_t,
                       self.diag)
        torch.cuda.synchronize()

    def desc(self, policy_mask=0x3F):
        inp = self.inp
        d = b.NormLinearDesc()
        d.norm_kind = self.kind
        d.dtype = b.BF16 if inp.dtype == "bf16" else b.F32
        d.T, d.C, d.O = self.T, self.C, self.O
        d.x, d.gamma, d.beta = b.ptr(self.x), b.ptr(self.gamma), b.ptr(self.beta)
        d.W, d.dY = b.ptr(self.W), b.ptr(self.dY)
        d.eps = inp.eps
        d.store_fmt, d.grad_fmt = inp.store_fmt, inp.grad_fmt
        d.forward_mode = b.ROUND_STOCHASTIC if inp.forward_mode == "sr" else b.ROUND_NEAREST
        d.seed, d.tensor_id, d.policy_mask = inp.seed, self.tensor_id, policy_mask
        return d


# ------------------------------------------------------------------ replica timing protocol


def max_over_ranks(ms: float, device="cpu") -> float:
    """Largest step time over all ranks (the job is as slow as its slowest replica).  Single
    process: the value itself."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_throughput(elements_per_step: int, steps: int, world: int, ms_total_max: float) -> float:
    """Whole-job throughput of `world` independent replicas, each doing `steps` steps of
    `elements_per_step` units, when the slowest replica took `ms_total_max` milliseconds."""
    return world * elements_per_step * steps / (ms_total_max * 1e-3)
