"""The fresh-read evaluations of the normalisation -> linear check with the K draws split over ranks.

One process per GPU.  Every rank prepares the same workload (the forward store, the incoming
gradient, the two reference gradients are identical everywhere: same seed, same keys), evaluates a
contiguous share of the K fresh draws of the gain use and of the weight use through the draw-range
entry points of the C ABI, and the shifted sums S1 = sum_k (g_k - g*), S2 = sum_k (g_k - g*)^2 are
then added over the ranks: one all-reduce (sum) per use is the only exchange.  The statistics are
finished on every rank from the merged sums with the total K.  A draw is keyed by (seed, tensor,
use, draw, element), so the draws a rank takes are the ones a single GPU would have taken at those
indices, and merged sums equal a single run's up to the order of FP32 additions.

Nothing of the method's arithmetic lives here: kernels through `binding`, the collective through
`torch.distributed` (NCCL on GPUs; the remote partial sums are reduced into local memory first and
read from there).
"""
from __future__ import annotations

import torch

from . import binding as b
from .harness import NormLinearGpu


def draw_range(K: int, world: int, rank: int):
    """(first draw, number of draws) of `rank`: contiguous shares, the first K % world one larger."""
    if K < 0 or world <= 0 or not 0 <= rank < world:
        raise ValueError("bad draw partition")
    base, rem = divmod(K, world)
    return rank * base + min(rank, rem), base + (1 if rank < rem else 0)


def merge_sums(tensors, group=None):
    """Sum each tensor over the ranks, in place (no-op in a single process).  One flat buffer, one
    collective."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return
    flat = torch.cat([t.reshape(-1) for t in tensors])
    dist.all_reduce(flat, op=dist.ReduceOp.SUM, group=group)
    off = 0
    for t in tensors:
        n = t.numel()
        t.copy_(flat[off:off + n].view_as(t))
        off += n


class ShardedFreshReads:
    """Gain use and weight use under the fresh read, draws [k0, k0 + nd) of K on this rank."""

    def __init__(self, g: NormLinearGpu, K: int, rank: int = 0, world: int = 1, draw_buffer_draws: int = 16):
        inp = g.inp
        self.g, self.K, self.rank, self.world = g, K, rank, world
        self.k0, self.nd = draw_range(K, world, rank)
        T, C, O = g.T, g.C, g.O
        dev = "cuda"
        act = torch.bfloat16 if inp.dtype == "bf16" else torch.float32
        self.du = torch.zeros(T * C, dtype=act, device=dev)
        self.dg_ref, self.db_ref = torch.zeros(C, device=dev), torch.zeros(C, device=dev)
        self.dW_ref = torch.zeros(O * C, device=dev)
        self.S1g, self.S2g = torch.zeros(C, device=dev), torch.zeros(C, device=dev)
        self.S1w, self.S2w = torch.zeros(O * C, device=dev), torch.zeros(O * C, device=dev)
        self.chunk = max(1, min(draw_buffer_draws, max(self.nd, 1)))
        self.fresh_t = torch.zeros(self.chunk * C * g.ld_t, dtype=torch.uint8, device=dev)
        self.ws_dgrad = b.workspace(b.bsp_linear_dgrad_workspace_bytes(T, O, C))
        self.ws_bwd = b.workspace(b.bsp_norm_bwd_workspace_bytes(T, C))
        self.ws_gain = b.workspace(b.bsp_norm_gain_mc_workspace_bytes(T, C, max(self.nd, 1)))
        self.ws_wgrad = b.workspace(max(b.bsp_linear_wgrad_workspace_bytes(T, O, C, b.READ_FORWARD), 256))
        self.ws_stats = b.workspace(b.bsp_mc_stats_workspace_bytes(O * C))
        self.qf = b.quant(inp.store_fmt, b.ROUND_STOCHASTIC, 1.0, g.scale)

    def prepare(self):
        """Once: du and the two reference gradients (gain use reads the original, weight use the
        forward's rounding).  Identical on every rank."""
        g, inp = self.g, self.g.inp
        T, C, O = g.T, g.C, g.O
        b.bsp_linear_dgrad(T, O, C, g.dy_codes, g.q_dy, g.W, self.du, self.ws_dgrad, g.diag)
        b.bsp_norm_bwd(g.kind, g.x, T, C, g.gamma, g.beta, g.rstd, g.mean, self.du, b.READ_ORIGINAL, None, g.q,
                       b.key(inp.seed, g.tensor_id, b.STREAM_GAIN, 0), self.dg_ref, self.db_ref, None, self.ws_bwd, g.diag)
        b.bsp_linear_wgrad(T, O, C, g.dy_codes_t, g.q_dy, b.READ_FORWARD, g.u_codes_t, g.q, g.ld_t, self.dW_ref,
                           ws=self.ws_wgrad, diag=g.diag)

    def local_sums(self):
        """This rank's draws into S1, S2 of both uses (cleared first)."""
        g, inp = self.g, self.g.inp
        T, C, O = g.T, g.C, g.O
        for t in (self.S1g, self.S2g, self.S1w, self.S2w):
            t.zero_()
        if self.nd == 0:
            return
        b.bsp_norm_gain_mc(g.kind, g.x, T, C, g.gamma, g.beta, g.rstd, g.mean, self.du, self.qf,
                           b.key(inp.seed, g.tensor_id, b.STREAM_GAIN, 0), self.k0, self.nd, self.dg_ref, self.S1g,
                           self.S2g, self.ws_gain, g.diag)
        kw = b.key(inp.seed, g.tensor_id, b.STREAM_WGRAD, 0)
        for c0 in range(0, self.nd, self.chunk):
            n = min(self.chunk, self.nd - c0)
            b.bsp_norm_fwd_draws(g.kind, g.x, T, C, g.gamma, g.beta, g.rstd, g.mean, self.qf, kw, self.k0 + c0, n,
                                 self.fresh_t, g.ld_t)
            b.bsp_linear_wgrad_mc(T, O, C, g.dy_codes_t, g.q_dy, self.fresh_t, self.qf, g.ld_t, n, self.dW_ref,
                                  self.S1w, self.S2w, g.diag)

    def merge(self, group=None):
        merge_sums([self.S1g, self.S2g, self.S1w, self.S2w], group)

    def statistics(self, rule=None):
        """(gain use, weight use) results from the merged sums and the total K."""
        g = self.g
        rg = b.bsp_mc_stats(self.dg_ref, self.S1g, self.S2g, g.C, self.K, 1, self.ws_stats, rule=rule)
        rw = b.bsp_mc_stats(self.dW_ref, self.S1w, self.S2w, g.O * g.C, self.K, 1, self.ws_stats, rule=rule)
        return rg, rw

    def step(self, group=None, rule=None):
        self.local_sums()
        self.merge(group)
        return self.statistics(rule)
