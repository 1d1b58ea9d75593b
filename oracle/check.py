"""The per-use check on one operator, run without training: the steps in the paper's order.

Reference (Section "Each use has a checkable requirement"): the gradient of the forward as it
ran with every rounding passed straight through -- gain use reads the original, the input
gradient uses unrounded values, the weight use reads the rounded value the layer multiplied,
and attention's D reads the original output.  Each (use, policy) is then evaluated with the
forward and the incoming gradient held fixed; a fresh read is averaged over K draws of its own
stream.

Test infrastructure: see the package docstring.
"""
from __future__ import annotations

import numpy as np

from . import attention, fp8, linear, mc, norm, philox

TENSOR_U = 1        # tensor id of the normalisation store in the generator key
TENSOR_O = 2        # tensor id of the attention output store

U, R, N = norm.READ_ORIGINAL, norm.READ_FORWARD, norm.READ_FRESH


def prepare_norm_linear(x, gamma, beta, W, dY, kind, eps, seed, act_dtype="f32",
                        store_fmt=fp8.E4M3, grad_fmt=fp8.E5M2, forward_mode=fp8.SR,
                        rstd32=None, mean32=None, du=None):
    """Everything that is computed once per workload: the forward with its store, the incoming
    gradient and du.  `rstd32`/`mean32` (the statistics the GPU saved) and `du` may be supplied
    so that both sides round exactly the same FP32 values and receive the same gradient."""
    fw = norm.forward(x, gamma, beta, kind, eps)
    if rstd32 is None:
        rstd32 = fw["rstd"].astype(np.float32)
    if mean32 is None:
        mean32 = fw["mean"].astype(np.float32)
    u32 = norm.store_value_fp32(x, gamma, beta, kind, rstd32, mean32, None)
    amax = np.float32(np.max(np.abs(u32)))
    scale, inv = fp8.scale_from_amax(amax, store_fmt)
    v32 = norm.store_value_fp32(x, gamma, beta, kind, rstd32, mean32, scale)
    codes, n_sat, n_nf = norm.store_codes(v32, store_fmt, forward_mode, seed, TENSOR_U,
                                          philox.STREAM_FORWARD, 0)
    g = linear.incoming_gradient(dY, grad_fmt)
    if du is None:
        du = linear.dgrad(g["value"], W)
        du = linear.bf16_round(du) if act_dtype == "bf16" else du.astype(np.float32).astype(np.float64)
    return dict(fw=fw, rstd32=rstd32, mean32=mean32, u32=u32, amax=amax, scale=np.float32(scale),
                inv_scale=np.float32(inv), v32=v32, codes=codes, n_saturated=n_sat,
                n_nonfinite=n_nf, dy=g, du=np.asarray(du, dtype=np.float64), store_fmt=store_fmt)


def fresh_copy(prep, seed, stream, draw, cols=None):
    """Policy N: decode(SR(v; words of (stream, draw))) * inv_scale, always stochastic, at the
    store's own scale.  `cols` restricts to a set of feature columns (all tokens)."""
    v32 = prep["v32"]
    if cols is None:
        codes, _, _ = norm.store_codes(v32, prep["store_fmt"], fp8.SR, seed, TENSOR_U, stream, draw)
    else:
        T, C = v32.shape
        cols = np.asarray(cols, dtype=np.uint64)
        elem = np.arange(T, dtype=np.uint64)[:, None] * np.uint64(C) + cols[None, :]
        codes, _, _ = norm.store_codes(v32[:, cols.astype(np.int64)], prep["store_fmt"], fp8.SR,
                                       seed, TENSOR_U, stream, draw, elem)
    return norm.read_value(codes, prep["store_fmt"], prep["inv_scale"]), codes


def gain_use(x, gamma, beta, kind, eps, prep, policy, K, seed, stream=philox.STREAM_GAIN):
    """dgamma (and dbeta) under one read at the gain use, against the reference (read U).
    Returns dict(ref, mean, m2, stats, dbeta)."""
    ref = norm.backward(x, gamma, beta, kind, eps, prep["du"])
    if policy == U:
        g = ref["dgamma"]
        return dict(ref=ref["dgamma"], mean=g, m2=None, dbeta=ref["dbeta"],
                    stats=mc.statistics(g, None, 1, ref["dgamma"], False))
    if policy == R:
        copy = norm.read_value(prep["codes"], prep["store_fmt"], prep["inv_scale"])
        g = norm.dgamma_from_copy(copy, gamma, beta, prep["du"])
        return dict(ref=ref["dgamma"], mean=g, m2=None, dbeta=ref["dbeta"],
                    stats=mc.statistics(g, None, 1, ref["dgamma"], False))
    acc = mc.Welford(ref["dgamma"].shape)
    for k in range(K):
        copy, _ = fresh_copy(prep, seed, stream, k)
        acc.add(norm.dgamma_from_copy(copy, gamma, beta, prep["du"]))
    return dict(ref=ref["dgamma"], mean=acc.mean, m2=acc.m2, dbeta=ref["dbeta"],
                stats=mc.statistics(acc.mean, acc.m2, K, ref["dgamma"], True))


def wgrad_use(prep, policy, K, seed, rows=None, cols=None, stream=philox.STREAM_WGRAD,
              operand_round=linear.bf16_round):
    """dW under one read at the weight use, against the reference (read R), optionally on the
    output sub-block rows x cols.  The original is rounded to the contraction's operand type
    (`operand_round`) before the product.  Returns dict(ref, mean, m2, stats)."""
    dyv = prep["dy"]["value"]
    xr = norm.read_value(prep["codes"], prep["store_fmt"], prep["inv_scale"])
    ref = linear.wgrad(dyv, xr, rows, cols)
    if policy == R:
        return dict(ref=ref, mean=ref, m2=None, stats=mc.statistics(ref, None, 1, ref, False))
    if policy == U:
        xu = operand_round(prep["u32"].astype(np.float64))
        g = linear.wgrad(dyv, xu, rows, cols)
        return dict(ref=ref, mean=g, m2=None, stats=mc.statistics(g, None, 1, ref, False))
    acc = mc.Welford(ref.shape)
    for k in range(K):
        copy, _ = fresh_copy(prep, seed, stream, k, cols)
        acc.add(linear.wgrad(dyv, copy, rows, None))
    return dict(ref=ref, mean=acc.mean, m2=acc.m2,
                stats=mc.statistics(acc.mean, acc.m2, K, ref, True))


# ------------------------------------------------------------------------------- attention


def prepare_attention_slice(q, k, v, dO, c, seed, slice_index, causal=True,
                            store_fmt=fp8.E4M3, forward_mode=fp8.SR, o32=None):
    """Once per (batch, head) slice: O_orig = P V (kept as FP32, the value the store rounds),
    its per-slice scale from its own amax, and the forward's codes.  Element indices are those
    of the full [B, H, S, d] tensor: slice_index * S * d + position.  `o32` may be supplied (the
    FP32 output the GPU stored) so both sides round the same values."""
    S, d = np.asarray(q).shape
    if o32 is None:
        o64, lse = attention.forward_output(q, k, v, c, causal)
        o32 = o64.astype(np.float32)
    else:
        _, lse = attention.probabilities(q, k, c, causal)
        o32 = np.asarray(o32, dtype=np.float32)
    amax = np.float32(np.max(np.abs(o32)))
    scale, inv = fp8.scale_from_amax(amax, store_fmt)
    v32 = (o32 * np.float32(scale)).astype(np.float32)
    elem = np.uint64(slice_index) * np.uint64(S * d) + np.arange(S * d, dtype=np.uint64).reshape(S, d)
    codes, n_sat, n_nf = norm.store_codes(v32, store_fmt, forward_mode, seed, TENSOR_O,
                                          philox.STREAM_FORWARD, 0, elem)
    return dict(o32=o32, lse=lse, amax=amax, scale=np.float32(scale), inv_scale=np.float32(inv),
                v32=v32, codes=codes, elem=elem, store_fmt=store_fmt, n_saturated=n_sat)


def attention_d_copy(prep, policy, seed, draw, stream=philox.STREAM_ATTN_D):
    """The copy of O that D reads under one policy (float64 [S, d])."""
    if policy == U:
        return prep["o32"].astype(np.float64)
    if policy == R:
        return norm.read_value(prep["codes"], prep["store_fmt"], prep["inv_scale"])
    codes, _, _ = norm.store_codes(prep["v32"], prep["store_fmt"], fp8.SR, seed, TENSOR_O, stream,
                                   draw, prep["elem"])
    return norm.read_value(codes, prep["store_fmt"], prep["inv_scale"])


def attention_d_use(q, k, v, dO, c, prep, policy, K, seed, causal=True, outputs=("D", "dq", "dk", "dv"),
                    operand_round=None, fp8_operands=False, scale_p=256.0, scale_ds=None):
    """Attention backward under one read at the D use, against the reference (D reads the original
    output).  BF16-operand mode by default (every product in float64 on the given operands,
    optionally with `operand_round` on P and dS); with `fp8_operands`, q, k, v, dO must be the
    dequantised FP8 operands and the emulated backward of Appendix "The forks" is evaluated
    (P rounded at scale_p before dV, dS rounded at scale_ds before dQ and dK).
    Returns {name: dict(ref, mean, m2, stats)}."""
    def bwd(copy):
        return attention.backward(q, k, v, dO, c, copy, causal, fp8_operands=fp8_operands, scale_p=scale_p,
                                  scale_ds=scale_ds, operand_round=operand_round)

    ref = bwd(attention_d_copy(prep, U, seed, 0))
    out = {}
    if policy in (U, R):
        g = bwd(attention_d_copy(prep, policy, seed, 0))
        for name in outputs:
            out[name] = dict(ref=ref[name], mean=g[name], m2=None,
                             stats=mc.statistics(g[name], None, 1, ref[name], False))
        return out
    accs = {name: mc.Welford(ref[name].shape) for name in outputs}
    for kk in range(K):
        g = bwd(attention_d_copy(prep, N, seed, kk))
        for name in outputs:
            accs[name].add(g[name])
    for name in outputs:
        a = accs[name]
        out[name] = dict(ref=ref[name], mean=a.mean, m2=a.m2,
                         stats=mc.statistics(a.mean, a.m2, K, ref[name], True))
    return out
