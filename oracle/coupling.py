"""Averaging over the forward's rounding: the mean-error / coupling split and the paired statistics.

Appendix "What the checker reads and reports": with the use's backward rule B h, the reference's
B* h and Delta = B - B*, averaging over the forward's rounding as well (inputs and weights fixed)
splits the use's average error into a mean error and a coupling,
    E[Delta h] = E[Delta] E[h] + E[(Delta - E Delta)(h - E h)].
Appendix "The same dependence in a normalization backward": for independent draws r and r' and
g(v) the incoming gradient when the forward consumes v, the paired statistic
    T = (1/2) <r - r', g(u + r) - g(u + r')>
averages to the difference between the errors from reading the consumed copy and an independent
copy; the control for the independent copy is <g(u + r), r'>.  With round-to-nearest the forwards
are identical and T is exactly zero.  Appendix "The normalization store" (continuation probes):
two forwards draw stores with errors r_a, r_b and incoming gradients dy_a, dy_b;
    X = -(1/2) (r_a - r_b)^T (dy_a - dy_b)
averages to the error at the weight use, -r^T dy.

Setting (the loss makes the incoming gradient depend on the consumed rounding, Section "One
tensor, two uses": "a looser test"): normalisation -> FP8 store -> y = u_q W^T, loss
(1/2) ||y||^2, so dy = y and du = dy W.  The gain use reading the forward's rounding errs by
sum_t (r / gamma) o du, the weight use reading the original by -dy^T r (as dW[O, C]).
Closed forms under stochastic rounding with per-entry variance sigma^2 (A = W^T W):
    E[gain error]_c = sum_t sigma^2[t, c] A[c, c] / gamma_c   (all coupling, no mean error),
    E[T] = sum_{t, c} sigma^2[t, c] A[c, c],   E[control] = 0,
    E[X] = E[-r^T dy] = -diag(sum_t sigma^2) W^T   (as [C, O]).

Readings: the forward's roundings are draws 0, 1, 2, ... of generator stream 0; pair k is draws
(2k, 2k + 1); a fresh read at the gain use takes stream 1 with the draw of the forward it goes
with; r = u_q - u with u the FP32 chain value the store rounds.

Test infrastructure: see the package docstring.
"""
from __future__ import annotations

import numpy as np

from . import fp8, norm, philox

TENSOR_U = 1


def prepare(x, gamma, beta, W, kind, eps, store_fmt=fp8.E4M3, rstd32=None, mean32=None):
    """What does not depend on the rounding: the FP32 chain value u32, the per-tensor scale, the
    scaled value v32 the store rounds, z, and the per-entry variance of one stochastic rounding."""
    fw = norm.forward(x, gamma, beta, kind, eps)
    if rstd32 is None:
        rstd32 = fw["rstd"].astype(np.float32)
    if mean32 is None:
        mean32 = fw["mean"].astype(np.float32)
    u32 = norm.store_value_fp32(x, gamma, beta, kind, rstd32, mean32, None)
    amax = np.float32(np.max(np.abs(u32)))
    scale, inv = fp8.scale_from_amax(amax, store_fmt)
    v32 = norm.store_value_fp32(x, gamma, beta, kind, rstd32, mean32, scale)
    lo, hi, _ = fp8.neighbours(v32, store_fmt)
    a = np.abs(v32.astype(np.float64))
    var = (a - lo) * (hi - a) * float(inv) ** 2
    return dict(fw=fw, u32=u32, v32=v32, scale=np.float32(scale), inv_scale=np.float32(inv), var=var,
                store_fmt=store_fmt, W=np.asarray(W, dtype=np.float64), gamma=np.asarray(gamma, dtype=np.float64))


def forward_draw(prep, seed: int, mode: int, stream: int, draw: int):
    """One rounding of the store: (u_q float64, r = u_q - u32)."""
    codes, _, _ = norm.store_codes(prep["v32"], prep["store_fmt"], mode, seed, TENSOR_U, stream, draw)
    uq = norm.read_value(codes, prep["store_fmt"], prep["inv_scale"])
    return uq, uq - prep["u32"].astype(np.float64)


def gradients(prep, uq):
    """The incoming gradients when the forward consumes uq under the loss ||y||^2 / 2: dy = y = uq W^T
    and du = dy W."""
    dy = uq @ prep["W"].T
    return dy, dy @ prep["W"]


def run(prep, seed: int, pairs: int, mode: int = fp8.SR):
    """`pairs` pairs of forwards (draws 2k and 2k + 1).  Returns per-pair T and control, and the
    averages over all 2 * pairs forwards of the gain-use error under read R (total, mean part,
    coupling) and under a fresh read, of the weight-use error -dy^T r (as [O, C]), and over the pairs
    of X (as [C, O])."""
    g = prep["gamma"][None, :]
    T_k, ctl_k = [], []
    n = 2 * pairs
    shape = prep["u32"].shape
    sum_r, sum_du = np.zeros(shape), np.zeros(shape)
    gain_tot = np.zeros(shape[1]); gain_fresh = np.zeros(shape[1])
    werr = np.zeros((prep["W"].shape[0], shape[1]))
    X = np.zeros((shape[1], prep["W"].shape[0]))
    for k in range(pairs):
        fw = []
        for d in (2 * k, 2 * k + 1):
            uq, r = forward_draw(prep, seed, mode, philox.STREAM_FORWARD, d)
            dy, du = gradients(prep, uq)
            _, rf = forward_draw(prep, seed, fp8.SR, philox.STREAM_GAIN, d)
            sum_r += r; sum_du += du
            gain_tot += np.sum(r / g * du, axis=0)
            gain_fresh += np.sum(rf / g * du, axis=0)
            werr += -(dy.T @ r)
            fw.append((r, dy, du))
        (ra, dya, dua), (rb, dyb, dub) = fw
        T_k.append(0.5 * np.sum((ra - rb) * (dua - dub)))
        ctl_k.append(np.sum(dua * rb))
        X += -0.5 * (ra - rb).T @ (dya - dyb)
    mean_part = np.sum((sum_r / n) / g * (sum_du / n), axis=0)
    total = gain_tot / n
    return dict(T=np.array(T_k), control=np.array(ctl_k), gain_total=total, gain_mean_part=mean_part,
                gain_coupling=total - mean_part, gain_fresh=gain_fresh / n, wgrad_error=werr / n, X=X / pairs)


def closed_forms(prep):
    A_diag = np.sum(prep["W"] ** 2, axis=0)                     # diag(W^T W)
    s2 = np.sum(prep["var"], axis=0)                            # sum over tokens, per column
    return dict(gain=s2 * A_diag / prep["gamma"], T=float(np.sum(s2 * A_diag)),
                X=-(s2[:, None] * prep["W"].T), wgrad_error=-(prep["W"] * s2[None, :]))
