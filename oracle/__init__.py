"""CPU oracle for the backward-state-policy operators and their per-use check.

TEST INFRASTRUCTURE, NOT PRODUCT.  Plain numpy, float64 unless a step is pinned to FP32, slow
and written to be checked against the paper by eye.  Only the tests, the smoke entry and the
benchmark's CPU-baseline leg may import this package; the CUDA library never does, and this
package imports nothing from it.  No blocking, fusion or reordering beyond what each definition
states.

Modules (each function cites the passage of the paper it follows):
  philox     Philox4x32-10 and the (seed, tensor, use, draw, element) keying
  fp8        E4M3 / E5M2 codec, round-to-nearest-even and stochastic rounding
  norm       RMSNorm / LayerNorm store forward, the three reads, backward
  linear     incoming gradient, weight gradient, input-gradient helper
  attention  causal attention forward statistics and backward with the D use
  mc         Monte-Carlo reduction, statistics z, R, Q', verdict
  store      the paper's own b-bit per-token store and its reads (incl. the U/R+eps read)
  logsoftmax log-softmax backward with a +-eps error in its saved output, two losses
  coupling   averages over the forward's rounding: mean-error / coupling split, statistics T and X
  probs      rounded attention probabilities as the saved tensor: exact enumeration and Monte-Carlo form

Parity unpinned (no value of the paper fixes them; only GPU == oracle): the verdict
thresholds of `mc.verdict`, and the quantisation points / P and dS scales of the FP8-operand
attention mode.
"""
