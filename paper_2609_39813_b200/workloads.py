"""Seeded synthetic inputs for the five benchmark configurations.

This module only *draws numbers*: it holds none of the method's arithmetic (no rounding to FP8,
no normalisation, no gradients).  Both the CUDA path and the CPU oracle are fed from the arrays
produced here, so that the two sides see byte-identical inputs.  numpy only; no torch import.

Recipe (host side, `numpy.random.Generator(PCG64(seed))`, tensors drawn in the order listed, each
cast once to its storage dtype):

  cfg 1  RMSNorm(eps 1e-6) -> Linear, tiny.  x[64,128] fp32 N(0,1); gamma = 1 + 0.1 N(0,1);
         W[128,128] N(0, var 1/128); dY[64,128] N(0,1).  K = 256.  data seed 0.
  cfg 2  RMSNorm -> Linear, 390M-model shapes.  x[4096,1024] bf16 N(0,1) with floor(0.01 C) = 10
         feature columns (first entries of a seeded column permutation) multiplied by 20;
         gamma fp32; W[4096,1024] bf16 N(0, var 1/1024); dY[4096,4096] bf16 N(0, var 1e-2).
         K = 64.  data seed 1002.
  cfg 3  causal attention backward.  Q,K,V [8,16,2048,64] bf16 N(0,1)/8; dO bf16 N(0,1);
         softmax scale 1/8.  K = 32.  data seed 1003.
  cfg 4  LayerNorm(eps 1e-5, bias) -> Linear.  x[8192,2048] fp32 Student-t(nu=4) drawn as
         N(0,1)/sqrt(chi2_4/4); gamma = 1 + 0.1 N; beta = 0.1 N; W[2048,2048] fp32
         N(0, var 1/2048); dY[8192,2048] fp32 N(0,1).  K = 1024.  data seed 1004.
  cfg 5  RMSNorm -> Linear, large MLP shape.  x[16384,4096] bf16 N(0,1); gamma; W[11008,4096] bf16
         N(0, var 1/4096); dY[16384,11008] bf16 N(0, var 1e-2).  K = 16.  data seed 1005.

Every config may be generated at reduced sizes (same distributions, same order) for parity
tests; the size overrides are explicit arguments, never silent.

bf16 tensors are returned as float32 arrays whose values are exactly representable in bf16
(`to_bf16_grid`), plus a helper that exposes the raw 16-bit patterns for upload.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, Optional

import numpy as np

FMT_E4M3 = 0
FMT_E5M2 = 1


def to_bf16_grid(a: np.ndarray) -> np.ndarray:
    """Round finite float32 values to the nearest bf16 value (ties to even); result stays float32."""
    out = np.array(a, dtype=np.float32, order="C", copy=True)
    b = out.view(np.uint32)
    lsb = (b >> np.uint32(16)) & np.uint32(1)
    lsb += np.uint32(0x7FFF)
    b += lsb                               # finite values: no carry out of the exponent field's top
    b &= np.uint32(0xFFFF0000)
    return out


def bf16_bits(a_on_grid: np.ndarray) -> np.ndarray:
    """Upper 16 bits of float32 values that already lie on the bf16 grid (uint16, same shape)."""
    a = np.ascontiguousarray(a_on_grid, dtype=np.float32)
    return (a.view(np.uint32) >> np.uint32(16)).astype(np.uint16).reshape(a.shape)


@dataclass
class NormLinearInputs:
    """Inputs of one normalisation -> linear workload (configs 1, 2, 4, 5)."""
    name: str
    norm: str                 # "rms" | "layer"
    eps: float
    dtype: str                # "f32" | "bf16": storage type of x, W, dY, du
    T: int
    C: int
    O: int
    K: int                    # fresh draws of the Monte-Carlo check
    seed: int                 # data seed = rounding seed
    x: np.ndarray             # [T, C] float32 (on the bf16 grid when dtype == "bf16")
    gamma: np.ndarray         # [C] float32
    beta: Optional[np.ndarray]  # [C] float32 or None (RMSNorm)
    W: np.ndarray             # [O, C] float32 (bf16 grid when dtype == "bf16")
    dY: np.ndarray            # [T, O] float32 (bf16 grid when dtype == "bf16")
    store_fmt: int = FMT_E4M3
    grad_fmt: int = FMT_E5M2
    forward_mode: str = "sr"  # rounding law of the forward's store


@dataclass
class AttentionInputs:
    """Inputs of the causal-attention backward workload (config 3)."""
    name: str
    B: int
    H: int
    S: int
    D: int
    K: int
    seed: int
    softmax_scale: float
    q: np.ndarray             # [B,H,S,D] float32 on the bf16 grid
    k: np.ndarray
    v: np.ndarray
    dO: np.ndarray
    store_fmt: int = FMT_E4M3
    forward_mode: str = "sr"
    causal: bool = True


def _normal(rng, shape, std=1.0):
    a = rng.standard_normal(shape, dtype=np.float32)
    if std != 1.0:
        a *= np.float32(std)
    return a


def _store(a, dtype):
    return to_bf16_grid(a) if dtype == "bf16" else a.astype(np.float32)


def config1(T=64, C=128, O=128, K=256, seed=0) -> NormLinearInputs:
    rng = np.random.Generator(np.random.PCG64(seed))
    x = _normal(rng, (T, C))
    gamma = (1.0 + 0.1 * _normal(rng, (C,))).astype(np.float32)
    W = _normal(rng, (O, C), std=float(np.sqrt(1.0 / C)))
    dY = _normal(rng, (T, O))
    return NormLinearInputs("cfg1_rms_tiny", "rms", 1e-6, "f32", T, C, O, K, seed,
                            x, gamma, None, W, dY)


def config2(T=4096, C=1024, O=4096, K=64, seed=1002) -> NormLinearInputs:
    rng = np.random.Generator(np.random.PCG64(seed))
    x = _normal(rng, (T, C))
    n_out = int(np.floor(0.01 * C))
    perm = rng.permutation(C)
    if n_out > 0:
        x[:, perm[:n_out]] *= np.float32(20.0)
    x = _store(x, "bf16")
    gamma = (1.0 + 0.1 * _normal(rng, (C,))).astype(np.float32)
    W = _store(_normal(rng, (O, C), std=float(np.sqrt(1.0 / C))), "bf16")
    dY = _store(_normal(rng, (T, O), std=0.1), "bf16")
    return NormLinearInputs("cfg2_rms_390m", "rms", 1e-6, "bf16", T, C, O, K, seed,
                            x, gamma, None, W, dY)


def config3(B=8, H=16, S=2048, D=64, K=32, seed=1003) -> AttentionInputs:
    rng = np.random.Generator(np.random.PCG64(seed))
    sc = 1.0 / np.sqrt(64.0)
    q = to_bf16_grid(_normal(rng, (B, H, S, D), std=sc))
    k = to_bf16_grid(_normal(rng, (B, H, S, D), std=sc))
    v = to_bf16_grid(_normal(rng, (B, H, S, D), std=sc))
    dO = to_bf16_grid(_normal(rng, (B, H, S, D)))
    return AttentionInputs("cfg3_attn_causal", B, H, S, D, K, seed, 1.0 / 8.0, q, k, v, dO)


def config4(T=8192, C=2048, O=2048, K=1024, seed=1004) -> NormLinearInputs:
    rng = np.random.Generator(np.random.PCG64(seed))
    g = rng.standard_normal((T, C), dtype=np.float32)
    chi = rng.chisquare(4.0, size=(T, C)).astype(np.float32)
    x = (g / np.sqrt(chi / np.float32(4.0))).astype(np.float32)
    gamma = (1.0 + 0.1 * _normal(rng, (C,))).astype(np.float32)
    beta = (0.1 * _normal(rng, (C,))).astype(np.float32)
    W = _normal(rng, (O, C), std=float(np.sqrt(1.0 / C)))
    dY = _normal(rng, (T, O))
    return NormLinearInputs("cfg4_layernorm_sweep", "layer", 1e-5, "f32", T, C, O, K, seed,
                            x, gamma, beta, W, dY)


def config5(T=16384, C=4096, O=11008, K=16, seed=1005) -> NormLinearInputs:
    rng = np.random.Generator(np.random.PCG64(seed))
    x = _store(_normal(rng, (T, C)), "bf16")
    gamma = (1.0 + 0.1 * _normal(rng, (C,))).astype(np.float32)
    W = _store(_normal(rng, (O, C), std=float(np.sqrt(1.0 / C))), "bf16")
    dY = _store(_normal(rng, (T, O), std=0.1), "bf16")
    return NormLinearInputs("cfg5_rms_large_mlp", "rms", 1e-6, "bf16", T, C, O, K, seed,
                            x, gamma, None, W, dY)


CONFIGS = {1: config1, 2: config2, 3: config3, 4: config4, 5: config5}
