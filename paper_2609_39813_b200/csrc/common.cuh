// Device-side building blocks shared by the kernels: Philox4x32-10, the FP8 codec, typed loads.
// Everything here is written for sm_100a; integer paths are bit-exact by construction.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/bsp.h"

#define BSP_CHECK_CUDA(expr)                      \
  do {                                            \
    cudaError_t _e = (expr);                      \
    if (_e != cudaSuccess) return BSP_ERR_CUDA;   \
  } while (0)

// Every kernel launch of the library is followed by this: it counts the launch (see
// bsp_launch_count) and turns a launch error into BSP_ERR_CUDA.
#define BSP_LAUNCH_CHECK()                   \
  do {                                       \
    ::bsp::count_launch();                   \
    BSP_CHECK_CUDA(cudaGetLastError());      \
  } while (0)

namespace bsp {

void count_launch();          // defined in mc.cu
void count_d2h(size_t bytes);  // bytes the library itself copies device -> host (mc.cu)

constexpr int kNumSMs = 148;

// The K-draw gain use behind bsp_norm_gain_mc; `thin` selects the kernel variant made to run beside
// a kernel that already fills the SMs (its slabs are shorter, so its workspace is larger).
// `grid_steps` (per-token steps [T]) switches the rounding law from the FP8 store to the b-bit
// per-token grid (q is then ignored apart from its format, which must still be valid).
size_t norm_gain_mc_workspace(int64_t T, int64_t C, int K, bool thin);
int norm_gain_mc_run(bool thin, int kind, const void* x, int dt, int64_t T, int64_t C, const float* gamma,
                     const float* beta, const float* rstd, const float* mean, const void* du, int du_dt, bsp_quant_t q,
                     bsp_key_t key, int draw0, int K, const float* g_ref, float* S1, float* S2, void* ws, size_t ws_bytes,
                     bsp_diag_t* diag, void* stream, const float* grid_steps = nullptr);

// Index of the current device into a per-device flag array of kMaxDevices entries (a function
// attribute such as the dynamic shared-memory limit is set once per device, not once per process).
constexpr int kMaxDevices = 64;
inline int device_slot() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) dev = 0;
  return dev % kMaxDevices;
}

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static inline size_t round_up(size_t a, size_t b) { return (a + b - 1) / b * b; }

// ------------------------------------------------------------------------------- Philox

struct PhiloxKey {
  uint32_t k0, k1;     // lo32(seed), hi32(seed)
  uint32_t c2, c3;     // draw, (tensor_id << 8) | stream
};

static inline PhiloxKey make_key(const bsp_key_t& k) {
  PhiloxKey p;
  p.k0 = (uint32_t)(k.seed & 0xFFFFFFFFull);
  p.k1 = (uint32_t)(k.seed >> 32);
  p.c2 = k.draw;
  p.c3 = (k.tensor_id << 8) | (k.stream & 0xFFu);
  return p;
}

// Ten rounds; counter (c0, c1, c2, c3), key (k0, k1).  Returns the four output words.
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               uint32_t k0, uint32_t k1) {
  constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    // one 32x32->64 multiply per lane pair (mul.wide.u32), one three-input XOR per new word
    const uint64_t p0 = (uint64_t)M0 * c0;
    const uint64_t p1 = (uint64_t)M1 * c2;
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ (k0 + (uint32_t)r * W0);
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ (k1 + (uint32_t)r * W1);
    c0 = n0; c1 = (uint32_t)p1; c2 = n2; c3 = (uint32_t)p0;
  }
  return make_uint4(c0, c1, c2, c3);
}

// Words of elements 4q .. 4q+3 of a tensor (q = element index >> 2).
__device__ __forceinline__ uint4 philox_block(const PhiloxKey& k, uint64_t q, uint32_t draw) {
  return philox4x32_10((uint32_t)q, (uint32_t)(q >> 32), draw, k.c3, k.k0, k.k1);
}

__device__ __forceinline__ uint32_t word_of(const uint4& w, uint32_t lane) {
  return lane == 0 ? w.x : lane == 1 ? w.y : lane == 2 ? w.z : w.w;
}

// ------------------------------------------------------------------------------- FP8 codec

template <int FMT> struct F8;
template <> struct F8<BSP_E4M3> {
  static constexpr int MB = 3, EMIN = -6, BIAS = 7;
  static constexpr uint32_t FMAX_BITS = 0x43E00000u;   // 448.0f
  static constexpr uint32_t MINNORM_BITS = 0x3C800000u;   // 2^-6
  static constexpr uint32_t TOP = 0x7Eu;
  static constexpr uint32_t EMASK = 0xFu;
};
template <> struct F8<BSP_E5M2> {
  static constexpr int MB = 2, EMIN = -14, BIAS = 15;
  static constexpr uint32_t FMAX_BITS = 0x47600000u;   // 57344.0f
  static constexpr uint32_t MINNORM_BITS = 0x38800000u;   // 2^-14
  static constexpr uint32_t TOP = 0x7Bu;
  static constexpr uint32_t EMASK = 0x1Fu;
};

// Per-thread counters, flushed to bsp_diag_t once per thread.
struct DiagCounters {
  uint32_t sat = 0, nonfinite = 0;
};

// Round an FP32 value to an FP8 code.  e = max(floor(log2|v|), EMIN), ulp = 2^(e-MB),
// n = floor(|v|/ulp), f = frac.  Nearest: up iff f > 1/2 or tie with n odd.  Stochastic: up iff
// U < floor(f * 2^32).  Saturating; the sign bit is kept even when the magnitude rounds to zero.
template <int FMT, bool STOCHASTIC>
__device__ __forceinline__ uint32_t f8_encode(float v, uint32_t U, DiagCounters& dc) {
  using F = F8<FMT>;
  const uint32_t b = __float_as_uint(v);
  const uint32_t sign = (b >> 24) & 0x80u;
  const uint32_t a = b & 0x7FFFFFFFu;
  if (a >= F::FMAX_BITS) {
    if (a > 0x7F800000u) { dc.nonfinite++; return 0x7Fu; }              // any NaN -> the one NaN code
    if (a == 0x7F800000u) dc.nonfinite++; else if (a > F::FMAX_BITS) dc.sat++;
    return sign | F::TOP;
  }
  uint32_t base, up;
  if (a >= F::MINNORM_BITS) {
    // normal range of the format: drop d low mantissa bits of the FP32 pattern
    constexpr int d = 23 - F::MB;
    const uint32_t rem = a & ((1u << d) - 1u);
    const uint32_t n = a >> d;                                             // exponent and kept mantissa
    base = n - ((uint32_t)(127 - F::BIAS) << F::MB);                       // re-bias the exponent
    if (STOCHASTIC) {
      up = U < (rem << (32 - d));
    } else {
      constexpr uint32_t half = 1u << (d - 1);
      up = (rem > half) | ((rem == half) & (n & 1u));
    }
  } else {
    // subnormal range: uniform grid of step 2^(EMIN-MB).  t = |v| / step is an exact FP32 product
    // (a power-of-two scaling), n = floor(t) < 2^MB, f = t - n exact, floor(f * 2^32) exact.
    const float t = __uint_as_float(a) * __uint_as_float((uint32_t)(F::MB - F::EMIN + 127) << 23);
    const uint32_t n = (uint32_t)t;
    const float f = t - (float)n;
    base = n;
    if (STOCHASTIC) {
      up = U < __float2uint_rd(f * 4294967296.0f);
    } else {
      up = (f > 0.5f) | ((f == 0.5f) & (n & 1u));
    }
  }
  return sign | (base + up);
}

// Value of the stochastic rounding of v as FP32, i.e. decode(encode_SR(v)) without the detour
// through the code: in the normal range the FP32 pattern is truncated and bumped in place.
template <int FMT>
__device__ __forceinline__ float f8_sr_value(float v, uint32_t U) {
  using F = F8<FMT>;
  const uint32_t b = __float_as_uint(v);
  const uint32_t a = b & 0x7FFFFFFFu;
  const uint32_t s = b & 0x80000000u;
  if (a >= F::FMAX_BITS) {
    if (a > 0x7F800000u) return __uint_as_float(0x7FC00000u);
    return __uint_as_float(s | F::FMAX_BITS);
  }
  if (a >= F::MINNORM_BITS) {
    constexpr int d = 23 - F::MB;
    const uint32_t rem = a & ((1u << d) - 1u);
    const uint32_t up = U < (rem << (32 - d));
    return __uint_as_float(s | ((a - rem) + (up << d)));
  }
  const float t = __uint_as_float(a) * __uint_as_float((uint32_t)(F::MB - F::EMIN + 127) << 23);
  const uint32_t n = (uint32_t)t;
  const float f = t - (float)n;
  const uint32_t up = U < __float2uint_rd(f * 4294967296.0f);
  const float mag = (float)(n + up) * __uint_as_float((uint32_t)(F::EMIN - F::MB + 127) << 23);
  return __uint_as_float(s | __float_as_uint(mag));
}

// The draw-independent part of the stochastic rounding of v: the threshold P such that the
// element rounds up (away from zero, by one code) exactly when its generator word U < P.  The same
// decision as f8_encode / f8_sr_value take: P = 0 when v is on the grid, saturates or is NaN.  With
// it, K draws of one element cost one comparison each: value(U) = value(~0) + (U < P) * step, and
// code(U) = code(~0) + (U < P).
template <int FMT>
__device__ __forceinline__ uint32_t f8_sr_threshold(float v) {
  using F = F8<FMT>;
  const uint32_t a = __float_as_uint(v) & 0x7FFFFFFFu;
  if (a >= F::FMAX_BITS) return 0u;
  if (a >= F::MINNORM_BITS) {
    constexpr int d = 23 - F::MB;
    return (a & ((1u << d) - 1u)) << (32 - d);
  }
  const float t = __uint_as_float(a) * __uint_as_float((uint32_t)(F::MB - F::EMIN + 127) << 23);
  const float f = t - (float)(uint32_t)t;
  return __float2uint_rd(f * 4294967296.0f);
}

// Nearest-even rounding of two in-range FP32 values (|v| below the format's maximum) to two codes
// with the hardware conversion: `lo` in bits 0..7, `hi` in bits 8..15.  NaN, infinities and
// magnitudes at or above the maximum never come here (the callers route those to f8_encode).
template <int FMT>
__device__ __forceinline__ uint32_t f8_encode_rn_pair_inrange(float lo, float hi) {
  uint16_t r;
  if (FMT == BSP_E4M3) asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  else asm("cvt.rn.satfinite.e5m2x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  return (uint32_t)r;
}

// Value of the nearest-even rounding of v as FP32, i.e. decode(encode_RN(v)); saturating.
template <int FMT>
__device__ __forceinline__ float f8_rn_value(float v) {
  using F = F8<FMT>;
  const uint32_t b = __float_as_uint(v);
  const uint32_t a = b & 0x7FFFFFFFu;
  const uint32_t s = b & 0x80000000u;
  if (a >= F::FMAX_BITS) {
    if (a > 0x7F800000u) return __uint_as_float(0x7FC00000u);
    return __uint_as_float(s | F::FMAX_BITS);
  }
  if (a >= F::MINNORM_BITS) {
    constexpr int d = 23 - F::MB;
    const uint32_t lsb = (a >> d) & 1u;
    const uint32_t r = (a + ((1u << (d - 1)) - 1u) + lsb) & ~((1u << d) - 1u);   // ties to even
    return __uint_as_float(s | r);
  }
  const float t = __uint_as_float(a) * __uint_as_float((uint32_t)(F::MB - F::EMIN + 127) << 23);
  const float n = rintf(t);                                                      // ties to even, t < 2^MB
  return __uint_as_float(s | __float_as_uint(n * __uint_as_float((uint32_t)(F::EMIN - F::MB + 127) << 23)));
}

// Exact FP32 value of a code.
template <int FMT>
__device__ __forceinline__ float f8_decode(uint32_t c) {
  using F = F8<FMT>;
  const uint32_t s = (c & 0x80u) << 24;
  const uint32_t ef = (c >> F::MB) & F::EMASK;
  const uint32_t m = c & ((1u << F::MB) - 1u);
  if (FMT == BSP_E4M3) {
    if ((c & 0x7Fu) == 0x7Fu) return __uint_as_float(s | 0x7FC00000u);
  } else {
    if (ef == 31u) return __uint_as_float(s | (m ? 0x7FC00000u : 0x7F800000u));
  }
  if (ef == 0) {
    // subnormal: m * 2^(EMIN - MB); m < 8 is exact in FP32
    const float mag = (float)m * __uint_as_float((uint32_t)(F::EMIN - F::MB + 127) << 23);
    return __uint_as_float(s | __float_as_uint(mag));
  }
  return __uint_as_float(s | ((ef - F::BIAS + 127u) << 23) | (m << (23 - F::MB)));
}

// Four codes (packed little-endian in one word) to FP32 with the hardware conversions: FP8 pair ->
// f16 pair (exact: every E4M3 / E5M2 value is an f16 value) -> FP32.  NaN and infinity codes come
// out as FP32 NaN / infinity.
template <int FMT>
__device__ __forceinline__ void f8_decode4(uint32_t packed, float (&out)[4]) {
  uint32_t h01, h23;
  const uint16_t lo = (uint16_t)(packed & 0xFFFFu), hi = (uint16_t)(packed >> 16);
  if (FMT == BSP_E4M3) {
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h01) : "h"(lo));
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h23) : "h"(hi));
  } else {
    asm("cvt.rn.f16x2.e5m2x2 %0, %1;" : "=r"(h01) : "h"(lo));
    asm("cvt.rn.f16x2.e5m2x2 %0, %1;" : "=r"(h23) : "h"(hi));
  }
  const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&h01));
  const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&h23));
  out[0] = a.x; out[1] = a.y; out[2] = b.x; out[3] = b.y;
}

__device__ __forceinline__ void diag_flush(bsp_diag_t* diag, const DiagCounters& dc) {
  if (diag == nullptr) return;
  if (dc.sat) atomicAdd(&diag->n_saturated, (unsigned long long)dc.sat);
  if (dc.nonfinite) {
    atomicAdd(&diag->n_nonfinite, (unsigned long long)dc.nonfinite);
    atomicMax(&diag->status, (int)BSP_ERR_NONFINITE);
  }
}

// Warp-aggregated flush: one atomic per warp.
__device__ __forceinline__ void diag_flush_warp(bsp_diag_t* diag, DiagCounters dc) {
  if (diag == nullptr) return;
  uint32_t sat = dc.sat, nf = dc.nonfinite;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    sat += __shfl_xor_sync(0xFFFFFFFFu, sat, o);
    nf += __shfl_xor_sync(0xFFFFFFFFu, nf, o);
  }
  if ((threadIdx.x & 31) == 0) {
    DiagCounters t; t.sat = sat; t.nonfinite = nf;
    diag_flush(diag, t);
  }
}

// ------------------------------------------------------------------------------- typed loads

__device__ __forceinline__ float bf16_bits_to_float(uint32_t h) { return __uint_as_float(h << 16); }

// Four consecutive elements starting at element index i (i % 4 == 0, pointer 16-byte aligned).
template <int DT>
__device__ __forceinline__ float4 load4(const void* p, size_t i) {
  if (DT == BSP_F32) {
    return __ldg(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(p) + i));
  } else {
    const uint2 r = __ldg(reinterpret_cast<const uint2*>(reinterpret_cast<const uint16_t*>(p) + i));
    return make_float4(bf16_bits_to_float(r.x & 0xFFFFu), bf16_bits_to_float(r.x >> 16),
                       bf16_bits_to_float(r.y & 0xFFFFu), bf16_bits_to_float(r.y >> 16));
  }
}

// Sixteen consecutive elements starting at element index i (i % 16 == 0, pointer 16-byte aligned),
// with 16-byte loads only: four for FP32, two for bf16.
template <int DT>
__device__ __forceinline__ void load16(const void* p, size_t i, float (&v)[16]) {
  if (DT == BSP_F32) {
    const float4* q = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(p) + i);
    const float4 a = __ldg(q), b = __ldg(q + 1), c = __ldg(q + 2), d = __ldg(q + 3);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    v[8] = c.x; v[9] = c.y; v[10] = c.z; v[11] = c.w; v[12] = d.x; v[13] = d.y; v[14] = d.z; v[15] = d.w;
  } else {
    const uint4* q = reinterpret_cast<const uint4*>(reinterpret_cast<const uint16_t*>(p) + i);
    const uint4 a = __ldg(q), b = __ldg(q + 1);
    const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      v[2 * j] = bf16_bits_to_float(w[j] & 0xFFFFu);
      v[2 * j + 1] = bf16_bits_to_float(w[j] >> 16);
    }
  }
}

template <int DT>
__device__ __forceinline__ float load1(const void* p, size_t i) {
  if (DT == BSP_F32) return __ldg(reinterpret_cast<const float*>(p) + i);
  return bf16_bits_to_float(__ldg(reinterpret_cast<const uint16_t*>(p) + i));
}

// Round-to-nearest-even float -> bf16 bit pattern (finite inputs).
__device__ __forceinline__ uint32_t float_to_bf16_bits(float f) {
  return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(f));
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
  return v;
}

}  // namespace bsp
