// The paper's own normalisation store (Appendix "The normalization store"): a b-bit uniform grid per
// token, step s = max_j |u_j| / (2^(b-1) - 1), u_q = s floor(u / s + xi), and the values its uses read:
// z | u_q / gamma | u_f / gamma at the gain use, u | u_q | u_f | u_q + (u_f - u) at the weight use.
//
// Arithmetic (fixed so that codes are a pure function of value and generator word): u is the FP32
// chain value of the normalisation, s = fl32(amax / M), t = fl32(u / s), n0 = floor(t),
// f = fl32(t - n0), P = min(floor(f 2^32), 2^32 - 1), n = n0 + [W < P] with W the element's 32-bit word.
//
// Kernels: store_fwd_kernel (one block per token: the row is held in registers between the maximum
// and the rounding), store_operand_kernel (the copy a weight use reads, FP32, split into two bf16
// terms hi + lo and written token-minor so that dW = [dY | dY] [X_hi | X_lo]^T runs on the BF16 tensor
// cores with the copy carried to 16 bits; 32 x 32 tiles through shared memory), and the host-side
// check.  The gain use under the b-bit law is the K-draw gain kernel of the FP8 store with the
// thresholds and step weights of this grid.
#include <string.h>

#include "common.cuh"
#include "gemm.cuh"
#include "mc_stats.cuh"

namespace bsp {

enum { STORE_READ_U = 0, STORE_READ_R = 1, STORE_READ_N = 2, STORE_READ_R_EPS = 3 };

// u = gamma z (+ beta) from the saved statistics: the chain of FP32 operations of the FP8 store.
__device__ __forceinline__ float store_chain(int kind, float x, float rs, float mu, float g, float b) {
  if (kind == BSP_RMSNORM) return __fmul_rn(__fmul_rn(x, rs), g);
  return __fadd_rn(__fmul_rn(__fmul_rn(__fsub_rn(x, mu), rs), g), b);
}

// Position of u on its token's grid: n0 = floor(u / s) and the threshold of rounding up.
__device__ __forceinline__ void grid_position(float u, float s, float& n0, uint32_t& P) {
  const float t = __fdiv_rn(u, s);
  n0 = floorf(t);
  P = __float2uint_rd(__fsub_rn(t, n0) * 4294967296.0f);      // saturates at 2^32 - 1
}

constexpr int kStoreThreads = 256;
constexpr int kStoreMaxPer = 32;                               // C <= 8192

template <int DT>
__global__ void __launch_bounds__(kStoreThreads)
store_fwd_kernel(int kind, const void* __restrict__ x, int64_t T, int64_t C, const float* __restrict__ gamma,
                 const float* __restrict__ beta, const float* __restrict__ rstd, const float* __restrict__ mean,
                 float levels, PhiloxKey key, int8_t* __restrict__ codes, float* __restrict__ steps) {
  __shared__ float red[kStoreThreads / 32];
  __shared__ float s_step;
  const int64_t r = blockIdx.x;
  const float rs = __ldg(rstd + r), mu = kind == BSP_LAYERNORM ? __ldg(mean + r) : 0.f;
  // thread t holds the groups of four columns 4 (t + 256 j)
  float u[kStoreMaxPer];
  float amax = 0.f;
#pragma unroll
  for (int j = 0; j < kStoreMaxPer / 4; ++j) {
    const int64_t c = 4 * ((int64_t)threadIdx.x + kStoreThreads * j);
    if (c < C) {
      const float4 xv = load4<DT>(x, (size_t)r * C + c);
      const float4 g4 = __ldg(reinterpret_cast<const float4*>(gamma + c));
      float4 b4 = make_float4(0.f, 0.f, 0.f, 0.f);
      if (kind == BSP_LAYERNORM) b4 = __ldg(reinterpret_cast<const float4*>(beta + c));
      u[4 * j] = store_chain(kind, xv.x, rs, mu, g4.x, b4.x);
      u[4 * j + 1] = store_chain(kind, xv.y, rs, mu, g4.y, b4.y);
      u[4 * j + 2] = store_chain(kind, xv.z, rs, mu, g4.z, b4.z);
      u[4 * j + 3] = store_chain(kind, xv.w, rs, mu, g4.w, b4.w);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float a = fabsf(u[4 * j + e]);
        if (a <= 3.4028234e38f) amax = fmaxf(amax, a);           // NaN and infinities do not set the step
      }
    }
  }
  amax = warp_max(amax);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = amax;
  __syncthreads();
  if (threadIdx.x == 0) {
    float m = 0.f;
    for (int w = 0; w < kStoreThreads / 32; ++w) m = fmaxf(m, red[w]);
    const float s = m > 0.f ? __fdiv_rn(m, levels) : 1.0f;
    s_step = s;
    steps[r] = s;
  }
  __syncthreads();
  const float s = s_step;
#pragma unroll
  for (int j = 0; j < kStoreMaxPer / 4; ++j) {
    const int64_t c = 4 * ((int64_t)threadIdx.x + kStoreThreads * j);
    if (c < C) {
      const size_t i0 = (size_t)r * C + c;
      const uint4 w = philox_block(key, (uint64_t)i0 >> 2, key.c2);
      const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
      int n[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float n0;
        uint32_t P;
        grid_position(u[4 * j + e], s, n0, P);
        n[e] = (int)n0 + (ww[e] < P ? 1 : 0);
      }
      const uint32_t packed = (uint32_t)(n[0] & 0xFF) | ((uint32_t)(n[1] & 0xFF) << 8) | ((uint32_t)(n[2] & 0xFF) << 16) |
                              ((uint32_t)(n[3] & 0xFF) << 24);
      *reinterpret_cast<uint32_t*>(codes + i0) = packed;
    }
  }
}

// The copy X a weight use reads, for a 64 x 64 tile of (tokens x columns): FP32 out (row-major, may be
// NULL) and the split bf16 operand out_t[c][t] = hi, out_t[c][ld_t + t] = lo (may be NULL), padding
// columns t in [T, ld_t) zeroed.  A thread forms 16 consecutive columns of one token (four generator
// blocks, no word wasted) and writes 16 consecutive tokens of one column of each half.
template <int DT>
__global__ void __launch_bounds__(256)
store_operand_kernel(int kind, const void* __restrict__ x, int64_t T, int64_t C, const float* __restrict__ gamma,
                     const float* __restrict__ beta, const float* __restrict__ rstd, const float* __restrict__ mean,
                     const int8_t* __restrict__ codes, const float* __restrict__ steps, int read, PhiloxKey key,
                     float* __restrict__ out_f32, uint16_t* __restrict__ out_t, int64_t ld_t) {
  constexpr int TS = 64, PITCH = TS + 2;
  __shared__ __align__(16) uint16_t s_hi[TS][PITCH], s_lo[TS][PITCH];
  const int64_t r0 = (int64_t)blockIdx.y * TS, c0 = (int64_t)blockIdx.x * TS;
  const int tr = threadIdx.x >> 2, tc = (threadIdx.x & 3) * 16;
  const int64_t r = r0 + tr, c = c0 + tc;
  float v[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) v[j] = 0.f;
  if (r < T && c < C) {
    const size_t i0 = (size_t)r * C + c;
    const float rs = __ldg(rstd + r), mu = kind == BSP_LAYERNORM ? __ldg(mean + r) : 0.f;
    const float s = __ldg(steps + r);
    float xv[16];
    load16<DT>(x, i0, xv);
    const bool fresh = read == STORE_READ_N || read == STORE_READ_R_EPS;
    const bool fwd = read == STORE_READ_R || read == STORE_READ_R_EPS;
    const uint4 cq = fwd ? __ldg(reinterpret_cast<const uint4*>(codes + i0)) : make_uint4(0, 0, 0, 0);
    const uint32_t cw[4] = {cq.x, cq.y, cq.z, cq.w};
#pragma unroll
    for (int b4 = 0; b4 < 4; ++b4) {
      uint4 w = make_uint4(0, 0, 0, 0);
      if (fresh) w = philox_block(key, ((uint64_t)i0 >> 2) + b4, key.c2);
      const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int j = 4 * b4 + e;
        const float u = store_chain(kind, xv[j], rs, mu, __ldg(gamma + c + j), kind == BSP_LAYERNORM ? __ldg(beta + c + j) : 0.f);
        float nf = 0.f;
        if (fresh) {
          float n0;
          uint32_t P;
          grid_position(u, s, n0, P);
          nf = n0 + (ww[e] < P ? 1.f : 0.f);
        }
        const float nq = fwd ? (float)(int8_t)((cw[b4] >> (8 * e)) & 0xFFu) : 0.f;
        if (read == STORE_READ_U) v[j] = u;
        else if (read == STORE_READ_R) v[j] = __fmul_rn(s, nq);
        else if (read == STORE_READ_N) v[j] = __fmul_rn(s, nf);
        else v[j] = __fsub_rn(__fmul_rn(s, nq + nf), u);            // u_q + (u_f - u) = s (n + n_f) - u
      }
    }
    if (out_f32) {
#pragma unroll
      for (int j = 0; j < 16; j += 4)
        *reinterpret_cast<float4*>(out_f32 + i0 + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
    }
  }
  if (!out_t) return;
  uint32_t* dh = reinterpret_cast<uint32_t*>(&s_hi[tr][tc]);
  uint32_t* dl = reinterpret_cast<uint32_t*>(&s_lo[tr][tc]);
#pragma unroll
  for (int j = 0; j < 16; j += 2) {
    const uint32_t h0 = float_to_bf16_bits(v[j]), h1 = float_to_bf16_bits(v[j + 1]);
    const uint32_t l0 = float_to_bf16_bits(v[j] - bf16_bits_to_float(h0)), l1 = float_to_bf16_bits(v[j + 1] - bf16_bits_to_float(h1));
    dh[j >> 1] = h0 | (h1 << 16);
    dl[j >> 1] = l0 | (l1 << 16);
  }
  __syncthreads();
  const int tcol = threadIdx.x >> 2, trow = (threadIdx.x & 3) * 16;
  const int64_t cc = c0 + tcol, rr = r0 + trow;
  if (cc < C && rr < ld_t) {
    uint32_t oh[8], ol[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const bool a = rr + 2 * j < T, b = rr + 2 * j + 1 < T;
      oh[j] = (a ? (uint32_t)s_hi[trow + 2 * j][tcol] : 0u) | ((b ? (uint32_t)s_hi[trow + 2 * j + 1][tcol] : 0u) << 16);
      ol[j] = (a ? (uint32_t)s_lo[trow + 2 * j][tcol] : 0u) | ((b ? (uint32_t)s_lo[trow + 2 * j + 1][tcol] : 0u) << 16);
    }
    uint4* ph = reinterpret_cast<uint4*>(out_t + (size_t)cc * (2 * ld_t) + rr);
    uint4* pl = reinterpret_cast<uint4*>(out_t + (size_t)cc * (2 * ld_t) + ld_t + rr);
    ph[0] = make_uint4(oh[0], oh[1], oh[2], oh[3]); ph[1] = make_uint4(oh[4], oh[5], oh[6], oh[7]);
    pl[0] = make_uint4(ol[0], ol[1], ol[2], ol[3]); pl[1] = make_uint4(ol[4], ol[5], ol[6], ol[7]);
  }
}

// dY's codes (token-minor [O][ld_t]) decoded to bf16 (exact) and written twice side by side:
// out[o][t] = out[o][ld_t + t] = decode(code[o][t]), the A operand that meets [X_hi | X_lo].
template <int FMT>
__global__ void decode_twice_kernel(const uint8_t* __restrict__ codes, int64_t ld_t, size_t n, uint16_t* __restrict__ out) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const size_t o = i / ld_t, t = i % ld_t;
  const uint16_t v = (uint16_t)(__float_as_uint(f8_decode<FMT>(codes[i])) >> 16);
  out[o * 2 * ld_t + t] = v;
  out[o * 2 * ld_t + ld_t + t] = v;
}

// The A operand of the K-draw weight-use contraction: dY's codes (token-minor [O][ld_t]) decoded and
// multiplied by the token's step, rounded to bf16: out[o][t] = bf16(decode(code[o][t]) * s_t).  The
// contraction it feeds forms *differences* to the reference gradient, so this rounding costs 2^-9 of
// the difference, not of the gradient.
template <int FMT>
__global__ void __launch_bounds__(256)
store_dys_kernel(const uint8_t* __restrict__ codes, const float* __restrict__ steps, int64_t T, int64_t ld_t, size_t n8,
                 uint16_t* __restrict__ out) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n8) return;
  const size_t e0 = i * 8;
  const int64_t t0 = (int64_t)(e0 % (size_t)ld_t);
  const uint2 c8 = __ldg(reinterpret_cast<const uint2*>(codes + e0));
  float d[8];
  f8_decode4<FMT>(c8.x, *reinterpret_cast<float(*)[4]>(&d[0]));
  f8_decode4<FMT>(c8.y, *reinterpret_cast<float(*)[4]>(&d[4]));
  uint32_t pk[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int64_t ta = t0 + 2 * j, tb = ta + 1;
    const uint32_t lo = ta < T ? float_to_bf16_bits(d[2 * j] * __ldg(steps + ta)) : 0u;
    const uint32_t hi = tb < T ? float_to_bf16_bits(d[2 * j + 1] * __ldg(steps + tb)) : 0u;
    pk[j] = lo | (hi << 16);
  }
  *reinterpret_cast<uint4*>(out + e0) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
}

// K fresh roundings of the store as differences to the reference's operand, in grid steps, token-minor
// bf16: out[d][c][t] = n_f - n_q (read N: the new code minus the forward's, a small integer) or
// n_f - u / s (read U/R+eps: u_q + (u_f - u) - u_q = s (n_f - t), |.| < 1).  An element's grid position
// is found once; a draw is one generator word and one comparison.  64 x 64 tiles, 256 threads: a thread
// forms 16 consecutive columns of one token and writes 16 consecutive tokens of one column.
template <int DT>
__global__ void __launch_bounds__(256)
store_diff_draws_kernel(int kind, const void* __restrict__ x, int64_t T, int64_t C, const float* __restrict__ gamma,
                        const float* __restrict__ beta, const float* __restrict__ rstd, const float* __restrict__ mean,
                        const int8_t* __restrict__ codes, const float* __restrict__ steps, int read, PhiloxKey key,
                        int draw0, int ndraws, uint16_t* __restrict__ out_t, int64_t ld_t) {
  constexpr int TS = 64, PITCH = TS + 2;
  __shared__ __align__(16) uint16_t s_tile[2][TS][PITCH];
  const int64_t r0 = (int64_t)blockIdx.y * TS, c0 = (int64_t)blockIdx.x * TS;
  const int tr = threadIdx.x >> 2, tc = (threadIdx.x & 3) * 16;
  const int64_t r = r0 + tr, c = c0 + tc;
  const bool active = r < T && c < C;
  const size_t i0 = (size_t)r * C + c;
  float base[16];
  uint32_t thr[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) { base[j] = 0.f; thr[j] = 0u; }
  if (active) {
    const float rs = __ldg(rstd + r), mu = kind == BSP_LAYERNORM ? __ldg(mean + r) : 0.f;
    const float s = __ldg(steps + r);
    float xv[16];
    load16<DT>(x, i0, xv);
    const uint4 cq = read == STORE_READ_N ? __ldg(reinterpret_cast<const uint4*>(codes + i0)) : make_uint4(0, 0, 0, 0);
    const uint32_t cw[4] = {cq.x, cq.y, cq.z, cq.w};
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const float u = store_chain(kind, xv[j], rs, mu, __ldg(gamma + c + j), kind == BSP_LAYERNORM ? __ldg(beta + c + j) : 0.f);
      const float t = __fdiv_rn(u, s);
      const float n0 = floorf(t);
      const float f = __fsub_rn(t, n0);
      thr[j] = __float2uint_rd(f * 4294967296.0f);
      if (read == STORE_READ_N) base[j] = n0 - (float)(int8_t)((cw[j >> 2] >> (8 * (j & 3))) & 0xFFu);
      else base[j] = -f;
    }
  }
  const int tcol = threadIdx.x >> 2, trow = (threadIdx.x & 3) * 16;
  const int64_t cc = c0 + tcol, rr = r0 + trow;
  const bool wr = cc < C && rr < ld_t;
  for (int d = 0; d < ndraws; ++d) {
    const int buf = d & 1;
    uint32_t pk[8];
#pragma unroll
    for (int b4 = 0; b4 < 4; ++b4) {
      uint4 w = make_uint4(0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu);
      if (active) w = philox_block(key, ((uint64_t)i0 >> 2) + b4, (uint32_t)(draw0 + d));
      const float v0 = active ? base[4 * b4 + 0] + (w.x < thr[4 * b4 + 0] ? 1.f : 0.f) : 0.f;
      const float v1 = active ? base[4 * b4 + 1] + (w.y < thr[4 * b4 + 1] ? 1.f : 0.f) : 0.f;
      const float v2 = active ? base[4 * b4 + 2] + (w.z < thr[4 * b4 + 2] ? 1.f : 0.f) : 0.f;
      const float v3 = active ? base[4 * b4 + 3] + (w.w < thr[4 * b4 + 3] ? 1.f : 0.f) : 0.f;
      pk[2 * b4] = float_to_bf16_bits(v0) | (float_to_bf16_bits(v1) << 16);
      pk[2 * b4 + 1] = float_to_bf16_bits(v2) | (float_to_bf16_bits(v3) << 16);
    }
    uint32_t* dst = reinterpret_cast<uint32_t*>(&s_tile[buf][tr][tc]);
#pragma unroll
    for (int j = 0; j < 8; ++j) dst[j] = pk[j];
    __syncthreads();
    if (wr) {
      uint32_t o[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint32_t lo = rr + 2 * j < T ? s_tile[buf][trow + 2 * j][tcol] : 0u;
        const uint32_t hi = rr + 2 * j + 1 < T ? s_tile[buf][trow + 2 * j + 1][tcol] : 0u;
        o[j] = lo | (hi << 16);
      }
      uint4* dstg = reinterpret_cast<uint4*>(out_t + ((size_t)d * C + cc) * ld_t + rr);
      dstg[0] = make_uint4(o[0], o[1], o[2], o[3]);
      dstg[1] = make_uint4(o[4], o[5], o[6], o[7]);
    }
  }
}

static bool valid_enum(int v, int hi) { return v >= 0 && v <= hi; }

static int store_levels(int bits) { return (1 << (bits - 1)) - 1; }

struct StoreBuffers {
  float *rstd, *mean, *amax_u, *steps, *amax_dy, *scale_dy;
  int8_t* codes;
  uint8_t *dy_codes, *dy_codes_t;
  uint16_t *dy_twice, *x_split, *dys_t, *diff_t;
  int chunk;
  void* du;
  float *dg_ref, *db_ref, *dg_pol, *S1g, *S2g, *dx, *zero_c;
  float *dW_ref, *dW_pol, *S1w, *S2w;
  void *ws_bwd, *ws_gain, *ws_dgrad, *ws_stats;
  size_t b_bwd, b_gain, b_dgrad, b_stats;
  int64_t ld_t;
};

static size_t store_carve(const bsp_store_desc_t* op, int K, char* base, StoreBuffers* out) {
  size_t off = 0;
  auto take = [&](size_t bytes) -> void* {
    void* p = base ? base + off : nullptr;
    off += round_up(bytes ? bytes : 1, 256);
    return p;
  };
  const size_t T = (size_t)op->T, C = (size_t)op->C, O = (size_t)op->O, ld_t = round_up(T, 16);
  const size_t eb = op->dtype == BSP_BF16 ? 2 : 4;
  StoreBuffers c;
  memset(&c, 0, sizeof(c));
  c.ld_t = (int64_t)ld_t;
  c.rstd = (float*)take(T * 4); c.mean = (float*)take(T * 4); c.amax_u = (float*)take(4); c.steps = (float*)take(T * 4);
  c.amax_dy = (float*)take(4); c.scale_dy = (float*)take(4);
  c.codes = (int8_t*)take(T * C);
  c.dy_codes = (uint8_t*)take(T * O); c.dy_codes_t = (uint8_t*)take(O * ld_t);
  c.dy_twice = (uint16_t*)take(O * 2 * ld_t * 2); c.x_split = (uint16_t*)take(C * 2 * ld_t * 2);
  // the K-draw contraction: dY o s once, and the difference operands of as many draws as fit 1 GiB
  {
    const size_t per = C * ld_t * 2;
    size_t fit = ((size_t)1 << 30) / (per ? per : 1);
    if (fit < 1) fit = 1;
    const size_t k = K > 0 ? (size_t)K : 1;
    if (fit >= k) c.chunk = (int)k;
    else { const size_t nch = (k + fit - 1) / fit; c.chunk = (int)((k + nch - 1) / nch); }
    c.dys_t = (uint16_t*)take(O * ld_t * 2);
    c.diff_t = (uint16_t*)take((size_t)c.chunk * per);
  }
  c.du = take(T * C * eb);
  c.dg_ref = (float*)take(C * 4); c.db_ref = (float*)take(C * 4); c.dg_pol = (float*)take(C * 4);
  c.S1g = (float*)take(C * 4); c.S2g = (float*)take(C * 4); c.zero_c = (float*)take(C * 4);
  c.dx = (float*)take(T * C * 4);
  c.dW_ref = (float*)take(O * C * 4); c.dW_pol = (float*)take(O * C * 4);
  c.S1w = (float*)take(O * C * 4); c.S2w = (float*)take(O * C * 4);
  c.b_bwd = bsp_norm_bwd_workspace_bytes(op->T, op->C);
  c.b_gain = norm_gain_mc_workspace(op->T, op->C, K > 0 ? K : 1, false);
  c.b_dgrad = bsp_linear_dgrad_workspace_bytes(op->T, op->O, op->C);
  c.b_stats = kMaxPendingStats * kStatSlotBytes;
  c.ws_bwd = take(c.b_bwd); c.ws_gain = take(c.b_gain); c.ws_dgrad = take(c.b_dgrad); c.ws_stats = take(c.b_stats);
  if (out) *out = c;
  return off;
}

}  // namespace bsp

using namespace bsp;

extern "C" {

int bsp_store_fwd(int kind, const void* x, int dt, int64_t T, int64_t C, const float* gamma, const float* beta,
                  const float* rstd, const float* mean, int bits, bsp_key_t key, int8_t* codes, float* steps,
                  void* stream) {
  if (!valid_enum(kind, 1) || !valid_enum(dt, 1) || bits < 2 || bits > 7 || T < 0 || C <= 0) return BSP_ERR_ARG;
  if (key.tensor_id >= (1u << 24) || key.stream > 255u || key.reserved != 0) return BSP_ERR_ARG;
  if (T == 0) return BSP_OK;
  if (!x || !gamma || !rstd || !codes || !steps || (kind == BSP_LAYERNORM && (!beta || !mean))) return BSP_ERR_ARG;
  if (C % 4 != 0 || C > 4 * kStoreThreads * (kStoreMaxPer / 4)) return BSP_ERR_UNSUPPORTED;
  if (!aligned16(x) || !aligned16(gamma) || !aligned16(beta) || (reinterpret_cast<uintptr_t>(codes) & 3u)) return BSP_ERR_ALIGN;
  const PhiloxKey pk = make_key(key);
  cudaStream_t st = (cudaStream_t)stream;
  if (dt == BSP_F32)
    store_fwd_kernel<BSP_F32><<<(unsigned)T, kStoreThreads, 0, st>>>(kind, x, T, C, gamma, beta, rstd, mean, (float)store_levels(bits), pk, codes, steps);
  else
    store_fwd_kernel<BSP_BF16><<<(unsigned)T, kStoreThreads, 0, st>>>(kind, x, T, C, gamma, beta, rstd, mean, (float)store_levels(bits), pk, codes, steps);
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

int bsp_store_read(int kind, const void* x, int dt, int64_t T, int64_t C, const float* gamma, const float* beta,
                   const float* rstd, const float* mean, const int8_t* codes, const float* steps, int read,
                   bsp_key_t key, float* copy_f32, void* copy_split_t, int64_t ld_t, void* stream) {
  if (!valid_enum(kind, 1) || !valid_enum(dt, 1) || !valid_enum(read, 3) || T < 0 || C <= 0) return BSP_ERR_ARG;
  if (key.tensor_id >= (1u << 24) || key.stream > 255u || key.reserved != 0) return BSP_ERR_ARG;
  if (T == 0 || (!copy_f32 && !copy_split_t)) return BSP_OK;
  if (!x || !gamma || !rstd || !steps || (kind == BSP_LAYERNORM && (!beta || !mean))) return BSP_ERR_ARG;
  if ((read == STORE_READ_R || read == STORE_READ_R_EPS) && !codes) return BSP_ERR_ARG;
  if (copy_split_t && (ld_t < T || ld_t % 16 != 0)) return BSP_ERR_ALIGN;
  if (C % 16 != 0) return BSP_ERR_UNSUPPORTED;
  if (!aligned16(x) || !aligned16(codes) || !aligned16(copy_f32) || !aligned16(copy_split_t)) return BSP_ERR_ALIGN;
  const PhiloxKey pk = make_key(key);
  cudaStream_t st = (cudaStream_t)stream;
  const int64_t rows = copy_split_t ? ld_t : T;                 // the padding columns are written too
  dim3 grid((unsigned)((C + 63) / 64), (unsigned)((rows + 63) / 64));
  if (dt == BSP_F32)
    store_operand_kernel<BSP_F32><<<grid, 256, 0, st>>>(kind, x, T, C, gamma, beta, rstd, mean, codes, steps, read, pk, copy_f32,
                                                        reinterpret_cast<uint16_t*>(copy_split_t), ld_t);
  else
    store_operand_kernel<BSP_BF16><<<grid, 256, 0, st>>>(kind, x, T, C, gamma, beta, rstd, mean, codes, steps, read, pk, copy_f32,
                                                         reinterpret_cast<uint16_t*>(copy_split_t), ld_t);
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

size_t bsp_store_wgrad_workspace_bytes(int64_t T, int64_t O) {
  if (T <= 0 || O <= 0) return 0;
  return round_up((size_t)O * 2 * round_up((size_t)T, 16) * 2, 256);
}

int bsp_store_wgrad(int64_t T, int64_t O, int64_t C, const uint8_t* dy_codes_t, bsp_quant_t q_dy, const void* copy_split_t,
                    int64_t ld_t, float* dW, void* ws, size_t ws_bytes, bsp_diag_t* diag, void* stream) {
  if (T <= 0 || O <= 0 || C <= 0 || !valid_enum(q_dy.fmt, 1)) return BSP_ERR_ARG;
  if (!dy_codes_t || !copy_split_t || !dW) return BSP_ERR_ARG;
  if (ld_t < T || ld_t % 16 != 0 || C % 4 != 0) return BSP_ERR_ALIGN;
  if (!ws || ws_bytes < bsp_store_wgrad_workspace_bytes(T, O) || (reinterpret_cast<uintptr_t>(ws) & 255u)) return BSP_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  uint16_t* a2 = reinterpret_cast<uint16_t*>(ws);
  const size_t n = (size_t)O * ld_t;
  if (q_dy.fmt == BSP_E5M2) decode_twice_kernel<BSP_E5M2><<<(unsigned)((n + 255) / 256), 256, 0, st>>>(dy_codes_t, ld_t, n, a2);
  else decode_twice_kernel<BSP_E4M3><<<(unsigned)((n + 255) / 256), 256, 0, st>>>(dy_codes_t, ld_t, n, a2);
  BSP_LAUNCH_CHECK();
  GemmArgs g;
  g.M = O; g.N = C; g.K = 2 * ld_t; g.nb = 1; g.fp8 = false; g.a_fmt = 0; g.b_fmt = 0;
  g.A = a2; g.B = copy_split_t; g.lda = 2 * ld_t; g.ldb = 2 * ld_t; g.b_batch_stride = (int64_t)C * 2 * ld_t;
  g.sa = q_dy.scale; g.sa_dev = q_dy.scale_dev; g.sb = 1.0f; g.sb_dev = nullptr;
  g.mode = EPI_STORE_F32; g.C = dW; g.ldc = C; g.diag = diag;
  return gemm_run(g, st);
}

size_t bsp_mc_check_store_workspace_bytes(const bsp_store_desc_t* op, int K) {
  if (!op || op->T <= 0 || op->C <= 0 || op->O <= 0) return 0;
  return store_carve(op, K, nullptr, nullptr);
}

#define BSP_TRY(expr)              \
  do {                             \
    int _rc = (expr);              \
    if (_rc != BSP_OK) return _rc; \
  } while (0)

int bsp_mc_check_store(const bsp_store_desc_t* op, int K, const bsp_verdict_rule_t* rule, bsp_use_result_t* results,
                       int* n_results, void* ws, size_t ws_bytes, bsp_diag_t* diag, void* stream) {
  if (!op || !results || !n_results || !rule_valid(rule)) return BSP_ERR_ARG;
  if (op->T <= 0 || op->C <= 0 || op->O <= 0 || K < 4 || op->bits < 2 || op->bits > 7) return BSP_ERR_ARG;
  if (!op->x || !op->gamma || !op->W || !op->dY || (op->norm_kind == BSP_LAYERNORM && !op->beta)) return BSP_ERR_ARG;
  if (!valid_enum(op->norm_kind, 1) || !valid_enum(op->dtype, 1) || !valid_enum(op->grad_fmt, 1)) return BSP_ERR_ARG;
  if (op->C % 16 != 0 || op->O % 16 != 0 || op->C > 8192) return BSP_ERR_UNSUPPORTED;
  if (!ws || ws_bytes < bsp_mc_check_store_workspace_bytes(op, K) || (reinterpret_cast<uintptr_t>(ws) & 255u))
    return BSP_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  StoreBuffers b;
  store_carve(op, K, reinterpret_cast<char*>(ws), &b);
  const int64_t T = op->T, C = op->C, O = op->O;
  const int dt = op->dtype, kind = op->norm_kind;
  *n_results = 0;

  // ---- once per call: statistics, the b-bit store (stream 0), the incoming gradient, du
  BSP_TRY(bsp_norm_stats(kind, op->x, dt, T, C, op->gamma, op->beta, op->eps, b.rstd, b.mean, b.amax_u, diag, st));
  bsp_key_t key;
  key.seed = op->seed; key.tensor_id = op->tensor_id; key.stream = BSP_STREAM_FORWARD; key.draw = 0; key.reserved = 0;
  BSP_TRY(bsp_store_fwd(kind, op->x, dt, T, C, op->gamma, op->beta, b.rstd, b.mean, op->bits, key, b.codes, b.steps, st));
  BSP_TRY(bsp_amax(op->dY, dt, 1, (size_t)T * O, b.amax_dy, diag, st));
  BSP_TRY(bsp_scale_from_amax(b.amax_dy, 1, op->grad_fmt, b.scale_dy, st));
  bsp_quant_t qdy;
  qdy.fmt = op->grad_fmt; qdy.mode = BSP_ROUND_NEAREST; qdy.scale = 1.f; qdy.scale_dev = b.scale_dy;
  bsp_key_t nokey;
  memset(&nokey, 0, sizeof(nokey));
  BSP_TRY(bsp_round_2d(op->dY, dt, T, O, qdy, nokey, b.dy_codes, b.dy_codes_t, b.ld_t, diag, st));
  BSP_TRY(bsp_linear_dgrad(T, O, C, b.dy_codes, qdy, op->W, dt, b.du, dt, b.ws_dgrad, b.b_dgrad, diag, st));

  PendingStats pend;
  pend.slots = reinterpret_cast<double*>(b.ws_stats);
  pend.st = st;
  pend.rule = rule;
  int nres = 0;
  auto emit = [&](int use, int out, int pol) -> bsp_use_result_t* {
    bsp_use_result_t* r = &results[nres++];
    memset(r, 0, sizeof(*r));
    r->use_id = use; r->output_id = out; r->policy = pol;
    return r;
  };
  bsp_quant_t qnone;                                             // the FP8 fields are unused under the grid law
  qnone.fmt = BSP_E4M3; qnone.mode = BSP_ROUND_STOCHASTIC; qnone.scale = 1.f; qnone.scale_dev = nullptr;

  // ---- gain use (reference: the original z)
  const uint32_t gain_mask = op->policy_mask & 7u;
  if (gain_mask) {
    BSP_TRY(bsp_norm_bwd(kind, op->x, dt, T, C, op->gamma, op->beta, b.rstd, b.mean, b.du, dt, BSP_READ_ORIGINAL,
                         BSP_READ_ORIGINAL, nullptr, qnone, key, b.dg_ref, b.db_ref, b.dx, b.ws_bwd, b.b_bwd, diag, st));
    if (gain_mask & 1u) BSP_TRY(pend.add(b.dg_ref, b.dg_ref, nullptr, C, 1, 0, emit(BSP_STREAM_GAIN, BSP_OUT_DGAMMA, BSP_READ_ORIGINAL)));
    if (gain_mask & 2u) {
      // u_q / gamma: the forward's own rounding, regenerated from its key (stream 0, draw 0): one "draw"
      // whose gradient lands in S1 against a zero reference
      BSP_CHECK_CUDA(cudaMemsetAsync(b.zero_c, 0, C * sizeof(float), st));
      BSP_CHECK_CUDA(cudaMemsetAsync(b.dg_pol, 0, C * sizeof(float), st));
      BSP_CHECK_CUDA(cudaMemsetAsync(b.S2g, 0, C * sizeof(float), st));
      BSP_TRY(norm_gain_mc_run(false, kind, op->x, dt, T, C, op->gamma, op->beta, b.rstd, b.mean, b.du, dt, qnone, key, 0, 1,
                               b.zero_c, b.dg_pol, b.S2g, b.ws_gain, b.b_gain, diag, st, b.steps));
      BSP_TRY(pend.add(b.dg_ref, b.dg_pol, nullptr, C, 1, 0, emit(BSP_STREAM_GAIN, BSP_OUT_DGAMMA, BSP_READ_FORWARD)));
    }
    if (gain_mask & 4u) {
      BSP_CHECK_CUDA(cudaMemsetAsync(b.S1g, 0, C * sizeof(float), st));
      BSP_CHECK_CUDA(cudaMemsetAsync(b.S2g, 0, C * sizeof(float), st));
      bsp_key_t gk = key;
      gk.stream = BSP_STREAM_GAIN;
      BSP_TRY(norm_gain_mc_run(false, kind, op->x, dt, T, C, op->gamma, op->beta, b.rstd, b.mean, b.du, dt, qnone, gk, 0, K,
                               b.dg_ref, b.S1g, b.S2g, b.ws_gain, b.b_gain, diag, st, b.steps));
      BSP_TRY(pend.add(b.dg_ref, b.S1g, b.S2g, C, K, 1, emit(BSP_STREAM_GAIN, BSP_OUT_DGAMMA, BSP_READ_FRESH)));
    }
  }

  // ---- weight use (reference: the rounded value the layer multiplied)
  const uint32_t w_mask = (op->policy_mask >> 3) & 15u;
  if (w_mask) {
    const size_t b_tw = bsp_store_wgrad_workspace_bytes(T, O);
    auto wgrad = [&](int read, int draw, float* out) -> int {
      bsp_key_t wk = key;
      wk.stream = BSP_STREAM_WGRAD; wk.draw = (uint32_t)draw;
      BSP_TRY(bsp_store_read(kind, op->x, dt, T, C, op->gamma, op->beta, b.rstd, b.mean, b.codes, b.steps, read, wk, nullptr,
                             b.x_split, b.ld_t, st));
      return bsp_store_wgrad(T, O, C, b.dy_codes_t, qdy, b.x_split, b.ld_t, out, b.dy_twice, b_tw, diag, st);
    };
    BSP_TRY(wgrad(STORE_READ_R, 0, b.dW_ref));
    if (w_mask & 1u) {
      BSP_TRY(wgrad(STORE_READ_U, 0, b.dW_pol));
      BSP_TRY(pend.add(b.dW_ref, b.dW_pol, nullptr, O * C, 1, 0, emit(BSP_STREAM_WGRAD, BSP_OUT_DW, BSP_READ_ORIGINAL)));
      // (the statistics pass above reads dW_pol before the draws below overwrite it: same stream)
    }
    if (w_mask & 2u) BSP_TRY(pend.add(b.dW_ref, b.dW_ref, nullptr, O * C, 1, 0, emit(BSP_STREAM_WGRAD, BSP_OUT_DW, BSP_READ_FORWARD)));
    if (w_mask & 12u) {
      const size_t n8 = (size_t)O * b.ld_t / 8;
      if (op->grad_fmt == BSP_E5M2)
        store_dys_kernel<BSP_E5M2><<<(unsigned)((n8 + 255) / 256), 256, 0, st>>>(b.dy_codes_t, b.steps, T, b.ld_t, n8, b.dys_t);
      else
        store_dys_kernel<BSP_E4M3><<<(unsigned)((n8 + 255) / 256), 256, 0, st>>>(b.dy_codes_t, b.steps, T, b.ld_t, n8, b.dys_t);
      BSP_LAUNCH_CHECK();
    }
    for (int which = 0; which < 2; ++which) {
      if (!((w_mask >> (2 + which)) & 1u)) continue;
      // Both fresh reads differ from the reference's operand u_q = s n_q by a multiple of the token's
      // step: s (n_f - n_q) under N, s (n_f - u / s) under U/R+eps.  So the K draws are one contraction
      // of (dY o s) with the K difference matrices, whose products are g_k - g* themselves: the shifted
      // sums take them as they come, no per-draw gradient is written, and the bf16 rounding of an
      // operand costs 2^-9 of the difference.
      const int read = which == 0 ? STORE_READ_N : STORE_READ_R_EPS;
      BSP_CHECK_CUDA(cudaMemsetAsync(b.S1w, 0, (size_t)O * C * sizeof(float), st));
      BSP_CHECK_CUDA(cudaMemsetAsync(b.S2w, 0, (size_t)O * C * sizeof(float), st));
      bsp_key_t wk = key;
      wk.stream = BSP_STREAM_WGRAD; wk.draw = 0;
      const PhiloxKey pk = make_key(wk);
      for (int k0 = 0; k0 < K; k0 += b.chunk) {
        const int nd = (K - k0) < b.chunk ? (K - k0) : b.chunk;
        dim3 grid((unsigned)((C + 63) / 64), (unsigned)((b.ld_t + 63) / 64));
        if (dt == BSP_F32)
          store_diff_draws_kernel<BSP_F32><<<grid, 256, 0, st>>>(kind, op->x, T, C, op->gamma, op->beta, b.rstd, b.mean, b.codes,
                                                                 b.steps, read, pk, k0, nd, b.diff_t, b.ld_t);
        else
          store_diff_draws_kernel<BSP_BF16><<<grid, 256, 0, st>>>(kind, op->x, T, C, op->gamma, op->beta, b.rstd, b.mean, b.codes,
                                                                  b.steps, read, pk, k0, nd, b.diff_t, b.ld_t);
        BSP_LAUNCH_CHECK();
        GemmArgs g;
        g.M = O; g.N = C; g.K = T; g.nb = nd; g.fp8 = false;
        g.A = b.dys_t; g.B = b.diff_t; g.lda = b.ld_t; g.ldb = b.ld_t; g.b_batch_stride = (int64_t)C * b.ld_t;
        g.sa = 1.f; g.sa_dev = b.scale_dy; g.sb = 1.f; g.sb_dev = nullptr;
        g.mode = EPI_MC; g.ldc = C; g.ref = nullptr; g.S1 = b.S1w; g.S2 = b.S2w; g.diag = diag;
        BSP_TRY(gemm_run(g, st));
      }
      BSP_TRY(pend.add(b.dW_ref, b.S1w, b.S2w, O * C, K, 1,
                       emit(BSP_STREAM_WGRAD, BSP_OUT_DW, which == 0 ? BSP_READ_FRESH : BSP_READ_FORWARD_PLUS_FRESH_ERROR)));
      // the two fresh reads share S1w / S2w: the first one's statistics pass is queued before the
      // second one clears them (same stream)
    }
  }
  *n_results = nres;
  return pend.flush();
}

}  // extern "C"
