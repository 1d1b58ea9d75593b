// Streamed normalisation backward: the arithmetic of norm_bwd_kernel, fed by a ring of bulk copies.
//
// Each block owns a contiguous range of rows and walks it in stages of kRS rows.  One elected
// thread keeps a ring of stages in flight with untiled bulk copies (x, du and, for the R read, the
// codes) that complete on an mbarrier, so tens of KB per SM are outstanding however long the
// per-row arithmetic takes.  A thread owns two groups of four columns, 4*(tid + NT*j): the column
// sums for dgamma / dbeta live in registers across the block's rows, z and gamma*du of a stage stay
// in registers across the one block barrier that publishes the stage's row sums, and dx is written
// with full 16-byte lines per lane.  The pass has about a dozen instructions per element to spend
// at HBM speed, so: the shape is restricted to whole stages and fully used blocks (no per-element
// predicates; other shapes take the plain kernel), the row sums of a stage are reduced together
// (several values per shuffle round), and the norm kind is a template parameter.
#pragma once

#include "tc.cuh"

namespace bsp {

constexpr int kRS = 2;    // rows per stage
constexpr int kNJ = 2;    // column groups per thread

// Four consecutive elements at column c of a staged row.
template <int DT>
__device__ __forceinline__ void lds4(const unsigned char* row, int c, float (&v)[4]) {
  if (DT == BSP_F32) {
    const float4 a = *reinterpret_cast<const float4*>(row + (size_t)c * 4);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
  } else {
    const uint2 a = *reinterpret_cast<const uint2*>(row + (size_t)c * 2);
    v[0] = __uint_as_float(a.x << 16); v[1] = __uint_as_float(a.x & 0xFFFF0000u);
    v[2] = __uint_as_float(a.y << 16); v[3] = __uint_as_float(a.y & 0xFFFF0000u);
  }
}

// Sums NV per-lane values over the warp in log2(32) rounds, halving the number of values carried
// while more than one is left.  Returns the total of value (lane / (32 / NV)); all lanes of that
// group of 32 / NV lanes hold it.
template <int NV>
__device__ __forceinline__ float warp_sum_packed(const float (&v)[NV], int lane) {
  static_assert(NV == 1 || NV == 2 || NV == 4, "one, two or four values");
  float r;
  if constexpr (NV == 4) {
    const bool hi = lane & 16;
    const float a0 = (hi ? v[2] : v[0]) + __shfl_xor_sync(0xFFFFFFFFu, hi ? v[0] : v[2], 16);
    const float a1 = (hi ? v[3] : v[1]) + __shfl_xor_sync(0xFFFFFFFFu, hi ? v[1] : v[3], 16);
    const bool h8 = lane & 8;
    r = (h8 ? a1 : a0) + __shfl_xor_sync(0xFFFFFFFFu, h8 ? a0 : a1, 8);
  } else if constexpr (NV == 2) {
    const bool hi = lane & 16;
    r = (hi ? v[1] : v[0]) + __shfl_xor_sync(0xFFFFFFFFu, hi ? v[0] : v[1], 16);
    r += __shfl_xor_sync(0xFFFFFFFFu, r, 8);
  } else {
    r = v[0] + __shfl_xor_sync(0xFFFFFFFFu, v[0], 16);
    r += __shfl_xor_sync(0xFFFFFFFFu, r, 8);
  }
  r += __shfl_xor_sync(0xFFFFFFFFu, r, 4);
  r += __shfl_xor_sync(0xFFFFFFFFu, r, 2);
  r += __shfl_xor_sync(0xFFFFFFFFu, r, 1);
  return r;
}

// Requires C == 8 * blockDim.x, T and rows_per_block multiples of kRS (see plan_stream).
template <int DT, int DU_DT, int FMT, int KIND>
__global__ void __launch_bounds__(512, 1)
norm_bwd_stream_kernel(const void* __restrict__ x, int64_t T, int64_t C, int64_t rows_per_block, int nstages_ring,
                       const float* __restrict__ gamma, const float* __restrict__ beta,
                       const float* __restrict__ rstd, const float* __restrict__ mean,
                       const void* __restrict__ du, int gain_read, const uint8_t* __restrict__ u_codes,
                       float scale_val, const float* __restrict__ scale_dev, PhiloxKey key,
                       float* __restrict__ part_g, float* __restrict__ part_b, float* __restrict__ dx,
                       bsp_diag_t* diag) {
  extern __shared__ __align__(128) unsigned char smem[];
  constexpr int ESX = DT == BSP_F32 ? 4 : 2, ESD = DU_DT == BSP_F32 ? 4 : 2;
  constexpr bool LN = KIND == BSP_LAYERNORM;
  constexpr int NV = LN ? 2 * kRS : kRS;          // row sums per stage: sum(dz*z), and sum(dz) for LayerNorm
  constexpr int GL = 32 / NV;                     // lanes that end up holding one of them
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, NT = blockDim.x, nwarp = NT >> 5;
  const int NS = nstages_ring;
  const bool use_codes = gain_read == BSP_READ_FORWARD;
  const size_t xrow = (size_t)C * ESX, drow = (size_t)C * ESD, crow = use_codes ? (size_t)C : 0;
  const size_t d_off = kRS * xrow, c_off = d_off + kRS * drow;
  const size_t stage_bytes = (c_off + kRS * crow + 127) / 128 * 128;
  unsigned char* tail = smem + (size_t)NS * stage_bytes;
  const uint32_t bar0 = smem_u32(tail);                                       // full[NS], 8 bytes each
  float* red = reinterpret_cast<float*>(tail + 8 * 8);                        // [2][4][16]
  volatile int* abort_flag = reinterpret_cast<volatile int*>(red + 2 * 4 * 16);

  const float scale = scale_dev ? __ldg(scale_dev) : scale_val;
  const float inv_scale = __fdiv_rn(1.0f, scale);
  const float invC = 1.0f / (float)C;
  int col[kNJ];
#pragma unroll
  for (int j = 0; j < kNJ; ++j) col[j] = 4 * (tid + NT * j);

  const int64_t r0 = (int64_t)blockIdx.x * rows_per_block;
  const int64_t r1 = r0 + rows_per_block < T ? r0 + rows_per_block : T;
  const int nst = r1 > r0 ? (int)((r1 - r0) / kRS) : 0;

  auto issue = [&](int i) {                                                   // thread 0 only
    const int s = i % NS;
    const int64_t rb = r0 + (int64_t)i * kRS;
    const uint32_t bar = bar0 + 8 * s;
    const uint32_t dst = smem_u32(smem + (size_t)s * stage_bytes);
    mbar_expect_tx(bar, (uint32_t)(kRS * (xrow + drow + crow)));
    bulk_load_1d(dst, reinterpret_cast<const unsigned char*>(x) + (size_t)rb * xrow, (uint32_t)(kRS * xrow), bar);
    bulk_load_1d(dst + (uint32_t)d_off, reinterpret_cast<const unsigned char*>(du) + (size_t)rb * drow,
                 (uint32_t)(kRS * drow), bar);
    if (use_codes) bulk_load_1d(dst + (uint32_t)c_off, u_codes + (size_t)rb * C, (uint32_t)(kRS * crow), bar);
  };

  if (tid == 0) {
    for (int s = 0; s < NS; ++s) mbar_init(bar0 + 8 * s, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    for (int i = 0; i < NS && i < nst; ++i) issue(i);
  }
  __syncthreads();

  float g[kNJ][4], b[kNJ][4], rg[kNJ][4], accg[kNJ][4], accb[kNJ][4];
#pragma unroll
  for (int j = 0; j < kNJ; ++j) {
    const float4 a = __ldg(reinterpret_cast<const float4*>(gamma + col[j]));
    g[j][0] = a.x; g[j][1] = a.y; g[j][2] = a.z; g[j][3] = a.w;
#pragma unroll
    for (int e = 0; e < 4; ++e) { b[j][e] = 0.f; accg[j][e] = 0.f; accb[j][e] = 0.f; }
    if (LN) {
      const float4 bb = __ldg(reinterpret_cast<const float4*>(beta + col[j]));
      b[j][0] = bb.x; b[j][1] = bb.y; b[j][2] = bb.z; b[j][3] = bb.w;
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) rg[j][e] = __fdiv_rn(1.0f, g[j][e]);
  }

  float rs_n[kRS], mu_n[kRS];
  auto fetch_stats = [&](int i) {
#pragma unroll
    for (int rr = 0; rr < kRS; ++rr) {
      const int64_t r = r0 + (int64_t)i * kRS + rr;
      rs_n[rr] = __ldg(rstd + r);
      mu_n[rr] = LN ? __ldg(mean + r) : 0.f;
    }
  };
  if (nst > 0) fetch_stats(0);

  bool failed = false;
  for (int i = 0; i < nst; ++i) {
    const int s = i % NS;
    const uint32_t par = (uint32_t)(i / NS) & 1u;
    const int64_t rb = r0 + (int64_t)i * kRS;
    float rs[kRS], mu[kRS];
#pragma unroll
    for (int rr = 0; rr < kRS; ++rr) { rs[rr] = rs_n[rr]; mu[rr] = mu_n[rr]; }
    if (i + 1 < nst) fetch_stats(i + 1);
    const unsigned char* st = smem + (size_t)s * stage_bytes;
    // after a failed wait the stage's contents are arbitrary; the results are discarded below
    const bool ok = mbar_wait_suspend(bar0 + 8 * s, par, abort_flag);

    // ---- column sums and the stage's row sums; z and gamma*du stay in registers for dx
    float z[kRS][kNJ][4], dz[kRS][kNJ][4], p[NV];
#pragma unroll
    for (int q = 0; q < NV; ++q) p[q] = 0.f;
#pragma unroll
    for (int rr = 0; rr < kRS; ++rr) {
#pragma unroll
      for (int j = 0; j < kNJ; ++j) {
        float xv[4], dv[4];
        lds4<DT>(st + rr * xrow, col[j], xv);
        lds4<DU_DT>(st + d_off + rr * drow, col[j], dv);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          z[rr][j][e] = LN ? __fmul_rn(__fsub_rn(xv[e], mu[rr]), rs[rr]) : __fmul_rn(xv[e], rs[rr]);
          dz[rr][j][e] = g[j][e] * dv[e];
          p[rr] = fmaf(dz[rr][j][e], z[rr][j][e], p[rr]);
          if (LN) p[NV - kRS + rr] += dz[rr][j][e];
        }
        if (gain_read == BSP_READ_ORIGINAL) {
#pragma unroll
          for (int e = 0; e < 4; ++e) accg[j][e] = fmaf(z[rr][j][e], dv[e], accg[j][e]);
        } else {
          float dec[4];
          if (gain_read == BSP_READ_FORWARD) {
            f8_decode4<FMT>(*reinterpret_cast<const uint32_t*>(st + c_off + rr * crow + col[j]), dec);
          } else {
            const uint64_t i0 = (uint64_t)(rb + rr) * (uint64_t)C + (uint64_t)col[j];
            const uint4 w = philox_block(key, i0 >> 2, key.c2);
            const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              float uu = __fmul_rn(z[rr][j][e], g[j][e]);
              if (LN) uu = __fadd_rn(uu, b[j][e]);
              dec[e] = f8_sr_value<FMT>(__fmul_rn(uu, scale), ww[e]);
            }
          }
          // (copy - beta) / gamma as a multiplication by the per-column reciprocal
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float zg = (dec[e] * inv_scale - b[j][e]) * rg[j][e];
            accg[j][e] = fmaf(zg, dv[e], accg[j][e]);
          }
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) accb[j][e] += dv[e];
      }
    }
    const int buf = i & 1;
    if (dx) {
      const float r = warp_sum_packed<NV>(p, lane);
      if ((lane & (GL - 1)) == 0) red[(buf * 4 + lane / GL) * 16 + warp] = r;
    }
    // one barrier per stage: publishes the row sums, agrees on failure, and tells thread 0 that
    // the stage read one iteration ago is no longer in use
    if (!__syncthreads_and(ok ? 1 : 0)) { failed = true; break; }
    if (tid == 0 && i >= 1 && i - 1 + NS < nst) issue(i - 1 + NS);

    if (dx) {
      // every warp sums the per-warp partials of all NV values: lane group q takes value q
      const int q = lane / GL, jl = lane & (GL - 1);
      float t = 0.f;
      for (int w = jl; w < nwarp; w += GL) t += red[(buf * 4 + q) * 16 + w];
#pragma unroll
      for (int o = GL / 2; o > 0; o >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, o);
      float tot[NV];
#pragma unroll
      for (int v = 0; v < NV; ++v) tot[v] = __shfl_sync(0xFFFFFFFFu, t, v * GL);
#pragma unroll
      for (int rr = 0; rr < kRS; ++rr) {
        const float m1 = tot[rr] * invC;
        const float m2 = LN ? tot[NV - kRS + rr] * invC : 0.f;
#pragma unroll
        for (int j = 0; j < kNJ; ++j) {
          float o[4];
#pragma unroll
          for (int e = 0; e < 4; ++e)
            o[e] = rs[rr] * (LN ? (dz[rr][j][e] - m2) - z[rr][j][e] * m1 : dz[rr][j][e] - z[rr][j][e] * m1);
          __stcs(reinterpret_cast<float4*>(dx + (size_t)(rb + rr) * C + col[j]), make_float4(o[0], o[1], o[2], o[3]));
        }
      }
    }
  }
  if (failed) {
    // a bounded wait ran out: the status says so, and the block's column partials are written as NaN
    // so that dgamma / dbeta come out recognisably invalid instead of being summed from whatever the
    // workspace held before
    if (tid == 0 && diag) atomicMax(&diag->status, (int)BSP_ERR_TIMEOUT);
    const float4 bad = make_float4(NAN, NAN, NAN, NAN);
#pragma unroll
    for (int j = 0; j < kNJ; ++j) {
      *reinterpret_cast<float4*>(part_g + (size_t)blockIdx.x * C + col[j]) = bad;
      if (part_b) *reinterpret_cast<float4*>(part_b + (size_t)blockIdx.x * C + col[j]) = bad;
    }
    return;
  }
#pragma unroll
  for (int j = 0; j < kNJ; ++j) {
    *reinterpret_cast<float4*>(part_g + (size_t)blockIdx.x * C + col[j]) =
        make_float4(accg[j][0], accg[j][1], accg[j][2], accg[j][3]);
    if (part_b)
      *reinterpret_cast<float4*>(part_b + (size_t)blockIdx.x * C + col[j]) =
          make_float4(accb[j][0], accb[j][1], accb[j][2], accb[j][3]);
  }
}

// The streamed kernel's launch shape.  ok == false (the plain kernel runs instead) unless rows are
// whole multiples of 256 columns and at most 4096 wide, T is a multiple of the stage height, and
// the addresses meet the bulk copy's 16-byte rule.
struct StreamPlan {
  bool ok;
  int threads, ring, grid;
  int64_t rows_per_block;
  size_t smem;
};

static inline StreamPlan plan_stream(int64_t T, int64_t C, int dt, int du_dt, int gain_read, const void* x,
                                     const void* du, const uint8_t* u_codes) {
  StreamPlan p{};
  const bool codes = gain_read == BSP_READ_FORWARD;
  if (C % (32 * 4 * kNJ) != 0 || C > 512 * 4 * kNJ || T % kRS != 0) return p;
  if (!aligned16(x) || !aligned16(du) || (codes && !aligned16(u_codes))) return p;
  p.threads = (int)(C / (4 * kNJ));
  const size_t row = (size_t)C * ((dt == BSP_F32 ? 4 : 2) + (du_dt == BSP_F32 ? 4 : 2) + (codes ? 1 : 0));
  const size_t stage = round_up(kRS * row, 128);
  const size_t tail = 64 + 2 * 4 * 16 * sizeof(float) + 16;
  int bps = 512 / p.threads;                        // 128 registers per thread at most
  if (bps > 4) bps = 4;
  const size_t budget = (size_t)227 * 1024 / bps - 1024;
  if (budget < 2 * stage + tail) return p;
  p.ring = (int)((budget - tail) / stage);
  if (p.ring > 8) p.ring = 8;
  p.smem = p.ring * stage + tail;
  const int64_t nstage_rows = T / kRS;
  const int64_t want = (int64_t)kNumSMs * bps;
  p.grid = (int)(nstage_rows < want ? nstage_rows : want);
  p.rows_per_block = ((T + p.grid - 1) / p.grid + kRS - 1) / kRS * kRS;
  p.ok = true;
  return p;
}

template <int DT, int DU_DT, int FMT>
static int launch_norm_bwd_stream(const StreamPlan& p, cudaStream_t st, int kind, const void* x, int64_t T, int64_t C,
                                  const float* gamma, const float* beta, const float* rstd, const float* mean,
                                  const void* du, int gain_read, const uint8_t* u_codes, bsp_quant_t q, PhiloxKey key,
                                  float* part_g, float* part_b, float* dx, bsp_diag_t* diag) {
#define BSP_NBS(KIND)                                                                                       \
  do {                                                                                                      \
    auto kfn = norm_bwd_stream_kernel<DT, DU_DT, FMT, KIND>;                                                \
    BSP_CHECK_CUDA(cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem));    \
    kfn<<<p.grid, p.threads, p.smem, st>>>(x, T, C, p.rows_per_block, p.ring, gamma, beta, rstd, mean, du,  \
                                            gain_read, u_codes, q.scale, q.scale_dev, key, part_g, part_b,  \
                                            dx, diag);                                                      \
  } while (0)
  if (kind == BSP_RMSNORM) BSP_NBS(BSP_RMSNORM);
  else BSP_NBS(BSP_LAYERNORM);
#undef BSP_NBS
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

}  // namespace bsp
