// Row statistics of the normalisation (rstd, mean) and the largest |u|, streamed like the backward:
// each block owns a contiguous range of rows and walks it RS rows at a time; one elected thread
// keeps a ring of stages in flight with untiled bulk copies that complete on an mbarrier.  A thread
// owns NJ groups of four columns, 4*(tid + NT*j), whose gains and biases stay in registers, and
// holds its RS x NJ x 4 elements of the stage in registers, so a row costs one pass over shared
// memory and the arithmetic of the value chain.  The row sums of a stage go through one block
// barrier (two for LayerNorm: the mean first, then the variance about it).  The pass has about ten
// instructions per element to spend at HBM speed: fat threads (64 elements per stage) keep the
// per-thread cost of the reductions, the divisions and the root small per element.
// Requires C == 4 * NJ * blockDim.x (a multiple of 128 * NJ), T a multiple of RS and 16-byte
// aligned rows; other shapes take norm_stats_kernel.
#pragma once

#include "norm_bwd_stream.cuh"

namespace bsp {

constexpr int kStatRS = 4;    // rows per stage
constexpr int kStatNJ = 4;    // column groups per thread

template <int DT, int KIND, int RS, int NJ>
__global__ void __launch_bounds__(512, 1)
norm_stats_stream_kernel(const void* __restrict__ x, int64_t T, int64_t C, int64_t rows_per_block, int nstages_ring,
                         const float* __restrict__ gamma, const float* __restrict__ beta, float eps,
                         float* __restrict__ rstd, float* __restrict__ mean, uint32_t* __restrict__ amax_bits,
                         bsp_diag_t* diag) {
  extern __shared__ __align__(128) unsigned char smem[];
  constexpr int ESX = DT == BSP_F32 ? 4 : 2;
  constexpr bool LN = KIND == BSP_LAYERNORM;
  constexpr int GL = 32 / RS;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, NT = blockDim.x, nwarp = NT >> 5;
  const int NS = nstages_ring;
  const size_t xrow = (size_t)C * ESX;
  const size_t stage_bytes = (RS * xrow + 127) / 128 * 128;
  unsigned char* tail = smem + (size_t)NS * stage_bytes;
  const uint32_t bar0 = smem_u32(tail);                                       // full[NS], 8 bytes each
  float* red = reinterpret_cast<float*>(tail + 8 * 8);                        // [2][RS][16]
  volatile int* abort_flag = reinterpret_cast<volatile int*>(red + 2 * RS * 16);
  const float fC = (float)C;
  int col[NJ];
#pragma unroll
  for (int j = 0; j < NJ; ++j) col[j] = 4 * (tid + NT * j);

  const int64_t r0 = (int64_t)blockIdx.x * rows_per_block;
  const int64_t r1 = r0 + rows_per_block < T ? r0 + rows_per_block : T;
  const int nst = r1 > r0 ? (int)((r1 - r0) / RS) : 0;

  auto issue = [&](int i) {                                                   // thread 0 only
    const int s = i % NS;
    const uint32_t bar = bar0 + 8 * s;
    mbar_expect_tx(bar, (uint32_t)(RS * xrow));
    bulk_load_1d(smem_u32(smem + (size_t)s * stage_bytes),
                 reinterpret_cast<const unsigned char*>(x) + (size_t)(r0 + (int64_t)i * RS) * xrow,
                 (uint32_t)(RS * xrow), bar);
  };
  if (tid == 0) {
    for (int s = 0; s < NS; ++s) mbar_init(bar0 + 8 * s, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    for (int i = 0; i < NS && i < nst; ++i) issue(i);
  }
  __syncthreads();

  float g[NJ][4], b[NJ][4];
#pragma unroll
  for (int j = 0; j < NJ; ++j) {
#pragma unroll
    for (int e = 0; e < 4; ++e) { g[j][e] = 1.f; b[j][e] = 0.f; }
    if (amax_bits) {
      const float4 a = __ldg(reinterpret_cast<const float4*>(gamma + col[j]));
      g[j][0] = a.x; g[j][1] = a.y; g[j][2] = a.z; g[j][3] = a.w;
      if (LN) {
        const float4 bb = __ldg(reinterpret_cast<const float4*>(beta + col[j]));
        b[j][0] = bb.x; b[j][1] = bb.y; b[j][2] = bb.z; b[j][3] = bb.w;
      }
    }
  }

  // sums of RS per-thread values over the block; slot alternates so that one barrier per call is enough
  int slot = 0;
  auto block_sum = [&](const float (&v)[RS], float (&tot)[RS], bool ok, bool& all_ok) {
    const float r = warp_sum_packed<RS>(v, lane);
    if ((lane & (GL - 1)) == 0) red[(slot * RS + lane / GL) * 16 + warp] = r;
    all_ok = __syncthreads_and(ok ? 1 : 0) != 0;
    const int q = lane / GL, jl = lane & (GL - 1);
    float t = 0.f;
    for (int w = jl; w < nwarp; w += GL) t += red[(slot * RS + q) * 16 + w];
#pragma unroll
    for (int o = GL / 2; o > 0; o >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, o);
#pragma unroll
    for (int k = 0; k < RS; ++k) tot[k] = __shfl_sync(0xFFFFFFFFu, t, k * GL);
    slot ^= 1;
  };

  float amax4[4] = {0.f, 0.f, 0.f, 0.f};
  uint32_t nf = 0;
  bool failed = false;
  for (int i = 0; i < nst; ++i) {
    const int s = i % NS;
    const uint32_t par = (uint32_t)(i / NS) & 1u;
    const int64_t rb = r0 + (int64_t)i * RS;
    const unsigned char* st = smem + (size_t)s * stage_bytes;
    // after a failed wait the stage's contents are arbitrary; the results are discarded below
    const bool ok = mbar_wait_suspend(bar0 + 8 * s, par, abort_flag);
    float xv[RS][NJ][4];
#pragma unroll
    for (int rr = 0; rr < RS; ++rr)
#pragma unroll
      for (int j = 0; j < NJ; ++j) lds4<DT>(st + rr * xrow, col[j], xv[rr][j]);

    bool all_ok = true;
    float mu[RS];
#pragma unroll
    for (int rr = 0; rr < RS; ++rr) mu[rr] = 0.f;
    bool refilled = false;
    if (LN) {
      float sv[RS], tot[RS];
#pragma unroll
      for (int rr = 0; rr < RS; ++rr) {
        sv[rr] = 0.f;
#pragma unroll
        for (int j = 0; j < NJ; ++j) sv[rr] += (xv[rr][j][0] + xv[rr][j][1]) + (xv[rr][j][2] + xv[rr][j][3]);
      }
      block_sum(sv, tot, ok, all_ok);
      if (!all_ok) { failed = true; break; }
      // every thread holds the stage in registers by now: its buffer can take the next copy
      if (tid == 0 && i + NS < nst) issue(i + NS);
      refilled = true;
#pragma unroll
      for (int rr = 0; rr < RS; ++rr) mu[rr] = __fdiv_rn(tot[rr], fC);
    }
    float sq[RS], tot[RS];
#pragma unroll
    for (int rr = 0; rr < RS; ++rr) {
      float a0 = 0.f, a1 = 0.f;
#pragma unroll
      for (int j = 0; j < NJ; ++j) {
        const float d0 = LN ? xv[rr][j][0] - mu[rr] : xv[rr][j][0], d1 = LN ? xv[rr][j][1] - mu[rr] : xv[rr][j][1];
        const float d2 = LN ? xv[rr][j][2] - mu[rr] : xv[rr][j][2], d3 = LN ? xv[rr][j][3] - mu[rr] : xv[rr][j][3];
        a0 = fmaf(d0, d0, a0); a1 = fmaf(d1, d1, a1); a0 = fmaf(d2, d2, a0); a1 = fmaf(d3, d3, a1);
      }
      sq[rr] = a0 + a1;
    }
    block_sum(sq, tot, ok, all_ok);
    if (!all_ok) { failed = true; break; }
    if (!refilled && tid == 0 && i + NS < nst) issue(i + NS);

    // lane rr of every warp takes the divisions and the root of row rr (one instruction sequence
    // for all rows of the stage); the others get the result by shuffle
    float my_tot = tot[0];
#pragma unroll
    for (int rr = 1; rr < RS; ++rr) my_tot = lane == rr ? tot[rr] : my_tot;
    const float my_rs = __fdiv_rn(1.0f, __fsqrt_rn(__fadd_rn(__fdiv_rn(my_tot, fC), eps)));
    float rs[RS];
#pragma unroll
    for (int rr = 0; rr < RS; ++rr) {
      rs[rr] = __shfl_sync(0xFFFFFFFFu, my_rs, rr);
      if (tid == 0) {
        if (!(tot[rr] <= 3.4028234663852886e38f)) nf += 1;        // NaN, infinity or overflow in this row
        rstd[rb + rr] = rs[rr];
        if (LN && mean) mean[rb + rr] = mu[rr];
      }
    }
    if (amax_bits) {
#pragma unroll
      for (int rr = 0; rr < RS; ++rr)
#pragma unroll
        for (int j = 0; j < NJ; ++j)
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float xe = xv[rr][j][e];
            const float u = LN ? __fadd_rn(__fmul_rn(__fmul_rn(__fsub_rn(xe, mu[rr]), rs[rr]), g[j][e]), b[j][e])
                               : __fmul_rn(__fmul_rn(xe, rs[rr]), g[j][e]);
            amax4[e] = fmaxf(amax4[e], fabsf(u));                // fmaxf drops a NaN operand
          }
    }
  }
  if (failed) {
    if (tid == 0 && diag) atomicMax(&diag->status, (int)BSP_ERR_TIMEOUT);
    return;
  }
  if (amax_bits) {
    const float amax = warp_max(fmaxf(fmaxf(amax4[0], amax4[1]), fmaxf(amax4[2], amax4[3])));
    if (lane == 0 && amax > 0.f) atomicMax(amax_bits, __float_as_uint(amax));
  }
  DiagCounters dc; dc.nonfinite = nf;
  diag_flush_warp(diag, dc);
}

struct StatsPlan {
  bool ok;
  int threads, ring, grid;
  int64_t rows_per_block;
  size_t smem;
};

static inline StatsPlan plan_stats_stream(int64_t T, int64_t C, int dt, const void* x) {
  StatsPlan p{};
  constexpr int RS = kStatRS, NJ = kStatNJ;
  if (C % (32 * 4 * NJ) != 0 || C > 512 * 4 * NJ || T % RS != 0 || !aligned16(x)) return p;
  p.threads = (int)(C / (4 * NJ));
  const size_t stage = round_up(RS * (size_t)C * (dt == BSP_F32 ? 4 : 2), 128);
  const size_t tail = 64 + 2 * RS * 16 * sizeof(float) + 16;
  int bps = 512 / p.threads;                        // 128 registers per thread at most
  if (bps > 4) bps = 4;
  const size_t budget = (size_t)227 * 1024 / bps - 1024;
  if (budget < 2 * stage + tail) return p;
  p.ring = (int)((budget - tail) / stage);
  if (p.ring > 8) p.ring = 8;
  p.smem = p.ring * stage + tail;
  const int64_t nstage_rows = T / RS;
  const int64_t want = (int64_t)kNumSMs * bps;
  p.grid = (int)(nstage_rows < want ? nstage_rows : want);
  p.rows_per_block = ((T + p.grid - 1) / p.grid + RS - 1) / RS * RS;
  p.ok = true;
  return p;
}

}  // namespace bsp
