// Normalisation backward under a per-use read policy, and the K-draw gain-use Monte-Carlo pass.
//
// norm_bwd_kernel: one row per block iteration; x and du are read once, dx is written once, the
// column sums for dgamma / dbeta are kept in registers across the block's rows and reduced over
// blocks by a second, deterministic kernel.  HBM-bound.  Shapes made of whole 256-column stages
// take norm_bwd_stream_kernel (same arithmetic, rows staged through shared memory by bulk copies).
// gain_mc_kernel: x and du are read once for all K draws; every draw costs one Philox block and
// four stochastic roundings per four elements, all in registers.  ALU-bound.
#include <mutex>

#include "norm_bwd_stream.cuh"

namespace bsp {

template <int FMT>
__device__ __forceinline__ float sr_value(float v, uint32_t U) { return f8_sr_value<FMT>(v, U); }

// ------------------------------------------------------------------------------- norm backward

// NT threads cover a row with JMAX groups of four columns each (NT * JMAX * 4 >= C).  Wide rows use
// wide blocks rather than more columns per thread: the per-thread state (column sums, gains, the
// current and the prefetched row) stays near 64 registers, which keeps 1024 threads resident.
template <int DT, int DU_DT, int FMT, int JMAX, int NT>
__global__ void __launch_bounds__(NT, 1024 / NT)
norm_bwd_kernel(int kind, const void* __restrict__ x, int64_t T, int64_t C, const float* __restrict__ gamma,
                const float* __restrict__ beta, const float* __restrict__ rstd, const float* __restrict__ mean,
                const void* __restrict__ du, int gain_read, int dx_read, const uint8_t* __restrict__ u_codes,
                float scale_val, const float* __restrict__ scale_dev, PhiloxKey key, PhiloxKey key_dx,
                float* __restrict__ part_g, float* __restrict__ part_b, float* __restrict__ dx) {
  __shared__ float red[2][2][NT / 32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float scale = scale_dev ? __ldg(scale_dev) : scale_val;
  const float inv_scale = __fdiv_rn(1.0f, scale);
  const float invC = 1.0f / (float)C;

  float4 g4[JMAX], b4[JMAX], accg[JMAX], accb[JMAX];
#pragma unroll
  for (int j = 0; j < JMAX; ++j) {
    const int64_t c = 4 * ((int64_t)tid + NT * j);
    g4[j] = make_float4(1.f, 1.f, 1.f, 1.f);
    b4[j] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (c < C) {
      g4[j] = __ldg(reinterpret_cast<const float4*>(gamma + c));
      if (kind == BSP_LAYERNORM) b4[j] = __ldg(reinterpret_cast<const float4*>(beta + c));
    }
    accg[j] = make_float4(0.f, 0.f, 0.f, 0.f);
    accb[j] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  float4 rg4[JMAX];
#pragma unroll
  for (int j = 0; j < JMAX; ++j)
    rg4[j] = make_float4(__fdiv_rn(1.0f, g4[j].x), __fdiv_rn(1.0f, g4[j].y), __fdiv_rn(1.0f, g4[j].z),
                         __fdiv_rn(1.0f, g4[j].w));

  // The next row's x and du are requested before this row's block-wide reduction, so the loads of
  // one row overlap the arithmetic and the barrier of the row before.
  float4 nx[JMAX], nd[JMAX];
  float nrs = 0.f, nmu = 0.f;
  auto fetch = [&](int64_t r) {
    nrs = __ldg(rstd + r);
    nmu = kind == BSP_LAYERNORM ? __ldg(mean + r) : 0.f;
#pragma unroll
    for (int j = 0; j < JMAX; ++j) {
      const int64_t c = 4 * ((int64_t)tid + NT * j);
      if (c < C) {
        nx[j] = load4<DT>(x, (size_t)r * C + c);
        nd[j] = load4<DU_DT>(du, (size_t)r * C + c);
      }
    }
  };
  if (blockIdx.x < T) fetch(blockIdx.x);
  int it = 0;
  for (int64_t r = blockIdx.x; r < T; r += gridDim.x, ++it) {
    const float rs = nrs, mu = nmu;
    float4 z[JMAX], dz[JMAX], d4[JMAX], xr[JMAX];
#pragma unroll
    for (int j = 0; j < JMAX; ++j) { xr[j] = nx[j]; d4[j] = nd[j]; }
    if (r + gridDim.x < T) fetch(r + gridDim.x);
    float p1 = 0.f, p2 = 0.f;
#pragma unroll
    for (int j = 0; j < JMAX; ++j) {
      const int64_t c = 4 * ((int64_t)tid + NT * j);
      z[j] = dz[j] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (c < C) {
        const size_t i0 = (size_t)r * C + c;
        const float4 xv = xr[j];
        if (kind == BSP_RMSNORM) {
          z[j] = make_float4(__fmul_rn(xv.x, rs), __fmul_rn(xv.y, rs), __fmul_rn(xv.z, rs), __fmul_rn(xv.w, rs));
        } else {
          z[j] = make_float4(__fmul_rn(__fsub_rn(xv.x, mu), rs), __fmul_rn(__fsub_rn(xv.y, mu), rs),
                             __fmul_rn(__fsub_rn(xv.z, mu), rs), __fmul_rn(__fsub_rn(xv.w, mu), rs));
        }
        dz[j] = make_float4(g4[j].x * d4[j].x, g4[j].y * d4[j].y, g4[j].z * d4[j].z, g4[j].w * d4[j].w);
        // z as a use reads it: the original, or (copy - beta) / gamma from the forward's codes (R)
        // or from a fresh stochastic rounding under the use's own generator stream (N)
        const float4 zo = z[j];
        auto z_read = [&](int policy, const PhiloxKey& kk) -> float4 {
          if (policy == BSP_READ_ORIGINAL) return zo;
          float dec[4];
          if (policy == BSP_READ_FORWARD) {
            const uint32_t pk = __ldg(reinterpret_cast<const uint32_t*>(u_codes + i0));
            f8_decode4<FMT>(pk, dec);
          } else {
            const uint4 w = philox_block(kk, (uint64_t)i0 >> 2, kk.c2);
            const float u[4] = {zo.x, zo.y, zo.z, zo.w};
            const float gg[4] = {g4[j].x, g4[j].y, g4[j].z, g4[j].w};
            const float bb[4] = {b4[j].x, b4[j].y, b4[j].z, b4[j].w};
            const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              float uu = __fmul_rn(u[e], gg[e]);
              if (kind == BSP_LAYERNORM) uu = __fadd_rn(uu, bb[e]);
              dec[e] = sr_value<FMT>(__fmul_rn(uu, scale), ww[e]);
            }
          }
          // (copy - beta) / gamma as a multiplication by the per-column reciprocal (one rounding
          // more than a division, far inside the FP32 tolerance; the division would cost ten
          // instructions per element on a pass that has about that many to spend)
          return make_float4((dec[0] * inv_scale - b4[j].x) * rg4[j].x, (dec[1] * inv_scale - b4[j].y) * rg4[j].y,
                             (dec[2] * inv_scale - b4[j].z) * rg4[j].z, (dec[3] * inv_scale - b4[j].w) * rg4[j].w);
        };
        const float4 zg = z_read(gain_read, key);
        if (dx) {
          if (dx_read != BSP_READ_ORIGINAL) z[j] = z_read(dx_read, key_dx);   // the input gradient's own read
          p1 += (dz[j].x * z[j].x + dz[j].y * z[j].y) + (dz[j].z * z[j].z + dz[j].w * z[j].w);
          p2 += (dz[j].x + dz[j].y) + (dz[j].z + dz[j].w);
        }
        accg[j].x = fmaf(zg.x, d4[j].x, accg[j].x); accg[j].y = fmaf(zg.y, d4[j].y, accg[j].y);
        accg[j].z = fmaf(zg.z, d4[j].z, accg[j].z); accg[j].w = fmaf(zg.w, d4[j].w, accg[j].w);
        accb[j].x += d4[j].x; accb[j].y += d4[j].y; accb[j].z += d4[j].z; accb[j].w += d4[j].w;
      }
    }
    if (dx) {
      const int buf = it & 1;
      p1 = warp_sum(p1);
      p2 = warp_sum(p2);
      if (lane == 0) { red[buf][0][warp] = p1; red[buf][1][warp] = p2; }
      __syncthreads();
      // every warp re-reduces the per-warp partials: one shared load per lane, then shuffles
      float s1 = lane < NT / 32 ? red[buf][0][lane] : 0.f;
      float s2 = lane < NT / 32 ? red[buf][1][lane] : 0.f;
      s1 = warp_sum(s1);
      s2 = warp_sum(s2);
      const float m1 = s1 * invC;
      const float m2 = kind == BSP_LAYERNORM ? s2 * invC : 0.f;
#pragma unroll
      for (int j = 0; j < JMAX; ++j) {
        const int64_t c = 4 * ((int64_t)tid + NT * j);
        if (c < C) {
          float4 o;
          o.x = rs * ((dz[j].x - m2) - z[j].x * m1);
          o.y = rs * ((dz[j].y - m2) - z[j].y * m1);
          o.z = rs * ((dz[j].z - m2) - z[j].z * m1);
          o.w = rs * ((dz[j].w - m2) - z[j].w * m1);
          *reinterpret_cast<float4*>(dx + (size_t)r * C + c) = o;
        }
      }
    }
  }
#pragma unroll
  for (int j = 0; j < JMAX; ++j) {
    const int64_t c = 4 * ((int64_t)tid + NT * j);
    if (c < C) {
      *reinterpret_cast<float4*>(part_g + (size_t)blockIdx.x * C + c) = accg[j];
      if (part_b) *reinterpret_cast<float4*>(part_b + (size_t)blockIdx.x * C + c) = accb[j];
    }
  }
}

// out[c] = sum over nparts of part[p*C + c], in a fixed order.  grid: (C/32, 1 or 2) blocks of
// 256 = 8 x 32 threads; blockIdx.y == 1 reduces the second pair (dbeta beside dgamma in one launch).
__global__ void __launch_bounds__(256)
column_reduce_kernel(const float* __restrict__ part0, float* __restrict__ out0, const float* __restrict__ part1,
                     float* __restrict__ out1, int nparts, int64_t C) {
  __shared__ float sm[8][33];
  const float* __restrict__ part = blockIdx.y ? part1 : part0;
  float* __restrict__ out = blockIdx.y ? out1 : out0;
  const int cl = threadIdx.x & 31, pl = threadIdx.x >> 5;
  const int64_t c = (int64_t)blockIdx.x * 32 + cl;
  float s = 0.f;
  if (c < C) {
    // four loads in flight per thread; the additions keep the order p = pl, pl + 8, ...
    int p = pl;
    for (; p + 24 < nparts; p += 32) {
      const float a0 = __ldg(part + (size_t)p * C + c), a1 = __ldg(part + (size_t)(p + 8) * C + c);
      const float a2 = __ldg(part + (size_t)(p + 16) * C + c), a3 = __ldg(part + (size_t)(p + 24) * C + c);
      s += a0; s += a1; s += a2; s += a3;
    }
    for (; p < nparts; p += 8) s += __ldg(part + (size_t)p * C + c);
  }
  sm[pl][cl] = s;
  __syncthreads();
  if (pl == 0 && c < C) {
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) t += sm[w][cl];
    out[c] = t;
  }
}

// ------------------------------------------------------------------------------- gain-use Monte Carlo

constexpr int kMcRows = 8;             // rows per thread
constexpr int kMcSlab = 8 * kMcRows;    // rows per block (8 warps)
constexpr int kMcCols = 128;            // columns per block (32 lanes x 4)
constexpr int kMcChunk = 64;            // draws per launch
constexpr size_t kMcSmemBytes = (size_t)2 * kMcRows * 256 * sizeof(float4);   // values + weights of a slab
constexpr int kMcThinWarps = 4, kMcThinRows = 4;     // the thin variant: 4 warps x 4 rows per thread
constexpr size_t kMcThinSmemBytes = (size_t)2 * kMcThinRows * kMcThinWarps * 32 * sizeof(float4);

template <int DT, int DU_DT, int FMT, int NW, int ROWS>
__global__ void __launch_bounds__(NW * 32, NW == 8 ? 3 : 4)
gain_mc_kernel(int kind, const void* __restrict__ x, int64_t T, int64_t C, const float* __restrict__ gamma,
               const float* __restrict__ beta, const float* __restrict__ rstd, const float* __restrict__ mean,
               const void* __restrict__ du, float scale_val, const float* __restrict__ scale_dev,
               const float* __restrict__ grid_steps, PhiloxKey key, int draw_begin, int ndraws,
               float* __restrict__ partial /* [ndraws][nslabs][C] */, bsp_diag_t* __restrict__ diag) {
  // A fresh rounding of an element is its round-down value plus, with probability frac, one grid
  // step: value(U) = lo + (U < P) * (hi - lo) with the threshold P of f8_sr_threshold.  So the
  // gain-use sum of draw k is  sum_t (lo/scale - beta)/gamma * du  (the same for every draw, summed
  // once) plus  sum_t [U_k,t < P_t] * (hi - lo)/scale/gamma * du : per element and draw one generator
  // word, one comparison and one conditional add.  The slab's thresholds and step weights live in
  // shared memory (each thread reads back only what it wrote), which keeps the register count low
  // enough for three blocks per SM: the draw loop is a chain of dependent integer multiplies, and it
  // is occupancy that hides their latency.
  // grid_steps != NULL selects the b-bit per-token store instead of the FP8 store: the element sits at
  // t = u / s on the uniform grid of its token's step s, lo = s floor(t), the step weight is s and the
  // threshold floor(frac(t) 2^32).  Everything after the prologue is the same.
  extern __shared__ __align__(16) float4 mc_smem[];
  uint4* sp = reinterpret_cast<uint4*>(mc_smem);   // [kMcRows][256] thresholds
  constexpr int NT = NW * 32;
  float4* sw = mc_smem + ROWS * NT;                // [ROWS][NT] step weights
  __shared__ __align__(16) float red[2][NW][kMcCols];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t c = (int64_t)blockIdx.x * kMcCols + lane * 4;
  const int64_t slab = blockIdx.y, nslabs = gridDim.y;
  const float scale = grid_steps ? 1.0f : (scale_dev ? __ldg(scale_dev) : scale_val);
  const float inv_scale = __fdiv_rn(1.0f, scale);
  const bool col_ok = c < C;

  float4 g4 = make_float4(1.f, 1.f, 1.f, 1.f), b4 = make_float4(0.f, 0.f, 0.f, 0.f);
  if (col_ok) {
    g4 = __ldg(reinterpret_cast<const float4*>(gamma + c));
    if (kind == BSP_LAYERNORM) b4 = __ldg(reinterpret_cast<const float4*>(beta + c));
  }
  // generator block index of this thread's four columns in row (slab*NW*ROWS + warp + NW*i) is
  // q0 + i*qstep; rows beyond T keep v = wgt = 0 and contribute nothing whatever word they draw
  const uint64_t q0 = (uint64_t)((slab * (NW * ROWS) + warp) * C + (col_ok ? c : 0)) >> 2;
  const uint64_t qstep = (uint64_t)(NW * C) / 4;
  float base[4] = {0.f, 0.f, 0.f, 0.f};                 // the draw-independent part of this thread's sums
  DiagCounters dc;                                       // non-finite x or du, counted once per element
#pragma unroll 1
  for (int i = 0; i < ROWS; ++i) {
    const int64_t r = slab * (NW * ROWS) + warp + NW * i;
    uint32_t thr[4] = {0u, 0u, 0u, 0u};
    float wgt[4] = {0.f, 0.f, 0.f, 0.f};
    if (r < T && col_ok) {
      const size_t i0 = (size_t)r * C + c;
      const float4 xv = load4<DT>(x, i0);
      const float4 dv = load4<DU_DT>(du, i0);
      const float rs = __ldg(rstd + r);
      const float mu = kind == BSP_LAYERNORM ? __ldg(mean + r) : 0.f;
      const float xs[4] = {xv.x, xv.y, xv.z, xv.w};
      const float ds[4] = {dv.x, dv.y, dv.z, dv.w};
      const float gg[4] = {g4.x, g4.y, g4.z, g4.w};
      const float bb[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float u;
        if (kind == BSP_RMSNORM) u = __fmul_rn(__fmul_rn(xs[e], rs), gg[e]);
        else u = __fadd_rn(__fmul_rn(__fmul_rn(__fsub_rn(xs[e], mu), rs), gg[e]), bb[e]);
        const float w = __fdiv_rn(ds[e], gg[e]);
        if (!isfinite(xs[e]) || !isfinite(ds[e])) dc.nonfinite++;
        if (grid_steps) {
          const float st = __ldg(grid_steps + r);
          const float t = __fdiv_rn(u, st);
          const float n0 = floorf(t);
          thr[e] = __float2uint_rd(__fsub_rn(t, n0) * 4294967296.0f);
          base[e] = fmaf(fmaf(st, n0, -bb[e]), w, base[e]);
          wgt[e] = thr[e] ? st * w : 0.f;
          continue;
        }
        const float v = __fmul_rn(u, scale);
        const float lo = sr_value<FMT>(v, 0xFFFFFFFFu), hi = sr_value<FMT>(v, 0u);   // never up / up whenever possible
        thr[e] = f8_sr_threshold<FMT>(v);
        base[e] = fmaf(fmaf(lo, inv_scale, -bb[e]), w, base[e]);
        wgt[e] = thr[e] ? (hi - lo) * inv_scale * w : 0.f;      // (NaN has threshold 0: it stays in base)
      }
    }
    sp[i * NT + tid] = make_uint4(thr[0], thr[1], thr[2], thr[3]);
    sw[i * NT + tid] = make_float4(wgt[0], wgt[1], wgt[2], wgt[3]);
  }
  diag_flush_warp(diag, dc);                             // (the host hands diag to the first chunk of draws only)
  for (int k = 0; k < ndraws; ++k) {
    const uint32_t draw = (uint32_t)(draw_begin + k);
    float acc[4] = {base[0], base[1], base[2], base[3]};
#pragma unroll 2
    for (int i = 0; i < ROWS; ++i) {
      const uint4 w = philox_block(key, q0 + (uint64_t)i * qstep, draw);
      const uint4 p4 = sp[i * NT + tid];
      const float4 w4 = sw[i * NT + tid];
      acc[0] += w.x < p4.x ? w4.x : 0.f;
      acc[1] += w.y < p4.y ? w4.y : 0.f;
      acc[2] += w.z < p4.z ? w4.z : 0.f;
      acc[3] += w.w < p4.w ? w4.w : 0.f;
    }
    const int buf = k & 1;
    *reinterpret_cast<float4*>(&red[buf][warp][lane * 4]) = make_float4(acc[0], acc[1], acc[2], acc[3]);
    __syncthreads();
    if (tid < kMcCols) {
      float s = 0.f;
#pragma unroll
      for (int w8 = 0; w8 < NW; ++w8) s += red[buf][w8][tid];
      const int64_t cc = (int64_t)blockIdx.x * kMcCols + tid;
      if (cc < C) partial[((size_t)k * nslabs + slab) * C + cc] = s;
    }
  }
}

// gk[k*C + c] = sum over slabs of partial[k][slab][c] in a fixed order.
__global__ void __launch_bounds__(256)
gain_mc_slab_reduce_kernel(const float* __restrict__ partial, int nslabs, int64_t C, float* __restrict__ gk) {
  __shared__ float sm[8][33];
  const int cl = threadIdx.x & 31, pl = threadIdx.x >> 5;
  const int64_t c = (int64_t)blockIdx.x * 32 + cl;
  const size_t k = blockIdx.y;
  float s = 0.f;
  if (c < C)
    for (int p = pl; p < nslabs; p += 8) s += partial[(k * nslabs + p) * C + c];
  sm[pl][cl] = s;
  __syncthreads();
  if (pl == 0 && c < C) {
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) t += sm[w][cl];
    gk[k * C + c] = t;
  }
}

// S1[c] += sum_k (gk - ref), S2[c] += sum_k (gk - ref)^2.
__global__ void gain_mc_accumulate_kernel(const float* __restrict__ gk, int ndraws, int64_t C,
                                          const float* __restrict__ ref, float* __restrict__ S1,
                                          float* __restrict__ S2) {
  const int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= C) return;
  const float g0 = ref[c];
  float s1 = 0.f, s2 = 0.f;
  for (int k = 0; k < ndraws; ++k) {
    const float d = gk[(size_t)k * C + c] - g0;
    s1 += d;
    s2 = fmaf(d, d, s2);
  }
  S1[c] += s1;
  S2[c] += s2;
}

static int bwd_grid(int64_t T) {
  const int64_t want = (int64_t)kNumSMs * 4;
  return (int)(T < want ? T : want);
}

template <int DT, int DU_DT, int FMT>
static int launch_norm_bwd(int jmax, int grid, cudaStream_t st, int kind, const void* x, int64_t T, int64_t C,
                           const float* gamma, const float* beta, const float* rstd, const float* mean,
                           const void* du, int gain_read, int dx_read, const uint8_t* u_codes, bsp_quant_t q,
                           PhiloxKey key, PhiloxKey key_dx, float* part_g, float* part_b, float* dx) {
  // jmax encodes the launch shape: C/4 column groups over 256, 512 or 1024 threads, two groups per
  // thread only beyond 4096 columns
  (void)jmax;
  const int64_t groups = C / 4;
#define BSP_NB(J, NT)                                                                                        \
  norm_bwd_kernel<DT, DU_DT, FMT, J, NT><<<grid, NT, 0, st>>>(kind, x, T, C, gamma, beta, rstd, mean, du,    \
                                                               gain_read, dx_read, u_codes, q.scale,           \
                                                               q.scale_dev, key, key_dx, part_g, part_b, dx)
  if (groups <= 256) BSP_NB(1, 256);
  else if (groups <= 512) BSP_NB(1, 512);
  else if (groups <= 1024) BSP_NB(1, 1024);
  else BSP_NB(2, 1024);
#undef BSP_NB
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

static bool valid_enum(int v, int hi) { return v >= 0 && v <= hi; }

}  // namespace bsp

using namespace bsp;

extern "C" {

size_t bsp_norm_bwd_workspace_bytes(int64_t T, int64_t C) {
  if (T <= 0 || C <= 0) return 0;
  return round_up((size_t)bwd_grid(T) * (size_t)C * sizeof(float), 256) * 2;
}

int bsp_norm_bwd(int kind, const void* x, int dt, int64_t T, int64_t C, const float* gamma, const float* beta,
                 const float* rstd, const float* mean, const void* du, int du_dt, int gain_read, int dx_read,
                 const uint8_t* u_codes, bsp_quant_t q, bsp_key_t key, float* dgamma, float* dbeta, float* dx,
                 void* ws, size_t ws_bytes, bsp_diag_t* diag, void* stream) {
  if (!valid_enum(kind, 1) || !valid_enum(dt, 1) || !valid_enum(du_dt, 1) || !valid_enum(gain_read, 2) ||
      !valid_enum(dx_read, 2) || !valid_enum(q.fmt, 1))
    return BSP_ERR_ARG;
  if (key.tensor_id >= (1u << 24) || key.stream > 255u || key.reserved != 0) return BSP_ERR_ARG;
  if (T < 0 || C <= 0) return BSP_ERR_ARG;
  if (!dgamma) return BSP_ERR_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if (T == 0) {
    BSP_CHECK_CUDA(cudaMemsetAsync(dgamma, 0, C * sizeof(float), st));
    if (dbeta) BSP_CHECK_CUDA(cudaMemsetAsync(dbeta, 0, C * sizeof(float), st));
    return BSP_OK;
  }
  if (!x || !gamma || !rstd || !du || (kind == BSP_LAYERNORM && (!beta || !mean))) return BSP_ERR_ARG;
  if (!dx) dx_read = BSP_READ_ORIGINAL;                        // no input gradient asked for: nothing reads
  if ((gain_read == BSP_READ_FORWARD || dx_read == BSP_READ_FORWARD) && !u_codes) return BSP_ERR_ARG;
  if (C % 4 != 0 || C > 8192) return BSP_ERR_UNSUPPORTED;
  if (!aligned16(x) || !aligned16(du) || !aligned16(gamma) || !aligned16(beta) || !aligned16(dx) ||
      (reinterpret_cast<uintptr_t>(u_codes) & 3u))
    return BSP_ERR_ALIGN;
  if (!ws || ws_bytes < bsp_norm_bwd_workspace_bytes(T, C) || (reinterpret_cast<uintptr_t>(ws) & 255u))
    return BSP_ERR_WORKSPACE;
  // whole stages of 256-column multiples take the streamed kernel, every other shape the plain one
  // (an input gradient that reads a copy is outside the reference and takes the plain kernel too)
  StreamPlan plan = plan_stream(T, C, dt, du_dt, gain_read, x, du, u_codes);
  if (dx_read != BSP_READ_ORIGINAL) plan.ok = false;
  const int grid = plan.ok ? plan.grid : bwd_grid(T);
  float* part_g = reinterpret_cast<float*>(ws);
  float* part_b = dbeta ? reinterpret_cast<float*>(reinterpret_cast<char*>(ws) +
                                                   round_up((size_t)grid * C * sizeof(float), 256))
                        : nullptr;
  const int64_t groups = (C / 4 + 255) / 256;
  const int jmax = groups <= 1 ? 1 : groups <= 2 ? 2 : groups <= 4 ? 4 : 8;
  const PhiloxKey pk = make_key(key);
  bsp_key_t key_dx = key;                                      // the input gradient's own generator stream
  key_dx.stream = BSP_STREAM_DX;
  const PhiloxKey pk_dx = make_key(key_dx);
  int rc;
#define BSP_CALL(DT, DU, FMT)                                                                                 \
  rc = plan.ok ? launch_norm_bwd_stream<DT, DU, FMT>(plan, st, kind, x, T, C, gamma, beta, rstd, mean, du,    \
                                                     gain_read, u_codes, q, pk, part_g, part_b, dx, diag)     \
               : launch_norm_bwd<DT, DU, FMT>(jmax, grid, st, kind, x, T, C, gamma, beta, rstd, mean, du,     \
                                              gain_read, dx_read, u_codes, q, pk, pk_dx, part_g, part_b, dx)
  if (q.fmt == BSP_E4M3) {
    if (dt == BSP_F32 && du_dt == BSP_F32) BSP_CALL(BSP_F32, BSP_F32, BSP_E4M3);
    else if (dt == BSP_F32) BSP_CALL(BSP_F32, BSP_BF16, BSP_E4M3);
    else if (du_dt == BSP_F32) BSP_CALL(BSP_BF16, BSP_F32, BSP_E4M3);
    else BSP_CALL(BSP_BF16, BSP_BF16, BSP_E4M3);
  } else {
    if (dt == BSP_F32 && du_dt == BSP_F32) BSP_CALL(BSP_F32, BSP_F32, BSP_E5M2);
    else if (dt == BSP_F32) BSP_CALL(BSP_F32, BSP_BF16, BSP_E5M2);
    else if (du_dt == BSP_F32) BSP_CALL(BSP_BF16, BSP_F32, BSP_E5M2);
    else BSP_CALL(BSP_BF16, BSP_BF16, BSP_E5M2);
  }
#undef BSP_CALL
  if (rc != BSP_OK) return rc;
  const unsigned rb = (unsigned)((C + 31) / 32);
  column_reduce_kernel<<<dim3(rb, dbeta ? 2 : 1), 256, 0, st>>>(part_g, dgamma, part_b, dbeta, grid, C);
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

size_t bsp_norm_gain_mc_workspace_bytes(int64_t T, int64_t C, int K) {
  return bsp::norm_gain_mc_workspace(T, C, K, false);
}

int bsp_norm_gain_mc(int kind, const void* x, int dt, int64_t T, int64_t C, const float* gamma, const float* beta,
                     const float* rstd, const float* mean, const void* du, int du_dt, bsp_quant_t q, bsp_key_t key,
                     int draw0, int K, const float* g_ref, float* S1, float* S2, void* ws, size_t ws_bytes,
                     bsp_diag_t* diag, void* stream) {
  return bsp::norm_gain_mc_run(false, kind, x, dt, T, C, gamma, beta, rstd, mean, du, du_dt, q, key, draw0, K, g_ref, S1,
                               S2, ws, ws_bytes, diag, stream);
}

}  // extern "C"

namespace bsp {

size_t norm_gain_mc_workspace(int64_t T, int64_t C, int K, bool thin) {
  if (T <= 0 || C <= 0 || K <= 0) return 0;
  const int slab_rows = thin ? kMcThinWarps * kMcThinRows : kMcSlab;
  const size_t nslabs = (size_t)((T + slab_rows - 1) / slab_rows);
  const size_t kc = (size_t)(K < kMcChunk ? K : kMcChunk);
  return round_up(kc * nslabs * (size_t)C * sizeof(float), 256) + round_up(kc * (size_t)C * sizeof(float), 256);
}

// thin: the variant of the kernel made to run beside a kernel that fills the SMs (128 threads, 16 KB
// of shared memory, 64 registers: one block fits next to a CTA of the Monte-Carlo contraction).
int norm_gain_mc_run(bool thin, int kind, const void* x, int dt, int64_t T, int64_t C, const float* gamma,
                     const float* beta, const float* rstd, const float* mean, const void* du, int du_dt, bsp_quant_t q,
                     bsp_key_t key, int draw0, int K, const float* g_ref, float* S1, float* S2, void* ws, size_t ws_bytes,
                     bsp_diag_t* diag, void* stream, const float* grid_steps) {
  if (!valid_enum(kind, 1) || !valid_enum(dt, 1) || !valid_enum(du_dt, 1) || !valid_enum(q.fmt, 1)) return BSP_ERR_ARG;
  if (key.tensor_id >= (1u << 24) || key.stream > 255u || key.reserved != 0) return BSP_ERR_ARG;
  if (T < 0 || C <= 0 || K < 0 || draw0 < 0) return BSP_ERR_ARG;
  if (!g_ref || !S1 || !S2) return BSP_ERR_ARG;
  if (K == 0) return BSP_OK;
  if (T > 0 && (!x || !gamma || !rstd || !du || (kind == BSP_LAYERNORM && (!beta || !mean)))) return BSP_ERR_ARG;
  if (C % 4 != 0) return BSP_ERR_UNSUPPORTED;
  if (!aligned16(x) || !aligned16(du) || !aligned16(gamma) || !aligned16(beta)) return BSP_ERR_ALIGN;
  if (!ws || ws_bytes < norm_gain_mc_workspace(T, C, K, thin) || (reinterpret_cast<uintptr_t>(ws) & 255u))
    return BSP_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  const int slab_rows = thin ? kMcThinWarps * kMcThinRows : kMcSlab;
  const int nslabs = (int)((T + slab_rows - 1) / slab_rows);
  const int kc_max = K < kMcChunk ? K : kMcChunk;
  float* partial = reinterpret_cast<float*>(ws);
  float* gk = reinterpret_cast<float*>(reinterpret_cast<char*>(ws) +
                                       round_up((size_t)kc_max * (nslabs > 0 ? nslabs : 1) * C * sizeof(float), 256));
  const PhiloxKey pk = make_key(key);
  for (int kb = 0; kb < K; kb += kMcChunk) {
    const int nd = (K - kb) < kMcChunk ? (K - kb) : kMcChunk;
    if (nslabs > 0) {
      dim3 grid((unsigned)((C + kMcCols - 1) / kMcCols), (unsigned)nslabs);
#define BSP_GM(DT, DU, FMT)                                                                                     \
  do {                                                                                                          \
    if (thin) {                                                                                                 \
      gain_mc_kernel<DT, DU, FMT, kMcThinWarps, kMcThinRows><<<grid, kMcThinWarps * 32, kMcThinSmemBytes, st>>>(kind, x, T, C, gamma, beta, rstd, mean, du, \
                                                                 q.scale, q.scale_dev, grid_steps, pk, draw0 + kb, nd, partial, kb == 0 ? diag : nullptr); \
      break;                                                                                                    \
    }                                                                                                           \
    BSP_CHECK_CUDA(cudaFuncSetAttribute(gain_mc_kernel<DT, DU, FMT, 8, kMcRows>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                        (int)kMcSmemBytes));                                                    \
    gain_mc_kernel<DT, DU, FMT, 8, kMcRows><<<grid, 256, kMcSmemBytes, st>>>(kind, x, T, C, gamma, beta, rstd, mean, du,    \
                                                                 q.scale, q.scale_dev, grid_steps, pk,           \
                                                                 draw0 + kb, nd, partial, kb == 0 ? diag : nullptr); \
  } while (0)
      if (q.fmt == BSP_E4M3) {
        if (dt == BSP_F32 && du_dt == BSP_F32) BSP_GM(BSP_F32, BSP_F32, BSP_E4M3);
        else if (dt == BSP_F32) BSP_GM(BSP_F32, BSP_BF16, BSP_E4M3);
        else if (du_dt == BSP_F32) BSP_GM(BSP_BF16, BSP_F32, BSP_E4M3);
        else BSP_GM(BSP_BF16, BSP_BF16, BSP_E4M3);
      } else {
        if (dt == BSP_F32 && du_dt == BSP_F32) BSP_GM(BSP_F32, BSP_F32, BSP_E5M2);
        else if (dt == BSP_F32) BSP_GM(BSP_F32, BSP_BF16, BSP_E5M2);
        else if (du_dt == BSP_F32) BSP_GM(BSP_BF16, BSP_F32, BSP_E5M2);
        else BSP_GM(BSP_BF16, BSP_BF16, BSP_E5M2);
      }
#undef BSP_GM
      BSP_LAUNCH_CHECK();
    }
    dim3 rgrid((unsigned)((C + 31) / 32), (unsigned)nd);
    gain_mc_slab_reduce_kernel<<<rgrid, 256, 0, st>>>(partial, nslabs, C, gk);
    BSP_LAUNCH_CHECK();
    gain_mc_accumulate_kernel<<<(unsigned)((C + 255) / 256), 256, 0, st>>>(gk, nd, C, g_ref, S1, S2);
    BSP_LAUNCH_CHECK();
  }
  return BSP_OK;
}

}  // namespace bsp

// ------------------------------------------------------------------------------- no-allocation variant

namespace bsp {

// Fixed scratch of bsp_norm_bwd_noalloc: lives in the library's device image, so every GPU that
// loads the library carries these 20 MiB until the process exits.  In host code the symbol below is
// only a handle; its device address is resolved with cudaGetSymbolAddress once per device.
constexpr size_t kNoAllocScratchBytes = BSP_NORM_BWD_NOALLOC_CAPACITY_BYTES;
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

static void* g_noalloc_ptr[kMaxDevices];          // resolved device addresses, by device ordinal
static std::mutex g_noalloc_mutex;

// Device address of the scratch array on the current device (resolved on first use).
static int noalloc_scratch(void** out) {
  int dev = -1;
  BSP_CHECK_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return BSP_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  if (g_noalloc_ptr[dev] == nullptr) {
    void* p = nullptr;
    BSP_CHECK_CUDA(cudaGetSymbolAddress(&p, g_noalloc_scratch));
    if (p == nullptr || (reinterpret_cast<uintptr_t>(p) & 255u)) return BSP_ERR_CUDA;
    g_noalloc_ptr[dev] = p;
  }
  *out = g_noalloc_ptr[dev];
  return BSP_OK;
}

}  // namespace bsp

extern "C" {

int bsp_norm_bwd_noalloc(int kind, const void* x, int dt, int64_t T, int64_t C, const float* gamma,
                         const float* beta, const float* rstd, const float* mean, const void* du, int du_dt,
                         int gain_read, int dx_read, const uint8_t* u_codes, bsp_quant_t q, bsp_key_t key,
                         float* dgamma, float* dbeta, float* dx, bsp_diag_t* diag, void* stream) {
  // size check first: pure host arithmetic, nothing is touched when the problem does not fit
  if (T < 0 || C <= 0) return BSP_ERR_ARG;
  const size_t need = bsp_norm_bwd_workspace_bytes(T, C);
  if (need > bsp::kNoAllocScratchBytes) return BSP_ERR_TOO_LARGE;
  void* scratch = nullptr;
  const int rc = bsp::noalloc_scratch(&scratch);
  if (rc != BSP_OK) return rc;
  // The column partials this pass keeps in scratch are written in full before they are read, so
  // whatever an earlier call left in the array is harmless and nothing has to be cleared.
  return bsp_norm_bwd(kind, x, dt, T, C, gamma, beta, rstd, mean, du, du_dt, gain_read, dx_read, u_codes, q, key,
                      dgamma, dbeta, dx, scratch, bsp::kNoAllocScratchBytes, diag, stream);
}

}  // extern "C"
