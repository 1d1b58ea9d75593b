// Rounded attention probabilities as the saved tensor (Appendix "Theory"): one row has probabilities
// p and values V; the forward rounds p to p_q and outputs o = V^T p_q; with L = ||o||^2 / 2 the row's
// incoming gradient is h = o and dp = V h.  The reference computes dV = p_q h^T and ds = J(p) dp,
// J(x) = diag(x) - x x^T.  A policy reads p_hat at the gradient of V and J_hat at the softmax's
// backward: Delta_V = (p_hat - p_q) h^T, Delta_s = (J_hat - J(p)) dp.  This kernel averages those
// errors over the forward's rounding and the new roundings, draw by draw, for many rows at once:
//   Delta_s for J_hat in { J(p_q), J(a), K(a), J2(a, b), J2(p_q, b) }  (a, b: new roundings;
//     K(a) = diag(a 1^T a) - a a^T, J2(a, b) = diag((a + b) / 2) - (a b^T + b a^T) / 2);
//   Delta_V for p_hat in { p, a }.
// One block per row, one thread per entry (n <= 256).  V (n x d, d <= 64) lies in shared memory for
// h = V^T p_q (every thread sums a slice of one column) and, row by row, in the threads' registers
// for dp = V h; a thread keeps its 2 x d sums of the gradient-of-V errors in registers for all draws.
// Per draw: three generator words per entry (the four threads of a generator block share its
// streams), 4 n d multiply-adds, five block-wide dot products, three block barriers.  CUDA cores
// only: bound by the FP32 multiply-add rate (4 n d per row and draw).
#include "common.cuh"

namespace bsp {

constexpr int kPrMaxN = 256, kPrMaxD = 64, kPrOps = 5;

__device__ __forceinline__ float probs_round(float p, int law, float param, uint32_t w) {
  if (law == 1) return p + ((w >> 31) ? param : -param);
  const float t = __fdiv_rn(p, param);
  const float n0 = floorf(t);
  const uint32_t P = __float2uint_rd(__fsub_rn(t, n0) * 4294967296.0f);
  return (n0 + (w < P ? 1.f : 0.f)) * param;
}

// Shared memory of a block: V as [npad][d] (rows beyond n are zero), the forward's rounding of the
// row pq[npad], and the partial sums of h = V^T p_q as [parts][64] (columns beyond d are zero).
struct ProbsSmem {
  int parts, per, npad;
  __host__ __device__ ProbsSmem(int n, int d, int threads) {
    parts = threads / d;
    if (parts > 4) parts = 4;
    if (parts < 1) parts = 1;
    per = ((n + parts - 1) / parts + 3) & ~3;
    npad = parts * per;
  }
  __host__ __device__ size_t floats(int d) const { return (size_t)npad * d + npad + (size_t)parts * kPrMaxD; }
};

// SHARE: n is a multiple of 4, so the four threads of entries 4q .. 4q+3 need words of the same
// generator blocks: each computes the block of one stream and they exchange words by shuffles.
template <bool SHARE>
__global__ void __launch_bounds__(kPrMaxN, 1)
probs_mc_kernel(const float* __restrict__ p_all, const float* __restrict__ V, int n, int d, int law, float param,
                PhiloxKey kq, PhiloxKey ka, PhiloxKey kb, int draw0, int K, float* __restrict__ ds_sum,
                float* __restrict__ ds_sq, float* __restrict__ dV_sum, size_t rows) {
  extern __shared__ __align__(16) float sm[];
  const ProbsSmem lay(n, d, blockDim.x);
  float* Vs = sm;                                  // [npad][d]
  float* pq_s = Vs + (size_t)lay.npad * d;         // [npad]
  float* hp_s = pq_s + lay.npad;                   // [parts][64]
  __shared__ float red[kPrMaxN / 32][5];
  const size_t row = blockIdx.x;
  const int j = threadIdx.x, lane = j & 31, nwarps = (blockDim.x + 31) / 32;
  const bool on = j < n;
  for (int i = threadIdx.x; i < lay.npad * d; i += blockDim.x) Vs[i] = i < n * d ? V[i] : 0.f;
  for (int i = threadIdx.x; i < lay.npad; i += blockDim.x) pq_s[i] = 0.f;
  for (int i = threadIdx.x; i < lay.parts * kPrMaxD; i += blockDim.x) hp_s[i] = 0.f;
  // this thread's row of V stays in registers: dp_j = sum_c V[j][c] h[c]
  float Vr[kPrMaxD];
#pragma unroll
  for (int c = 0; c < kPrMaxD; ++c) Vr[c] = (on && c < d) ? V[(size_t)j * d + c] : 0.f;
  const float p = on ? p_all[row * n + j] : 0.f;
  const size_t e = row * n + (on ? j : 0);
  float acc_s[kPrOps] = {0.f, 0.f, 0.f, 0.f, 0.f}, acc_q[kPrOps] = {0.f, 0.f, 0.f, 0.f, 0.f};
  float acc_vu[kPrMaxD], acc_va[kPrMaxD];
#pragma unroll
  for (int c = 0; c < kPrMaxD; ++c) acc_vu[c] = acc_va[c] = 0.f;
  // the partial sum of h this thread forms: column hc over the entries [i0, i0 + per)
  const bool h_worker = j < lay.parts * d;
  const int hc = j % d, hpart = j / d, i0 = hpart * lay.per;
  // sum_j p_j - 1 in double, once per row (K(a) needs 1^T a - 1 = sum (a - p) + (sum p - 1))
  __shared__ double red_d[kPrMaxN / 32];
  {
    double t = (double)p;
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, o);
    if (lane == 0) red_d[j >> 5] = t;
  }
  __syncthreads();
  float sum_p_m1;
  {
    double t = 0.0;
    for (int w = 0; w < nwarps; ++w) t += red_d[w];
    sum_p_m1 = (float)(t - 1.0);
  }
  for (int k = draw0; k < draw0 + K; ++k) {
    uint32_t wq, wa, wb;
    if (SHARE) {
      const int pos = j & 3;
      const uint64_t q = (row * (size_t)n + (size_t)j) >> 2;             // the same for the four threads of a group
      const uint32_t c3 = (kq.c3 & ~0xFFu) | (uint32_t)pos;               // streams 0, 1, 2 (3: unused)
      const uint4 w = philox4x32_10((uint32_t)q, (uint32_t)(q >> 32), (uint32_t)k, c3, kq.k0, kq.k1);
      wq = wa = wb = 0u;
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        // round r: every thread sends word (pos + r) & 3 and reads from the group's thread (pos - r) & 3,
        // which is that thread's word `pos`
        const int src = (pos - r) & 3;
        const uint32_t got = __shfl_sync(0xFFFFFFFFu, word_of(w, (uint32_t)((pos + r) & 3)), (lane & ~3) | src);
        if (src == 0) wq = got; else if (src == 1) wa = got; else if (src == 2) wb = got;
      }
    } else {
      wq = word_of(philox_block(kq, e >> 2, (uint32_t)k), (uint32_t)(e & 3));
      wa = word_of(philox_block(ka, e >> 2, (uint32_t)k), (uint32_t)(e & 3));
      wb = word_of(philox_block(kb, e >> 2, (uint32_t)k), (uint32_t)(e & 3));
    }
    float pq = 0.f, a = 0.f, b = 0.f;
    if (on) {
      pq = probs_round(p, law, param, wq);
      a = probs_round(p, law, param, wa);
      b = probs_round(p, law, param, wb);
      pq_s[j] = pq;
    }
    __syncthreads();
    if (h_worker) {                                // h = V^T p_q, in `parts` partial sums per column
      float t0 = 0.f, t1 = 0.f, t2 = 0.f, t3 = 0.f;
      const float* vcol = Vs + (size_t)i0 * d + hc;
      for (int i = 0; i < lay.per; i += 4) {
        const float4 q4 = *reinterpret_cast<const float4*>(pq_s + i0 + i);
        t0 = fmaf(vcol[(size_t)(i + 0) * d], q4.x, t0);
        t1 = fmaf(vcol[(size_t)(i + 1) * d], q4.y, t1);
        t2 = fmaf(vcol[(size_t)(i + 2) * d], q4.z, t2);
        t3 = fmaf(vcol[(size_t)(i + 3) * d], q4.w, t3);
      }
      hp_s[hpart * kPrMaxD + hc] = (t0 + t1) + (t2 + t3);
    }
    __syncthreads();
    // dp = V h and the two gradient-of-V errors (p_hat - p_q) h^T in one walk over the columns
    const float eu = p - pq, ea = a - pq;
    float dp = 0.f;
#pragma unroll
    for (int c0 = 0; c0 < kPrMaxD; c0 += 4) {
      if (c0 < d) {
        float4 h4 = *reinterpret_cast<const float4*>(hp_s + c0);
        for (int pp = 1; pp < lay.parts; ++pp) {
          const float4 g4 = *reinterpret_cast<const float4*>(hp_s + pp * kPrMaxD + c0);
          h4.x += g4.x; h4.y += g4.y; h4.z += g4.z; h4.w += g4.w;
        }
        dp = fmaf(Vr[c0], h4.x, dp); dp = fmaf(Vr[c0 + 1], h4.y, dp);
        dp = fmaf(Vr[c0 + 2], h4.z, dp); dp = fmaf(Vr[c0 + 3], h4.w, dp);
        acc_vu[c0] = fmaf(eu, h4.x, acc_vu[c0]); acc_vu[c0 + 1] = fmaf(eu, h4.y, acc_vu[c0 + 1]);
        acc_vu[c0 + 2] = fmaf(eu, h4.z, acc_vu[c0 + 2]); acc_vu[c0 + 3] = fmaf(eu, h4.w, acc_vu[c0 + 3]);
        acc_va[c0] = fmaf(ea, h4.x, acc_va[c0]); acc_va[c0 + 1] = fmaf(ea, h4.y, acc_va[c0 + 1]);
        acc_va[c0 + 2] = fmaf(ea, h4.z, acc_va[c0 + 2]); acc_va[c0 + 3] = fmaf(ea, h4.w, acc_va[c0 + 3]);
      }
    }
    // the block-wide sums the operators need, taken on the differences to p so that no operator's
    // error is formed as a small difference of large terms:
    //   s0 = p.dp, Dq = (pq - p).dp, Da = (a - p).dp, Db = (b - p).dp, Sa = sum (a - p)
    const float dq = pq - p, da = a - p, db = b - p;
    float dots[5] = {p * dp, dq * dp, da * dp, db * dp, da};
#pragma unroll
    for (int i = 0; i < 5; ++i) dots[i] = warp_sum(dots[i]);
    if (lane == 0)
      for (int i = 0; i < 5; ++i) red[j >> 5][i] = dots[i];
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 5; ++i) {
      float t = 0.f;
      for (int w = 0; w < nwarps; ++w) t += red[w][i];
      dots[i] = t;
    }
    if (on) {
      // with J(x) dp = x o dp - x (x.dp) and x = p + dx:  (J(x) - J(p)) dp = dx (dp - s0) - x (dx.dp)
      const float c = dp - dots[0];
      float err[kPrOps];
      err[0] = dq * c - pq * dots[1];                                            // J(p_q)
      err[1] = da * c - a * dots[2];                                             // J(a)
      err[2] = a * (dots[4] + sum_p_m1) * dp + err[1];                           // K(a): + a (1^T a - 1) dp
      err[3] = 0.5f * ((da + db) * c - (a * dots[3] + b * dots[2]));             // J2(a, b)
      err[4] = 0.5f * ((dq + db) * c - (pq * dots[3] + b * dots[1]));            // J2(p_q, b)
#pragma unroll
      for (int i = 0; i < kPrOps; ++i) { acc_s[i] += err[i]; acc_q[i] = fmaf(err[i], err[i], acc_q[i]); }
    }
    // red[] and pq_s are written again only after the next draw's first barrier, hp_s after its second
  }
  if (!on) return;
#pragma unroll
  for (int i = 0; i < kPrOps; ++i) {
    ds_sum[((size_t)i * rows + row) * n + j] = acc_s[i];
    if (ds_sq) ds_sq[((size_t)i * rows + row) * n + j] = acc_q[i];
  }
  float* o_u = dV_sum + (((size_t)0 * rows + row) * n + j) * d;
  float* o_a = dV_sum + (((size_t)1 * rows + row) * n + j) * d;
  if ((d & 3) == 0) {
#pragma unroll
    for (int c = 0; c < kPrMaxD; c += 4)
      if (c < d) {
        *reinterpret_cast<float4*>(o_u + c) = make_float4(acc_vu[c], acc_vu[c + 1], acc_vu[c + 2], acc_vu[c + 3]);
        *reinterpret_cast<float4*>(o_a + c) = make_float4(acc_va[c], acc_va[c + 1], acc_va[c + 2], acc_va[c + 3]);
      }
  } else {
#pragma unroll
    for (int c = 0; c < kPrMaxD; ++c)
      if (c < d) { o_u[c] = acc_vu[c]; o_a[c] = acc_va[c]; }
  }
}

// The same sums for rows of 128 entries and 64 value columns (an attention key block at head width 64),
// eight draws at a time: 256 threads, one warp per draw.
//   Phase 1 (a warp, its draw): a lane owns four consecutive entries, i.e. exactly one generator block
//   per stream (no word wasted).  An entry's grid position is found once per row; a draw is a
//   comparison.  h = V^T p_q with the lane owning two columns (V row-major in shared memory, p_q
//   broadcast), dp = V h with the lane's four entries read from a transposed copy of V (one 16-byte
//   load per column).  The five dot products are warp sums.  Errors, p - p_q, a - p_q and h go to
//   shared memory.
//   Phase 2 (the block): thread (entry j, column half) owns 2 x 32 sums of the gradient-of-V errors and
//   the sums of two or three operators' errors of its entry, and adds the eight draws to them.
constexpr int kPfN = 128, kPfD = 64, kPfDraws = 8, kPfThreads = 256;
constexpr size_t kPfSmemFloats = (size_t)2 * kPfN * kPfD + kPfDraws * kPfN /*pq*/ + kPfDraws * kPfD /*h*/ +
                                 2 * kPfDraws * kPfN /*eu, ea*/ + (size_t)kPfDraws * kPrOps * kPfN /*err*/;

__global__ void __launch_bounds__(kPfThreads, 2)
probs_mc_128x64_kernel(const float* __restrict__ p_all, const float* __restrict__ V, int law, float param,
                       PhiloxKey kq, int draw0, int K, float* __restrict__ ds_sum, float* __restrict__ ds_sq,
                       float* __restrict__ dV_sum, size_t rows) {
  extern __shared__ __align__(16) float sm[];
  float* Vs = sm;                                   // [128][64]
  float* Vt = Vs + kPfN * kPfD;                     // [64][128]: Vt[c][j] = V[j][c]
  float* pq_s = Vt + kPfN * kPfD;                   // [8][128]
  float* h_s = pq_s + kPfDraws * kPfN;              // [8][64]
  float* eu_s = h_s + kPfDraws * kPfD;              // [8][128]
  float* ea_s = eu_s + kPfDraws * kPfN;             // [8][128]
  float* err_s = ea_s + kPfDraws * kPfN;            // [8][5][128]
  __shared__ double red_d[kPfThreads / 32];
  const size_t row = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
  for (int i = tid; i < kPfN * kPfD; i += kPfThreads) {
    const float v = V[i];
    Vs[i] = v;
    Vt[(i % kPfD) * kPfN + i / kPfD] = v;
  }
  // this lane's four entries (the same for every warp): values, and where they sit on the grid
  const float4 p4 = *reinterpret_cast<const float4*>(p_all + row * kPfN + 4 * lane);
  const float pv[4] = {p4.x, p4.y, p4.z, p4.w};
  float lo[4], hi[4];
  uint32_t thr[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    if (law == 1) {
      lo[e] = pv[e] - param; hi[e] = pv[e] + param; thr[e] = 0x80000000u;     // up iff the word's top bit is set
    } else {
      const float t = __fdiv_rn(pv[e], param);
      const float n0 = floorf(t);
      thr[e] = __float2uint_rd(__fsub_rn(t, n0) * 4294967296.0f);
      lo[e] = n0 * param;
      hi[e] = (n0 + 1.f) * param;
    }
  }
  // sum_j p_j - 1 in double, once per row (threads of warp 0 cover the row)
  {
    double t = w == 0 ? ((double)pv[0] + (double)pv[1]) + ((double)pv[2] + (double)pv[3]) : 0.0;
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, o);
    if (tid == 0) red_d[0] = t;
  }
  __syncthreads();
  const float sum_p_m1 = (float)(red_d[0] - 1.0);
  // phase-2 ownership
  const int j2 = tid & (kPfN - 1), hh = tid >> 7;
  float acc_u[32], acc_a[32], acc_s[3] = {0.f, 0.f, 0.f}, acc_q[3] = {0.f, 0.f, 0.f};
#pragma unroll
  for (int c = 0; c < 32; ++c) acc_u[c] = acc_a[c] = 0.f;
  const uint64_t q = (uint64_t)row * (kPfN / 4) + (uint64_t)lane;       // generator block of this lane's entries
  const uint32_t c3 = kq.c3 & ~0xFFu;

  for (int k0 = 0; k0 < K; k0 += kPfDraws) {
    const int nd = K - k0 < kPfDraws ? K - k0 : kPfDraws;
    if (w < nd) {
      const uint32_t k = (uint32_t)(draw0 + k0 + w);
      const uint4 wq = philox4x32_10((uint32_t)q, (uint32_t)(q >> 32), k, c3 | 0u, kq.k0, kq.k1);
      const uint4 wa = philox4x32_10((uint32_t)q, (uint32_t)(q >> 32), k, c3 | 1u, kq.k0, kq.k1);
      const uint4 wb = philox4x32_10((uint32_t)q, (uint32_t)(q >> 32), k, c3 | 2u, kq.k0, kq.k1);
      const uint32_t uq[4] = {wq.x, wq.y, wq.z, wq.w}, ua[4] = {wa.x, wa.y, wa.z, wa.w}, ub[4] = {wb.x, wb.y, wb.z, wb.w};
      float pq[4], a[4], b[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        // law 0: up iff word < threshold; law 1: up iff the top bit is set, i.e. word >= 2^31
        const bool u0 = law == 1 ? uq[e] >= thr[e] : uq[e] < thr[e];
        const bool u1 = law == 1 ? ua[e] >= thr[e] : ua[e] < thr[e];
        const bool u2 = law == 1 ? ub[e] >= thr[e] : ub[e] < thr[e];
        pq[e] = u0 ? hi[e] : lo[e];
        a[e] = u1 ? hi[e] : lo[e];
        b[e] = u2 ? hi[e] : lo[e];
      }
      float* pqw = pq_s + w * kPfN;
      *reinterpret_cast<float4*>(pqw + 4 * lane) = make_float4(pq[0], pq[1], pq[2], pq[3]);
      __syncwarp();
      // h = V^T p_q: columns 2 lane, 2 lane + 1
      float h0 = 0.f, h1 = 0.f, g0 = 0.f, g1 = 0.f;
#pragma unroll 4
      for (int j = 0; j < kPfN; j += 4) {
        const float4 x = *reinterpret_cast<const float4*>(pqw + j);
        const float2 v0 = *reinterpret_cast<const float2*>(Vs + (j + 0) * kPfD + 2 * lane);
        const float2 v1 = *reinterpret_cast<const float2*>(Vs + (j + 1) * kPfD + 2 * lane);
        const float2 v2 = *reinterpret_cast<const float2*>(Vs + (j + 2) * kPfD + 2 * lane);
        const float2 v3 = *reinterpret_cast<const float2*>(Vs + (j + 3) * kPfD + 2 * lane);
        h0 = fmaf(v0.x, x.x, h0); h1 = fmaf(v0.y, x.x, h1);
        g0 = fmaf(v1.x, x.y, g0); g1 = fmaf(v1.y, x.y, g1);
        h0 = fmaf(v2.x, x.z, h0); h1 = fmaf(v2.y, x.z, h1);
        g0 = fmaf(v3.x, x.w, g0); g1 = fmaf(v3.y, x.w, g1);
      }
      float* hw = h_s + w * kPfD;
      *reinterpret_cast<float2*>(hw + 2 * lane) = make_float2(h0 + g0, h1 + g1);
      __syncwarp();
      // dp = V h for the lane's four entries
      float dp[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
      for (int c = 0; c < kPfD; c += 4) {
        const float4 hv = *reinterpret_cast<const float4*>(hw + c);
        const float4 t0 = *reinterpret_cast<const float4*>(Vt + (c + 0) * kPfN + 4 * lane);
        const float4 t1 = *reinterpret_cast<const float4*>(Vt + (c + 1) * kPfN + 4 * lane);
        const float4 t2 = *reinterpret_cast<const float4*>(Vt + (c + 2) * kPfN + 4 * lane);
        const float4 t3 = *reinterpret_cast<const float4*>(Vt + (c + 3) * kPfN + 4 * lane);
        dp[0] = fmaf(t0.x, hv.x, dp[0]); dp[1] = fmaf(t0.y, hv.x, dp[1]); dp[2] = fmaf(t0.z, hv.x, dp[2]); dp[3] = fmaf(t0.w, hv.x, dp[3]);
        dp[0] = fmaf(t1.x, hv.y, dp[0]); dp[1] = fmaf(t1.y, hv.y, dp[1]); dp[2] = fmaf(t1.z, hv.y, dp[2]); dp[3] = fmaf(t1.w, hv.y, dp[3]);
        dp[0] = fmaf(t2.x, hv.z, dp[0]); dp[1] = fmaf(t2.y, hv.z, dp[1]); dp[2] = fmaf(t2.z, hv.z, dp[2]); dp[3] = fmaf(t2.w, hv.z, dp[3]);
        dp[0] = fmaf(t3.x, hv.w, dp[0]); dp[1] = fmaf(t3.y, hv.w, dp[1]); dp[2] = fmaf(t3.z, hv.w, dp[2]); dp[3] = fmaf(t3.w, hv.w, dp[3]);
      }
      // the sums over the row the operators need (on the differences to p: see probs_mc_kernel)
      float dots[5] = {0.f, 0.f, 0.f, 0.f, 0.f};
      float dq[4], da[4], db[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        dq[e] = pq[e] - pv[e]; da[e] = a[e] - pv[e]; db[e] = b[e] - pv[e];
        dots[0] = fmaf(pv[e], dp[e], dots[0]);
        dots[1] = fmaf(dq[e], dp[e], dots[1]);
        dots[2] = fmaf(da[e], dp[e], dots[2]);
        dots[3] = fmaf(db[e], dp[e], dots[3]);
        dots[4] += da[e];
      }
#pragma unroll
      for (int i = 0; i < 5; ++i) dots[i] = warp_sum(dots[i]);
      float er[kPrOps][4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float c = dp[e] - dots[0];
        er[0][e] = dq[e] * c - pq[e] * dots[1];
        er[1][e] = da[e] * c - a[e] * dots[2];
        er[2][e] = a[e] * (dots[4] + sum_p_m1) * dp[e] + er[1][e];
        er[3][e] = 0.5f * ((da[e] + db[e]) * c - (a[e] * dots[3] + b[e] * dots[2]));
        er[4][e] = 0.5f * ((dq[e] + db[e]) * c - (pq[e] * dots[3] + b[e] * dots[1]));
      }
      *reinterpret_cast<float4*>(eu_s + w * kPfN + 4 * lane) = make_float4(-dq[0], -dq[1], -dq[2], -dq[3]);   // p - p_q
      *reinterpret_cast<float4*>(ea_s + w * kPfN + 4 * lane) =
          make_float4(a[0] - pq[0], a[1] - pq[1], a[2] - pq[2], a[3] - pq[3]);
#pragma unroll
      for (int op = 0; op < kPrOps; ++op)
        *reinterpret_cast<float4*>(err_s + ((size_t)w * kPrOps + op) * kPfN + 4 * lane) =
            make_float4(er[op][0], er[op][1], er[op][2], er[op][3]);
    }
    __syncthreads();
    // phase 2
    for (int d8 = 0; d8 < nd; ++d8) {
      const float eu = eu_s[d8 * kPfN + j2], ea = ea_s[d8 * kPfN + j2];
      const float* hd = h_s + d8 * kPfD + 32 * hh;
#pragma unroll
      for (int c = 0; c < 32; c += 4) {
        const float4 hv = *reinterpret_cast<const float4*>(hd + c);
        acc_u[c] = fmaf(eu, hv.x, acc_u[c]); acc_u[c + 1] = fmaf(eu, hv.y, acc_u[c + 1]);
        acc_u[c + 2] = fmaf(eu, hv.z, acc_u[c + 2]); acc_u[c + 3] = fmaf(eu, hv.w, acc_u[c + 3]);
        acc_a[c] = fmaf(ea, hv.x, acc_a[c]); acc_a[c + 1] = fmaf(ea, hv.y, acc_a[c + 1]);
        acc_a[c + 2] = fmaf(ea, hv.z, acc_a[c + 2]); acc_a[c + 3] = fmaf(ea, hv.w, acc_a[c + 3]);
      }
      // operators 0, 1, 2 in the first column half's threads, 3 and 4 in the second's
#pragma unroll
      for (int i = 0; i < 3; ++i) {
        const int op = hh == 0 ? i : 3 + i;
        if (op < kPrOps) {
          const float v = err_s[((size_t)d8 * kPrOps + op) * kPfN + j2];
          acc_s[i] += v;
          acc_q[i] = fmaf(v, v, acc_q[i]);
        }
      }
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 3; ++i) {
    const int op = hh == 0 ? i : 3 + i;
    if (op < kPrOps) {
      ds_sum[((size_t)op * rows + row) * kPfN + j2] = acc_s[i];
      if (ds_sq) ds_sq[((size_t)op * rows + row) * kPfN + j2] = acc_q[i];
    }
  }
  float* o_u = dV_sum + (((size_t)0 * rows + row) * kPfN + j2) * kPfD + 32 * hh;
  float* o_a = dV_sum + (((size_t)1 * rows + row) * kPfN + j2) * kPfD + 32 * hh;
#pragma unroll
  for (int c = 0; c < 32; c += 4) {
    *reinterpret_cast<float4*>(o_u + c) = make_float4(acc_u[c], acc_u[c + 1], acc_u[c + 2], acc_u[c + 3]);
    *reinterpret_cast<float4*>(o_a + c) = make_float4(acc_a[c], acc_a[c + 1], acc_a[c + 2], acc_a[c + 3]);
  }
}

}  // namespace bsp

using namespace bsp;

extern "C" {

int bsp_probs_mc(const float* p, const float* V, int64_t rows, int n, int d, int law, float param, uint64_t seed,
                 uint32_t tensor_id, int draw0, int K, float* ds_sum, float* ds_sq, float* dV_sum, void* stream) {
  if (!p || !V || !ds_sum || !dV_sum || rows < 0 || n <= 0 || d <= 0 || K < 0 || draw0 < 0 || (law != 0 && law != 1) ||
      !(param > 0.f) || tensor_id >= (1u << 24))
    return BSP_ERR_ARG;
  if (n > kPrMaxN || d > kPrMaxD || d > n) return BSP_ERR_UNSUPPORTED;
  if (rows == 0) return BSP_OK;
  bsp_key_t k;
  k.seed = seed; k.tensor_id = tensor_id; k.draw = 0; k.reserved = 0;
  k.stream = 0; const PhiloxKey kq = make_key(k);
  k.stream = 1; const PhiloxKey ka = make_key(k);
  k.stream = 2; const PhiloxKey kb = make_key(k);
  if (n == kPfN && d == kPfD && (reinterpret_cast<uintptr_t>(p) & 15u) == 0 && (reinterpret_cast<uintptr_t>(dV_sum) & 15u) == 0) {
    const size_t smem_f = kPfSmemFloats * sizeof(float);
    BSP_CHECK_CUDA(cudaFuncSetAttribute(probs_mc_128x64_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_f));
    probs_mc_128x64_kernel<<<(unsigned)rows, kPfThreads, smem_f, (cudaStream_t)stream>>>(p, V, law, param, kq, draw0, K, ds_sum,
                                                                                      ds_sq, dV_sum, (size_t)rows);
    BSP_LAUNCH_CHECK();
    return BSP_OK;
  }
  const int threads = (n + 31) / 32 * 32;
  const ProbsSmem lay(n, d, threads);
  const size_t smem = lay.floats(d) * sizeof(float);
  const bool share = (n & 3) == 0;
  auto kern = share ? probs_mc_kernel<true> : probs_mc_kernel<false>;
  if (smem > 48 * 1024)
    BSP_CHECK_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  kern<<<(unsigned)rows, threads, smem, (cudaStream_t)stream>>>(p, V, n, d, law, param, kq, ka, kb, draw0, K, ds_sum, ds_sq,
                                                               dV_sum, (size_t)rows);
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

}  // extern "C"
