// Rounded attention probabilities as the saved tensor (Appendix "Theory"): one row has probabilities
// p and values V; the forward rounds p to p_q and outputs o = V^T p_q; with L = ||o||^2 / 2 the row's
// incoming gradient is h = o and dp = V h.  The reference computes dV = p_q h^T and ds = J(p) dp,
// J(x) = diag(x) - x x^T.  A policy reads p_hat at the gradient of V and J_hat at the softmax's
// backward: Delta_V = (p_hat - p_q) h^T, Delta_s = (J_hat - J(p)) dp.  This kernel averages those
// errors over the forward's rounding and the new roundings, draw by draw, for many rows at once:
//   Delta_s for J_hat in { J(p_q), J(a), K(a), J2(a, b), J2(p_q, b) }  (a, b: new roundings;
//     K(a) = diag(a 1^T a) - a a^T, J2(a, b) = diag((a + b) / 2) - (a b^T + b a^T) / 2);
//   Delta_V for p_hat in { p, a }.
// One block per row, one thread per entry (n <= 256), V (n x d, d <= 64) in shared memory; per draw
// three generator words per entry, two small dense products (h = V^T p_q, dp = V h) and five
// block-wide dot products.  CUDA cores only: the rows are far too small for tensor tiles.
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

// Sum over the block of up to five values per thread (warp shuffles, then one shared-memory pass).
template <int NV>
__device__ __forceinline__ void block_sums(float (&v)[NV], float (*red)[NV], int nwarps) {
#pragma unroll
  for (int i = 0; i < NV; ++i) v[i] = warp_sum(v[i]);
  __syncthreads();
  if ((threadIdx.x & 31) == 0)
    for (int i = 0; i < NV; ++i) red[threadIdx.x >> 5][i] = v[i];
  __syncthreads();
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    float t = 0.f;
    for (int w = 0; w < nwarps; ++w) t += red[w][i];
    v[i] = t;
  }
}

__global__ void __launch_bounds__(kPrMaxN)
probs_mc_kernel(const float* __restrict__ p_all, const float* __restrict__ V, int n, int d, int law, float param,
                PhiloxKey kq, PhiloxKey ka, PhiloxKey kb, int draw0, int K, float* __restrict__ ds_sum,
                float* __restrict__ ds_sq, float* __restrict__ dV_sum, size_t rows) {
  extern __shared__ float sm[];
  float* Vs = sm;                                  // [n][d]
  float* pq_s = Vs + (size_t)n * d;                // [n]
  float* h_s = pq_s + n;                           // [d]
  __shared__ float red[kPrMaxN / 32][6];
  const size_t row = blockIdx.x;
  const int j = threadIdx.x, nwarps = (blockDim.x + 31) / 32;
  const bool on = j < n;
  for (int i = threadIdx.x; i < n * d; i += blockDim.x) Vs[i] = V[i];
  const float p = on ? p_all[row * n + j] : 0.f;
  const size_t e = row * n + (on ? j : 0);
  float acc_s[kPrOps] = {0.f, 0.f, 0.f, 0.f, 0.f}, acc_q[kPrOps] = {0.f, 0.f, 0.f, 0.f, 0.f};
  float acc_vu[kPrMaxD], acc_va[kPrMaxD];
#pragma unroll
  for (int c = 0; c < kPrMaxD; ++c) acc_vu[c] = acc_va[c] = 0.f;
  __syncthreads();
  for (int k = draw0; k < draw0 + K; ++k) {
    float pq = 0.f, a = 0.f, b = 0.f;
    if (on) {
      pq = probs_round(p, law, param, word_of(philox_block(kq, e >> 2, (uint32_t)k), (uint32_t)(e & 3)));
      a = probs_round(p, law, param, word_of(philox_block(ka, e >> 2, (uint32_t)k), (uint32_t)(e & 3)));
      b = probs_round(p, law, param, word_of(philox_block(kb, e >> 2, (uint32_t)k), (uint32_t)(e & 3)));
    }
    __syncthreads();                               // the previous draw's readers of pq_s / h_s are done
    if (on) pq_s[j] = pq;
    __syncthreads();
    if (j < d) {                                   // h = V^T p_q
      float t = 0.f;
      for (int i = 0; i < n; ++i) t = fmaf(Vs[i * d + j], pq_s[i], t);
      h_s[j] = t;
    }
    __syncthreads();
    float dp = 0.f;                                // dp = V h
    if (on)
      for (int c = 0; c < d; ++c) dp = fmaf(Vs[j * d + c], h_s[c], dp);
    // the dot products the operators need: p.dp, pq.dp, a.dp, b.dp, sum a
    float dots[5] = {p * dp, pq * dp, a * dp, b * dp, a};
    block_sums<5>(dots, reinterpret_cast<float(*)[5]>(&red[0][0]), nwarps);
    if (on) {
      const float ref = p * dp - p * dots[0];                                   // J(p) dp
      float err[kPrOps];
      err[0] = (pq * dp - pq * dots[1]) - ref;                                   // J(p_q)
      err[1] = (a * dp - a * dots[2]) - ref;                                     // J(a)
      err[2] = (a * dots[4] * dp - a * dots[2]) - ref;                           // K(a)
      err[3] = (0.5f * (a + b) * dp - 0.5f * (a * dots[3] + b * dots[2])) - ref; // J2(a, b)
      err[4] = (0.5f * (pq + b) * dp - 0.5f * (pq * dots[3] + b * dots[1])) - ref;   // J2(p_q, b)
#pragma unroll
      for (int i = 0; i < kPrOps; ++i) { acc_s[i] += err[i]; acc_q[i] = fmaf(err[i], err[i], acc_q[i]); }
      const float eu = p - pq, ea = a - pq;
#pragma unroll
      for (int c = 0; c < kPrMaxD; ++c)
        if (c < d) { acc_vu[c] = fmaf(eu, h_s[c], acc_vu[c]); acc_va[c] = fmaf(ea, h_s[c], acc_va[c]); }
    }
  }
  if (!on) return;
#pragma unroll
  for (int i = 0; i < kPrOps; ++i) {
    ds_sum[((size_t)i * rows + row) * n + j] = acc_s[i];
    if (ds_sq) ds_sq[((size_t)i * rows + row) * n + j] = acc_q[i];
  }
#pragma unroll
  for (int c = 0; c < kPrMaxD; ++c)
    if (c < d) {
      dV_sum[(((size_t)0 * rows + row) * n + j) * d + c] = acc_vu[c];
      dV_sum[(((size_t)1 * rows + row) * n + j) * d + c] = acc_va[c];
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
  const int threads = (n + 31) / 32 * 32;
  const size_t smem = ((size_t)n * d + n + d) * sizeof(float);
  if (smem > 48 * 1024)
    BSP_CHECK_CUDA(cudaFuncSetAttribute(probs_mc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  probs_mc_kernel<<<(unsigned)rows, threads, smem, (cudaStream_t)stream>>>(p, V, n, d, law, param, kq, ka, kb, draw0, K, ds_sum,
                                                                          ds_sq, dV_sum, (size_t)rows);
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

}  // extern "C"
