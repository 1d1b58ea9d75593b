// Log-softmax backward with a +-eps error injected into its saved output (Appendix "Log-softmax").
//
// The operator's backward takes the incoming gradient h and the saved output S and returns
// h - exp(S) (1^T h).  The saved output is S = l + r, r_j = +-eps independently; under reuse the
// backward reads this S, under an independent copy l + r'.  With p = exp(l), g the returned gradient
// and g* what the operator returns from l with the same h, a trial's statistic is the mean over rows
// and classes of (g_j - g*_j) / p_j, under two losses: the likelihood with a fixed target (h = -e_y)
// and the constructed loss whose incoming gradient is the error itself (h = r).  Six statistics per
// trial (see bsp_lsm_stat_id), then mean, standard error over trials and z.
//
// lsm_prep_kernel: l and p once per row.  lsm_trial_kernel: one block per trial walks the rows; a
// thread owns groups of four classes (one generator block per group and stream), the row's sum of
// errors is a block reduction of sign counts, the backward is evaluated as the operator defines it.
// lsm_reduce_kernel: per-column sums over trials in double.  Generator-bound; no tensor cores.
#include "common.cuh"

namespace bsp {

constexpr int kLsmThreads = 256;
constexpr int kLsmStats = 6, kLsmCols = 8;

__global__ void __launch_bounds__(kLsmThreads)
lsm_prep_kernel(const float* __restrict__ logits, int classes, float* __restrict__ l, float* __restrict__ p) {
  __shared__ float red[kLsmThreads / 32];
  __shared__ float bc;
  const size_t row = blockIdx.x;
  const float* x = logits + row * classes;
  float m = -INFINITY;
  for (int j = threadIdx.x; j < classes; j += kLsmThreads) m = fmaxf(m, x[j]);
  m = warp_max(m);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = red[0];
    for (int w = 1; w < kLsmThreads / 32; ++w) t = fmaxf(t, red[w]);
    bc = t;
  }
  __syncthreads();
  m = bc;
  float s = 0.f;
  for (int j = threadIdx.x; j < classes; j += kLsmThreads) s += expf(x[j] - m);
  s = warp_sum(s);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int w = 0; w < kLsmThreads / 32; ++w) t += red[w];
    bc = logf(t);
  }
  __syncthreads();
  const float lz = bc;
  for (int j = threadIdx.x; j < classes; j += kLsmThreads) {
    const float v = (x[j] - m) - lz;
    l[row * classes + j] = v;
    p[row * classes + j] = expf(v);
  }
}

__global__ void __launch_bounds__(kLsmThreads)
lsm_trial_kernel(const float* __restrict__ l, const float* __restrict__ p, const int32_t* __restrict__ target, int rows,
                 int classes, float eps, PhiloxKey key_reuse, PhiloxKey key_copy, float* __restrict__ per_trial) {
  __shared__ int cnt_s[2][kLsmThreads / 32];
  __shared__ float acc_s[kLsmThreads / 32][kLsmStats];
  const uint32_t trial = blockIdx.x;
  const int groups = classes / 4;
  const float inv_c = 1.0f / coshf(eps);
  float acc[kLsmStats] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  for (int row = 0; row < rows; ++row) {
    // signs of this thread's classes (bit e of `sg`: class 4 * group + e of the thread's n-th group)
    uint32_t sg = 0, sg2 = 0;
    int cnt = 0, nb = 0;
    for (int gq = threadIdx.x; gq < groups; gq += kLsmThreads, nb += 4) {
      const uint64_t q = ((uint64_t)row * classes) / 4 + gq;      // classes % 4 == 0: groups never straddle rows
      const uint4 w = philox_block(key_reuse, q, trial), w2 = philox_block(key_copy, q, trial);
      const uint32_t b = (w.x >> 31) | ((w.y >> 31) << 1) | ((w.z >> 31) << 2) | ((w.w >> 31) << 3);
      const uint32_t b2 = (w2.x >> 31) | ((w2.y >> 31) << 1) | ((w2.z >> 31) << 2) | ((w2.w >> 31) << 3);
      sg |= b << nb; sg2 |= b2 << nb;
      cnt += __popc(b);
    }
    // 1^T h of the constructed loss: the sum of the consumed errors over the row
    cnt = __reduce_add_sync(0xFFFFFFFFu, cnt);
    const int buf = row & 1;
    if ((threadIdx.x & 31) == 0) cnt_s[buf][threadIdx.x >> 5] = cnt;
    __syncthreads();
    int total = 0;
#pragma unroll
    for (int w = 0; w < kLsmThreads / 32; ++w) total += cnt_s[buf][w];
    const float sum_r = eps * (float)(2 * total - classes);
    const int y = __ldg(target + row);
    nb = 0;
    for (int gq = threadIdx.x; gq < groups; gq += kLsmThreads, nb += 4) {
      const size_t i0 = (size_t)row * classes + 4 * (size_t)gq;
      const float4 lv = __ldg(reinterpret_cast<const float4*>(l + i0)), pv = __ldg(reinterpret_cast<const float4*>(p + i0));
      const float ls[4] = {lv.x, lv.y, lv.z, lv.w}, ps[4] = {pv.x, pv.y, pv.z, pv.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float r = (sg >> (nb + e)) & 1u ? eps : -eps, r2 = (sg2 >> (nb + e)) & 1u ? eps : -eps;
        const float eS = expf(ls[e] + r), eS2 = expf(ls[e] + r2), pj = ps[e], ipj = 1.0f / pj;
        const float h_lik = (4 * gq + e) == y ? -1.0f : 0.f;
        // the operator: g = h - exp(S) * (1^T h); likelihood: 1^T h = -1; constructed: h = r, 1^T h = sum_r
        const float gs_lik = h_lik + pj, gs_con = r - pj * sum_r;
        acc[0] += ((h_lik + eS) - gs_lik) * ipj;
        acc[1] += ((h_lik + eS2) - gs_lik) * ipj;
        acc[2] += ((r - eS * sum_r) - gs_con) * ipj;
        acc[3] += ((r - eS2 * sum_r) - gs_con) * ipj;
        acc[4] += ((h_lik + eS * inv_c) - gs_lik) * ipj;
        acc[5] += ((r - eS * inv_c * sum_r) - gs_con) * ipj;
      }
    }
  }
#pragma unroll
  for (int i = 0; i < kLsmStats; ++i) acc[i] = warp_sum(acc[i]);
  if ((threadIdx.x & 31) == 0)
    for (int i = 0; i < kLsmStats; ++i) acc_s[threadIdx.x >> 5][i] = acc[i];
  __syncthreads();
  if (threadIdx.x < kLsmStats) {
    double t = 0.0;
    for (int w = 0; w < kLsmThreads / 32; ++w) t += (double)acc_s[w][threadIdx.x];
    per_trial[(size_t)trial * kLsmStats + threadIdx.x] = (float)(t / ((double)rows * classes));
  }
}

// Column c < 6: the statistic itself; 6 and 7: the paired contrasts reuse - independent (likelihood,
// constructed).  out[2c], out[2c + 1] = sum and sum of squares over trials, in double.
__global__ void __launch_bounds__(256)
lsm_reduce_kernel(const float* __restrict__ per_trial, int trials, double* __restrict__ out) {
  // thread t sums the trials t, t + 256, ... of every column; the 256 partial sums are then added
  // pairwise in a fixed tree, so the result does not depend on scheduling
  __shared__ double sh[2 * kLsmCols][256];
  double s1[kLsmCols], s2[kLsmCols];
#pragma unroll
  for (int c = 0; c < kLsmCols; ++c) s1[c] = s2[c] = 0.0;
  for (int t = threadIdx.x; t < trials; t += 256) {
    const float* v = per_trial + (size_t)t * kLsmStats;
    double x[kLsmCols];
#pragma unroll
    for (int c = 0; c < kLsmStats; ++c) x[c] = (double)v[c];
    x[6] = x[0] - x[1];
    x[7] = x[2] - x[3];
#pragma unroll
    for (int c = 0; c < kLsmCols; ++c) { s1[c] += x[c]; s2[c] += x[c] * x[c]; }
  }
#pragma unroll
  for (int c = 0; c < kLsmCols; ++c) { sh[2 * c][threadIdx.x] = s1[c]; sh[2 * c + 1][threadIdx.x] = s2[c]; }
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if ((int)threadIdx.x < o)
      for (int c = 0; c < 2 * kLsmCols; ++c) sh[c][threadIdx.x] += sh[c][threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x < 2 * kLsmCols) out[threadIdx.x] = sh[threadIdx.x][0];
}

}  // namespace bsp

using namespace bsp;

extern "C" {

size_t bsp_lsm_check_workspace_bytes(int rows, int classes, int trials) {
  if (rows <= 0 || classes <= 0 || trials <= 0) return 0;
  const size_t n = (size_t)rows * classes;
  return 2 * round_up(n * 4, 256) + round_up((size_t)trials * kLsmStats * 4, 256) + 256;
}

int bsp_lsm_check(const float* logits, const int32_t* target, int rows, int classes, float eps, int trials, uint64_t seed,
                  uint32_t tensor_id, float* per_trial, bsp_lsm_stat_t* stats, void* ws, size_t ws_bytes, void* stream) {
  if (!logits || !target || !stats || rows <= 0 || classes <= 0 || trials < 2 || !(eps > 0.f) || tensor_id >= (1u << 24))
    return BSP_ERR_ARG;
  if (classes % 4 != 0 || classes > 32 * 4 * kLsmThreads / 4) return BSP_ERR_UNSUPPORTED;   // <= 32 classes per thread
  if (!aligned16(logits)) return BSP_ERR_ALIGN;
  if (!ws || ws_bytes < bsp_lsm_check_workspace_bytes(rows, classes, trials) || (reinterpret_cast<uintptr_t>(ws) & 255u))
    return BSP_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t n = (size_t)rows * classes;
  char* base = reinterpret_cast<char*>(ws);
  float* l = reinterpret_cast<float*>(base);
  float* p = reinterpret_cast<float*>(base + round_up(n * 4, 256));
  float* pt = reinterpret_cast<float*>(base + 2 * round_up(n * 4, 256));
  double* sums = reinterpret_cast<double*>(base + 2 * round_up(n * 4, 256) + round_up((size_t)trials * kLsmStats * 4, 256));
  if (per_trial) pt = per_trial;
  bsp_key_t k;
  k.seed = seed; k.tensor_id = tensor_id; k.stream = BSP_STREAM_FORWARD; k.draw = 0; k.reserved = 0;
  const PhiloxKey kr = make_key(k);
  k.stream = BSP_STREAM_GAIN;                                       // the independent copy's own stream
  const PhiloxKey kc = make_key(k);
  lsm_prep_kernel<<<(unsigned)rows, kLsmThreads, 0, st>>>(logits, classes, l, p);
  BSP_LAUNCH_CHECK();
  lsm_trial_kernel<<<(unsigned)trials, kLsmThreads, 0, st>>>(l, p, target, rows, classes, eps, kr, kc, pt);
  BSP_LAUNCH_CHECK();
  lsm_reduce_kernel<<<1, 256, 0, st>>>(pt, trials, sums);
  BSP_LAUNCH_CHECK();
  double host[2 * kLsmCols];
  BSP_CHECK_CUDA(cudaMemcpyAsync(host, sums, sizeof(host), cudaMemcpyDeviceToHost, st));
  count_d2h(sizeof(host));
  BSP_CHECK_CUDA(cudaStreamSynchronize(st));
  for (int c = 0; c < kLsmCols; ++c) {
    const double mean = host[2 * c] / trials;
    double var = (host[2 * c + 1] - host[2 * c] * mean) / (trials - 1);
    if (var < 0) var = 0;
    const double se = sqrt(var / trials);
    stats[c].mean = mean;
    stats[c].se = se;
    stats[c].z = se > 0 ? fabs(mean) / se : (mean == 0 ? 0.0 : INFINITY);
  }
  return BSP_OK;
}

}  // extern "C"
