// Monte-Carlo statistics and the host-side orchestration of the per-use check.
#include <math.h>
#include <string.h>

#include <atomic>
#include <vector>

#include "common.cuh"
#include "mc_stats.cuh"
#include "tc.cuh"

namespace bsp {

static std::atomic<unsigned long long> g_launches{0};
void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }
static std::atomic<unsigned long long> g_d2h_bytes{0};
void count_d2h(size_t bytes) { g_d2h_bytes.fetch_add(bytes, std::memory_order_relaxed); }


__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}
__device__ __forceinline__ double warp_max_d(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
  return v;
}

// Per element: err = mean - g*; fresh: mean - g* = S1/K, M2 = S2 - S1^2/K, se^2 = M2/(K-1)/K,
// z = err/se.  An element whose draws all coincide (no variance: the read is deterministic there,
// e.g. every entry it touches already lies on the grid) is judged as a deterministic read: z = 0
// when |err| <= det_tol |g*|, else +-infinity.  M2 below the resolution of the FP32 sums (1e-6 of
// S2) counts as no variance.  Block partials in double, summed on the host in block order.
__global__ void __launch_bounds__(256)
mc_stats_kernel(const float* __restrict__ g_ref, const float* __restrict__ g, const float* __restrict__ S2,
                int64_t n, int K, int fresh, float det_tol, double* __restrict__ partials) {
  // Per-element arithmetic in FP32 (M2 = S2 - S1^2/K as one fused multiply-add), per-thread partial
  // sums in FP32 over the few hundred elements a thread visits, everything above that in double:
  // FP64 division and square root per element would make this pass compute-bound.
  float f_err2 = 0.f, f_ref2 = 0.f, f_se2 = 0.f, f_z2 = 0.f, f_zs = 0.f, f_zmax = 0.f, f_cnt = 0.f;
  const float invK = 1.0f / (float)K;
  const float invKK = fresh ? 1.0f / ((float)(K - 1) * (float)K) : 0.f;
  auto one = [&](float r, float a, float s2) {
    f_ref2 = fmaf(r, r, f_ref2);
    if (!fresh) {
      const float e = a - r;
      f_err2 = fmaf(e, e, f_err2);
    } else {
      const float e = a * invK;
      float m2 = fmaxf(fmaf(-a, e, s2), 0.f);
      if (m2 <= 1e-6f * s2) m2 = 0.f;
      const float se2 = m2 * invKK;
      float z;
      if (se2 > 0.f) z = e * rsqrtf(se2);
      else z = fabsf(e) <= det_tol * fabsf(r) ? 0.f : copysignf(INFINITY, e);
      f_err2 = fmaf(e, e, f_err2);
      f_se2 += se2;
      f_z2 = fmaf(z, z, f_z2);
      f_zs += z;
      f_zmax = fmaxf(f_zmax, fabsf(z));
      f_cnt += fabsf(z) > 3.0f ? 1.f : 0.f;
    }
  };
  const int64_t n4 = n / 4, stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
    const float4 r = __ldg(reinterpret_cast<const float4*>(g_ref) + i);
    const float4 a = __ldg(reinterpret_cast<const float4*>(g) + i);
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    if (fresh) s = __ldg(reinterpret_cast<const float4*>(S2) + i);
    one(r.x, a.x, s.x); one(r.y, a.y, s.y); one(r.z, a.z, s.z); one(r.w, a.w, s.w);
  }
  for (int64_t i = n4 * 4 + (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride)
    one(g_ref[i], g[i], fresh ? S2[i] : 0.f);
  double err2 = f_err2, ref2 = f_ref2, se2s = f_se2, z2 = f_z2, zs = f_zs, zmax = f_zmax, cnt = f_cnt;
  __shared__ double sm[8][kStatFields];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  err2 = warp_sum_d(err2); ref2 = warp_sum_d(ref2); se2s = warp_sum_d(se2s); z2 = warp_sum_d(z2);
  zs = warp_sum_d(zs); zmax = warp_max_d(zmax); cnt = warp_sum_d(cnt);
  if (lane == 0) {
    sm[warp][0] = err2; sm[warp][1] = ref2; sm[warp][2] = se2s; sm[warp][3] = z2;
    sm[warp][4] = zs; sm[warp][5] = zmax; sm[warp][6] = cnt; sm[warp][7] = 0;
  }
  __syncthreads();
  if (threadIdx.x < kStatFields) {
    double a = 0;
    for (int w = 0; w < 8; ++w) a = threadIdx.x == 5 ? fmax(a, sm[w][5]) : a + sm[w][threadIdx.x];
    partials[(size_t)blockIdx.x * kStatFields + threadIdx.x] = a;
  }
}


static const bsp_verdict_rule_t kDefaultRule = {1e-4, 2.0, 3.0, 4.0, 6.0, 0.0};
const bsp_verdict_rule_t* default_rule() { return &kDefaultRule; }
bool rule_valid(const bsp_verdict_rule_t* r) {
  if (!r) return true;
  return r->rel_tol_deterministic >= 0.0 && r->qprime_hold >= 0.0 && r->r_hold >= 0.0 && r->rel_hold >= 0.0 &&
         r->qprime_fail >= r->qprime_hold && r->r_fail >= r->r_hold;
}

// Launches the statistics pass over n elements into one slot of block partials; returns the number
// of blocks whose partials the slot then holds.
int mc_stats_launch(const float* g_ref, const float* g, const float* S2, int64_t n, int K, int fresh,
                    const bsp_verdict_rule_t* rule, double* partials, cudaStream_t st, int* blocks_out) {
  int blocks = (int)((n + 255) / 256);
  if (blocks > kStatBlocks) blocks = kStatBlocks;
  *blocks_out = blocks;
  if (blocks > 0) {
    const float det_tol = (float)(rule ? rule : default_rule())->rel_tol_deterministic;
    mc_stats_kernel<<<blocks, 256, 0, st>>>(g_ref, g, S2, n, K, fresh, det_tol, partials);
    BSP_LAUNCH_CHECK();
  }
  return BSP_OK;
}

// Sums a slot's block partials on the host, in block order, and fills the result of the use.
void mc_stats_finish(const double* host, int blocks, int64_t n, int K, int fresh, const bsp_verdict_rule_t* rule,
                     bsp_use_result_t* result) {
  if (!rule) rule = &kDefaultRule;
  double f[kStatFields] = {0, 0, 0, 0, 0, 0, 0, 0};
  for (int b = 0; b < blocks; ++b)
    for (int j = 0; j < kStatFields; ++j)
      f[j] = j == 5 ? fmax(f[j], host[b * kStatFields + j]) : f[j] + host[b * kStatFields + j];
  const double num = sqrt(f[0]), den = sqrt(f[1]);
  result->n_elements = n;
  result->rel_l2_mean_err = num == 0.0 ? 0.0 : (den > 0.0 ? num / den : INFINITY);
  if (!fresh) {
    result->K = 1;
    result->R = result->Qprime = result->mean_z = result->rms_z = result->max_abs_z = result->frac_abs_z_gt3 = 0.0;
    result->verdict = result->rel_l2_mean_err <= rule->rel_tol_deterministic ? BSP_HOLDS : BSP_FAILS;
    return;
  }
  const double nn = n > 0 ? (double)n : 1.0;
  result->K = K;
  result->R = f[0] == 0.0 ? 0.0 : (f[2] > 0.0 ? f[0] / f[2] : INFINITY);
  result->Qprime = f[3] / nn * (double)(K - 3) / (double)(K - 1);
  result->mean_z = f[4] / nn;
  result->rms_z = sqrt(f[3] / nn);
  result->max_abs_z = f[5];
  result->frac_abs_z_gt3 = f[6] / nn;
  const bool small = rule->rel_hold <= 0.0 || result->rel_l2_mean_err <= rule->rel_hold;
  if (result->Qprime >= rule->qprime_fail || result->R >= rule->r_fail) result->verdict = BSP_FAILS;
  else if (result->Qprime <= rule->qprime_hold && result->R <= rule->r_hold && small) result->verdict = BSP_HOLDS;
  else result->verdict = BSP_UNDECIDED;
}

// Fork / join of the caller's side stream inside one call; whatever path leaves the call, the side
// stream is idle and the events are gone when this goes out of scope.
struct SideWork {
  cudaStream_t side = nullptr;
  cudaEvent_t fork = nullptr, join = nullptr;
  bool launched = false;
  ~SideWork() {
    if (launched) cudaStreamSynchronize(side);
    if (fork) cudaEventDestroy(fork);
    if (join) cudaEventDestroy(join);
  }
};

struct Bump {
  char* base;
  size_t off;
  void* take(size_t bytes) {
    void* p = base ? base + off : nullptr;
    off += round_up(bytes ? bytes : 1, 256);
    return p;
  }
};

// Draws per re-round + contraction launch pair: as many as fit the code buffer (1 GiB unless the
// caller gives a budget), balanced so that the chunks are of near-equal size.
static int draw_chunk(int64_t C, int64_t ld_t, int K, size_t budget) {
  const int64_t per = C * ld_t;
  const int64_t room = budget ? (int64_t)budget : ((int64_t)1 << 30);
  int64_t fit = room / (per > 0 ? per : 1);
  if (fit < 1) fit = 1;
  if (fit >= K) return K > 0 ? K : 1;
  const int64_t nchunks = (K + fit - 1) / fit;
  return (int)((K + nchunks - 1) / nchunks);
}

struct CheckBuffers {
  float *rstd, *mean, *amax_u, *scale_u, *amax_dy, *scale_dy;
  uint8_t *u_codes, *u_codes_t, *fresh_t, *dy_codes, *dy_codes_t;
  uint16_t* u_bf16_t;
  void* du;
  float *dg_ref, *db_ref, *dg_pol, *S1g, *S2g, *dx;
  float *dW_ref, *dW_pol, *S2w;
  void *ws_bwd, *ws_gain, *ws_wgrad, *ws_dgrad, *ws_stats;
  size_t b_bwd, b_gain, b_wgrad, b_dgrad, b_stats;
  int64_t ld_t;
};

static size_t carve(const bsp_norm_linear_desc_t* op, int K, char* base, CheckBuffers* cb) {
  Bump b{base, 0};
  const size_t T = (size_t)op->T, C = (size_t)op->C, O = (size_t)op->O;
  const size_t ld_t = round_up(T, 16);
  const size_t eb = op->dtype == BSP_BF16 ? 2 : 4;
  CheckBuffers c;
  memset(&c, 0, sizeof(c));
  c.ld_t = (int64_t)ld_t;
  c.rstd = (float*)b.take(T * 4); c.mean = (float*)b.take(T * 4);
  c.amax_u = (float*)b.take(4); c.scale_u = (float*)b.take(4);
  c.amax_dy = (float*)b.take(4); c.scale_dy = (float*)b.take(4);
  c.u_codes = (uint8_t*)b.take(T * C); c.u_codes_t = (uint8_t*)b.take(C * ld_t);
  c.fresh_t = (uint8_t*)b.take(C * ld_t * (size_t)draw_chunk((int64_t)C, (int64_t)ld_t, K > 0 ? K : 1, op->draw_buffer_bytes));
  c.dy_codes = (uint8_t*)b.take(T * O); c.dy_codes_t = (uint8_t*)b.take(O * ld_t);
  c.u_bf16_t = (uint16_t*)b.take(C * ld_t * 2);
  c.du = b.take(T * C * eb);
  c.dg_ref = (float*)b.take(C * 4); c.db_ref = (float*)b.take(C * 4); c.dg_pol = (float*)b.take(C * 4);
  c.S1g = (float*)b.take(C * 4); c.S2g = (float*)b.take(C * 4);
  c.dx = (float*)b.take(T * C * 4);
  c.dW_ref = (float*)b.take(O * C * 4); c.dW_pol = (float*)b.take(O * C * 4); c.S2w = (float*)b.take(O * C * 4);
  c.b_bwd = bsp_norm_bwd_workspace_bytes(op->T, op->C);
  c.b_gain = norm_gain_mc_workspace(op->T, op->C, K > 0 ? K : 1, true);   // room for either kernel variant
  c.b_wgrad = bsp_linear_wgrad_workspace_bytes(op->T, op->O, op->C, BSP_READ_ORIGINAL);
  c.b_dgrad = bsp_linear_dgrad_workspace_bytes(op->T, op->O, op->C);
  c.b_stats = kMaxPendingStats * kStatSlotBytes;
  c.ws_bwd = b.take(c.b_bwd); c.ws_gain = b.take(c.b_gain); c.ws_wgrad = b.take(c.b_wgrad);
  c.ws_dgrad = b.take(c.b_dgrad); c.ws_stats = b.take(c.b_stats);
  if (cb) *cb = c;
  return b.off;
}

// mean = g* + S1/K, var = (S2 - S1^2/K)/(K-1), z = (S1/K)/sqrt(var/K), elementwise.
__global__ void __launch_bounds__(256)
mc_moments_kernel(const float* __restrict__ g_ref, const float* __restrict__ S1, const float* __restrict__ S2, size_t n,
                  int K, float* __restrict__ mean, float* __restrict__ var, float* __restrict__ z) {
  const float invK = 1.0f / (float)K, invK1 = 1.0f / (float)(K - 1);
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
    const float a = S1[i], e = a * invK;
    const float v = fmaxf(fmaf(-a, e, S2[i]), 0.f) * invK1;
    if (mean) mean[i] = g_ref[i] + e;
    if (var) var[i] = v;
    if (z) {
      const float se2 = v * invK;
      z[i] = se2 > 0.f ? e * rsqrtf(se2) : (e == 0.f ? 0.f : copysignf(INFINITY, e));
    }
  }
}

// One warp waits, with the library's bounded wait and the given limit, on a barrier that nothing
// completes; the wait gives up, the status is raised, the kernel returns.
__global__ void bounded_wait_selftest_kernel(uint64_t limit_ns, bsp_diag_t* diag) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  bool ok = true;
  if (threadIdx.x < 32) ok = mbar_wait_limit(smem_u32(&bar), 0, &abort_flag, limit_ns);
  __syncthreads();
  if (threadIdx.x == 0 && (!ok || abort_flag)) atomicMax(&diag->status, (int)BSP_ERR_TIMEOUT);
}


}  // namespace bsp

using namespace bsp;

extern "C" {

const char* bsp_status_string(int status) {
  switch (status) {
    case BSP_OK: return "ok";
    case BSP_ERR_ARG: return "invalid argument";
    case BSP_ERR_ALIGN: return "pointer or leading dimension not 16-byte aligned";
    case BSP_ERR_UNSUPPORTED: return "unsupported shape or option";
    case BSP_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case BSP_ERR_NONFINITE: return "non-finite value met in an input";
    case BSP_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case BSP_ERR_CUDA: return "CUDA runtime or driver call failed";
    case BSP_ERR_TOO_LARGE: return "problem exceeds the fixed scratch capacity of the no-allocation entry point";
    default: return "unknown status";
  }
}

unsigned long long bsp_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }
unsigned long long bsp_d2h_byte_count(void) { return g_d2h_bytes.load(std::memory_order_relaxed); }

size_t bsp_mc_stats_workspace_bytes(int64_t n) {
  (void)n;
  return round_up((size_t)kStatBlocks * kStatFields * sizeof(double), 256);
}

int bsp_mc_stats(const float* g_ref, const float* g, const float* S2, int64_t n, int K, int fresh,
                 const bsp_verdict_rule_t* rule, bsp_use_result_t* result, void* ws, size_t ws_bytes, void* stream) {
  if (!g_ref || !g || !result || n < 0 || (fresh && (!S2 || K < 4)) || !rule_valid(rule)) return BSP_ERR_ARG;
  if (!aligned16(g_ref) || !aligned16(g) || !aligned16(S2)) return BSP_ERR_ALIGN;
  if (!ws || ws_bytes < bsp_mc_stats_workspace_bytes(n) || (reinterpret_cast<uintptr_t>(ws) & 255u))
    return BSP_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  double* partials = reinterpret_cast<double*>(ws);
  int blocks = 0;
  int rc = mc_stats_launch(g_ref, g, S2, n, K, fresh, rule, partials, st, &blocks);
  if (rc != BSP_OK) return rc;
  double host[kStatSlotDoubles];
  if (blocks > 0) {
    BSP_CHECK_CUDA(cudaMemcpyAsync(host, partials, (size_t)blocks * kStatFields * sizeof(double),
                                   cudaMemcpyDeviceToHost, st));
    count_d2h((size_t)blocks * kStatFields * sizeof(double));
  }
  BSP_CHECK_CUDA(cudaStreamSynchronize(st));
  mc_stats_finish(host, blocks, n, K, fresh, rule, result);
  result->informational = 0;
  return BSP_OK;
}

int bsp_mc_moments(const float* g_ref, const float* S1, const float* S2, size_t n, int K, float* mean, float* var,
                   float* z, void* stream) {
  if (!g_ref || !S1 || !S2 || K < 2) return BSP_ERR_ARG;
  if (n == 0 || (!mean && !var && !z)) return BSP_OK;
  const unsigned grid = (unsigned)((n + 255) / 256 < 148 * 16 ? (n + 255) / 256 : 148 * 16);
  mc_moments_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>(g_ref, S1, S2, n, K, mean, var, z);
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

int bsp_selftest_bounded_wait(uint64_t limit_ns, bsp_diag_t* diag, void* stream) {
  if (!diag || limit_ns == 0 || limit_ns > 100000000ull) return BSP_ERR_ARG;
  bounded_wait_selftest_kernel<<<1, 64, 0, (cudaStream_t)stream>>>(limit_ns, diag);
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

size_t bsp_mc_check_workspace_bytes(const bsp_norm_linear_desc_t* op, int K) {
  if (!op || op->T <= 0 || op->C <= 0 || op->O <= 0) return 0;
  return carve(op, K, nullptr, nullptr);
}

int bsp_mc_check_layout(const bsp_norm_linear_desc_t* op, int K, bsp_mc_layout_t* layout) {
  if (!op || !layout || op->T <= 0 || op->C <= 0 || op->O <= 0 || K < 1) return BSP_ERR_ARG;
  CheckBuffers b;
  char* const base = reinterpret_cast<char*>((uintptr_t)4096);      // any non-null base: only differences are used
  carve(op, K, base, &b);
  auto off = [&](const void* p) { return (size_t)(reinterpret_cast<const char*>(p) - base); };
  layout->dgamma_ref = off(b.dg_ref); layout->dbeta_ref = off(b.db_ref); layout->dgamma_forward = off(b.dg_pol);
  layout->dgamma_S1 = off(b.S1g); layout->dgamma_S2 = off(b.S2g);
  layout->dW_ref = off(b.dW_ref); layout->dW_S1 = off(b.dW_pol); layout->dW_S2 = off(b.S2w);
  layout->dx = off(b.dx); layout->rstd = off(b.rstd); layout->mean = off(b.mean); layout->u_codes = off(b.u_codes);
  layout->scale_u = off(b.scale_u); layout->scale_dy = off(b.scale_dy); layout->du = off(b.du);
  return BSP_OK;
}

#define BSP_TRY(expr)            \
  do {                           \
    int _rc = (expr);            \
    if (_rc != BSP_OK) return _rc; \
  } while (0)

int bsp_mc_check(const bsp_norm_linear_desc_t* op, int K, const bsp_verdict_rule_t* rule, bsp_use_result_t* results,
                 int* n_results, void* ws, size_t ws_bytes, bsp_diag_t* diag, void* stream) {
  if (!op || !results || !n_results || !rule_valid(rule)) return BSP_ERR_ARG;
  if (op->T <= 0 || op->C <= 0 || op->O <= 0 || K < 4) return BSP_ERR_ARG;
  if (!op->x || !op->gamma || !op->W || !op->dY || (op->norm_kind == BSP_LAYERNORM && !op->beta)) return BSP_ERR_ARG;
  if (op->norm_kind < 0 || op->norm_kind > 1 || op->dtype < 0 || op->dtype > 1) return BSP_ERR_ARG;
  if (op->C % 16 != 0 || op->O % 16 != 0 || op->C > 8192) return BSP_ERR_UNSUPPORTED;
  if (!ws || ws_bytes < bsp_mc_check_workspace_bytes(op, K) || (reinterpret_cast<uintptr_t>(ws) & 255u))
    return BSP_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  CheckBuffers b;
  carve(op, K, reinterpret_cast<char*>(ws), &b);
  const int64_t T = op->T, C = op->C, O = op->O;
  const int dt = op->dtype;
  *n_results = 0;

  // ---- once per call: statistics, scale, forward store, incoming gradient, du
  BSP_TRY(bsp_norm_stats(op->norm_kind, op->x, dt, T, C, op->gamma, op->beta, op->eps, b.rstd, b.mean, b.amax_u,
                         diag, st));
  BSP_TRY(bsp_scale_from_amax(b.amax_u, 1, op->store_fmt, b.scale_u, st));
  bsp_quant_t qu;
  qu.fmt = op->store_fmt; qu.mode = op->forward_mode; qu.scale = 1.f; qu.scale_dev = b.scale_u;
  bsp_key_t key;
  key.seed = op->seed; key.tensor_id = op->tensor_id; key.stream = BSP_STREAM_FORWARD; key.draw = 0; key.reserved = 0;
  const bool want_wu = (op->policy_mask >> 3) & 1u;
  BSP_TRY(bsp_norm_fwd(op->norm_kind, op->x, dt, T, C, op->gamma, op->beta, b.rstd, b.mean, qu, key, b.u_codes,
                       b.u_codes_t, b.ld_t, nullptr, want_wu ? b.u_bf16_t : nullptr, diag, st));
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
  auto stats = [&](const float* g_ref, const float* g, const float* S2, int64_t n, int Kd, int fresh,
                   bsp_use_result_t* r) -> int { return pend.add(g_ref, g, S2, n, Kd, fresh, r); };
  int nres = 0;
  auto emit = [&](int use, int out, int pol) -> bsp_use_result_t* {
    bsp_use_result_t* r = &results[nres++];
    memset(r, 0, sizeof(*r));
    r->use_id = use; r->output_id = out; r->policy = pol;
    return r;
  };
  // dbeta = sum_t du reads no saved tensor: under every read it is the reference itself
  auto emit_dbeta = [&](int pol) {
    bsp_use_result_t* r = emit(BSP_STREAM_GAIN, BSP_OUT_DBETA, pol);
    if (pol == BSP_READ_FRESH) pend.add_exact_fresh(C, K, r);
    else pend.add(b.db_ref, b.db_ref, nullptr, C, 1, 0, r);
  };

  // When both uses ask for the fresh read and the caller gave a side stream, the K-draw gain kernel
  // runs there beside the first K-draw contraction of the weight use: one is bound by the integer
  // pipes, the other by the tensor pipes, and the thin variant of the gain kernel fits next to the
  // contraction's CTA.
  const bool overlap_gain = op->side_stream && (op->policy_mask & 4u) && ((op->policy_mask >> 3) & 4u);
  SideWork sw;
  bsp_use_result_t* gain_n_result = nullptr;
  bsp_key_t gain_key = key;

  // ---- gain use (reference: the original)
  const uint32_t gain_mask = op->policy_mask & 7u;
  if (gain_mask) {
    key.stream = BSP_STREAM_GAIN;
    BSP_TRY(bsp_norm_bwd(op->norm_kind, op->x, dt, T, C, op->gamma, op->beta, b.rstd, b.mean, b.du, dt,
                         BSP_READ_ORIGINAL, BSP_READ_ORIGINAL, nullptr, qu, key, b.dg_ref, b.db_ref, b.dx, b.ws_bwd,
                         b.b_bwd, diag, st));
    if (gain_mask & 1u) {
      bsp_use_result_t* r = emit(BSP_STREAM_GAIN, BSP_OUT_DGAMMA, BSP_READ_ORIGINAL);
      BSP_TRY(stats(b.dg_ref, b.dg_ref, nullptr, C, 1, 0, r));
      emit_dbeta(BSP_READ_ORIGINAL);
    }
    if (gain_mask & 2u) {
      BSP_TRY(bsp_norm_bwd(op->norm_kind, op->x, dt, T, C, op->gamma, op->beta, b.rstd, b.mean, b.du, dt,
                           BSP_READ_FORWARD, BSP_READ_ORIGINAL, b.u_codes, qu, key, b.dg_pol, nullptr, nullptr,
                           b.ws_bwd, b.b_bwd, diag, st));
      bsp_use_result_t* r = emit(BSP_STREAM_GAIN, BSP_OUT_DGAMMA, BSP_READ_FORWARD);
      BSP_TRY(stats(b.dg_ref, b.dg_pol, nullptr, C, 1, 0, r));
      emit_dbeta(BSP_READ_FORWARD);
    }
    if (gain_mask & 4u) {
      BSP_CHECK_CUDA(cudaMemsetAsync(b.S1g, 0, C * sizeof(float), st));
      BSP_CHECK_CUDA(cudaMemsetAsync(b.S2g, 0, C * sizeof(float), st));
      gain_n_result = emit(BSP_STREAM_GAIN, BSP_OUT_DGAMMA, BSP_READ_FRESH);
      emit_dbeta(BSP_READ_FRESH);
      gain_key = key;
      if (!overlap_gain) {
        BSP_TRY(bsp_norm_gain_mc(op->norm_kind, op->x, dt, T, C, op->gamma, op->beta, b.rstd, b.mean, b.du, dt, qu,
                                 gain_key, 0, K, b.dg_ref, b.S1g, b.S2g, b.ws_gain, b.b_gain, diag, st));
        BSP_TRY(stats(b.dg_ref, b.S1g, b.S2g, C, K, 1, gain_n_result));
      }
    }
  }

  // ---- weight use (reference: the rounded value the layer multiplied)
  const uint32_t w_mask = (op->policy_mask >> 3) & 7u;
  if (w_mask) {
    BSP_TRY(bsp_linear_wgrad(T, O, C, b.dy_codes_t, qdy, BSP_READ_FORWARD, b.u_codes_t, qu, b.ld_t, b.dW_ref, nullptr,
                             nullptr, nullptr, b.ws_wgrad, b.b_wgrad, diag, st));
    if (w_mask & 1u) {
      BSP_TRY(bsp_linear_wgrad(T, O, C, b.dy_codes_t, qdy, BSP_READ_ORIGINAL, b.u_bf16_t, qu, b.ld_t, b.dW_pol,
                               nullptr, nullptr, nullptr, b.ws_wgrad, b.b_wgrad, diag, st));
      bsp_use_result_t* r = emit(BSP_STREAM_WGRAD, BSP_OUT_DW, BSP_READ_ORIGINAL);
      BSP_TRY(stats(b.dW_ref, b.dW_pol, nullptr, O * C, 1, 0, r));
    }
    if (w_mask & 2u) {
      bsp_use_result_t* r = emit(BSP_STREAM_WGRAD, BSP_OUT_DW, BSP_READ_FORWARD);
      BSP_TRY(stats(b.dW_ref, b.dW_ref, nullptr, O * C, 1, 0, r));
    }
    if (w_mask & 4u) {
      float* S1w = b.dW_pol;   // the U result has been reduced already
      BSP_CHECK_CUDA(cudaMemsetAsync(S1w, 0, (size_t)O * C * sizeof(float), st));
      BSP_CHECK_CUDA(cudaMemsetAsync(b.S2w, 0, (size_t)O * C * sizeof(float), st));
      bsp_quant_t qf = qu;
      qf.mode = BSP_ROUND_STOCHASTIC;
      key.stream = BSP_STREAM_WGRAD;
      // draws in chunks: one re-rounding launch writes the chunk's code matrices, one contraction
      // launch walks them with the running sums resident in tensor memory
      const int chunk = draw_chunk(C, b.ld_t, K, op->draw_buffer_bytes);
      key.draw = 0;
      for (int k0 = 0; k0 < K; k0 += chunk) {
        const int nd = (K - k0) < chunk ? (K - k0) : chunk;
        BSP_TRY(bsp_norm_fwd_draws(op->norm_kind, op->x, dt, T, C, op->gamma, op->beta, b.rstd, b.mean, qf, key, k0,
                                   nd, b.fresh_t, b.ld_t, st));
        if (overlap_gain && k0 == 0) {
          // fork: everything the gain kernel reads (du, the statistics, the reference, the cleared
          // sums) has been queued on the main stream before this point
          sw.side = (cudaStream_t)op->side_stream;
          BSP_CHECK_CUDA(cudaEventCreateWithFlags(&sw.fork, cudaEventDisableTiming));
          BSP_CHECK_CUDA(cudaEventCreateWithFlags(&sw.join, cudaEventDisableTiming));
          BSP_CHECK_CUDA(cudaEventRecord(sw.fork, st));
        }
        BSP_TRY(bsp_linear_wgrad_mc(T, O, C, b.dy_codes_t, qdy, b.fresh_t, qf, b.ld_t, nd, b.dW_ref, S1w, b.S2w, diag,
                                    st));
        if (overlap_gain && k0 == 0) {
          // the contraction is queued first, so its CTAs take the SMs first; the gain blocks fill in
          BSP_CHECK_CUDA(cudaStreamWaitEvent(sw.side, sw.fork, 0));
          sw.launched = true;
          BSP_TRY(norm_gain_mc_run(true, op->norm_kind, op->x, dt, T, C, op->gamma, op->beta, b.rstd, b.mean, b.du, dt,
                                   qu, gain_key, 0, K, b.dg_ref, b.S1g, b.S2g, b.ws_gain, b.b_gain, diag, sw.side));
          BSP_CHECK_CUDA(cudaEventRecord(sw.join, sw.side));
        }
      }
      if (overlap_gain) {
        BSP_CHECK_CUDA(cudaStreamWaitEvent(st, sw.join, 0));
        BSP_TRY(stats(b.dg_ref, b.S1g, b.S2g, C, K, 1, gain_n_result));
      }
      bsp_use_result_t* r = emit(BSP_STREAM_WGRAD, BSP_OUT_DW, BSP_READ_FRESH);
      BSP_TRY(stats(b.dW_ref, S1w, b.S2w, O * C, K, 1, r));
    }
  }
  *n_results = nres;
  return pend.flush();
}

}  // extern "C"
