// Averages over the forward's rounding (Appendix "What the checker reads and reports"; Appendix "The
// same dependence in a normalization backward"; the continuation probes of Appendix "The
// normalization store").
//
// Setting: normalisation -> FP8 store u_q = u + r -> y = u_q W^T with the loss ||y||^2 / 2, so that the
// incoming gradients dy = y and du = dy W depend on the rounding the forward consumed.  The forward
// is drawn again and again (generator stream 0, draws 0, 1, 2, ...; pair k = draws 2k, 2k + 1) and
// the following are averaged:
//   * the gain-use error under read R, sum_t (r / gamma) o du, with its split into a mean part
//     sum_t (E r / gamma) o E du and a coupling (the rest); and the same error under a fresh read;
//   * per pair T = <r_a - r_b, du_a - du_b> / 2 and the control <du_a, r_b>;
//   * X = -(r_a - r_b)^T (dy_a - dy_b) / 2, which averages to the weight-use error -r^T dy.
//
// Tensor cores carry the three contractions with no operand rounded below 16 bits: u_q (decoded
// codes) and W are bf16 values, dy is split into hi + lo bf16 terms against [W^T | W^T], and for X
// the difference of two roundings of one value is a single grid step (exact in bf16) against the
// hi + lo split of dy_a - dy_b.  Everything else is streaming FP32 work on CUDA cores.
#include <string.h>

#include <vector>

#include "common.cuh"
#include "gemm.cuh"

namespace bsp {

// r = decode(code) / scale - u; uq (bf16) = decode(code) (exact); sum_r += r (when given).
template <int FMT>
__global__ void __launch_bounds__(256)
cp_resid_kernel(const uint8_t* __restrict__ codes, const float* __restrict__ scale_dev, const float* __restrict__ u,
                size_t n4, float* __restrict__ r, uint16_t* __restrict__ uq, float* __restrict__ sum_r) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n4) return;
  const float inv = __fdiv_rn(1.0f, __ldg(scale_dev));
  float dec[4];
  f8_decode4<FMT>(__ldg(reinterpret_cast<const uint32_t*>(codes) + i), dec);
  const float4 uv = __ldg(reinterpret_cast<const float4*>(u) + i);
  const float4 rv = make_float4(dec[0] * inv - uv.x, dec[1] * inv - uv.y, dec[2] * inv - uv.z, dec[3] * inv - uv.w);
  if (r) reinterpret_cast<float4*>(r)[i] = rv;
  if (uq)
    reinterpret_cast<uint2*>(uq)[i] = make_uint2(float_to_bf16_bits(dec[0]) | (float_to_bf16_bits(dec[1]) << 16),
                                                 float_to_bf16_bits(dec[2]) | (float_to_bf16_bits(dec[3]) << 16));
  if (sum_r) {
    float4 s = reinterpret_cast<float4*>(sum_r)[i];
    s.x += rv.x; s.y += rv.y; s.z += rv.z; s.w += rv.w;
    reinterpret_cast<float4*>(sum_r)[i] = s;
  }
}

// out[row][0 .. n) = hi(in[row]), out[row][n .. 2n) = lo(in[row]) as bf16.  n a multiple of 4: a thread
// takes four consecutive columns of row blockIdx.x.
__global__ void __launch_bounds__(256)
cp_split_rows_kernel(const float* __restrict__ in, int64_t rows, int64_t n, uint16_t* __restrict__ out) {
  const int64_t c = 4 * ((int64_t)blockIdx.y * blockDim.x + threadIdx.x), row = blockIdx.x;
  if (c >= n || row >= rows) return;
  const float4 v = __ldg(reinterpret_cast<const float4*>(in + (size_t)row * n + c));
  const float f[4] = {v.x, v.y, v.z, v.w};
  uint32_t hi[4], lo[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    hi[e] = float_to_bf16_bits(f[e]);
    lo[e] = float_to_bf16_bits(f[e] - bf16_bits_to_float(hi[e]));
  }
  uint16_t* o = out + (size_t)row * 2 * n + c;
  *reinterpret_cast<uint2*>(o) = make_uint2(hi[0] | (hi[1] << 16), hi[2] | (hi[3] << 16));
  *reinterpret_cast<uint2*>(o + n) = make_uint2(lo[0] | (lo[1] << 16), lo[2] | (lo[3] << 16));
}

// Wt2[c][o] = Wt2[c][O + o] = bf16(W[o][c]) and Wb[o][c] = bf16(W[o][c]).
template <int DT>
__global__ void cp_weight_kernel(const void* __restrict__ W, int64_t O, int64_t C, uint16_t* __restrict__ Wb,
                                 uint16_t* __restrict__ Wt2) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (size_t)O * C) return;
  const size_t o = i / C, c = i % C;
  const uint16_t v = (uint16_t)float_to_bf16_bits(load1<DT>(W, i));
  Wb[i] = v;
  Wt2[c * 2 * O + o] = v;
  Wt2[c * 2 * O + O + o] = v;
}

// out[c] += sum_t w[t][c] * du[t][c] / gamma[c], w = r (given) or the residual of `codes` (a fresh
// rounding, formed on the fly); and sum_du += du when given.  Block (x, y) walks the y-th slab of rows
// for 32 columns (eight rows at a time) and writes one partial per column; cp_gain_final_kernel adds
// the slabs in order, so every output has one writer and a fixed order of additions.
constexpr int kCpSlabs = 64;
template <int FMT>
__global__ void __launch_bounds__(256)
cp_gain_kernel(const float* __restrict__ r, const uint8_t* __restrict__ codes, const float* __restrict__ scale_dev,
               const float* __restrict__ u, const float* __restrict__ du, int64_t T, int64_t C, int64_t slab_rows,
               float* __restrict__ partial /* [gridDim.y][C] */, float* __restrict__ sum_du) {
  __shared__ float sm[8][33];
  const int cl = threadIdx.x & 31, rl = threadIdx.x >> 5;
  const int64_t c = (int64_t)blockIdx.x * 32 + cl;
  const float inv = codes ? __fdiv_rn(1.0f, __ldg(scale_dev)) : 0.f;
  const int64_t t_begin = (int64_t)blockIdx.y * slab_rows;
  const int64_t t_end = t_begin + slab_rows < T ? t_begin + slab_rows : T;
  float s = 0.f;
  if (c < C) {
    for (int64_t t = t_begin + rl; t < t_end; t += 8) {
      const size_t i = (size_t)t * C + c;
      const float d = du[i];
      const float w = codes ? f8_decode<FMT>(codes[i]) * inv - u[i] : r[i];
      s = fmaf(w, d, s);
      if (sum_du) sum_du[i] += d;
    }
  }
  sm[rl][cl] = s;
  __syncthreads();
  if (rl == 0 && c < C) {
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) t += sm[w][cl];
    partial[(size_t)blockIdx.y * C + c] = t;
  }
}

__global__ void __launch_bounds__(256)
cp_gain_final_kernel(const float* __restrict__ partial, int nslabs, const float* __restrict__ gamma, int64_t C,
                     float* __restrict__ out, float scale = 1.f, bool accumulate = true) {
  const int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= C) return;
  float t = 0.f;
  for (int y = 0; y < nslabs; ++y) t += partial[(size_t)y * C + c];
  const float v = t * scale / gamma[c];
  out[c] = accumulate ? out[c] + v : v;
}

// partial[b] = { sum (ra - rb)(dua - dub), sum dua * rb } over the block's grid-stride share, in double.
__global__ void __launch_bounds__(256)
cp_dots_kernel(const float* __restrict__ ra, const float* __restrict__ rb, const float* __restrict__ dua,
               const float* __restrict__ dub, size_t n, double* __restrict__ partial) {
  // a thread's share (a few dozen groups of four) in FP32, four chains each; everything above a thread
  // in double (double arithmetic is scarce on this part: the per-element work stays out of it)
  float a4[4] = {0.f, 0.f, 0.f, 0.f}, b4[4] = {0.f, 0.f, 0.f, 0.f};
  const size_t n4 = n / 4;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
    const float4 xa = __ldg(reinterpret_cast<const float4*>(ra) + i), xb = __ldg(reinterpret_cast<const float4*>(rb) + i);
    const float4 ya = __ldg(reinterpret_cast<const float4*>(dua) + i), yb = __ldg(reinterpret_cast<const float4*>(dub) + i);
    a4[0] = fmaf(xa.x - xb.x, ya.x - yb.x, a4[0]); a4[1] = fmaf(xa.y - xb.y, ya.y - yb.y, a4[1]);
    a4[2] = fmaf(xa.z - xb.z, ya.z - yb.z, a4[2]); a4[3] = fmaf(xa.w - xb.w, ya.w - yb.w, a4[3]);
    b4[0] = fmaf(ya.x, xb.x, b4[0]); b4[1] = fmaf(ya.y, xb.y, b4[1]);
    b4[2] = fmaf(ya.z, xb.z, b4[2]); b4[3] = fmaf(ya.w, xb.w, b4[3]);
  }
  double a = ((double)a4[0] + (double)a4[1]) + ((double)a4[2] + (double)a4[3]);
  double b = ((double)b4[0] + (double)b4[1]) + ((double)b4[2] + (double)b4[3]);
  if (blockIdx.x == 0 && threadIdx.x == 0)
    for (size_t i = n4 * 4; i < n; ++i) {                      // a tail of fewer than four
      a += (double)(ra[i] - rb[i]) * (double)(dua[i] - dub[i]);
      b += (double)dua[i] * (double)rb[i];
    }
  __shared__ double sa[256], sb[256];
  sa[threadIdx.x] = a; sb[threadIdx.x] = b;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if ((int)threadIdx.x < o) { sa[threadIdx.x] += sa[threadIdx.x + o]; sb[threadIdx.x] += sb[threadIdx.x + o]; }
    __syncthreads();
  }
  if (threadIdx.x == 0) { partial[2 * blockIdx.x] = sa[0]; partial[2 * blockIdx.x + 1] = sb[0]; }
}
__global__ void cp_dots_final_kernel(const double* __restrict__ partial, int nblocks, double* __restrict__ out) {
  if (threadIdx.x != 0) return;
  double a = 0.0, b = 0.0;
  for (int i = 0; i < nblocks; ++i) { a += partial[2 * i]; b += partial[2 * i + 1]; }
  out[0] = 0.5 * a;
  out[1] = b;
}

// Token-minor operands of X over a 32 x 32 tile.  mode 0: out[c][t] = out[c][ld + t] = bf16(decode(ca) -
// decode(cb)) (the difference of two roundings of one value: zero or one grid step, exact); mode 1:
// out[c][t] = hi, out[c][ld + t] = lo of a[t][c] - b[t][c].  Padding t in [T, ld) zeroed.
template <int FMT>
__global__ void __launch_bounds__(256)
cp_delta_t_kernel(int mode, const uint8_t* __restrict__ ca, const uint8_t* __restrict__ cb, const float* __restrict__ a,
                  const float* __restrict__ b, int64_t T, int64_t N, uint16_t* __restrict__ out, int64_t ld) {
  __shared__ float tile[32][33];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int64_t r0 = (int64_t)blockIdx.y * 32, c0 = (int64_t)blockIdx.x * 32;
  for (int i = ty; i < 32; i += 8) {
    const int64_t t = r0 + i, c = c0 + tx;
    float v = 0.f;
    if (t < T && c < N) {
      const size_t k = (size_t)t * N + c;
      v = mode == 0 ? f8_decode<FMT>(ca[k]) - f8_decode<FMT>(cb[k]) : a[k] - b[k];
    }
    tile[i][tx] = v;
  }
  __syncthreads();
  for (int i = ty; i < 32; i += 8) {
    const int64_t c = c0 + i, t = r0 + tx;
    if (c < N && t < ld) {
      const float v = t < T ? tile[tx][i] : 0.f;
      const uint32_t hi = float_to_bf16_bits(v);
      out[(size_t)c * 2 * ld + t] = (uint16_t)hi;
      out[(size_t)c * 2 * ld + ld + t] = mode == 0 ? (uint16_t)hi : (uint16_t)float_to_bf16_bits(v - bf16_bits_to_float(hi));
    }
  }
}

// out[i] += a[i]; sq[i] += a[i]^2.
__global__ void cp_accumulate_kernel(const float* __restrict__ a, size_t n, float* __restrict__ out, float* __restrict__ sq) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const float v = a[i];
  out[i] += v;
  sq[i] = fmaf(v, v, sq[i]);
}

__global__ void cp_scale_kernel(float* __restrict__ a, size_t n, float f) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) a[i] *= f;
}

constexpr int kCpDotBlocks = 296;

struct CouplingBuffers {
  float *rstd, *mean, *amax, *scale, *u;
  uint8_t* codes[2];
  uint8_t* codes_f;
  uint16_t *uq, *Wb, *Wt2, *ysplit, *dr_t, *dy_t;
  float *r[2], *y[2], *du[2], *sum_r, *sum_du, *xk;
  float *gain_total, *gain_mean_part, *gain_fresh, *X, *X_sq, *gain_partial;
  double *dot_partial, *dots;
  int64_t ld_t;
};

static size_t coupling_carve(const bsp_coupling_desc_t* op, int pairs, char* base, CouplingBuffers* out) {
  size_t off = 0;
  auto take = [&](size_t bytes) -> void* {
    void* p = base ? base + off : nullptr;
    off += round_up(bytes ? bytes : 1, 256);
    return p;
  };
  const size_t T = (size_t)op->T, C = (size_t)op->C, O = (size_t)op->O, ld = round_up(T, 16);
  CouplingBuffers c;
  memset(&c, 0, sizeof(c));
  c.ld_t = (int64_t)ld;
  c.rstd = (float*)take(T * 4); c.mean = (float*)take(T * 4); c.amax = (float*)take(4); c.scale = (float*)take(4);
  c.u = (float*)take(T * C * 4);
  c.codes[0] = (uint8_t*)take(T * C); c.codes[1] = (uint8_t*)take(T * C); c.codes_f = (uint8_t*)take(T * C);
  c.uq = (uint16_t*)take(T * C * 2); c.Wb = (uint16_t*)take(O * C * 2); c.Wt2 = (uint16_t*)take(C * 2 * O * 2);
  c.ysplit = (uint16_t*)take(T * 2 * O * 2); c.dr_t = (uint16_t*)take(C * 2 * ld * 2); c.dy_t = (uint16_t*)take(O * 2 * ld * 2);
  for (int i = 0; i < 2; ++i) { c.r[i] = (float*)take(T * C * 4); c.y[i] = (float*)take(T * O * 4); c.du[i] = (float*)take(T * C * 4); }
  c.sum_r = (float*)take(T * C * 4); c.sum_du = (float*)take(T * C * 4); c.xk = (float*)take(C * O * 4);
  c.gain_total = (float*)take(C * 4); c.gain_mean_part = (float*)take(C * 4); c.gain_fresh = (float*)take(C * 4);
  c.X = (float*)take(C * O * 4); c.X_sq = (float*)take(C * O * 4);
  c.dot_partial = (double*)take(kCpDotBlocks * 2 * sizeof(double));
  c.dots = (double*)take((size_t)(pairs > 0 ? pairs : 1) * 2 * sizeof(double));
  c.gain_partial = (float*)take((size_t)kCpSlabs * C * 4);
  if (out) *out = c;
  return off;
}

}  // namespace bsp

using namespace bsp;

extern "C" {

size_t bsp_coupling_check_workspace_bytes(const bsp_coupling_desc_t* op, int pairs) {
  if (!op || op->T <= 0 || op->C <= 0 || op->O <= 0 || pairs <= 0) return 0;
  return coupling_carve(op, pairs, nullptr, nullptr);
}

int bsp_coupling_layout(const bsp_coupling_desc_t* op, int pairs, bsp_coupling_layout_t* layout) {
  if (!op || !layout || op->T <= 0 || op->C <= 0 || op->O <= 0 || pairs <= 0) return BSP_ERR_ARG;
  CouplingBuffers b;
  char* const base = reinterpret_cast<char*>((uintptr_t)4096);
  coupling_carve(op, pairs, base, &b);
  auto off = [&](const void* p) { return (size_t)(reinterpret_cast<const char*>(p) - base); };
  layout->gain_total = off(b.gain_total); layout->gain_mean_part = off(b.gain_mean_part); layout->gain_fresh = off(b.gain_fresh);
  layout->X = off(b.X); layout->X_sq = off(b.X_sq);
  return BSP_OK;
}

#define BSP_TRY(expr)              \
  do {                             \
    int _rc = (expr);              \
    if (_rc != BSP_OK) return _rc; \
  } while (0)

int bsp_coupling_check(const bsp_coupling_desc_t* op, int pairs, double* T_out, double* control_out, void* ws,
                       size_t ws_bytes, bsp_diag_t* diag, void* stream) {
  if (!op || !T_out || !control_out || pairs <= 0) return BSP_ERR_ARG;
  if (op->T <= 0 || op->C <= 0 || op->O <= 0) return BSP_ERR_ARG;
  if (!op->x || !op->gamma || !op->W || (op->norm_kind == BSP_LAYERNORM && !op->beta)) return BSP_ERR_ARG;
  if (op->norm_kind < 0 || op->norm_kind > 1 || op->dtype < 0 || op->dtype > 1 || op->store_fmt < 0 || op->store_fmt > 1 ||
      op->forward_mode < 0 || op->forward_mode > 1)
    return BSP_ERR_ARG;
  if (op->C % 16 != 0 || op->O % 16 != 0 || op->C > 8192) return BSP_ERR_UNSUPPORTED;
  if (!ws || ws_bytes < bsp_coupling_check_workspace_bytes(op, pairs) || (reinterpret_cast<uintptr_t>(ws) & 255u))
    return BSP_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  CouplingBuffers b;
  coupling_carve(op, pairs, reinterpret_cast<char*>(ws), &b);
  const int64_t T = op->T, C = op->C, O = op->O;
  const size_t n = (size_t)T * C, no = (size_t)T * O;
  const int dt = op->dtype, kind = op->norm_kind, fmt = op->store_fmt;

  BSP_TRY(bsp_norm_stats(kind, op->x, dt, T, C, op->gamma, op->beta, op->eps, b.rstd, b.mean, b.amax, diag, st));
  BSP_TRY(bsp_scale_from_amax(b.amax, 1, fmt, b.scale, st));
  if (dt == BSP_BF16) cp_weight_kernel<BSP_BF16><<<(unsigned)(((size_t)O * C + 255) / 256), 256, 0, st>>>(op->W, O, C, b.Wb, b.Wt2);
  else cp_weight_kernel<BSP_F32><<<(unsigned)(((size_t)O * C + 255) / 256), 256, 0, st>>>(op->W, O, C, b.Wb, b.Wt2);
  BSP_LAUNCH_CHECK();
  for (float* z : {b.sum_r, b.sum_du}) BSP_CHECK_CUDA(cudaMemsetAsync(z, 0, n * 4, st));
  for (float* z : {b.gain_total, b.gain_fresh}) BSP_CHECK_CUDA(cudaMemsetAsync(z, 0, (size_t)C * 4, st));
  for (float* z : {b.X, b.X_sq}) BSP_CHECK_CUDA(cudaMemsetAsync(z, 0, (size_t)C * O * 4, st));

  bsp_quant_t q;
  q.fmt = fmt; q.mode = op->forward_mode; q.scale = 1.f; q.scale_dev = b.scale;
  bsp_quant_t qf = q;
  qf.mode = BSP_ROUND_STOCHASTIC;
  bsp_key_t key;
  key.seed = op->seed; key.tensor_id = op->tensor_id; key.reserved = 0;
  const unsigned g4 = (unsigned)((n / 4 + 255) / 256), gcol = (unsigned)((C + 31) / 32);
  const int64_t slab_rows = ((T + kCpSlabs - 1) / kCpSlabs + 7) & ~(int64_t)7;
  const int nslabs = (int)((T + slab_rows - 1) / slab_rows);
  const dim3 ggain(gcol, (unsigned)nslabs);

  auto forward = [&](int draw, int slot) -> int {
    key.stream = BSP_STREAM_FORWARD; key.draw = (uint32_t)draw;
    BSP_TRY(bsp_norm_fwd(kind, op->x, dt, T, C, op->gamma, op->beta, b.rstd, b.mean, q, key, b.codes[slot], nullptr, 0,
                         draw == 0 ? b.u : nullptr, nullptr, diag, st));
    if (fmt == BSP_E4M3) cp_resid_kernel<BSP_E4M3><<<g4, 256, 0, st>>>(b.codes[slot], b.scale, b.u, n / 4, b.r[slot], b.uq, b.sum_r);
    else cp_resid_kernel<BSP_E5M2><<<g4, 256, 0, st>>>(b.codes[slot], b.scale, b.u, n / 4, b.r[slot], b.uq, b.sum_r);
    BSP_LAUNCH_CHECK();
    // y = u_q W^T (decoded codes times bf16 W, the store's scale in the epilogue); dy = y
    GemmArgs g;
    g.M = T; g.N = O; g.K = C; g.nb = 1; g.fp8 = false;
    g.A = b.uq; g.lda = C; g.B = b.Wb; g.ldb = C; g.b_batch_stride = O * C;
    g.sa = 1.f; g.sa_dev = b.scale; g.sb = 1.f; g.mode = EPI_STORE_F32; g.C = b.y[slot]; g.ldc = O; g.diag = diag;
    BSP_TRY(gemm_run(g, st));
    // du = dy W with dy split into hi + lo against [W^T | W^T]
    cp_split_rows_kernel<<<dim3((unsigned)T, (unsigned)((O / 4 + 255) / 256)), 256, 0, st>>>(b.y[slot], T, O, b.ysplit);
    BSP_LAUNCH_CHECK();
    GemmArgs h;
    h.M = T; h.N = C; h.K = 2 * O; h.nb = 1; h.fp8 = false;
    h.A = b.ysplit; h.lda = 2 * O; h.B = b.Wt2; h.ldb = 2 * O; h.b_batch_stride = C * 2 * O;
    h.sa = 1.f; h.sb = 1.f; h.mode = EPI_STORE_F32; h.C = b.du[slot]; h.ldc = C; h.diag = diag;
    BSP_TRY(gemm_run(h, st));
    // gain-use errors: read R (this forward's own error) and a fresh read (stream 1, same draw)
    if (fmt == BSP_E4M3) cp_gain_kernel<BSP_E4M3><<<ggain, 256, 0, st>>>(b.r[slot], nullptr, b.scale, b.u, b.du[slot], T, C, slab_rows, b.gain_partial, b.sum_du);
    else cp_gain_kernel<BSP_E5M2><<<ggain, 256, 0, st>>>(b.r[slot], nullptr, b.scale, b.u, b.du[slot], T, C, slab_rows, b.gain_partial, b.sum_du);
    cp_gain_final_kernel<<<(unsigned)((C + 255) / 256), 256, 0, st>>>(b.gain_partial, nslabs, op->gamma, C, b.gain_total);
    BSP_LAUNCH_CHECK();
    key.stream = BSP_STREAM_GAIN;
    BSP_TRY(bsp_norm_fwd(kind, op->x, dt, T, C, op->gamma, op->beta, b.rstd, b.mean, qf, key, b.codes_f, nullptr, 0, nullptr,
                         nullptr, diag, st));
    if (fmt == BSP_E4M3) cp_gain_kernel<BSP_E4M3><<<ggain, 256, 0, st>>>(nullptr, b.codes_f, b.scale, b.u, b.du[slot], T, C, slab_rows, b.gain_partial, nullptr);
    else cp_gain_kernel<BSP_E5M2><<<ggain, 256, 0, st>>>(nullptr, b.codes_f, b.scale, b.u, b.du[slot], T, C, slab_rows, b.gain_partial, nullptr);
    cp_gain_final_kernel<<<(unsigned)((C + 255) / 256), 256, 0, st>>>(b.gain_partial, nslabs, op->gamma, C, b.gain_fresh);
    BSP_LAUNCH_CHECK();
    return BSP_OK;
  };

  for (int k = 0; k < pairs; ++k) {
    BSP_TRY(forward(2 * k, 0));
    BSP_TRY(forward(2 * k + 1, 1));
    cp_dots_kernel<<<kCpDotBlocks, 256, 0, st>>>(b.r[0], b.r[1], b.du[0], b.du[1], n, b.dot_partial);
    BSP_LAUNCH_CHECK();
    cp_dots_final_kernel<<<1, 32, 0, st>>>(b.dot_partial, kCpDotBlocks, b.dots + 2 * k);
    BSP_LAUNCH_CHECK();
    // X_k = -(r_a - r_b)^T (dy_a - dy_b) / 2 as [C, O]
    dim3 gr((unsigned)((C + 31) / 32), (unsigned)((b.ld_t + 31) / 32)), gy((unsigned)((O + 31) / 32), (unsigned)((b.ld_t + 31) / 32));
    if (fmt == BSP_E4M3) {
      cp_delta_t_kernel<BSP_E4M3><<<gr, 256, 0, st>>>(0, b.codes[0], b.codes[1], nullptr, nullptr, T, C, b.dr_t, b.ld_t);
      cp_delta_t_kernel<BSP_E4M3><<<gy, 256, 0, st>>>(1, nullptr, nullptr, b.y[0], b.y[1], T, O, b.dy_t, b.ld_t);
    } else {
      cp_delta_t_kernel<BSP_E5M2><<<gr, 256, 0, st>>>(0, b.codes[0], b.codes[1], nullptr, nullptr, T, C, b.dr_t, b.ld_t);
      cp_delta_t_kernel<BSP_E5M2><<<gy, 256, 0, st>>>(1, nullptr, nullptr, b.y[0], b.y[1], T, O, b.dy_t, b.ld_t);
    }
    BSP_LAUNCH_CHECK();
    GemmArgs x;
    x.M = C; x.N = O; x.K = 2 * b.ld_t; x.nb = 1; x.fp8 = false;
    x.A = b.dr_t; x.lda = 2 * b.ld_t; x.B = b.dy_t; x.ldb = 2 * b.ld_t; x.b_batch_stride = O * 2 * b.ld_t;
    x.sa = 1.f; x.sa_dev = b.scale; x.sb = -2.0f;                   // alpha = -1 / (2 scale): the codes' scale and the -1/2
    x.mode = EPI_STORE_F32; x.C = b.xk; x.ldc = O; x.diag = diag;
    BSP_TRY(gemm_run(x, st));
    cp_accumulate_kernel<<<(unsigned)(((size_t)C * O + 255) / 256), 256, 0, st>>>(b.xk, (size_t)C * O, b.X, b.X_sq);
    BSP_LAUNCH_CHECK();
  }
  const float inv_n = 1.0f / (float)(2 * pairs);
  // mean part of the gain error, sum_t (sum_r / n) (sum_du / n) / gamma: the same column sums over row slabs
  cp_gain_kernel<BSP_E4M3><<<ggain, 256, 0, st>>>(b.sum_r, nullptr, b.scale, b.u, b.sum_du, T, C, slab_rows, b.gain_partial, nullptr);
  cp_gain_final_kernel<<<(unsigned)((C + 255) / 256), 256, 0, st>>>(b.gain_partial, nslabs, op->gamma, C, b.gain_mean_part,
                                                                     inv_n * inv_n, false);
  BSP_LAUNCH_CHECK();
  // sums over the forwards / pairs to averages
  cp_scale_kernel<<<(unsigned)((C + 255) / 256), 256, 0, st>>>(b.gain_total, (size_t)C, inv_n);
  cp_scale_kernel<<<(unsigned)((C + 255) / 256), 256, 0, st>>>(b.gain_fresh, (size_t)C, inv_n);
  cp_scale_kernel<<<(unsigned)(((size_t)C * O + 255) / 256), 256, 0, st>>>(b.X, (size_t)C * O, 1.0f / (float)pairs);
  cp_scale_kernel<<<(unsigned)(((size_t)C * O + 255) / 256), 256, 0, st>>>(b.X_sq, (size_t)C * O, 1.0f / (float)pairs);
  BSP_LAUNCH_CHECK();
  std::vector<double> host((size_t)pairs * 2);
  BSP_CHECK_CUDA(cudaMemcpyAsync(host.data(), b.dots, host.size() * sizeof(double), cudaMemcpyDeviceToHost, st));
  count_d2h(host.size() * sizeof(double));
  BSP_CHECK_CUDA(cudaStreamSynchronize(st));
  for (int k = 0; k < pairs; ++k) { T_out[k] = host[2 * k]; control_out[k] = host[2 * k + 1]; }
  return BSP_OK;
}

}  // extern "C"
