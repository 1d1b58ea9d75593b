// Rounding kernels: raw generator words, group amax, scales, flat / grouped / 2-D rounding, and
// the normalisation store's rounding pass (forward store and fresh re-rounding).
//
// All of these are streaming kernels: every element is read once and one byte is written, with
// 128-bit loads and stores; stochastic rounding costs one Philox4x32-10 block per four elements.
#include "common.cuh"
#include "norm_stats_stream.cuh"

namespace bsp {

// ------------------------------------------------------------------------------- philox fill

// Four generator blocks per thread, a warp's 16-byte stores contiguous: the four chains of dependent
// multiplies overlap, which is what the draw kernels also rely on.
__global__ void __launch_bounds__(256)
philox_fill_kernel(PhiloxKey key, size_t n, uint32_t* __restrict__ out) {
  const size_t nq = (n + 3) / 4;
  const size_t q0 = (size_t)blockIdx.x * (blockDim.x * 4) + threadIdx.x;
  uint4 w[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) w[j] = philox_block(key, q0 + (size_t)j * blockDim.x, key.c2);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const size_t q = q0 + (size_t)j * blockDim.x, i = q * 4;
    if (q >= nq) continue;
    if (i + 4 <= n) {
      reinterpret_cast<uint4*>(out)[q] = w[j];
    } else {
      for (uint32_t l = 0; i + l < n; ++l) out[i + l] = word_of(w[j], l);
    }
  }
}

// ------------------------------------------------------------------------------- amax

template <int DT>
__global__ void amax_kernel(const void* __restrict__ x, size_t group_size, uint32_t* __restrict__ amax_bits,
                            bsp_diag_t* diag) {
  // grid: (blocks_per_group, n_groups); amax_bits pre-cleared to 0.
  const size_t g = blockIdx.y;
  const size_t base = g * group_size;
  float m = 0.f;
  uint32_t nf = 0;
  // 16-byte loads, four of them in flight per thread and iteration
  constexpr int EPV = DT == BSP_F32 ? 4 : 8;                 // elements per 16-byte vector
  const size_t nvec = group_size / EPV;
  const bool vec_ok = ((base % EPV) == 0);
  if (vec_ok) {
    const uint4* xv = reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(x) + base * (16 / EPV));
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    auto take = [&](const uint4& r) {
      float a[8];
      if (DT == BSP_F32) {
        a[0] = __uint_as_float(r.x); a[1] = __uint_as_float(r.y); a[2] = __uint_as_float(r.z); a[3] = __uint_as_float(r.w);
      } else {
        a[0] = bf16_bits_to_float(r.x & 0xFFFFu); a[1] = bf16_bits_to_float(r.x >> 16);
        a[2] = bf16_bits_to_float(r.y & 0xFFFFu); a[3] = bf16_bits_to_float(r.y >> 16);
        a[4] = bf16_bits_to_float(r.z & 0xFFFFu); a[5] = bf16_bits_to_float(r.z >> 16);
        a[6] = bf16_bits_to_float(r.w & 0xFFFFu); a[7] = bf16_bits_to_float(r.w >> 16);
      }
#pragma unroll
      for (int j = 0; j < EPV; ++j) {
        const float v = fabsf(a[j]);
        if (v <= 3.4028234663852886e38f) m = fmaxf(m, v); else nf++;
      }
    };
    size_t v = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (; v + 3 * stride < nvec; v += 4 * stride) {
      const uint4 r0 = __ldg(xv + v), r1 = __ldg(xv + v + stride), r2 = __ldg(xv + v + 2 * stride),
                  r3 = __ldg(xv + v + 3 * stride);
      take(r0); take(r1); take(r2); take(r3);
    }
    for (; v < nvec; v += stride) take(__ldg(xv + v));
    for (size_t i = nvec * EPV + (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < group_size;
         i += (size_t)gridDim.x * blockDim.x) {
      const float a = fabsf(load1<DT>(x, base + i));
      if (a <= 3.4028234663852886e38f) m = fmaxf(m, a); else nf++;
    }
  } else {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < group_size; i += (size_t)gridDim.x * blockDim.x) {
      const float a = fabsf(load1<DT>(x, base + i));
      if (a <= 3.4028234663852886e38f) m = fmaxf(m, a); else nf++;
    }
  }
  m = warp_max(m);
  if ((threadIdx.x & 31) == 0) atomicMax(&amax_bits[g], __float_as_uint(m));
  DiagCounters dc; dc.nonfinite = nf;
  diag_flush_warp(diag, dc);
}

__global__ void scale_from_amax_kernel(const float* __restrict__ amax, size_t n, int fmt, float* __restrict__ scale) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const float a = amax[i];
  const float fmax = fmt == BSP_E4M3 ? 448.f : 57344.f;
  float s = 1.f;
  if (a > 0.f && a <= 3.4028234663852886e38f) {
    s = __fdiv_rn(fmax, a);
    if (!(s <= 3.4028234663852886e38f)) s = 1.f;
  }
  scale[i] = s;
}

// ------------------------------------------------------------------------------- flat rounding

// Encodes 16 consecutive values whose first element has logical index e0 (e0 % 4 == 0).
template <int FMT, int MODE>
__device__ __forceinline__ uint4 encode16(const float (&v)[16], const PhiloxKey& key, uint32_t draw, uint64_t e0,
                                          DiagCounters& dc) {
  uint32_t packed[4];
  if (MODE == BSP_ROUND_NEAREST) {
    // nearest-even: the hardware conversion, unless the chunk holds a value at or above the
    // format's maximum (saturation, infinity, NaN), which goes through the counting encoder below
    uint32_t amax_bits = 0;
#pragma unroll
    for (int j = 0; j < 16; ++j) amax_bits = max(amax_bits, __float_as_uint(v[j]) & 0x7FFFFFFFu);
    if (amax_bits < F8<FMT>::FMAX_BITS) {
#pragma unroll
      for (int b = 0; b < 4; ++b)
        packed[b] = f8_encode_rn_pair_inrange<FMT>(v[4 * b], v[4 * b + 1]) |
                    (f8_encode_rn_pair_inrange<FMT>(v[4 * b + 2], v[4 * b + 3]) << 16);
      return make_uint4(packed[0], packed[1], packed[2], packed[3]);
    }
  }
#pragma unroll
  for (int b = 0; b < 4; ++b) {
    uint4 w = make_uint4(0, 0, 0, 0);
    if (MODE == BSP_ROUND_STOCHASTIC) w = philox_block(key, (e0 >> 2) + b, draw);
    const uint32_t c0 = f8_encode<FMT, MODE == BSP_ROUND_STOCHASTIC>(v[4 * b + 0], w.x, dc);
    const uint32_t c1 = f8_encode<FMT, MODE == BSP_ROUND_STOCHASTIC>(v[4 * b + 1], w.y, dc);
    const uint32_t c2 = f8_encode<FMT, MODE == BSP_ROUND_STOCHASTIC>(v[4 * b + 2], w.z, dc);
    const uint32_t c3 = f8_encode<FMT, MODE == BSP_ROUND_STOCHASTIC>(v[4 * b + 3], w.w, dc);
    packed[b] = c0 | (c1 << 8) | (c2 << 16) | (c3 << 24);
  }
  return make_uint4(packed[0], packed[1], packed[2], packed[3]);
}

// One thread per 16 elements; group_size % 16 == 0 and elem_offset % 4 == 0 on this path.
template <int DT, int FMT, int MODE>
__global__ void __launch_bounds__(256)
round_vec_kernel(const void* __restrict__ x, size_t n16, size_t group_size, float scale_val,
                 const float* __restrict__ scales, PhiloxKey key, uint64_t elem_offset,
                 uint8_t* __restrict__ codes, bsp_diag_t* diag) {
  // grid-stride over 16-element chunks, two chunks' loads in flight per thread
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  DiagCounters dc;
  auto finish = [&](size_t t, float (&v)[16]) {
    const size_t i0 = t * 16;
    const float s = scales ? __ldg(scales + (group_size ? i0 / group_size : 0)) : scale_val;
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = __fmul_rn(v[j], s);
    reinterpret_cast<uint4*>(codes)[t] = encode16<FMT, MODE>(v, key, key.c2, elem_offset + i0, dc);
  };
  size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  for (; t + stride < n16; t += 2 * stride) {
    float a[16], b[16];
    load16<DT>(x, t * 16, a);
    load16<DT>(x, (t + stride) * 16, b);
    finish(t, a);
    finish(t + stride, b);
  }
  if (t < n16) {
    float a[16];
    load16<DT>(x, t * 16, a);
    finish(t, a);
  }
  diag_flush_warp(diag, dc);
}

// General path: one thread per element (tails, odd group sizes, unaligned offsets).
template <int DT, int FMT, int MODE>
__global__ void round_scalar_kernel(const void* __restrict__ x, size_t i_begin, size_t n, size_t group_size,
                                    float scale_val, const float* __restrict__ scales, PhiloxKey key,
                                    uint64_t elem_offset, uint8_t* __restrict__ codes, bsp_diag_t* diag) {
  const size_t i = i_begin + (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  DiagCounters dc;
  if (i < n) {
    const float s = scales ? __ldg(scales + (group_size ? i / group_size : 0)) : scale_val;
    const float v = __fmul_rn(load1<DT>(x, i), s);
    uint32_t U = 0;
    if (MODE == BSP_ROUND_STOCHASTIC) {
      const uint64_t e = elem_offset + i;
      U = word_of(philox_block(key, e >> 2, key.c2), (uint32_t)(e & 3));
    }
    codes[i] = (uint8_t)f8_encode<FMT, MODE == BSP_ROUND_STOCHASTIC>(v, U, dc);
  }
  diag_flush_warp(diag, dc);
}

// ------------------------------------------------------------------------------- 2-D tile rounding

// Produces the FP32 value *before scaling* of element (r, c) from the loaded input value.
struct PlainProducer {
  static constexpr bool kCopies = false;   // no FP32 / transposed-bf16 copies of the value on this path
  __device__ __forceinline__ void row(int64_t) {}
  __device__ __forceinline__ float value(float xin, int64_t) const { return xin; }
};

struct NormProducer {
  static constexpr bool kCopies = true;
  int kind;
  const float* __restrict__ gamma;
  const float* __restrict__ beta;
  const float* __restrict__ rstd;
  const float* __restrict__ mean;
  float r_, m_;
  __device__ __forceinline__ void row(int64_t r) {
    r_ = __ldg(rstd + r);
    m_ = kind == BSP_LAYERNORM ? __ldg(mean + r) : 0.f;
  }
  // RMS: fl(fl(x*rstd)*gamma).  LN: fl(fl(fl(fl(x-mean)*rstd)*gamma)+beta).
  __device__ __forceinline__ float value(float xin, int64_t c) const {
    if (kind == BSP_RMSNORM) return __fmul_rn(__fmul_rn(xin, r_), __ldg(gamma + c));
    return __fadd_rn(__fmul_rn(__fmul_rn(__fsub_rn(xin, m_), r_), __ldg(gamma + c)), __ldg(beta + c));
  }
};

constexpr int kTile = 64;   // 64 x 64 tile, 256 threads, 16 consecutive columns per thread

// Requires cols % 16 == 0.  Outputs may each be NULL.
template <class Producer, int DT, int FMT, int MODE>
__global__ void __launch_bounds__(256)
quant_tile_kernel(Producer prod, const void* __restrict__ x, int64_t rows, int64_t cols, float scale_val,
                  const float* __restrict__ scale_dev, PhiloxKey key, uint8_t* __restrict__ codes,
                  uint8_t* __restrict__ codes_t, int64_t ld_t, float* __restrict__ u_f32,
                  uint16_t* __restrict__ u_bf16_t, bsp_diag_t* diag) {
  __shared__ __align__(16) uint8_t s_codes[kTile][kTile + 4];
  __shared__ __align__(16) uint16_t s_bf16[Producer::kCopies ? kTile : 1][kTile + 2];
  const int64_t r0 = (int64_t)blockIdx.y * kTile, c0 = (int64_t)blockIdx.x * kTile;
  const int tr = threadIdx.x >> 2, tc = (threadIdx.x & 3) * 16;
  const int64_t r = r0 + tr, c = c0 + tc;
  const float s = scale_dev ? __ldg(scale_dev) : scale_val;
  DiagCounters dc;
  const bool active = (r < rows) && (c < cols);
  if (active) {
    prod.row(r);
    const size_t i0 = (size_t)r * cols + c;
    float u[16], v[16];
    load16<DT>(x, i0, u);
#pragma unroll
    for (int j = 0; j < 16; ++j) u[j] = prod.value(u[j], c + j);
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = __fmul_rn(u[j], s);
    if (Producer::kCopies && u_f32) {
#pragma unroll
      for (int j = 0; j < 4; ++j)
        reinterpret_cast<float4*>(u_f32 + i0)[j] = make_float4(u[4 * j], u[4 * j + 1], u[4 * j + 2], u[4 * j + 3]);
    }
    if (codes || codes_t) {
      const uint4 pk = encode16<FMT, MODE>(v, key, key.c2, (uint64_t)i0, dc);
      if (codes) *reinterpret_cast<uint4*>(codes + i0) = pk;
      if (codes_t) {
        uint32_t* dst = reinterpret_cast<uint32_t*>(&s_codes[tr][tc]);
        dst[0] = pk.x; dst[1] = pk.y; dst[2] = pk.z; dst[3] = pk.w;
      }
    }
    if (Producer::kCopies && u_bf16_t) {
#pragma unroll
      for (int j = 0; j < 16; ++j) s_bf16[tr][tc + j] = (uint16_t)float_to_bf16_bits(u[j]);
    }
  }
  if (codes_t || (Producer::kCopies && u_bf16_t)) {
    __syncthreads();
    if (codes_t) {
      // transposed codes: a thread takes a 4 x 4 block (rows 4*rb.., columns 4*g..) as four words,
      // transposes it with eight byte permutes, and writes one word to each of its four columns;
      // sixteen neighbouring lanes cover the 64 rows of a column (64 contiguous bytes)
      const int rb = threadIdx.x & 15, g = threadIdx.x >> 4;
      const int64_t rr = r0 + 4 * rb, cg = c0 + 4 * g;
      // rows up to the next multiple of 16 past `rows` are written as zeros (ld_t covers them)
      if (cg < cols && rr < ((rows + 15) & ~(int64_t)15)) {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
          w[i] = rr + i < rows ? *reinterpret_cast<const uint32_t*>(&s_codes[4 * rb + i][4 * g]) : 0u;
        const uint32_t t0 = __byte_perm(w[0], w[1], 0x5140), t1 = __byte_perm(w[2], w[3], 0x5140);
        const uint32_t t2 = __byte_perm(w[0], w[1], 0x7362), t3 = __byte_perm(w[2], w[3], 0x7362);
        const uint32_t o[4] = {__byte_perm(t0, t1, 0x5410), __byte_perm(t0, t1, 0x7632),
                               __byte_perm(t2, t3, 0x5410), __byte_perm(t2, t3, 0x7632)};
#pragma unroll
        for (int i = 0; i < 4; ++i)
          *reinterpret_cast<uint32_t*>(codes_t + (size_t)(cg + i) * ld_t + rr) = o[i];
      }
    }
    // transposed bf16 copy: thread -> column tcol, 16 consecutive rows
    const int tcol = threadIdx.x >> 2, trow = (threadIdx.x & 3) * 16;
    const int64_t cc = c0 + tcol, rr = r0 + trow;
    if (cc < cols && rr < rows) {
      const int nvalid = (int)((rows - rr) < 16 ? (rows - rr) : 16);
      if (Producer::kCopies && u_bf16_t) {
        uint32_t pk[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const uint32_t lo = (2 * j) < nvalid ? s_bf16[trow + 2 * j][tcol] : 0u;
          const uint32_t hi = (2 * j + 1) < nvalid ? s_bf16[trow + 2 * j + 1][tcol] : 0u;
          pk[j] = lo | (hi << 16);
        }
        uint4* dst = reinterpret_cast<uint4*>(u_bf16_t + (size_t)cc * ld_t + rr);
        dst[0] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        dst[1] = make_uint4(pk[4], pk[5], pk[6], pk[7]);
      }
    }
  }
  diag_flush_warp(diag, dc);
}

// Fresh re-roundings of the normalisation output for `ndraws` consecutive draws in one pass: the
// FP32 value of every element is formed once, then rounded stochastically once per draw; only the
// transposed code matrices are written: codes_t[d][c][r], d-th matrix at d * cols * ld_t.
template <int DT, int FMT>
__global__ void __launch_bounds__(256, 3)
reround_draws_kernel(NormProducer prod, const void* __restrict__ x, int64_t rows, int64_t cols, float scale_val,
                     const float* __restrict__ scale_dev, PhiloxKey key, int draw0, int ndraws,
                     uint8_t* __restrict__ codes_t, int64_t ld_t) {
  __shared__ __align__(16) uint8_t s_codes[2][kTile][kTile + 4];
  const int64_t r0 = (int64_t)blockIdx.y * kTile, c0 = (int64_t)blockIdx.x * kTile;
  const int tr = threadIdx.x >> 2, tc = (threadIdx.x & 3) * 16;
  const int64_t r = r0 + tr, c = c0 + tc;
  const float s = scale_dev ? __ldg(scale_dev) : scale_val;
  const bool active = (r < rows) && (c < cols);
  const size_t i0 = (size_t)r * cols + c;
  float v[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) v[j] = 0.f;
  if (active) {
    prod.row(r);
    load16<DT>(x, i0, v);
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = __fmul_rn(prod.value(v[j], c + j), s);
  }
  const int tcol = threadIdx.x >> 2, trow = (threadIdx.x & 3) * 16;
  const int64_t cc = c0 + tcol, rr = r0 + trow;
  const bool wr = cc < cols && rr < rows;
  const int nvalid = wr ? (int)((rows - rr) < 16 ? (rows - rr) : 16) : 0;
  // A fresh rounding of an element is its round-down code plus one exactly when the element's
  // generator word falls below the threshold of f8_sr_threshold: both are fixed across draws, so a
  // draw costs one generator block, four comparisons and four conditional adds per four elements.
  // (A code that can round up is below the format's top code, so the add never carries out of its byte.)
  uint32_t thr[16], lo4[4] = {0u, 0u, 0u, 0u};
  {
    DiagCounters dc;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      thr[j] = f8_sr_threshold<FMT>(v[j]);
      lo4[j >> 2] |= f8_encode<FMT, true>(v[j], 0xFFFFFFFFu, dc) << (8 * (j & 3));
    }
  }
  for (int d = 0; d < ndraws; ++d) {
    const int buf = d & 1;
    if (active) {
      uint32_t pk[4];
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const uint4 w = philox_block(key, ((uint64_t)i0 >> 2) + b, (uint32_t)(draw0 + d));
        uint32_t c4 = lo4[b];
        c4 += w.x < thr[4 * b + 0] ? 0x1u : 0u;
        c4 += w.y < thr[4 * b + 1] ? 0x100u : 0u;
        c4 += w.z < thr[4 * b + 2] ? 0x10000u : 0u;
        c4 += w.w < thr[4 * b + 3] ? 0x1000000u : 0u;
        pk[b] = c4;
      }
      uint32_t* dst = reinterpret_cast<uint32_t*>(&s_codes[buf][tr][tc]);
      dst[0] = pk[0]; dst[1] = pk[1]; dst[2] = pk[2]; dst[3] = pk[3];
    }
    __syncthreads();
    if (wr) {
      uint32_t pk[4] = {0, 0, 0, 0};
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const uint32_t b = j < nvalid ? s_codes[buf][trow + j][tcol] : 0u;
        pk[j >> 2] |= b << (8 * (j & 3));
      }
      *reinterpret_cast<uint4*>(codes_t + ((size_t)d * cols + cc) * ld_t + rr) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
    }
  }
}

// ------------------------------------------------------------------------------- norm statistics

// One warp per row.  RMS: rstd = 1/sqrt(mean x^2 + eps).  LN: mean, biased variance.
// Optionally the largest |u| with u from the same FP32 chain the rounding pass uses.
// Kept lean on purpose: at 2 bytes per element the HBM roofline leaves about ten instructions per
// element, so non-finite inputs are detected once per row (a non-finite sum of squares), not per
// element, and the norm kind is a template parameter.
template <int DT, int kind>
__global__ void __launch_bounds__(256)
norm_stats_kernel(const void* __restrict__ x, int64_t T, int64_t C, const float* __restrict__ gamma,
                  const float* __restrict__ beta, float eps, float* __restrict__ rstd, float* __restrict__ mean,
                  uint32_t* __restrict__ amax_bits, bsp_diag_t* diag) {
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  float amax = 0.f;
  uint32_t nf = 0;
  if (row < T) {
    const size_t base = (size_t)row * C;
    const int64_t nvec = C / 4;
    // the first pass over the row sets the HBM traffic (later passes hit L1): four 16-byte loads in
    // flight per lane.  Quads of four elements are visited in the same order by every pass.
    auto first_pass = [&](auto&& fn) {
      int64_t v = lane;
      for (; v + 96 < nvec; v += 128) {
        const float4 f0 = load4<DT>(x, base + v * 4), f1 = load4<DT>(x, base + (v + 32) * 4),
                     f2 = load4<DT>(x, base + (v + 64) * 4), f3 = load4<DT>(x, base + (v + 96) * 4);
        fn(f0); fn(f1); fn(f2); fn(f3);
      }
      for (; v < nvec; v += 32) fn(load4<DT>(x, base + v * 4));
    };
    float mu = 0.f;
    if (kind == BSP_LAYERNORM) {
      float s = 0.f;
      first_pass([&](const float4& f) { s += (f.x + f.y) + (f.z + f.w); });
      mu = __fdiv_rn(warp_sum(s), (float)C);
    }
    float ss = 0.f;
    first_pass([&](const float4& f) {
      if (kind == BSP_LAYERNORM) {
        const float a = f.x - mu, b = f.y - mu, c = f.z - mu, d = f.w - mu;
        ss += (a * a + b * b) + (c * c + d * d);
      } else {
        ss += (f.x * f.x + f.y * f.y) + (f.z * f.z + f.w * f.w);
      }
    });
    ss = warp_sum(ss);
    if (lane == 0 && !(ss <= 3.4028234663852886e38f)) nf = 1;     // NaN, infinity or overflow in this row
    const float rs = __fdiv_rn(1.0f, __fsqrt_rn(__fadd_rn(__fdiv_rn(ss, (float)C), eps)));
    if (lane == 0) {
      rstd[row] = rs;
      if (mean && kind == BSP_LAYERNORM) mean[row] = mu;
    }
    if (amax_bits) {
      for (int64_t v = lane; v < nvec; v += 32) {
        const float4 f = load4<DT>(x, base + v * 4);
        const float4 g = __ldg(reinterpret_cast<const float4*>(gamma) + v);
        float u0, u1, u2, u3;
        if (kind == BSP_RMSNORM) {
          u0 = __fmul_rn(__fmul_rn(f.x, rs), g.x); u1 = __fmul_rn(__fmul_rn(f.y, rs), g.y);
          u2 = __fmul_rn(__fmul_rn(f.z, rs), g.z); u3 = __fmul_rn(__fmul_rn(f.w, rs), g.w);
        } else {
          const float4 b = __ldg(reinterpret_cast<const float4*>(beta) + v);
          u0 = __fadd_rn(__fmul_rn(__fmul_rn(__fsub_rn(f.x, mu), rs), g.x), b.x);
          u1 = __fadd_rn(__fmul_rn(__fmul_rn(__fsub_rn(f.y, mu), rs), g.y), b.y);
          u2 = __fadd_rn(__fmul_rn(__fmul_rn(__fsub_rn(f.z, mu), rs), g.z), b.z);
          u3 = __fadd_rn(__fmul_rn(__fmul_rn(__fsub_rn(f.w, mu), rs), g.w), b.w);
        }
        // fmaxf drops a NaN operand; an infinite |u| makes amax infinite and the scale falls back to 1
        amax = fmaxf(fmaxf(amax, fabsf(u0)), fmaxf(fabsf(u1), fmaxf(fabsf(u2), fabsf(u3))));
      }
    }
  }
  if (amax_bits) {
    amax = warp_max(amax);
    if (lane == 0 && amax > 0.f) atomicMax(amax_bits, __float_as_uint(amax));
  }
  DiagCounters dc; dc.nonfinite = nf;
  diag_flush_warp(diag, dc);
}

// ------------------------------------------------------------------------------- dispatch helpers

template <class Producer, int DT, int FMT>
static void launch_tile_mode(int mode, dim3 grid, cudaStream_t st, Producer prod, const void* x, int64_t rows,
                             int64_t cols, float scale, const float* scale_dev, PhiloxKey key, uint8_t* codes,
                             uint8_t* codes_t, int64_t ld_t, float* u_f32, uint16_t* u_bf16_t, bsp_diag_t* diag) {
  if (mode == BSP_ROUND_STOCHASTIC)
    quant_tile_kernel<Producer, DT, FMT, BSP_ROUND_STOCHASTIC><<<grid, 256, 0, st>>>(
        prod, x, rows, cols, scale, scale_dev, key, codes, codes_t, ld_t, u_f32, u_bf16_t, diag);
  else
    quant_tile_kernel<Producer, DT, FMT, BSP_ROUND_NEAREST><<<grid, 256, 0, st>>>(
        prod, x, rows, cols, scale, scale_dev, key, codes, codes_t, ld_t, u_f32, u_bf16_t, diag);
}

template <class Producer>
static int launch_tile(int dt, int fmt, int mode, cudaStream_t st, Producer prod, const void* x, int64_t rows,
                       int64_t cols, float scale, const float* scale_dev, PhiloxKey key, uint8_t* codes,
                       uint8_t* codes_t, int64_t ld_t, float* u_f32, uint16_t* u_bf16_t, bsp_diag_t* diag) {
  dim3 grid((unsigned)((cols + kTile - 1) / kTile), (unsigned)((rows + kTile - 1) / kTile));
#define BSP_TILE_CASE(DT, FMT)                                                                              \
  launch_tile_mode<Producer, DT, FMT>(mode, grid, st, prod, x, rows, cols, scale, scale_dev, key, codes,   \
                                      codes_t, ld_t, u_f32, u_bf16_t, diag)
  if (dt == BSP_F32 && fmt == BSP_E4M3) BSP_TILE_CASE(BSP_F32, BSP_E4M3);
  else if (dt == BSP_F32 && fmt == BSP_E5M2) BSP_TILE_CASE(BSP_F32, BSP_E5M2);
  else if (dt == BSP_BF16 && fmt == BSP_E4M3) BSP_TILE_CASE(BSP_BF16, BSP_E4M3);
  else BSP_TILE_CASE(BSP_BF16, BSP_E5M2);
#undef BSP_TILE_CASE
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

template <int DT, int FMT, int MODE>
static int launch_round_flat(const void* x, size_t n, size_t group_size, float scale, const float* scales,
                             PhiloxKey key, uint64_t elem_offset, uint8_t* codes, bsp_diag_t* diag,
                             cudaStream_t st) {
  const bool vec_ok = (elem_offset % 4 == 0) && (group_size == 0 || group_size % 16 == 0);
  size_t n16 = vec_ok ? n / 16 : 0;
  if (n16) {
    const size_t want = (n16 + 511) / 512;                      // two chunks per thread
    const size_t cap = (size_t)kNumSMs * 8;                     // eight 256-thread blocks per SM
    const unsigned blocks = (unsigned)(want < cap ? want : cap);
    round_vec_kernel<DT, FMT, MODE><<<blocks, 256, 0, st>>>(x, n16, group_size, scale, scales, key, elem_offset,
                                                           codes, diag);
    BSP_LAUNCH_CHECK();
  }
  const size_t done = n16 * 16;
  if (done < n) {
    const unsigned blocks = (unsigned)((n - done + 255) / 256);
    round_scalar_kernel<DT, FMT, MODE><<<blocks, 256, 0, st>>>(x, done, n, group_size, scale, scales, key,
                                                              elem_offset, codes, diag);
    BSP_LAUNCH_CHECK();
  }
  return BSP_OK;
}

static int dispatch_round_flat(int dt, int fmt, int mode, const void* x, size_t n, size_t group_size, float scale,
                               const float* scales, PhiloxKey key, uint64_t elem_offset, uint8_t* codes,
                               bsp_diag_t* diag, cudaStream_t st) {
#define BSP_FLAT(DT, FMT, MODE) \
  return launch_round_flat<DT, FMT, MODE>(x, n, group_size, scale, scales, key, elem_offset, codes, diag, st)
  if (dt == BSP_F32) {
    if (fmt == BSP_E4M3) { if (mode) BSP_FLAT(BSP_F32, BSP_E4M3, 1); else BSP_FLAT(BSP_F32, BSP_E4M3, 0); }
    else { if (mode) BSP_FLAT(BSP_F32, BSP_E5M2, 1); else BSP_FLAT(BSP_F32, BSP_E5M2, 0); }
  } else {
    if (fmt == BSP_E4M3) { if (mode) BSP_FLAT(BSP_BF16, BSP_E4M3, 1); else BSP_FLAT(BSP_BF16, BSP_E4M3, 0); }
    else { if (mode) BSP_FLAT(BSP_BF16, BSP_E5M2, 1); else BSP_FLAT(BSP_BF16, BSP_E5M2, 0); }
  }
#undef BSP_FLAT
}

static bool valid_enum(int v, int hi) { return v >= 0 && v <= hi; }

}  // namespace bsp

using namespace bsp;

extern "C" {

int bsp_diag_clear(bsp_diag_t* diag, void* stream) {
  if (!diag) return BSP_ERR_ARG;
  BSP_CHECK_CUDA(cudaMemsetAsync(diag, 0, sizeof(bsp_diag_t), (cudaStream_t)stream));
  return BSP_OK;
}

int bsp_philox_fill(bsp_key_t key, size_t n, uint32_t* out, void* stream) {
  if (!out && n) return BSP_ERR_ARG;
  if (key.tensor_id >= (1u << 24) || key.stream > 255u || key.reserved != 0) return BSP_ERR_ARG;
  if (!aligned16(out)) return BSP_ERR_ALIGN;
  if (n == 0) return BSP_OK;
  const size_t nq = (n + 3) / 4;
  philox_fill_kernel<<<(unsigned)((nq + 1023) / 1024), 256, 0, (cudaStream_t)stream>>>(make_key(key), n, out);
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

int bsp_amax(const void* x, int dt, size_t n_groups, size_t group_size, float* amax, bsp_diag_t* diag,
             void* stream) {
  if (!amax || !valid_enum(dt, 1)) return BSP_ERR_ARG;
  if (n_groups == 0) return BSP_OK;
  if (!x && group_size) return BSP_ERR_ARG;
  if (!aligned16(x)) return BSP_ERR_ALIGN;
  if (n_groups > 65535) return BSP_ERR_UNSUPPORTED;
  cudaStream_t st = (cudaStream_t)stream;
  BSP_CHECK_CUDA(cudaMemsetAsync(amax, 0, n_groups * sizeof(float), st));
  if (group_size == 0) return BSP_OK;
  size_t per = (group_size / 4 + 255) / 256;
  size_t want = (size_t)kNumSMs * 8 / n_groups + 1;
  unsigned bx = (unsigned)(per < want ? (per ? per : 1) : want);
  dim3 grid(bx, (unsigned)n_groups);
  if (dt == BSP_F32) amax_kernel<BSP_F32><<<grid, 256, 0, st>>>(x, group_size, reinterpret_cast<uint32_t*>(amax), diag);
  else amax_kernel<BSP_BF16><<<grid, 256, 0, st>>>(x, group_size, reinterpret_cast<uint32_t*>(amax), diag);
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

int bsp_scale_from_amax(const float* amax, size_t n, int fmt, float* scale, void* stream) {
  if (!amax || !scale || !valid_enum(fmt, 1)) return BSP_ERR_ARG;
  if (n == 0) return BSP_OK;
  scale_from_amax_kernel<<<(unsigned)((n + 255) / 256), 256, 0, (cudaStream_t)stream>>>(amax, n, fmt, scale);
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

int bsp_round(const void* x, int dt, size_t n, bsp_quant_t q, bsp_key_t key, uint64_t elem_offset,
              uint8_t* codes, bsp_diag_t* diag, void* stream) {
  if (!valid_enum(dt, 1) || !valid_enum(q.fmt, 1) || !valid_enum(q.mode, 1)) return BSP_ERR_ARG;
  if (key.tensor_id >= (1u << 24) || key.stream > 255u || key.reserved != 0) return BSP_ERR_ARG;
  if (n == 0) return BSP_OK;
  if (!x || !codes) return BSP_ERR_ARG;
  if (!aligned16(x) || !aligned16(codes)) return BSP_ERR_ALIGN;
  // a device scale is a scale array with group size 0: every element reads entry 0
  return dispatch_round_flat(dt, q.fmt, q.mode, x, n, 0, q.scale, q.scale_dev,
                             make_key(key), elem_offset, codes, diag, (cudaStream_t)stream);
}

int bsp_round_grouped(const void* x, int dt, size_t n_groups, size_t group_size, int fmt, int mode,
                      const float* scales, bsp_key_t key, uint8_t* codes, bsp_diag_t* diag, void* stream) {
  if (!valid_enum(dt, 1) || !valid_enum(fmt, 1) || !valid_enum(mode, 1)) return BSP_ERR_ARG;
  if (key.tensor_id >= (1u << 24) || key.stream > 255u || key.reserved != 0) return BSP_ERR_ARG;
  if (n_groups == 0 || group_size == 0) return BSP_OK;
  if (!x || !codes || !scales) return BSP_ERR_ARG;
  if (!aligned16(x) || !aligned16(codes)) return BSP_ERR_ALIGN;
  return dispatch_round_flat(dt, fmt, mode, x, n_groups * group_size, group_size, 1.f, scales, make_key(key), 0,
                             codes, diag, (cudaStream_t)stream);
}

int bsp_round_2d(const void* x, int dt, int64_t rows, int64_t cols, bsp_quant_t q, bsp_key_t key,
                 uint8_t* codes, uint8_t* codes_t, int64_t ld_t, bsp_diag_t* diag, void* stream) {
  if (!valid_enum(dt, 1) || !valid_enum(q.fmt, 1) || !valid_enum(q.mode, 1)) return BSP_ERR_ARG;
  if (key.tensor_id >= (1u << 24) || key.stream > 255u || key.reserved != 0) return BSP_ERR_ARG;
  if (rows < 0 || cols < 0) return BSP_ERR_ARG;
  if (rows == 0 || cols == 0) return BSP_OK;
  if (!x || (!codes && !codes_t)) return BSP_ERR_ARG;
  if (cols % 16 != 0) return BSP_ERR_UNSUPPORTED;
  if (codes_t && (ld_t < rows || ld_t % 16 != 0)) return BSP_ERR_ALIGN;
  if (!aligned16(x) || !aligned16(codes) || !aligned16(codes_t)) return BSP_ERR_ALIGN;
  return launch_tile(dt, q.fmt, q.mode, (cudaStream_t)stream, PlainProducer(), x, rows, cols, q.scale, q.scale_dev,
                     make_key(key), codes, codes_t, ld_t, nullptr, nullptr, diag);
}

int bsp_norm_stats(int kind, const void* x, int dt, int64_t T, int64_t C, const float* gamma, const float* beta,
                   float eps, float* rstd, float* mean, float* amax, bsp_diag_t* diag, void* stream) {
  if (!valid_enum(kind, 1) || !valid_enum(dt, 1) || T < 0 || C <= 0) return BSP_ERR_ARG;
  if (T == 0) return BSP_OK;
  if (!x || !rstd || (kind == BSP_LAYERNORM && !mean)) return BSP_ERR_ARG;
  if (amax && (!gamma || (kind == BSP_LAYERNORM && !beta))) return BSP_ERR_ARG;
  if (C % 4 != 0) return BSP_ERR_UNSUPPORTED;
  if (!aligned16(x) || !aligned16(gamma) || !aligned16(beta)) return BSP_ERR_ALIGN;
  cudaStream_t st = (cudaStream_t)stream;
  if (amax) BSP_CHECK_CUDA(cudaMemsetAsync(amax, 0, sizeof(float), st));
  uint32_t* ab = reinterpret_cast<uint32_t*>(amax);
  // whole stages of 256-column multiples take the streamed kernel
  const StatsPlan sp = plan_stats_stream(T, C, dt, x);
  if (sp.ok) {
#define BSP_NSS(DT, KIND)                                                                                    \
  do {                                                                                                       \
    auto kfn = norm_stats_stream_kernel<DT, KIND, kStatRS, kStatNJ>;                                                          \
    BSP_CHECK_CUDA(cudaFuncSetAttribute(kfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sp.smem));    \
    kfn<<<sp.grid, sp.threads, sp.smem, st>>>(x, T, C, sp.rows_per_block, sp.ring, gamma, beta, eps, rstd,   \
                                               mean, ab, diag);                                              \
  } while (0)
    if (dt == BSP_F32) { if (kind == BSP_RMSNORM) BSP_NSS(BSP_F32, BSP_RMSNORM); else BSP_NSS(BSP_F32, BSP_LAYERNORM); }
    else { if (kind == BSP_RMSNORM) BSP_NSS(BSP_BF16, BSP_RMSNORM); else BSP_NSS(BSP_BF16, BSP_LAYERNORM); }
#undef BSP_NSS
    BSP_LAUNCH_CHECK();
    return BSP_OK;
  }
  const unsigned blocks = (unsigned)((T + 7) / 8);
#define BSP_NS(DT, KIND) norm_stats_kernel<DT, KIND><<<blocks, 256, 0, st>>>(x, T, C, gamma, beta, eps, rstd, mean, ab, diag)
  if (dt == BSP_F32) { if (kind == BSP_RMSNORM) BSP_NS(BSP_F32, BSP_RMSNORM); else BSP_NS(BSP_F32, BSP_LAYERNORM); }
  else { if (kind == BSP_RMSNORM) BSP_NS(BSP_BF16, BSP_RMSNORM); else BSP_NS(BSP_BF16, BSP_LAYERNORM); }
#undef BSP_NS
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

int bsp_norm_fwd(int kind, const void* x, int dt, int64_t T, int64_t C, const float* gamma, const float* beta,
                 const float* rstd, const float* mean, bsp_quant_t q, bsp_key_t key, uint8_t* u_codes,
                 uint8_t* u_codes_t, int64_t ld_t, float* u_f32, void* u_bf16_t, bsp_diag_t* diag, void* stream) {
  if (!valid_enum(kind, 1) || !valid_enum(dt, 1) || !valid_enum(q.fmt, 1) || !valid_enum(q.mode, 1)) return BSP_ERR_ARG;
  if (key.tensor_id >= (1u << 24) || key.stream > 255u || key.reserved != 0) return BSP_ERR_ARG;
  if (T < 0 || C <= 0) return BSP_ERR_ARG;
  if (T == 0) return BSP_OK;
  if (!x || !gamma || !rstd || (kind == BSP_LAYERNORM && (!beta || !mean))) return BSP_ERR_ARG;
  if (!u_codes && !u_codes_t && !u_f32 && !u_bf16_t) return BSP_ERR_ARG;
  if (C % 16 != 0) return BSP_ERR_UNSUPPORTED;
  if ((u_codes_t || u_bf16_t) && (ld_t < T || ld_t % 16 != 0)) return BSP_ERR_ALIGN;
  if (!aligned16(x) || !aligned16(u_codes) || !aligned16(u_codes_t) || !aligned16(u_f32) || !aligned16(u_bf16_t))
    return BSP_ERR_ALIGN;
  NormProducer prod;
  prod.kind = kind; prod.gamma = gamma; prod.beta = beta; prod.rstd = rstd; prod.mean = mean;
  prod.r_ = 0.f; prod.m_ = 0.f;
  return launch_tile(dt, q.fmt, q.mode, (cudaStream_t)stream, prod, x, T, C, q.scale, q.scale_dev, make_key(key),
                     u_codes, u_codes_t, ld_t, u_f32, reinterpret_cast<uint16_t*>(u_bf16_t), diag);
}

int bsp_norm_fwd_draws(int kind, const void* x, int dt, int64_t T, int64_t C, const float* gamma, const float* beta,
                       const float* rstd, const float* mean, bsp_quant_t q, bsp_key_t key, int draw0, int n_draws,
                       uint8_t* u_codes_t_draws, int64_t ld_t, void* stream) {
  if (!valid_enum(kind, 1) || !valid_enum(dt, 1) || !valid_enum(q.fmt, 1)) return BSP_ERR_ARG;
  if (key.tensor_id >= (1u << 24) || key.stream > 255u || key.reserved != 0) return BSP_ERR_ARG;
  if (T < 0 || C <= 0 || draw0 < 0 || n_draws < 0) return BSP_ERR_ARG;
  if (T == 0 || n_draws == 0) return BSP_OK;
  if (!x || !gamma || !rstd || !u_codes_t_draws || (kind == BSP_LAYERNORM && (!beta || !mean))) return BSP_ERR_ARG;
  if (C % 16 != 0) return BSP_ERR_UNSUPPORTED;
  if (ld_t < T || ld_t % 16 != 0) return BSP_ERR_ALIGN;
  if (!aligned16(x) || !aligned16(u_codes_t_draws)) return BSP_ERR_ALIGN;
  NormProducer prod;
  prod.kind = kind; prod.gamma = gamma; prod.beta = beta; prod.rstd = rstd; prod.mean = mean;
  prod.r_ = 0.f; prod.m_ = 0.f;
  dim3 grid((unsigned)((C + kTile - 1) / kTile), (unsigned)((T + kTile - 1) / kTile));
  cudaStream_t st = (cudaStream_t)stream;
  const PhiloxKey pk = make_key(key);
#define BSP_RR(DT, FMT)                                                                                          \
  reround_draws_kernel<DT, FMT><<<grid, 256, 0, st>>>(prod, x, T, C, q.scale, q.scale_dev, pk, draw0, n_draws,   \
                                                      u_codes_t_draws, ld_t)
  if (dt == BSP_F32 && q.fmt == BSP_E4M3) BSP_RR(BSP_F32, BSP_E4M3);
  else if (dt == BSP_F32) BSP_RR(BSP_F32, BSP_E5M2);
  else if (q.fmt == BSP_E4M3) BSP_RR(BSP_BF16, BSP_E4M3);
  else BSP_RR(BSP_BF16, BSP_E5M2);
#undef BSP_RR
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

}  // extern "C"
