// Pieces shared by the attention kernels: tile constants, small PTX helpers, the tensor maps of the
// [B*H, S, 64] operands and outputs, and the internal entry points one translation unit offers the
// other.
#pragma once

#include "common.cuh"
#include "tc.cuh"

namespace bsp {

enum { AT_DKV = 0, AT_DQ = 1, AT_FWD = 2 };

constexpr int AT_BLK = 128, AT_D = 64;
constexpr int kAtTile = AT_BLK * AT_D * 2;        // 16 KB: one 128 x 64 bf16 tile
constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// 2^x on the special-function unit (2^-inf = 0): one instruction per probability.
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Two FP32 products in one instruction (packed pair operands).
__device__ __forceinline__ void mul_f32x2(float& x0, float& x1, float a0, float a1, float b0, float b1) {
  asm("{\n\t.reg .b64 ra, rb, rc;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
      "mul.rn.f32x2 rc, ra, rb;\n\tmov.b64 {%0, %1}, rc;\n\t}"
      : "=f"(x0), "=f"(x1) : "f"(a0), "f"(a1), "f"(b0), "f"(b1));
}

__device__ __forceinline__ void fma_f32x2(float& x0, float& x1, float a0, float a1, float b0, float b1, float c0, float c1) {
  asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\tmov.b64 rc, {%6, %7};\n\t"
      "fma.rn.f32x2 rd, ra, rb, rc;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(x0), "=f"(x1) : "f"(a0), "f"(a1), "f"(b0), "f"(b1), "f"(c0), "f"(c1));
}

// Two floats to one packed bf16 pair (round to nearest even): `lo` in bits 0..15, `hi` in 16..31.
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}

// tcgen05.ld of 32 columns without the wait, so several loads can be in flight before one wait.
__device__ __forceinline__ void tmem_ld32_nowait(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}

// FP32 output [BH][S][64] as two 32-column boxes per 128-row block (128-byte swizzle).
static inline int make_out_map(CUtensorMap* map, const void* base, int BH, int S) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return BSP_ERR_CUDA;
  cuuint64_t gdim[3] = {(cuuint64_t)AT_D, (cuuint64_t)S, (cuuint64_t)BH};
  cuuint64_t gstr[2] = {(cuuint64_t)AT_D * 4, (cuuint64_t)S * AT_D * 4};
  cuuint32_t box[3] = {32u, (cuuint32_t)AT_BLK, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(base), gdim, gstr, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? BSP_OK : BSP_ERR_CUDA;
}

static inline int make_head_map(CUtensorMap* map, const void* base, int BH, int S) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return BSP_ERR_CUDA;
  cuuint64_t gdim[3] = {(cuuint64_t)AT_D, (cuuint64_t)S, (cuuint64_t)BH};
  cuuint64_t gstr[2] = {(cuuint64_t)AT_D * 2, (cuuint64_t)S * AT_D * 2};
  cuuint32_t box[3] = {(cuuint32_t)AT_D, (cuuint32_t)AT_BLK, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), gdim, gstr, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? BSP_OK : BSP_ERR_CUDA;
}

// The operands' FP8 codes, uint8 [BH][S][64]: tiles of 128 rows of 64 bytes, 64-byte swizzle.
static inline int make_head_map_u8(CUtensorMap* map, const void* base, int BH, int S) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return BSP_ERR_CUDA;
  cuuint64_t gdim[3] = {(cuuint64_t)AT_D, (cuuint64_t)S, (cuuint64_t)BH};
  cuuint64_t gstr[2] = {(cuuint64_t)AT_D, (cuuint64_t)S * AT_D};
  cuuint32_t box[3] = {(cuuint32_t)AT_D, (cuuint32_t)AT_BLK, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void*>(base), gdim, gstr, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? BSP_OK : BSP_ERR_CUDA;
}

inline int check_attn_shape(int B, int H, int S, int Dh, int dt) {
  if (B <= 0 || H <= 0 || S <= 0) return BSP_ERR_ARG;
  if (Dh != AT_D || dt != BSP_BF16) return BSP_ERR_UNSUPPORTED;
  if ((int64_t)B * H > 65535 * 16) return BSP_ERR_UNSUPPORTED;
  return BSP_OK;
}

// Number of SMs of the current device (the persistent kernels launch one CTA per SM).
inline int sm_count_or_default() {
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) == cudaSuccess &&
      cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0)
    return n;
  return kNumSMs;
}

// Internal entry points of attn.cu used by the per-use check (attn_mc.cu).  `f` = NULL: BF16-operand
// mode; otherwise the FP8-operand mode with the operands holding decoded codes.
int attn_fwd_impl(int B, int H, int S, int Dh, int causal, float softmax_scale, const void* q, const void* k,
                  const void* v, int dt, const bsp_attn_fp8_t* f, float* o, float* lse, bsp_diag_t* diag, void* stream,
                  const float* lse_known = nullptr);   // rows' LSE given: one pass over the keys, `lse` may be NULL
int attn_dterm_impl(int B, int H, int S, int Dh, const void* dO, int dt, const float* do_scales, const float* o_orig,
                    const uint8_t* o_codes, const float* o_scales, int o_fmt, int d_read, bsp_key_t key, int draw0,
                    int n_draws, float* d_out, void* stream);
int attn_bwd_dterm_impl(int B, int H, int S, int Dh, int causal, float softmax_scale, const void* q, const void* k,
                        const void* v, const void* dO, int dt, const bsp_attn_fp8_t* f, const float* lse,
                        const float* dterm, float* dq, float* dk, float* dv, bsp_diag_t* diag, void* stream);
int attn_bwd_dterm_mc(int B, int H, int S, int Dh, int causal, float softmax_scale, const void* q, const void* k,
                      const void* v, const void* dO, int dt, const bsp_attn_fp8_t* f, const float* lse,
                      const float* dterm, int nd, const float* ref_dq, float* S1q, float* S2q, const float* ref_dk,
                      float* S1k, float* S2k, bsp_diag_t* diag, void* stream);

}  // namespace bsp
