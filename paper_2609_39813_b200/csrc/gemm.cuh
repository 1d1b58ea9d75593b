// Internal interface of the tensor-core contraction used by the weight-gradient, input-gradient
// and Monte-Carlo entry points.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/bsp.h"

namespace bsp {

enum { EPI_STORE_F32 = 0, EPI_STORE_BF16 = 1, EPI_MC = 2 };

// C[b][M][ldc] = alpha * A[M][K] * B[b][N][K]^T, alpha = (1/sa) * (1/sb); operands K-major.
// EPI_MC: S1 += C - ref, S2 += (C - ref)^2 for every batch in order (single [M][ldc] buffers).
struct GemmArgs {
  int64_t M = 0, N = 0, K = 0;
  int nb = 1;
  bool fp8 = true;
  int a_fmt = 0, b_fmt = 0;            // bsp_format_t of A and B when fp8
  const void* A = nullptr;
  const void* B = nullptr;
  bool a_mn = false, b_mn = false;     // operand stored [K][M] / [K][N] (pitch lda / ldb) instead
  int64_t lda = 0, ldb = 0;            // row pitch in elements
  int64_t b_batch_stride = 0;          // elements between batches of B
  float sa = 1.f, sb = 1.f;
  const float* sa_dev = nullptr;
  const float* sb_dev = nullptr;
  int mode = EPI_STORE_F32;
  void* C = nullptr;
  int64_t ldc = 0;
  const float* ref = nullptr;
  float* S1 = nullptr;
  float* S2 = nullptr;
  bsp_diag_t* diag = nullptr;
};

int gemm_run(const GemmArgs& g, cudaStream_t st);

}  // namespace bsp
