// The per-use check of the attention D use, and the kernels that evaluate a fresh read of the saved
// output through Eq. dterm itself.
//
// dS = P o (dP - D) is affine in the correction term D, and so are dQ = c dS K and dK = c dS^T Q.
// With D_k = rowsum(dO o O_k) the term under the k-th fresh rounding of the saved output and D* the
// reference's (from the original output), draw k differs from the reference gradient by
//
//     dQ_k - dQ* = -c diag(D_k - D*) (P K)            dK_k - dK* = -c P^T diag(D_k - D*) Q
//
// and dV does not move at all.  The Monte-Carlo check needs exactly these differences (its sums are
// S1 = sum_k (g_k - g*), S2 = sum_k (g_k - g*)^2), so the kernels here form them directly:
//   * dQ: row i of the difference is the row of P K scaled by (D_k - D*)[i], hence
//     S1 = -c (P K) o rowwise sum_k (D_k - D*),  S2 = c^2 (P K)^2 o rowwise sum_k (D_k - D*)^2:
//     one pass for P K (the forward kernel with K in place of V) and an elementwise kernel, whatever K;
//   * dK: one contraction per draw, P^T against the rows of Q scaled by -c (D_k - D*).  The
//     probabilities are formed once per step for four draws: the scaled Q tiles of the four draws lie
//     side by side as one 128 x 256 B operand, so a step is one product for S^T, one pass of the exp2
//     unit, and one 128 x 256 x 128 product.
// Rounding an operand to bf16 now costs 2^-9 of the *difference*, not of the whole dS, so the
// statistics see the read and not the operand format, and no per-draw gradient is ever written.
//
// attn_dk_diff_kernel: persistent, one CTA per SM walking (key block, head) items, heaviest first.
// 320 threads: warp 0 TMA producer, warp 1 MMA issuer, warps 2..9 probabilities, operand scaling and
// epilogue.  Tensor memory: S^T 128 columns, P^T operand 64, four accumulators of 64.  -LSE enters
// S^T through one extra K = 16 product step (a tile of ones against rows holding -LSE/c as three
// bf16 terms), as in the dK/dV kernel of the plain backward.  Every wait is bounded.
#include <string.h>

#include <atomic>

#include "attn_common.cuh"
#include "mc_stats.cuh"

namespace bsp {

constexpr int kDkThreads = 320;
constexpr int kDkND = 4;                           // draws per launch
constexpr uint32_t kDkStages = 3;                  // ring of streamed Q tiles
constexpr int kDkBiasTile = AT_BLK * 16 * 2;       // 4 KB: one 128 x 16 bf16 tile of the extra K = 16 step
// shared memory: K tiles [2], Q ring [3], two buffers of the scaled Q tiles [2][4] (the first one is
// also the epilogue's 64 KB of staging), barriers, then the ones tile and three buffers of the -LSE tile
constexpr int kDkSmem = 1024 + (2 + (int)kDkStages + 2 * kDkND) * kAtTile + 1024 + 4 * kDkBiasTile;
static_assert(kDkSmem <= 232448, "dynamic shared memory of attn_dk_diff_kernel exceeds the SM's");

struct DkDiffParams {
  int BH, S, nblk, causal;
  float c;                       // softmax scale
  const float* lse;              // [BH*S]
  const float* d_ref;            // [BH*S]      the reference's correction term
  const float* d_draws;          // [nd][BH*S]  the draws' correction terms
  int nd;                        // draws in this launch, 1 .. kDkND (the rest contribute zeros)
  bsp_diag_t* diag;
};

__device__ __forceinline__ uint32_t mul_bf16x2(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}

__global__ void __launch_bounds__(kDkThreads, 1)
attn_dk_diff_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_s1, const __grid_constant__ CUtensorMap tm_s2,
                    DkDiffParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  const uint32_t res_base = base;                                   // K tile of the item, two buffers
  const uint32_t q0 = base + 2 * kAtTile;                           // stage s: q0 + s * kAtTile
  const uint32_t bs0 = q0 + kDkStages * kAtTile;                    // buffer pb, draw d: bs0 + (4 pb + d) * kAtTile
  const uint32_t bars = bs0 + 2 * kDkND * kAtTile;
  // P^T and the scaled tiles are double-buffered (buffer = step & 1), so the probabilities of step
  // j + 1 are formed while the accumulating product of step j runs
  const uint32_t b_res = bars, b_res_empty = bars + 16, b_sfull = bars + 32, b_sempty = bars + 56,
                 b_sdp_full = bars + 80, b_sdp_free = bars + 88, b_pds_ready = bars + 96 /* [2] */,
                 b_pds_free = bars + 112 /* [2] */, b_acc = bars + 128, b_acc_free = bars + 136, b_bias = bars + 144;
  const uint32_t bias0 = bars + 1024;                               // ones tile; buffer b: the -LSE tile at 1 + b
  uint8_t* bars_gen = smem_raw + (bars - raw);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bars_gen + 176);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars_gen + 180);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nitems = p.nblk * p.BH;
  // the CTA's n-th item: rounds of gridDim.x items, walked forwards and backwards in turn
  auto item_at = [&](int n) -> int {
    const int b = (int)blockIdx.x, G = (int)gridDim.x;
    return n * G + ((n & 1) ? G - 1 - b : b);
  };
  auto decode_item = [&](int w, int& blk, int& bh, int& it_begin, int& nsteps) {
    blk = w / p.BH;                                                 // key block j: steps i = j .. nblk-1 (causal)
    bh = w % p.BH;
    it_begin = p.causal ? blk : 0;
    nsteps = p.nblk - it_begin;
  };

  if (threadIdx.x == 0) {
    for (int s = 0; s < 2; ++s) { mbar_init(b_res + 8 * s, 1); mbar_init(b_res_empty + 8 * s, 1); }
    for (uint32_t s = 0; s < kDkStages; ++s) { mbar_init(b_sfull + 8 * s, 1); mbar_init(b_sempty + 8 * s, 1); }
    for (uint32_t s = 0; s < 3; ++s) mbar_init(b_bias + 8 * s, 8);
    mbar_init(b_sdp_full, 1); mbar_init(b_sdp_free, 8);
    for (int s = 0; s < 2; ++s) { mbar_init(b_pds_ready + 8 * s, 8); mbar_init(b_pds_free + 8 * s, 1); }
    mbar_init(b_acc, 1); mbar_init(b_acc_free, 8);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // S^T 128 columns, two P^T operands of 64, the accumulator of draw d at t_acc + 64 d
  const uint32_t t_s = tmem, t_p = tmem + 128, t_acc = tmem + 256;

  const uint32_t id_s = make_idesc(1u, 1u, 128, 128);                          // A, B K-major
  const uint32_t id_acc = make_idesc(1u, 1u, 128, 64 * kDkND) | (1u << 16);    // A from tensor memory, B MN-major

  if (warp == 0) {
    // ------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_k);
      bool ok = true;
      uint32_t itg = 0;
      int item = 0;
      for (int w = item_at(0); w < nitems && ok; w = item_at(++item)) {
        int blk, bh, it_begin, nsteps;
        decode_item(w, blk, bh, it_begin, nsteps);
        const uint32_t rb = item & 1u, rph = (item >> 1) & 1u;
        if (!mbar_wait(b_res_empty + 8 * rb, rph ^ 1u, abort_flag)) { ok = false; break; }
        mbar_expect_tx(b_res + 8 * rb, kAtTile);
        tma_load_3d(res_base + rb * kAtTile, &tm_k, b_res + 8 * rb, 0, blk * AT_BLK, bh);
        for (int it = 0; it < nsteps; ++it, ++itg) {
          const uint32_t s = itg % kDkStages, ph = (itg / kDkStages) & 1u;
          if (!mbar_wait(b_sempty + 8 * s, ph ^ 1u, abort_flag)) { ok = false; break; }
          mbar_expect_tx(b_sfull + 8 * s, kAtTile);
          tma_load_3d(q0 + s * kAtTile, &tm_q, b_sfull + 8 * s, 0, (it_begin + it) * AT_BLK, bh);
        }
      }
      if (!ok) for (int i = 0; i < 200; ++i) __nanosleep(1000);     // let copies in flight land
    }
  } else if (warp == 1) {
    // ------------------------------------------------ MMA issuer
    if (lane == 0) {
      bool ok = true;
      uint32_t itg = 0;
      int item = 0;
      for (int w = item_at(0); w < nitems && ok; w = item_at(++item)) {
        int blk, bh, it_begin, nsteps;
        decode_item(w, blk, bh, it_begin, nsteps);
        const uint32_t rb = item & 1u, iph = (item >> 1) & 1u, aph = (uint32_t)item & 1u;
        const uint32_t k_t = res_base + rb * kAtTile;
        if (!mbar_wait(b_res + 8 * rb, iph, abort_flag)) { ok = false; break; }
        // S^T = K Q^T of global step jt (rows = keys), plus the K = 16 step that subtracts LSE / c.
        // Issued one step ahead: the other warps hand the S^T columns back as soon as they hold them
        // in registers.
        auto issue_s = [&](uint32_t jt) -> bool {
          const uint32_t s = jt % kDkStages, ph = (jt / kDkStages) & 1u;
          if (!mbar_wait(b_sfull + 8 * s, ph, abort_flag)) return false;
          if (!mbar_wait(b_sdp_free, (jt & 1u) ^ 1u, abort_flag)) return false;
          tc_fence_after();
          const uint64_t a = make_smem_desc(k_t), b = make_smem_desc(q0 + s * kAtTile);
#pragma unroll
          for (int k = 0; k < 4; ++k) tc_mma<false>(t_s, a + 2u * k, b + 2u * k, id_s, k != 0);
          const uint32_t bb = jt % 3u;
          if (!mbar_wait(b_bias + 8 * bb, (jt / 3u) & 1u, abort_flag)) return false;
          tc_mma<false>(t_s, make_smem_desc_k16(bias0), make_smem_desc_k16(bias0 + (1u + bb) * kDkBiasTile), id_s, 1u);
          tc_commit(b_sdp_full);
          return true;
        };
        if (nsteps > 0) ok = issue_s(itg);
        for (int it = 0; it < nsteps && ok; ++it) {
          const uint32_t jg = itg + (uint32_t)it;
          const uint32_t s = jg % kDkStages, pb = jg & 1u, pph = (jg >> 1) & 1u;
          if (it + 1 < nsteps && !issue_s(jg + 1)) { ok = false; break; }
          if (!mbar_wait(b_pds_ready + 8 * pb, pph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          // the accumulators are free once the epilogue of the item before has read them
          if (it == 0 && !mbar_wait(b_acc_free, aph ^ 1u, abort_flag)) { ok = false; break; }
          // all four draws at once: P^T (tensor memory, eight columns per 16 queries) against the four
          // scaled Q tiles side by side (MN-major, one 128-byte atom of 64 columns per draw)
          const uint64_t bq = make_smem_desc_mn(bs0 + pb * kDkND * kAtTile, (uint32_t)kAtTile);
#pragma unroll
          for (int k = 0; k < 8; ++k) tc_mma_ts(t_acc, t_p + 64u * pb + 8u * k, bq + 128u * k, id_acc, (it != 0) | (k != 0));
          tc_commit(b_pds_free + 8 * pb);
          tc_commit(b_sempty + 8 * s);
        }
        itg += (uint32_t)nsteps;
        if (ok) tc_commit(b_acc);
      }
    }
  } else {
    // ------------------------------------------------ probabilities, operand scaling, epilogue
    const int q4 = warp & 3, h = (warp - 2) >> 2;
    const int r = q4 * 32 + lane;                                   // row of the 128-row block: a key (S^T), a query (Q tile)
    const uint32_t lane_off = (uint32_t)(q4 * 32) << 16;
    const int ts = (int)threadIdx.x - 64;                           // 0 .. 255
    {
      // constant parts of the four extra tiles: thread ts clears 16 bytes of each (row ts & 127, half
      // ts >> 7); the first three columns of the ones tile are 1
      const uint32_t off = (uint32_t)((ts & 127) >> 3) * 256u + (uint32_t)(ts >> 7) * 128u + (uint32_t)(ts & 7) * 16u;
#pragma unroll
      for (uint32_t t = 0; t < 4; ++t) {
        const bool one = t == 0 && ts < 128;
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %3};" ::"r"(bias0 + t * kDkBiasTile + off),
                     "r"(one ? 0x3F803F80u : 0u), "r"(one ? 0x00003F80u : 0u), "r"(0u) : "memory");
      }
      named_bar_sync(1, 256);
    }
    const float c2 = p.c * kLog2e;
    const float bias_mul = -kLog2e / c2;                            // the accumulator holds s - LSE / c
    const size_t rows_total = (size_t)p.BH * p.S;
    bool ok = true;
    bool store_pending = false;                                     // the epilogue's bulk adds may still read the staging
    uint32_t bias_written = 0, itg = 0;
    int item = 0;
    // the -LSE row of one step: threads ts < 128 own query ts of the tile
    auto bias_fetch = [&](int tbh, int step) -> float {
      if (ts >= 128) return 0.f;
      const int q = step * AT_BLK + ts;
      return q < p.S ? __ldg(p.lse + (size_t)tbh * p.S + q) : 0.f;
    };
    // (fenced = false: the caller issues the proxy fence itself, after other stores that need one too)
    auto bias_put = [&](uint32_t jt, float rawv, bool fenced = true) {
      if (ts < 128) {
        const float x = rawv * bias_mul;
        const __nv_bfloat16 h1 = __float2bfloat16_rn(x);
        const float r1 = x - __bfloat162float(h1);
        const __nv_bfloat16 h2 = __float2bfloat16_rn(r1);
        const __nv_bfloat16 h3 = __float2bfloat16_rn(r1 - __bfloat162float(h2));
        const uint32_t w0 = (uint32_t)__bfloat16_as_ushort(h1) | ((uint32_t)__bfloat16_as_ushort(h2) << 16);
        const uint32_t w1 = (uint32_t)__bfloat16_as_ushort(h3);
        const uint32_t tile = bias0 + (1u + jt % 3u) * kDkBiasTile;
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %3};" ::"r"(tile + (uint32_t)(ts >> 3) * 256u + (uint32_t)(ts & 7) * 16u),
                     "r"(w0), "r"(w1), "r"(0u) : "memory");
        if (fenced) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      }
      if (!fenced) return;
      __syncwarp();
      if (lane == 0) mbar_arrive(b_bias + 8 * (jt % 3u));
    };
    for (int w = item_at(0); w < nitems && ok; w = item_at(++item)) {
      int blk, bh, it_begin, nsteps;
      decode_item(w, blk, bh, it_begin, nsteps);
      const uint32_t rb = (uint32_t)item & 1u, aph = (uint32_t)item & 1u;
      // the next item's head and first step: its first two -LSE rows are written under this item's tail
      int nx_bh = 0, nx_begin = 0, nx_total = 0;
      {
        const int wn = item_at(item + 1);
        if (wn < nitems) { int nb; decode_item(wn, nb, nx_bh, nx_begin, nx_total); }
      }
      while (bias_written < itg + (uint32_t)(nsteps < 2 ? nsteps : 2)) {
        const int l = (int)(bias_written - itg);
        bias_put(bias_written, bias_fetch(bh, it_begin + l));
        ++bias_written;
      }
      auto bias_target = [&](int it, int& tbh, int& tstep) -> bool {
        const int t = it + 2;
        if (t < nsteps) { tbh = bh; tstep = it_begin + t; return true; }
        if (t - nsteps < nx_total) { tbh = nx_bh; tstep = nx_begin + (t - nsteps); return true; }
        return false;
      };
      const int key = blk * AT_BLK + r;                             // this thread's row of S^T
      for (int it = 0; it < nsteps && ok; ++it) {
        const int step = it_begin + it;
        const uint32_t jt = itg + (uint32_t)it, ip = jt & 1u, pb = jt & 1u, pph = (jt >> 1) & 1u;
        const uint32_t t_pb = t_p + 64u * pb, bsb = bs0 + pb * kDkND * kAtTile;
        // this step's correction terms of query step*128 + r: requested here, first used after the
        // exponentials (nothing may depend on these loads before then, or the in-order warp sits out
        // their latency)
        float draw_raw[kDkND], dref_raw;
        const bool q_in = step * AT_BLK + r < p.S;
        {
          const size_t qi = (size_t)bh * p.S + (q_in ? step * AT_BLK + r : 0);
          dref_raw = __ldg(p.d_ref + qi);
#pragma unroll
          for (int d = 0; d < kDkND; ++d) draw_raw[d] = d < p.nd ? __ldg(p.d_draws + (size_t)d * rows_total + qi) : 0.f;
        }
        int bias_bh = 0, bias_step = 0;
        const bool bias_due = bias_written == jt + 2u && bias_target(it, bias_bh, bias_step);
        float bias_next = 0.f;
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(b_sdp_full, ip, abort_flag));
        if (!ok) break;
        tc_fence_after();
        uint32_t sv[64];
        tmem_ld32_nowait(t_s + lane_off + h * 64, *reinterpret_cast<uint32_t(*)[32]>(&sv[0]));
        tmem_ld32_nowait(t_s + lane_off + h * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[32]));
        // the step's Q tile has landed long ago (S^T read it); this thread still has to see its barrier
        // before it reads the tile further down: the test goes out here, under the tensor-memory load
        const uint32_t q_seen = mbar_try_wait(b_sfull + 8 * (jt % kDkStages), (jt / kDkStages) & 1u);
        tmem_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(b_sdp_free);
        if (bias_due) bias_next = bias_fetch(bias_bh, bias_step);

        const int col0 = step * AT_BLK + h * 64;                    // first query of this thread's 64 columns
        const bool edge = (p.causal && blk == step) || (blk + 1) * AT_BLK > p.S || (step + 1) * AT_BLK > p.S;
        auto valid_at = [&](int j) {
          const int qy = col0 + j;
          return key < p.S && qy < p.S && (!p.causal || key <= qy);
        };
        uint32_t pk[32];
        auto pair_at = [&](int j, bool masked) {
          float a0, a1;
          mul_f32x2(a0, a1, __uint_as_float(sv[j]), __uint_as_float(sv[j + 1]), c2, c2);
          if (masked) {
            if (!valid_at(j)) a0 = -INFINITY;
            if (!valid_at(j + 1)) a1 = -INFINITY;
          }
          pk[j >> 1] = pack_bf16x2(ex2_approx(a0), ex2_approx(a1));
        };
        if (!edge) {
#pragma unroll
          for (int j = 0; j < 32; j += 2) pair_at(j, false);
        } else {
#pragma unroll
          for (int j = 0; j < 32; j += 2) pair_at(j, true);
        }
        // this buffer of the P^T operand and of the scaled tiles is free once the product of two steps
        // ago has read it
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(b_pds_free + 8 * pb, pph ^ 1u, abort_flag));
        if (!ok) break;
        tmem_st16(t_pb + lane_off + h * 32, *reinterpret_cast<const uint32_t(*)[16]>(&pk[0]));
        if (!edge) {
#pragma unroll
          for (int j = 32; j < 64; j += 2) pair_at(j, false);
        } else {
#pragma unroll
          for (int j = 32; j < 64; j += 2) pair_at(j, true);
        }
        tmem_st16(t_pb + lane_off + h * 32 + 16, *reinterpret_cast<const uint32_t(*)[16]>(&pk[16]));
        // ---- the B operand: row r of the streamed Q tile times this row's factor of each draw, written
        // at the same (swizzled) place of the draw's tile.  Thread (r, h) takes the four 16-byte chunks
        // whose logical index is 4h .. 4h+3; chunk c of row r sits at position c ^ (r & 7), so the lanes
        // of a warp (consecutive rows) spread over all banks.
        if (store_pending) {
          if (warp == 2 && lane == 0) tma_store_wait_read();
          named_bar_sync(2, 256);
          store_pending = false;
        }
        {
          const uint32_t s = jt % kDkStages, ph = (jt / kDkStages) & 1u;
          if (!__all_sync(0xFFFFFFFFu, q_seen)) {
            ok = __all_sync(0xFFFFFFFFu, mbar_wait(b_sfull + 8 * s, ph, abort_flag));
            if (!ok) break;
          }
          // the row factors -c (D_k - D*) of the draws (zero for a draw this launch does not have)
          uint32_t f2[kDkND];
          asm volatile("" : "+f"(dref_raw));
#pragma unroll
          for (int d = 0; d < kDkND; ++d) {
            asm volatile("" : "+f"(draw_raw[d]));
            const float fk = (q_in && d < p.nd) ? -p.c * (draw_raw[d] - dref_raw) : 0.f;
            f2[d] = pack_bf16x2(fk, fk);
          }
          const uint32_t row_off = (uint32_t)r * 128u;
#pragma unroll
          for (int cch = 0; cch < 4; ++cch) {
            uint32_t a0, a1, a2, a3;
            const uint32_t off = row_off + ((uint32_t)((4 * h + cch) ^ (r & 7)) << 4);
            asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(a0), "=r"(a1), "=r"(a2), "=r"(a3) : "r"(q0 + s * kAtTile + off));
#pragma unroll
            for (int d = 0; d < kDkND; ++d)
              asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(bsb + (uint32_t)d * kAtTile + off),
                           "r"(mul_bf16x2(a0, f2[d])), "r"(mul_bf16x2(a1, f2[d])), "r"(mul_bf16x2(a2, f2[d])),
                           "r"(mul_bf16x2(a3, f2[d])) : "memory");
          }
        }
        tmem_wait_st();
        tc_fence_before();
        if (bias_due) {
          // the -LSE row two steps ahead goes out under the same proxy fence as the scaled tiles (a
          // fence waits for the thread's shared-memory stores to drain: one per step, not two)
          asm volatile("" : "+f"(bias_next));                       // keeps the first use of the load here
          bias_put(bias_written, bias_next, false);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(b_pds_ready + 8 * pb);
          if (bias_due) mbar_arrive(b_bias + 8 * (bias_written % 3u));
        }
        if (bias_due) ++bias_written;
      }
      itg += (uint32_t)nsteps;
      // ---- epilogue: the four accumulators hold the draws' differences; their sum and sum of squares
      // leave through the (now idle) scaled-tile buffers as bulk adds into S1 and S2
      if (ok) ok = __all_sync(0xFFFFFFFFu, mbar_wait(b_acc, aph, abort_flag));
      if (ok) {
        tc_fence_after();
        float s1[32], s2[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) s1[e] = s2[e] = 0.f;
#pragma unroll
        for (int d = 0; d < kDkND; ++d) {
          uint32_t a[32];
          tmem_ld32(t_acc + 64u * d + lane_off + h * 32, a);
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const float v = __uint_as_float(a[e]);
            s1[e] += v;
            s2[e] = fmaf(v, v, s2[e]);
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(b_acc_free);
        if (warp == 2 && lane == 0) mbar_arrive(b_res_empty + 8 * rb);   // the item's K tile is no longer read
#pragma unroll
        for (int t = 0; t < 8; ++t) {
          const uint32_t off = (uint32_t)h * 16384u + (uint32_t)r * 128u + ((uint32_t)(t ^ (r & 7)) << 4);
          asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(bs0 + off), "f"(s1[4 * t]), "f"(s1[4 * t + 1]),
                       "f"(s1[4 * t + 2]), "f"(s1[4 * t + 3]) : "memory");
          asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(bs0 + 32768u + off), "f"(s2[4 * t]),
                       "f"(s2[4 * t + 1]), "f"(s2[4 * t + 2]), "f"(s2[4 * t + 3]) : "memory");
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        named_bar_sync(3, 256);
        if (warp == 2 && lane == 0) {
          tma_reduce_add_3d(&tm_s1, bs0, 0, blk * AT_BLK, bh);
          tma_reduce_add_3d(&tm_s1, bs0 + 16384u, 32, blk * AT_BLK, bh);
          tma_reduce_add_3d(&tm_s2, bs0 + 32768u, 0, blk * AT_BLK, bh);
          tma_reduce_add_3d(&tm_s2, bs0 + 49152u, 32, blk * AT_BLK, bh);
          tma_store_commit();
        }
        store_pending = true;
      }
    }
    if (warp == 2 && lane == 0) tma_store_wait_all();
  }

  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag && p.diag) atomicMax(&p.diag->status, (int)BSP_ERR_TIMEOUT);
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

// S1[i, :] = -c PK[i, :] a[i], S2[i, :] = c^2 PK[i, :]^2 b[i] with a = sum_k (D_k - D*), b = sum_k (D_k - D*)^2
// (the rowwise sums of the correction term itself): the K draws of dQ in one elementwise pass.
__global__ void __launch_bounds__(256)
attn_dq_sums_kernel(const float* __restrict__ pk, const float* __restrict__ S1d, const float* __restrict__ S2d, float c,
                    float* __restrict__ S1q, float* __restrict__ S2q, size_t n4) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n4) return;
  const size_t row = i / (AT_D / 4);
  const float4 v = __ldg(reinterpret_cast<const float4*>(pk) + i);
  const float a = -c * __ldg(S1d + row), b = c * c * __ldg(S2d + row);
  reinterpret_cast<float4*>(S1q)[i] = make_float4(v.x * a, v.y * a, v.z * a, v.w * a);
  reinterpret_cast<float4*>(S2q)[i] = make_float4(v.x * v.x * b, v.y * v.y * b, v.z * v.z * b, v.w * v.w * b);
}

// S1 += times * (g - ref), S2 += times * (g - ref)^2, elementwise (times = 1: one draw).
__global__ void mc_accumulate_kernel(const float* __restrict__ g, const float* __restrict__ ref, float* __restrict__ S1,
                                     float* __restrict__ S2, size_t n4, float times) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n4) return;
  const float4 a = __ldg(reinterpret_cast<const float4*>(g) + i), r = __ldg(reinterpret_cast<const float4*>(ref) + i);
  float4 s1 = reinterpret_cast<float4*>(S1)[i], s2 = reinterpret_cast<float4*>(S2)[i];
  const float d0 = a.x - r.x, d1 = a.y - r.y, d2 = a.z - r.z, d3 = a.w - r.w;
  s1.x = fmaf(times, d0, s1.x); s1.y = fmaf(times, d1, s1.y); s1.z = fmaf(times, d2, s1.z); s1.w = fmaf(times, d3, s1.w);
  s2.x = fmaf(times * d0, d0, s2.x); s2.y = fmaf(times * d1, d1, s2.y);
  s2.z = fmaf(times * d2, d2, s2.z); s2.w = fmaf(times * d3, d3, s2.w);
  reinterpret_cast<float4*>(S1)[i] = s1;
  reinterpret_cast<float4*>(S2)[i] = s2;
}

// The same over nd draws held back to back (g[d * stride + i]), in draw order: one launch instead of
// nd for a tensor as small as the correction term.  Any n (no vector accesses).
__global__ void mc_accumulate_draws_kernel(const float* __restrict__ g, size_t stride, int nd,
                                           const float* __restrict__ ref, float* __restrict__ S1,
                                           float* __restrict__ S2, size_t n) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const float r = __ldg(ref + i);
  float s1 = S1[i], s2 = S2[i];
  for (int d = 0; d < nd; ++d) {
    const float e = __ldg(g + (size_t)d * stride + i) - r;
    s1 += e;
    s2 = fmaf(e, e, s2);
  }
  S1[i] = s1;
  S2[i] = s2;
}

// nd (1 .. 4) draws of the dK difference, added to the running sums.
static int attn_dk_diff(int BH, int S, int causal, float c, const void* q, const void* k, const float* lse,
                        const float* d_ref, const float* d_draws, int nd, float* S1k, float* S2k, bsp_diag_t* diag,
                        cudaStream_t st) {
  if (nd < 1 || nd > kDkND) return BSP_ERR_ARG;
  CUtensorMap mq, mk, m1, m2;
  int rc;
  if ((rc = make_head_map(&mq, q, BH, S)) != BSP_OK) return rc;
  if ((rc = make_head_map(&mk, k, BH, S)) != BSP_OK) return rc;
  if ((rc = make_out_map(&m1, S1k, BH, S)) != BSP_OK) return rc;
  if ((rc = make_out_map(&m2, S2k, BH, S)) != BSP_OK) return rc;
  static std::atomic<bool> attr_set_dev[kMaxDevices];
  std::atomic<bool>& attr_set = attr_set_dev[device_slot()];
  if (!attr_set.load(std::memory_order_acquire)) {
    BSP_CHECK_CUDA(cudaFuncSetAttribute(attn_dk_diff_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kDkSmem));
    attr_set.store(true, std::memory_order_release);
  }
  DkDiffParams p;
  p.BH = BH; p.S = S; p.nblk = (S + AT_BLK - 1) / AT_BLK; p.causal = causal ? 1 : 0; p.c = c;
  p.lse = lse; p.d_ref = d_ref; p.d_draws = d_draws; p.nd = nd; p.diag = diag;
  const int nsm = sm_count_or_default();
  const int64_t nitems = (int64_t)p.nblk * BH;
  const unsigned grid = (unsigned)(nitems < nsm ? nitems : nsm);
  attn_dk_diff_kernel<<<grid, kDkThreads, kDkSmem, st>>>(mq, mk, m1, m2, p);
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

struct AttnCheckBuffers {
  float *o, *lse, *amax, *scales, *d_ref, *d_pol, *d_draws;
  uint8_t* codes;
  float *g_ref[3], *g_pol[3], *S1[2], *S2[2], *S1d, *S2d;
  // FP8-operand mode: the rounded operands (decoded codes as bf16) and their per-slice scales
  void* op8[4];
  uint8_t* opc[4];                                // the operands' codes (FP8-operand mode)
  float *op_amax[4], *op_scale[4];
  void* ws_stats;
  size_t b_stats;
};

static size_t attn_carve(const bsp_attn_desc_t* op, int K, char* base, AttnCheckBuffers* out) {
  size_t off = 0;
  auto take = [&](size_t bytes) -> void* {
    void* p = base ? base + off : nullptr;
    off += round_up(bytes ? bytes : 1, 256);
    return p;
  };
  const size_t BH = (size_t)op->B * op->H, rows = BH * op->S, n = rows * op->Dh;
  AttnCheckBuffers c;
  memset(&c, 0, sizeof(c));
  c.o = (float*)take(n * 4); c.lse = (float*)take(rows * 4);
  c.amax = (float*)take(BH * 4); c.scales = (float*)take(BH * 4);
  c.d_ref = (float*)take(rows * 4); c.d_pol = (float*)take(rows * 4);
  c.d_draws = (float*)take(rows * 4 * (size_t)(K > 0 ? K : 1));
  c.codes = (uint8_t*)take(n);
  for (int t = 0; t < 3; ++t) { c.g_ref[t] = (float*)take(n * 4); c.g_pol[t] = (float*)take(n * 4); }
  for (int t = 0; t < 2; ++t) { c.S1[t] = (float*)take(n * 4); c.S2[t] = (float*)take(n * 4); }
  c.S1d = (float*)take(rows * 4); c.S2d = (float*)take(rows * 4);
  if (op->fp8_operands) {
    for (int t = 0; t < 4; ++t) {
      c.op8[t] = take(n * 2); c.opc[t] = (uint8_t*)take(n); c.op_amax[t] = (float*)take(BH * 4); c.op_scale[t] = (float*)take(BH * 4);
    }
  }
  c.b_stats = kMaxPendingStats * kStatSlotBytes;
  c.ws_stats = take(c.b_stats);
  if (out) *out = c;
  return off;
}

}  // namespace bsp

using namespace bsp;

extern "C" {

int bsp_mc_accumulate(const float* g, const float* g_ref, float* S1, float* S2, size_t n, void* stream) {
  if (!g || !g_ref || !S1 || !S2) return BSP_ERR_ARG;
  if (n % 4 != 0) return BSP_ERR_UNSUPPORTED;
  if (!aligned16(g) || !aligned16(g_ref) || !aligned16(S1) || !aligned16(S2)) return BSP_ERR_ALIGN;
  if (n == 0) return BSP_OK;
  const size_t n4 = n / 4;
  mc_accumulate_kernel<<<(unsigned)((n4 + 255) / 256), 256, 0, (cudaStream_t)stream>>>(g, g_ref, S1, S2, n4, 1.0f);
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

size_t bsp_mc_check_attn_workspace_bytes(const bsp_attn_desc_t* op, int K) {
  if (!op || op->B <= 0 || op->H <= 0 || op->S <= 0 || op->Dh <= 0) return 0;
  return attn_carve(op, K, nullptr, nullptr);
}

#define BSP_TRY(expr)              \
  do {                             \
    int _rc = (expr);              \
    if (_rc != BSP_OK) return _rc; \
  } while (0)

int bsp_mc_check_attn(const bsp_attn_desc_t* op, int K, const bsp_verdict_rule_t* rule, bsp_use_result_t* results,
                      int* n_results, void* ws, size_t ws_bytes, bsp_diag_t* diag, void* stream) {
  if (!op || !results || !n_results || K < 4 || !rule_valid(rule)) return BSP_ERR_ARG;
  if (!op->q || !op->k || !op->v || !op->dO) return BSP_ERR_ARG;
  int rc = check_attn_shape(op->B, op->H, op->S, op->Dh, op->dtype);
  if (rc != BSP_OK) return rc;
  const bool fp8 = op->fp8_operands != 0;
  if (fp8 && (!(op->p_scale > 0.f) || !(op->ds_scale > 0.f))) return BSP_ERR_ARG;
  if (!ws || ws_bytes < bsp_mc_check_attn_workspace_bytes(op, K) || (reinterpret_cast<uintptr_t>(ws) & 255u))
    return BSP_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  AttnCheckBuffers b;
  attn_carve(op, K, reinterpret_cast<char*>(ws), &b);
  const int B = op->B, H = op->H, S = op->S, Dh = op->Dh, dt = op->dtype;
  const size_t BH = (size_t)B * H, rows = BH * S, n = rows * Dh;
  const float c = op->softmax_scale;
  *n_results = 0;

  // ---- FP8-operand mode: the operands as the emulated backward sees them
  const void *q = op->q, *k = op->k, *v = op->v, *dO = op->dO;
  bsp_attn_fp8_t f8;
  const bsp_attn_fp8_t* f = nullptr;
  if (fp8) {
    const void* src[4] = {op->q, op->k, op->v, op->dO};
    for (int t = 0; t < 4; ++t)
      BSP_TRY(bsp_attn_quantize(src[t], (int)BH, (size_t)S * Dh, t == 3 ? BSP_E5M2 : BSP_E4M3, b.op8[t], b.opc[t],
                                b.op_amax[t], b.op_scale[t], diag, st));
    q = b.op8[0]; k = b.op8[1]; v = b.op8[2]; dO = b.op8[3];
    f8.q_scale = b.op_scale[0]; f8.k_scale = b.op_scale[1]; f8.v_scale = b.op_scale[2]; f8.do_scale = b.op_scale[3];
    f8.p_scale = op->p_scale; f8.ds_scale = op->ds_scale;
    f8.q_codes = b.opc[0]; f8.k_codes = b.opc[1]; f8.v_codes = b.opc[2]; f8.do_codes = b.opc[3];
    f = &f8;
  }
  const float* do_scales = fp8 ? f8.do_scale : nullptr;

  // ---- once: forward output and LSE, the output store (per-(b,h) amax scale, stream 0)
  BSP_TRY(attn_fwd_impl(B, H, S, Dh, op->causal, c, q, k, v, dt, f, b.o, b.lse, diag, st));
  BSP_TRY(bsp_amax(b.o, BSP_F32, BH, (size_t)S * Dh, b.amax, diag, st));
  BSP_TRY(bsp_scale_from_amax(b.amax, BH, op->store_fmt, b.scales, st));
  bsp_key_t key;
  key.seed = op->seed; key.tensor_id = op->tensor_id; key.stream = BSP_STREAM_FORWARD; key.draw = 0; key.reserved = 0;
  BSP_TRY(bsp_round_grouped(b.o, BSP_F32, BH, (size_t)S * Dh, op->store_fmt, op->forward_mode, b.scales, key, b.codes,
                            diag, st));
  key.stream = BSP_STREAM_ATTN_D;

  // ---- reference: D reads the original output
  BSP_TRY(attn_dterm_impl(B, H, S, Dh, dO, dt, do_scales, b.o, b.codes, b.scales, op->store_fmt, BSP_READ_ORIGINAL,
                          key, 0, 1, b.d_ref, st));
  BSP_TRY(attn_bwd_dterm_impl(B, H, S, Dh, op->causal, c, q, k, v, dO, dt, f, b.lse, b.d_ref, b.g_ref[0], b.g_ref[1],
                              b.g_ref[2], diag, st));
  // the statistics passes are read behind one synchronisation at the end
  PendingStats pend;
  pend.slots = reinterpret_cast<double*>(b.ws_stats);
  pend.st = st;
  pend.rule = rule;
  int nres = 0;
  const int out_ids[4] = {BSP_OUT_D, BSP_OUT_DQ, BSP_OUT_DK, BSP_OUT_DV};
  auto emit = [&](int out, int pol) -> bsp_use_result_t* {
    bsp_use_result_t* r = &results[nres++];
    memset(r, 0, sizeof(*r));
    r->use_id = BSP_STREAM_ATTN_D; r->output_id = out; r->policy = pol;
    // FP8 operands: dQ and dK pass through the nearest rounding of dS, which is not linear in D
    r->informational = (fp8 && pol == BSP_READ_FRESH && (out == BSP_OUT_DQ || out == BSP_OUT_DK)) ? 1 : 0;
    return r;
  };
  for (int pol = 0; pol < 2; ++pol) {
    if (!((op->policy_mask >> pol) & 1u)) continue;
    const float* dsrc = b.d_ref;
    float* const* gsrc = b.g_ref;
    if (pol == BSP_READ_FORWARD) {
      BSP_TRY(attn_dterm_impl(B, H, S, Dh, dO, dt, do_scales, b.o, b.codes, b.scales, op->store_fmt, BSP_READ_FORWARD,
                              key, 0, 1, b.d_pol, st));
      BSP_TRY(attn_bwd_dterm_impl(B, H, S, Dh, op->causal, c, q, k, v, dO, dt, f, b.lse, b.d_pol, b.g_pol[0],
                                  b.g_pol[1], b.g_pol[2], diag, st));
      dsrc = b.d_pol;
      gsrc = b.g_pol;
    }
    BSP_TRY(pend.add(b.d_ref, dsrc, nullptr, (int64_t)rows, 1, 0, emit(out_ids[0], pol)));
    for (int t = 0; t < 3; ++t)
      BSP_TRY(pend.add(b.g_ref[t], gsrc[t], nullptr, (int64_t)n, 1, 0, emit(out_ids[t + 1], pol)));
  }
  if ((op->policy_mask >> 2) & 1u) {
    // fresh read: all K correction terms in one pass, and the sums of D itself in one launch
    BSP_TRY(attn_dterm_impl(B, H, S, Dh, dO, dt, do_scales, b.o, b.codes, b.scales, op->store_fmt, BSP_READ_FRESH, key,
                            0, K, b.d_draws, st));
    BSP_CHECK_CUDA(cudaMemsetAsync(b.S1d, 0, rows * 4, st));
    BSP_CHECK_CUDA(cudaMemsetAsync(b.S2d, 0, rows * 4, st));
    mc_accumulate_draws_kernel<<<(unsigned)((rows + 255) / 256), 256, 0, st>>>(b.d_draws, rows, K, b.d_ref, b.S1d, b.S2d,
                                                                              rows);
    BSP_LAUNCH_CHECK();
    for (int t = 0; t < 2; ++t) {
      BSP_CHECK_CUDA(cudaMemsetAsync(b.S1[t], 0, n * 4, st));
      BSP_CHECK_CUDA(cudaMemsetAsync(b.S2[t], 0, n * 4, st));
    }
    if (!fp8) {
      // dQ: P K once (the forward kernel with K in place of V and the rows' LSE given, so it takes one
      // pass over the keys; g_pol[0] is free by now), then the K draws collapse to one elementwise pass
      BSP_TRY(attn_fwd_impl(B, H, S, Dh, op->causal, c, q, k, k, dt, nullptr, b.g_pol[0], nullptr, diag, st, b.lse));
      attn_dq_sums_kernel<<<(unsigned)((n / 4 + 255) / 256), 256, 0, st>>>(b.g_pol[0], b.S1d, b.S2d, c, b.S1[0], b.S2[0],
                                                                          n / 4);
      BSP_LAUNCH_CHECK();
      // dK: four draws per launch
      for (int k0 = 0; k0 < K; k0 += kDkND) {
        const int nd = K - k0 < kDkND ? K - k0 : kDkND;
        BSP_TRY(attn_dk_diff((int)BH, S, op->causal, c, q, k, b.lse, b.d_ref, b.d_draws + (size_t)k0 * rows, nd, b.S1[1],
                             b.S2[1], diag, st));
      }
    } else {
      // the rounded backward once per draw; dQ and dK go from the accumulators straight into their sums
      // (two draws per launch: the scores, dP and the exponentials are formed once for both)
      for (int k0 = 0; k0 < K; k0 += 2)
        BSP_TRY(attn_bwd_dterm_mc(B, H, S, Dh, op->causal, c, q, k, v, dO, dt, f, b.lse, b.d_draws + (size_t)k0 * rows,
                                  K - k0 >= 2 ? 2 : 1, b.g_ref[0], b.S1[0], b.S2[0], b.g_ref[1], b.S1[1], b.S2[1], diag, st));
    }
    BSP_TRY(pend.add(b.d_ref, b.S1d, b.S2d, (int64_t)rows, K, 1, emit(out_ids[0], BSP_READ_FRESH)));
    for (int t = 0; t < 2; ++t)
      BSP_TRY(pend.add(b.g_ref[t], b.S1[t], b.S2[t], (int64_t)n, K, 1, emit(out_ids[t + 1], BSP_READ_FRESH)));
    // dV does not read the correction term: every draw is the reference itself
    pend.add_exact_fresh((int64_t)n, K, emit(out_ids[3], BSP_READ_FRESH));
  }
  *n_results = nres;
  return pend.flush();
}

}  // extern "C"
