// Causal softmax attention on the tensor cores: forward statistics and the backward whose
// correction term D = rowsum(dO o O_copy) reads a copy of the saved output chosen by policy.
//
//   P = softmax(c Q K^T), O = P V;  dV = P^T dO, dP = dO V^T, dS = P o (dP - D),
//   dQ = c dS K, dK = c dS^T Q.
//
// One kernel template, three modes, one CTA per (batch*head, 128-row block):
//   AT_DKV  the CTA owns key block j: K_j, V_j resident, streams (Q_i, dO_i) for i >= j,
//           accumulates dV_j and dK_j in tensor memory;
//   AT_DQ   the CTA owns query block i: Q_i, dO_i resident, streams (K_j, V_j) for j <= i,
//           accumulates dQ_i;
//   AT_FWD  the CTA owns query block i and takes one pass over j: per row and half of 64 keys a
//           running maximum m_h (moved lazily, only past 2^8) and O_h += exp(S - m_h) V in an
//           accumulator of its own, rescaled when m_h moves; the halves meet in the epilogue,
//           O_i = (w_0 O_0 + w_1 O_1), which also gives the row's log-sum-exp.
// No cross-CTA reduction exists in these modes, so results are bit-reproducible (the one-kernel
// form of the backward, further down, is the exception).
//
// Per inner step: S = Q K^T and dP = dO V^T (128x128x64 each; the dK/dV mode forms the transposes) land
// in TMEM columns [0,128) and [128,256); eight softmax warps (two per TMEM lane quarter, 64 columns
// each) turn them into P and dS and write those back into tensor memory as packed bf16 pairs (FP8-
// operand mode: as codes), where the accumulating products read them as their A operand, row per
// lane; the TMA-loaded 128 x 64 tiles are the MN-major B operands.  320 threads: warp 0 TMA, warp 1
// MMA (the whole warp walks the loop, one elected lane issues), warps 2..9 softmax + epilogue.
// Head dimension 64, bf16 inputs, FP32 outputs.  Every wait is bounded.
#include <string.h>

#include <atomic>


#include "attn_common.cuh"
#include "mc_stats.cuh"

namespace bsp {

constexpr int kAtThreads = 320;
constexpr int kAtSoftWarp0 = 2;                   // first softmax warp
constexpr int kAtSoftThread0 = kAtSoftWarp0 * 32;
// shared memory: 12 tiles of 16 KB (resident, ring, staging), barriers and small buffers, the extra-step tiles
constexpr int kAtBiasTile = AT_BLK * 16 * 2;      // 4 KB: one 128 x 16 bf16 tile of the extra K = 16 step (DKV)
constexpr int kAtBias = 7 * kAtBiasTile;          // a tile of ones, then three buffers of (LSE tile, D tile)
constexpr int kAtSmem = 12 * kAtTile + 1024 /*alignment*/ + 4096 /*barriers, exchange*/ +
                        kAtBias;

struct AttnParams {
  int BH, S, nblk;
  int causal;
  float c;                       // softmax scale
  const float* lse;              // [BH*S]  (DKV, DQ: input; FWD: unused)
  const float* dterm;            // [BH*S]  (DKV, DQ)
  float* out0;                   // DKV: dV   DQ: dQ   FWD: O      [BH*S*64]
  float* out1;                   // DKV: dK                         [BH*S*64]
  float* out2;                   // DKV with the fused dQ: dQ (zero at launch), else NULL
  float* lse_out;                // FWD
  // Monte-Carlo epilogue (DQ, and DKV without dV): instead of storing the gradient g, the kernel adds
  // g - mc_ref to out0 and (g - mc_ref)^2 to out1 (the running sums S1, S2 of that gradient)
  const float* mc_ref;           // [BH*S*64] or NULL
  int nd;                        // draws per launch (1; 2 in the Monte-Carlo dQ kernel: dterm holds [2][BH*S])
  bsp_diag_t* diag;
  // FP8-operand mode: q, k, v, dO hold decoded FP8 codes (exact in bf16); their per-(b,h) scales
  // are folded into the softmax argument, dP and the outputs; P and dS are rounded onto the E4M3 /
  // E5M2 grids (at p_scale / ds_scale) before their products.  All NULL / 0 in BF16-operand mode.
  int fp8;
  const float* sc_q;             // [BH]
  const float* sc_k;
  const float* sc_v;
  const float* sc_do;
  float p_scale, ds_scale;
  const uint8_t *cq, *ck, *cv, *cdo;   // the operands' codes: what the backward modes load in FP8-operand mode
};

// Two floats rounded to the nearest FP8 grid value (ties to even, saturating: what f8_rn_value
// gives) and packed as a bf16 pair, through the hardware conversions: f32 pair -> FP8 pair -> f16 pair
// (every FP8 value is an f16 value) -> f32 -> bf16 pair (every FP8 value is a bf16 value too).
template <int FMT>
__device__ __forceinline__ uint32_t f8_grid_bf16x2(float lo, float hi) {
  const uint16_t c = (uint16_t)f8_encode_rn_pair_inrange<FMT>(lo, hi);
  uint32_t h2;
  if (FMT == BSP_E4M3) asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(c));
  else asm("cvt.rn.f16x2.e5m2x2 %0, %1;" : "=r"(h2) : "h"(c));
  const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&h2));
  return pack_bf16x2(f.x, f.y);
}

// FP8: the FP8-operand mode (per-head operand scales, P and dS rounded onto the FP8 grids); a
// template parameter because its tests and extra multiplications sit in the innermost loop.
// DV (dK/dV mode only): false leaves dV out (its product, the P operand and its store): dV does
// not read the correction term, so the draws of a fresh read need it once, not K times.
// MC: the Monte-Carlo epilogue (see AttnParams::mc_ref); a template parameter so that the plain
// kernels carry none of its registers.
// ND (Monte-Carlo dQ and dK kernels only): draws per launch.  S, dP and P do not depend on the correction
// term, so with ND = 2 a step forms them once and builds two dS operands, one per draw's D (at
// p.dterm and p.dterm + BH*S), into two accumulators; the epilogue adds both draws to the sums.
// DQF (dK/dV mode, BF16 operands only): the same CTA also forms the step's share of dQ, dS_ij K_j, and
// adds it to dQ in global memory (one tiled bulk reduce-add per step and column half), so S, dP and
// the exponentials are formed once per score tile for all three gradients.  dS^T then goes to
// shared memory instead of tensor memory (K-major A operand of dK, MN-major A operand of dQ) and
// the tile ring has two stages.  dQ must hold zeros at launch; the order of its FP32 additions is
// not fixed, so dQ is not bit-reproducible in this form.
template <int MODE, bool FP8, bool DV, bool MC, int ND, bool DQF = false>
__global__ void __launch_bounds__(kAtThreads, 1)
attn_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
            const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
            const __grid_constant__ CUtensorMap tm_o0, const __grid_constant__ CUtensorMap tm_o1,
            const __grid_constant__ CUtensorMap tm_o2, AttnParams p) {
  static_assert(!DQF || (MODE == AT_DKV && !FP8 && DV && !MC && ND == 1), "fused dQ: plain BF16 dK/dV kernel only");
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  // shared memory, in 16 KB tiles: resident tiles [2 buffers][2 tiles]; the ring of streamed tiles
  // [3 stages][2 tiles] (the one-kernel form: 2 stages, the third's space holds dS^T); 32 KB of staging
  // (second output of the dK/dV epilogue, dQ shares of the one-kernel form); barriers and small buffers
  const uint32_t res_base = base;
  const uint32_t str0 = base + 4 * kAtTile;                 // stage s: str0 + s*2*kAtTile (+kAtTile for the 2nd tile)
  const uint32_t bars = base + 12 * kAtTile;
  // barriers (8 bytes each): res_full[2], res_empty[2], str_full[2], str_empty[2], sdp_full, sdp_free,
  // pds_ready, pds_free, acc_full[2], acc_free[2]
  const uint32_t b_res = bars, b_res_empty = bars + 16, b_sfull = bars + 32, b_sempty = bars + 64,
                 b_sdp_full = bars + 96, b_sdp_free = bars + 104, b_pds_ready = bars + 112, b_pds_free = bars + 120,
                 b_acc = bars + 128, b_acc_free = bars + 144;
  constexpr uint32_t kStg = DQF ? 2u : 3u;
  auto stage_at = [&](uint32_t s) -> uint32_t { return str0 + s * 2u * kAtTile; };
  const uint32_t dst_buf = str0 + 2u * 2u * kAtTile;         // DQF: dS^T [128 keys][2 halves of 64 queries], 32 KB
  const uint32_t stage2 = str0 + 3u * 2u * kAtTile;
  uint8_t* gen = smem_raw + (base - raw);
  uint8_t* bars_gen = gen + 12 * kAtTile;
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bars_gen + 160);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars_gen + 164);
  float* xchg = reinterpret_cast<float*>(bars_gen + 176);   // FWD: row max / sum exchange between column halves
  // DKV: per-query terms enter the scores through the products themselves.  A thread of that mode
  // owns a key row, so the query's -LSE and -D would be per-column values (a shared-memory load in
  // front of every exponential: measured at twice the arithmetic time).  Instead S^T = K Q^T takes one
  // more K = 16 step, ones[keys x 16] times X[queries x 16]^T, where row q of X holds
  // -LSE[q] * log2(e) / c2 split into three bf16 terms (24 bits) and zeros, so the accumulator
  // already is s - LSE/c; likewise dP^T with -D[q].  The tiles are K-major without swizzle: 8-row
  // groups 256 bytes apart, the two 8-element halves of a row 128 bytes apart, 16 bytes per row.
  const uint32_t b_bias = bars + 2240;                       // three barriers, one per buffer
  const uint32_t bias0 = bars + 4096;                        // ones tile; buffer b: X_lse at 1 + 2b, X_d at 2 + 2b

  // dK kernel with two draws: the extra product step carries the first draw's -D; the second draw
  // needs, per query (a column of S^T), delta = D_first - D_second, kept as FP32 in three buffers of
  // 128 values that the threads writing the X tiles fill alongside them
  const uint32_t delta0 = bars + 2304;
  // DQF: the step's dQ share is complete / has been read out of tensor memory
  const uint32_t b_dq_full = bars + 3848, b_dq_free = bars + 3856;
  // Plain dQ kernel: the two halves of 64 keys of a step are two pipelines (their own S and dP
  // products, 128 x 64 each, their own hand-over barriers with the four softmax warps that own those
  // columns, their own share of the dQ product), issued in turn by the one MMA warp, so that one half's
  // hand-overs run under the other half's work.
  constexpr bool PP = (MODE == AT_DQ || MODE == AT_FWD) && !FP8 && !MC && ND == 1;
  const uint32_t b_sdp_full1 = bars + 3864, b_sdp_free1 = bars + 3872, b_pds_ready1 = bars + 3880, b_pds_free1 = bars + 3888;
  const uint32_t id_sdp64 = make_idesc(1u, 1u, 128, 64);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Persistent CTA: work items w = item_at(0), item_at(1), ... of nblk * BH, heavy blocks first
  // (item rank 0 is the block with most inner steps).  Resident tiles and accumulators are
  // double-buffered across items, so the next item's loads and first products run under this
  // item's tail and epilogue; barrier phases simply keep counting across items.
  const int nitems = p.nblk * p.BH;
  // the CTA's n-th item: rounds of gridDim.x items, walked forwards and backwards in turn, so the CTA
  // that got the heaviest item of one round gets the lightest of the next
  auto item_at = [&](int n) -> int {
    const int b = (int)blockIdx.x, G = (int)gridDim.x;
    return n * G + ((n & 1) ? G - 1 - b : b);
  };
  auto decode_item = [&](int w, int& blk, int& bh, int& it_begin, int& nsteps) {
    const int rank = w / p.BH;
    bh = w % p.BH;
    int it_end;
    if (MODE == AT_DKV) {
      blk = rank;                                            // key block j: steps i = j .. nblk-1 (causal)
      it_begin = p.causal ? blk : 0; it_end = p.nblk;
    } else {
      blk = p.nblk - 1 - rank;                               // query block i: steps j = 0 .. i (causal)
      it_begin = 0; it_end = p.causal ? blk + 1 : p.nblk;
    }
    nsteps = it_end - it_begin;
  };
  // FWD takes one pass over the keys with a running maximum per row and column half (the two halves
  // of a row keep separate accumulators, so no maximum crosses warps); with the rows' log-sum-exp
  // already known (p.lse) the shift is fixed: P = exp(s - LSE) directly
  const bool lse_known = MODE == AT_FWD && p.lse != nullptr;
  constexpr int npass = 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < 2; ++s) {
      mbar_init(b_res + 8 * s, 1); mbar_init(b_res_empty + 8 * s, 1);
      mbar_init(b_acc + 8 * s, 1); mbar_init(b_acc_free + 8 * s, 8);
    }
    for (uint32_t s = 0; s < kStg; ++s) { mbar_init(b_sfull + 8 * s, 1); mbar_init(b_sempty + 8 * s, 1); }
    for (uint32_t s = 0; s < 3; ++s) mbar_init(b_bias + 8 * s, 8);
    mbar_init(b_sdp_full, 1); mbar_init(b_sdp_free, PP ? 4 : 8); mbar_init(b_pds_ready, PP ? 4 : 8); mbar_init(b_pds_free, 1);
    mbar_init(b_sdp_full1, 1); mbar_init(b_sdp_free1, 4); mbar_init(b_pds_ready1, 4); mbar_init(b_pds_free1, 1);
    mbar_init(b_dq_full, 1); mbar_init(b_dq_free, 8);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // TMEM columns: S [0,128), dP [128,256).  FWD: accumulator buffer ab at 256 + 128*ab.  DKV / DQ: the
  // bf16 operands P and dS as the softmax warps write them back (64 columns each: two elements per
  // column) at [256,320) and [320,384), and one accumulator buffer of two 64-column halves at 384.
  const uint32_t t_s = tmem, t_dp = tmem + 128, t_p = tmem + 256, t_ds = tmem + 320;
  // two draws (dQ kernel): the second draw's dS operand takes the P columns (no product reads P
  // there) and its accumulator the second half of the accumulator buffer
  const uint32_t t_ds2 = tmem + 256;
  const uint32_t t_dq = tmem + 320;                           // DQF: the step's dQ share (dS^T is in shared memory)
  const uint32_t t_accbase = MODE == AT_FWD ? tmem + 256 : tmem + 384;
  constexpr bool kAccDouble = MODE == AT_FWD;   // accumulators double-buffered across items

  // instruction descriptors (bf16 operands, FP32 accumulation)
  const uint32_t id_sdp = make_idesc(1u, 1u, 128, 128);                                   // A, B K-major
  const uint32_t id_kmn = make_idesc(1u, 1u, 128, 64) | (1u << 16);                       // A K-major, B MN-major
  const uint32_t id_mn = make_idesc(1u, 1u, 128, 64) | (1u << 15) | (1u << 16);           // A, B MN-major
  // FP8-operand mode of the backward: every product is an FP8 tensor-core product (kind::f8f6f4) on the
  // codes themselves.  The streamed and resident tiles are 128 rows of 64 bytes (64-byte swizzle), a
  // K step is 32 elements, and P (E4M3) and dS (E5M2) go back into tensor memory four codes per column.
  constexpr bool F8K = FP8 && MODE != AT_FWD;
  constexpr uint32_t kTileB = F8K ? (uint32_t)(AT_BLK * AT_D) : (uint32_t)kAtTile;        // bytes a tile load brings
  // operand formats (E4M3 = 0, E5M2 = 1): S from Q and K; dP from dO (E5M2) and V
  const uint32_t id8_s = make_idesc(0u, 0u, 128, 128);
  const uint32_t id8_dp = MODE == AT_DKV ? make_idesc(0u, 1u, 128, 128) : make_idesc(1u, 0u, 128, 128);
  const uint32_t id8_pdo = make_idesc(0u, 1u, 128, 64) | (1u << 16);                      // P^T (E4M3) x dO (E5M2, MN-major)
  const uint32_t id8_ds = make_idesc(1u, 0u, 128, 64) | (1u << 16);                       // dS (E5M2) x Q or K (E4M3, MN-major)

  if (warp == 0) {
    // ------------------------------------------------ TMA producer
    if (lane == 0) {
      tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_k); tma_prefetch_desc(&tm_v); tma_prefetch_desc(&tm_do);
      bool ok = true;
      uint32_t itg = 0;                                       // step counter across items
      int item = 0;
      for (int w = item_at(0); w < nitems && ok; w = item_at(++item)) {
        int blk, bh, it_begin, nsteps;
        decode_item(w, blk, bh, it_begin, nsteps);
        // resident tiles of this item, into the buffer the item before last has released
        const uint32_t rb = item & 1u, rph = (item >> 1) & 1u;
        if (!mbar_wait(b_res_empty + 8 * rb, rph ^ 1u, abort_flag)) { ok = false; break; }
        const uint32_t r0 = res_base + rb * 2 * kAtTile, r1 = r0 + kAtTile;
        mbar_expect_tx(b_res + 8 * rb, (MODE == AT_FWD ? 1 : 2) * kTileB);
        if (MODE == AT_DKV) {
          tma_load_3d(r0, &tm_k, b_res + 8 * rb, 0, blk * AT_BLK, bh);
          tma_load_3d(r1, &tm_v, b_res + 8 * rb, 0, blk * AT_BLK, bh);
        } else {
          tma_load_3d(r0, &tm_q, b_res + 8 * rb, 0, blk * AT_BLK, bh);
          if (MODE == AT_DQ) tma_load_3d(r1, &tm_do, b_res + 8 * rb, 0, blk * AT_BLK, bh);
        }
        const int total = nsteps * npass;
        for (int it = 0; it < total; ++it, ++itg) {
          const int step = it_begin + (it % nsteps);
          const uint32_t s = itg % kStg, ph = (itg / kStg) & 1u;
          if (!mbar_wait(b_sempty + 8 * s, ph ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t d0 = stage_at(s), d1 = d0 + kAtTile;
          mbar_expect_tx(b_sfull + 8 * s, 2 * kTileB);
          if (MODE == AT_DKV) {
            tma_load_3d(d0, &tm_q, b_sfull + 8 * s, 0, step * AT_BLK, bh);
            tma_load_3d(d1, &tm_do, b_sfull + 8 * s, 0, step * AT_BLK, bh);
          } else {
            tma_load_3d(d0, &tm_k, b_sfull + 8 * s, 0, step * AT_BLK, bh);
            tma_load_3d(d1, &tm_v, b_sfull + 8 * s, 0, step * AT_BLK, bh);
          }
        }
      }
      if (!ok) for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
  } else if (warp == 1) {
    // ------------------------------------------------ MMA issuer
    {
      // the whole warp walks the loop (loop control and descriptor arithmetic stay warp-uniform); one
      // lane issues.  Measured: a 128 x 64 x 16 product with A in tensor memory issues every 32 cycles
      // this way, every 45 from a single-lane branch.
      const uint32_t leader = elect_one() ? 1u : 0u;
      auto wait_all = [&](uint32_t bar, uint32_t parity) -> bool {
        return __all_sync(0xFFFFFFFFu, mbar_wait(bar, parity, abort_flag));
      };
      bool ok = true;
      uint32_t itg = 0;                                       // step counter across items
      int item = 0;
      for (int w = item_at(0); w < nitems && ok; w = item_at(++item)) {
      int blk, bh, it_begin, nsteps;
      decode_item(w, blk, bh, it_begin, nsteps);
      const int total = nsteps * npass;
      const uint32_t rb = item & 1u, iph = (item >> 1) & 1u;  // resident buffer and its phase
      // accumulator buffer and its phase: alternating with the items (FWD), else the one buffer
      const uint32_t ab = kAccDouble ? rb : 0u, aph = kAccDouble ? iph : ((uint32_t)item & 1u);
      const uint32_t res0 = res_base + rb * 2 * kAtTile, res1 = res0 + kAtTile;
      const uint32_t t_acc0 = t_accbase + ab * 128, t_acc1 = t_acc0 + 64;
      if (!wait_all(b_res + 8 * rb, iph)) { ok = false; break; }
      // the accumulators are free once the epilogue that last used them is done: with two buffers
      // that is checked here, with one just before the item's first accumulating product, so the
      // first S and dP of this item already run under the epilogue of the item before
      if (kAccDouble && !wait_all(b_acc_free + 8 * ab, aph ^ 1u)) { ok = false; break; }
      // S = Q K^T (and dP = dO V^T) of global step `jt`: both operands K-major, 64 = 4 x 16 along K.
      // Issued one step ahead: the softmax warps release the S / dP columns as soon as they hold
      // them in registers, so these products overlap the softmax arithmetic of the step before.
      auto issue_sdp = [&](uint32_t jt) -> bool {
        const uint32_t s = jt % kStg, ph = (jt / kStg) & 1u;
        if (!wait_all(b_sfull + 8 * s, ph)) return false;
        if (!wait_all(b_sdp_free, (jt & 1u) ^ 1u)) return false;
        tc_fence_after();
        const uint32_t st0 = stage_at(s), st1 = st0 + kAtTile;
        const uint32_t q_t = MODE == AT_DKV ? st0 : res0, k_t = MODE == AT_DKV ? res0 : st0;
        const uint32_t do_t = MODE == AT_DKV ? st1 : res1, v_t = MODE == AT_DKV ? res1 : st1;
        // DKV forms the transposes, S^T = K Q^T and dP^T = V dO^T (rows = keys), so that P^T and dS^T
        // come out of the softmax warps as the row-per-lane A operands of dV = P^T dO, dK = dS^T Q
        if (F8K) {
          // 64 bytes of K per row: two steps of 32 elements
          const uint64_t a = make_smem_desc_sw64(MODE == AT_DKV ? k_t : q_t), b = make_smem_desc_sw64(MODE == AT_DKV ? q_t : k_t);
#pragma unroll
          for (int k = 0; k < 2; ++k) tc_mma_l<true>(leader, t_s, a + 2u * k, b + 2u * k, id8_s, k != 0);
          const uint64_t a2 = make_smem_desc_sw64(MODE == AT_DKV ? v_t : do_t), b2 = make_smem_desc_sw64(MODE == AT_DKV ? do_t : v_t);
#pragma unroll
          for (int k = 0; k < 2; ++k) tc_mma_l<true>(leader, t_dp, a2 + 2u * k, b2 + 2u * k, id8_dp, k != 0);
        } else {
          {
            const uint64_t a = make_smem_desc(MODE == AT_DKV ? k_t : q_t), b = make_smem_desc(MODE == AT_DKV ? q_t : k_t);
#pragma unroll
            for (int k = 0; k < 4; ++k) tc_mma_l<false>(leader, t_s, a + 2u * k, b + 2u * k, id_sdp, k != 0);
          }
          if (MODE != AT_FWD) {
            const uint64_t a = make_smem_desc(MODE == AT_DKV ? v_t : do_t), b = make_smem_desc(MODE == AT_DKV ? do_t : v_t);
#pragma unroll
            for (int k = 0; k < 4; ++k) tc_mma_l<false>(leader, t_dp, a + 2u * k, b + 2u * k, id_sdp, k != 0);
          }
        }
        if (MODE == AT_DKV) {
          // the extra K = 16 step: minus LSE/c into S^T, minus D into dP^T (see the X tiles)
          const uint32_t bb = jt % 3u;
          if (!wait_all(b_bias + 8 * bb, (jt / 3u) & 1u)) return false;
          const uint64_t ones = make_smem_desc_k16(bias0);
          tc_mma_l<false>(leader, t_s, ones, make_smem_desc_k16(bias0 + (1u + 2u * bb) * kAtBiasTile), id_sdp, 1u);
          tc_mma_l<false>(leader, t_dp, ones, make_smem_desc_k16(bias0 + (2u + 2u * bb) * kAtBiasTile), id_sdp, 1u);
        }
        tc_commit_l(leader, b_sdp_full);
        return true;
      };
      // PP: S and dP of half hh (keys 64 hh .. 64 hh + 63 of the step's tiles) of global step jt
      auto issue_half = [&](uint32_t jt, uint32_t hh) -> bool {
        const uint32_t s = jt % kStg, ph = (jt / kStg) & 1u;
        if (hh == 0 && !wait_all(b_sfull + 8 * s, ph)) return false;   // (the second half follows the first: the tiles have landed)
        if (!wait_all(hh ? b_sdp_free1 : b_sdp_free, (jt & 1u) ^ 1u)) return false;
        tc_fence_after();
        const uint32_t st0 = stage_at(s), st1 = st0 + kAtTile;
        const uint64_t a = make_smem_desc(res0), b = make_smem_desc(st0 + hh * 8192u);
#pragma unroll
        for (int k = 0; k < 4; ++k) tc_mma_l<false>(leader, t_s + 64u * hh, a + 2u * k, b + 2u * k, id_sdp64, k != 0);
        if (MODE != AT_FWD) {
          const uint64_t a2 = make_smem_desc(res1), b2 = make_smem_desc(st1 + hh * 8192u);
#pragma unroll
          for (int k = 0; k < 4; ++k) tc_mma_l<false>(leader, t_dp + 64u * hh, a2 + 2u * k, b2 + 2u * k, id_sdp64, k != 0);
        }
        tc_commit_l(leader, hh ? b_sdp_full1 : b_sdp_full);
        return true;
      };
      if (PP) {
        if (ok && total > 0) ok = issue_half(itg, 0u) && issue_half(itg, 1u);
        for (int it = 0; it < total && ok; ++it) {
          const uint32_t jg = itg + (uint32_t)it;
          const uint32_t s = jg % kStg, ip = jg & 1u;
          const uint64_t bk = make_smem_desc_mn(stage_at(s) + (MODE == AT_FWD ? kAtTile : 0u), 16384u);   // dQ: K; forward: V
          // in turn: the next step's S and dP of a half, then this step's dQ share of that half (taking
          // both halves' S and dP first, or giving each half an MMA warp of its own, measured slower)
#pragma unroll
          for (uint32_t hh = 0; hh < 2; ++hh) {
            if (it + 1 < total && !issue_half(jg + 1, hh)) { ok = false; break; }
            if (!wait_all(hh ? b_pds_ready1 : b_pds_ready, ip)) { ok = false; break; }
            tc_fence_after();
            if (!kAccDouble && it == 0 && hh == 0 && !wait_all(b_acc_free + 8 * ab, aph ^ 1u)) { ok = false; break; }
            if (MODE == AT_FWD) {
              // O_hh += P_hh V_hh into the half's own accumulator
#pragma unroll
              for (uint32_t k = 0; k < 4; ++k)
                tc_mma_ts_l<false>(leader, hh ? t_acc1 : t_acc0, t_dp + 32u * hh + 8u * k, bk + 128u * (4u * hh + k), id_kmn,
                                   (it != 0 || k != 0) ? 1u : 0u);
            } else {
              // dQ += dS_hh K_hh: 64 keys = 4 x 16 along K
#pragma unroll
              for (uint32_t k = 0; k < 4; ++k)
                tc_mma_ts_l<false>(leader, t_acc0, t_ds + 32u * hh + 8u * k, bk + 128u * (4u * hh + k), id_kmn,
                                   (it != 0 || hh != 0 || k != 0) ? 1u : 0u);
            }
            tc_commit_l(leader, hh ? b_pds_free1 : b_pds_free);
          }
          if (!ok) break;
          tc_commit_l(leader, b_sempty + 8 * s);
        }
      } else {
      if (ok && total > 0) ok = issue_sdp(itg);
      for (int it = 0; it < total && ok; ++it) {
        const uint32_t jg = itg + (uint32_t)it;
        const uint32_t s = jg % kStg, ip = jg & 1u;
        const uint32_t st0 = stage_at(s), st1 = st0 + kAtTile;
        if (it + 1 < total && !issue_sdp(jg + 1)) { ok = false; break; }
        if (!wait_all(b_pds_ready, ip)) { ok = false; break; }
        tc_fence_after();
        const uint32_t first = it == 0 ? 0u : 1u;             // overwrite on the first product
        if (!kAccDouble && it == 0 && !wait_all(b_acc_free + 8 * ab, aph ^ 1u)) { ok = false; break; }
        if (F8K && MODE == AT_DKV) {
          // the same products on the codes: eight columns per 32 queries, 128 queries = 4 x 32 along K
          const uint64_t bdo = make_smem_desc_mn_sw64(st1), bq = make_smem_desc_mn_sw64(st0);
          if (DV) {
#pragma unroll
            for (int k = 0; k < 4; ++k) tc_mma_ts_l<true>(leader, t_acc0, t_p + 8u * k, bdo + 128u * k, id8_pdo, first | (k != 0));
          }
#pragma unroll
          for (int k = 0; k < 4; ++k) tc_mma_ts_l<true>(leader, t_acc1, t_ds + 8u * k, bq + 128u * k, id8_ds, first | (k != 0));
          if (ND == 2 && !DV) {
#pragma unroll
            for (int k = 0; k < 4; ++k) tc_mma_ts_l<true>(leader, t_acc0, t_ds2 + 8u * k, bq + 128u * k, id8_ds, first | (k != 0));
          }
        } else if (F8K && MODE == AT_DQ) {
          const uint64_t bk = make_smem_desc_mn_sw64(st0);
#pragma unroll
          for (int k = 0; k < 4; ++k) tc_mma_ts_l<true>(leader, t_acc0, t_ds + 8u * k, bk + 128u * k, id8_ds, first | (k != 0));
          if (ND == 2) {
#pragma unroll
            for (int k = 0; k < 4; ++k) tc_mma_ts_l<true>(leader, t_acc1, t_ds2 + 8u * k, bk + 128u * k, id8_ds, first | (k != 0));
          }
        } else if (DQF) {
          // dV += P^T dO with P^T from tensor memory; dK += dS^T Q with dS^T K-major from shared memory
          // (two halves of 64 queries, four K = 16 steps each); then the step's dQ share = dS K_j: the same
          // buffer read MN-major (128 queries wide, 16 keys per step), K_j = the resident tile, MN-major
          const uint64_t bdo = make_smem_desc_mn(st1, 16384u), bq = make_smem_desc_mn(st0, 16384u);
#pragma unroll
          for (int k = 0; k < 8; ++k) tc_mma_ts_l<false>(leader, t_acc0, t_p + 8u * k, bdo + 128u * k, id_kmn, first | (k != 0));
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const uint64_t a = make_smem_desc(dst_buf + (k >> 2) * 16384u + (k & 3) * 32u);
            tc_mma_l<false>(leader, t_acc1, a, bq + 128u * k, id_kmn, first | (k != 0));
          }
          // the share of the step before has left tensor memory
          if (!wait_all(b_dq_free, (jg & 1u) ^ 1u)) { ok = false; break; }
          tc_fence_after();
          const uint64_t ads = make_smem_desc_mn(dst_buf, 16384u), bk = make_smem_desc_mn(res0, 16384u);
#pragma unroll
          for (int k = 0; k < 8; ++k) tc_mma_l<false>(leader, t_dq, ads + 128u * k, bk + 128u * k, id_mn, k != 0);
          tc_commit_l(leader, b_dq_full);
        } else if (MODE == AT_DKV) {
          // dV += P^T dO, dK += dS^T Q : A from tensor memory (row = key, eight columns per 16
          // queries), B MN-major = the streamed 128 x 64 tiles; 128 queries = 8 x 16 along K
          const uint64_t bdo = make_smem_desc_mn(st1, 16384u), bq = make_smem_desc_mn(st0, 16384u);
          if (DV) {
#pragma unroll
            for (int k = 0; k < 8; ++k) tc_mma_ts_l<false>(leader, t_acc0, t_p + 8u * k, bdo + 128u * k, id_kmn, first | (k != 0));
          }
#pragma unroll
          for (int k = 0; k < 8; ++k) tc_mma_ts_l<false>(leader, t_acc1, t_ds + 8u * k, bq + 128u * k, id_kmn, first | (k != 0));
          if (ND == 2 && !DV) {
            // second draw: its dS^T operand sits in the P columns, its dK in the dV accumulator
#pragma unroll
            for (int k = 0; k < 8; ++k) tc_mma_ts_l<false>(leader, t_acc0, t_ds2 + 8u * k, bq + 128u * k, id_kmn, first | (k != 0));
          }
        } else if (MODE == AT_DQ) {
          // dQ += dS K : A from tensor memory (row = query, eight columns per 16 keys), B MN-major = streamed K
          const uint64_t bk = make_smem_desc_mn(st0, 16384u);
#pragma unroll
          for (int k = 0; k < 8; ++k) tc_mma_ts_l<false>(leader, t_acc0, t_ds + 8u * k, bk + 128u * k, id_kmn, first | (k != 0));
          if (ND == 2) {
#pragma unroll
            for (int k = 0; k < 8; ++k) tc_mma_ts_l<false>(leader, t_acc1, t_ds2 + 8u * k, bk + 128u * k, id_kmn, first | (k != 0));
          }
        } else {
          // O_h += P_h V_h for the two halves of 64 keys, each into its own accumulator (its own running
          // maximum): A = P from tensor memory (eight columns per 16 keys), B MN-major = streamed V
          const uint64_t bk = make_smem_desc_mn(st1, 16384u);
#pragma unroll
          for (int k = 0; k < 8; ++k)
            tc_mma_ts_l<false>(leader, k < 4 ? t_acc0 : t_acc1, t_dp + 8u * k, bk + 128u * k, id_kmn, first | ((k & 3) != 0));
        }
        tc_commit_l(leader, b_pds_free);
        tc_commit_l(leader, b_sempty + 8 * s);
      }
      }
      itg += (uint32_t)total;
      if (ok) {
        // this item's accumulators are complete (and its resident tiles no longer read: the epilogue
        // stages the output through their buffer and releases it)
        tc_commit_l(leader, b_acc + 8 * ab);
      }
      }  // items
    }
  } else if (warp >= kAtSoftWarp0) {
    // ------------------------------------------------ softmax / dS warps, then the epilogue
    const int q4 = warp & 3, h = (warp - kAtSoftWarp0) >> 2;
    const int r = q4 * 32 + lane;                             // row inside the 128-row block (a query)
    const uint32_t lane_off = (uint32_t)(q4 * 32) << 16;
    if (MODE == AT_DKV) {
      // the constant parts of the seven extra tiles: thread ts sets 16 bytes of each (row ts & 127,
      // half ts >> 7): the first three columns of the ones tile to 1, everything else to 0
      const int ts0 = (int)threadIdx.x - kAtSoftThread0;
      const uint32_t off = (uint32_t)((ts0 & 127) >> 3) * 256u + (uint32_t)(ts0 >> 7) * 128u + (uint32_t)(ts0 & 7) * 16u;
#pragma unroll
      for (uint32_t t = 0; t < 7; ++t) {
        const bool one = t == 0 && ts0 < 128;
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %3};" ::"r"(bias0 + t * kAtBiasTile + off),
                     "r"(one ? 0x3F803F80u : 0u), "r"(one ? 0x00003F80u : 0u), "r"(0u) : "memory");
      }
      named_bar_sync(1, 256);   // before any thread overwrites a row's first half with a step's terms
    }
    bool ok = true;
    uint32_t bias_written = 0;                                // DKV: rows of the X tiles written so far (global steps)
    bool store_pending = false;                               // warp 2, lane 0: an epilogue's bulk stores are in flight
    bool red_pending = false;                                 // warp 2, lane 0 (DQF): a dQ share's reduce-adds are in flight
    uint32_t itg = 0;                                         // step counter across items
    int item = 0;
    for (int w = item_at(0); w < nitems && ok; w = item_at(++item)) {
    int blk, bh, it_begin, nsteps;
    decode_item(w, blk, bh, it_begin, nsteps);
    const int total = nsteps * npass;
    // accumulator buffer of this item and its phase (see the MMA issuer)
    const uint32_t ab = kAccDouble ? (item & 1u) : 0u;
    const uint32_t iph = kAccDouble ? ((item >> 1) & 1u) : ((uint32_t)item & 1u);
    const uint32_t t_acc0 = t_accbase + ab * 128, t_acc1 = t_acc0 + 64;
    float inv_q = 1.f, inv_k = 1.f, inv_v = 1.f, inv_do = 1.f;
    if (FP8) {
      inv_q = __fdiv_rn(1.0f, __ldg(p.sc_q + bh)); inv_k = __fdiv_rn(1.0f, __ldg(p.sc_k + bh));
      inv_v = __fdiv_rn(1.0f, __ldg(p.sc_v + bh)); inv_do = __fdiv_rn(1.0f, __ldg(p.sc_do + bh));
    }
    const float c2 = FP8 ? p.c * kLog2e * inv_q * inv_k : p.c * kLog2e;   // scores arrive as products of decoded codes
    const float dp_mul = FP8 ? inv_do * inv_v : 1.0f;                     // likewise dP
    // DKV: softmax thread ts owns row (ts & 127) of the X tiles: the LSE tile for ts < 128, the D tile
    // above.  bias_fetch reads the raw value of a step's query (nothing may depend on that load
    // before the step's arithmetic is done, or the in-order warp sits out its latency); bias_put
    // writes the three-term row into buffer (global step) % 3 and signals the MMA issuer.
    const int ts = (int)threadIdx.x - kAtSoftThread0;
    const float* bias_src = ts < 128 ? p.lse : p.dterm;
    const float bias_mul = ts < 128 ? -kLog2e / c2 : -1.0f / dp_mul;
    float nx_mul = bias_mul;                                  // the same factor for the next item's head
    auto bias_fetch = [&](int tbh, int step) -> float {
      const int q = step * AT_BLK + (ts & 127);
      return __ldg(bias_src + (size_t)tbh * p.S + (q < p.S ? q : 0));
    };
    // the second draw's correction term of the same query (threads of the D tile only)
    auto bias_fetch2 = [&](int tbh, int step) -> float {
      if (ND != 2 || ts < 128) return 0.f;
      const int q = step * AT_BLK + (ts & 127);
      return __ldg(p.dterm + (size_t)p.BH * p.S + (size_t)tbh * p.S + (q < p.S ? q : 0));
    };
    auto bias_put = [&](int step, uint32_t jt, float raw, float mul, float raw2) {
      const int q = ts & 127;
      if (ND == 2 && ts >= 128) {
        const float dl = step * AT_BLK + q < p.S ? raw - raw2 : 0.f;
        asm volatile("st.shared.f32 [%0], %1;" ::"r"(delta0 + ((jt % 3u) * 128u + (uint32_t)q) * 4u), "f"(dl) : "memory");
      }
      const float x = step * AT_BLK + q < p.S ? raw * mul : 0.f;
      const __nv_bfloat16 h1 = __float2bfloat16_rn(x);
      const float r1 = x - __bfloat162float(h1);
      const __nv_bfloat16 h2 = __float2bfloat16_rn(r1);
      const __nv_bfloat16 h3 = __float2bfloat16_rn(r1 - __bfloat162float(h2));
      const uint32_t w0 = (uint32_t)__bfloat16_as_ushort(h1) | ((uint32_t)__bfloat16_as_ushort(h2) << 16);
      const uint32_t w1 = (uint32_t)__bfloat16_as_ushort(h3);
      const uint32_t tile = bias0 + (1u + 2u * (jt % 3u) + (ts < 128 ? 0u : 1u)) * kAtBiasTile;
      asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %3};" ::"r"(tile + (uint32_t)(q >> 3) * 256u + (uint32_t)(q & 7) * 16u),
                   "r"(w0), "r"(w1), "r"(0u) : "memory");
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(b_bias + 8 * (jt % 3u));
    };
    // The rows are written two steps ahead of their use, in the order of the CTA's global step count
    // (bias_written rows so far), across item boundaries: the last two steps of an item write the first
    // two rows of the next one, so its first S and dP run under this item's epilogue.  Rows that are
    // still missing at an item's start (the first item, or after a one-step item) are written here.
    int nx_bh = 0, nx_begin = 0, nx_total = 0;                // DKV: the next item's head, first step, step count
    if (MODE == AT_DKV) {
      const int wn = item_at(item + 1);
      if (wn < nitems) {
        int nb, ns;
        decode_item(wn, nb, nx_bh, nx_begin, ns);
        nx_total = ns;
        if (FP8) {                                            // per-head operand scales
          const float nq = __fdiv_rn(1.0f, __ldg(p.sc_q + nx_bh)), nk = __fdiv_rn(1.0f, __ldg(p.sc_k + nx_bh));
          const float nv = __fdiv_rn(1.0f, __ldg(p.sc_v + nx_bh)), ndo = __fdiv_rn(1.0f, __ldg(p.sc_do + nx_bh));
          nx_mul = ts < 128 ? -kLog2e / (p.c * kLog2e * nq * nk) : -1.0f / (ndo * nv);
        }
      }
      while (bias_written < itg + (uint32_t)(total < 2 ? total : 2)) {
        const int l = (int)(bias_written - itg);
        bias_put(it_begin + l, bias_written, bias_fetch(bh, it_begin + l), bias_mul, bias_fetch2(bh, it_begin + l));
        ++bias_written;
      }
    }
    // the row that step `it` of this item is to write: global step itg + it + 2
    auto bias_target = [&](int it, int& tbh, int& tstep) -> bool {
      const int t = it + 2;
      if (t < total) { tbh = bh; tstep = it_begin + t; return true; }
      if (t - total < nx_total) { tbh = nx_bh; tstep = nx_begin + (t - total); return true; }
      return false;
    };
    float lse2 = 0.f, dq = 0.f, dq2 = 0.f;                    // this row's LSE*log2e and D (dq2: the second draw's D)
    int qrow = 0;                                             // global query index of this thread's row
    if (MODE != AT_DKV) {
      qrow = blk * AT_BLK + r;
      if (MODE == AT_DQ && qrow < p.S) {
        lse2 = __ldg(p.lse + (size_t)bh * p.S + qrow) * kLog2e;
        dq = __ldg(p.dterm + (size_t)bh * p.S + qrow);
        if (ND == 2) dq2 = __ldg(p.dterm + (size_t)p.BH * p.S + (size_t)bh * p.S + qrow);
      }
      if (lse_known && qrow < p.S) lse2 = __ldg(p.lse + (size_t)bh * p.S + qrow) * kLog2e;
    }
    // FWD: the shift in use (log2 units) and the sum of exp2(c2 s - shift) of this row and column half
    float run_m = lse_known ? lse2 : -INFINITY, run_l = 0.f;
    // DQF: the dQ share of global step jd (queries of block qblk): tensor memory -> registers (rows =
    // queries, this thread's 32 columns of half h) -> scaled by c into the swizzled staging boxes ->
    // two tiled bulk reduce-adds into dQ.  The staging buffer is the one the epilogue uses for dK.
    auto drain_dq = [&](uint32_t jd, int qblk) -> bool {
      if (!__all_sync(0xFFFFFFFFu, mbar_wait(b_dq_full, jd & 1u, abort_flag))) return false;
      tc_fence_after();
      uint32_t a[32];
      tmem_ld32(t_dq + lane_off + h * 32, a);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(b_dq_free);
      // the bulk operations that last read the staging buffer (the share before, or an epilogue) are done with it
      if (warp == kAtSoftWarp0 && lane == 0 && (store_pending || red_pending)) tma_store_wait_read();
      named_bar_sync(2, 256);
#pragma unroll
      for (int t = 0; t < 8; ++t) {
        const uint32_t off = (uint32_t)h * 16384u + (uint32_t)r * 128u + ((uint32_t)(t ^ (r & 7)) << 4);
        asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(stage2 + off), "f"(__uint_as_float(a[4 * t]) * p.c),
                     "f"(__uint_as_float(a[4 * t + 1]) * p.c), "f"(__uint_as_float(a[4 * t + 2]) * p.c),
                     "f"(__uint_as_float(a[4 * t + 3]) * p.c) : "memory");
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      named_bar_sync(4, 256);
      if (warp == kAtSoftWarp0 && lane == 0) {
        tma_reduce_add_3d(&tm_o2, stage2, 0, qblk * AT_BLK, bh);
        tma_reduce_add_3d(&tm_o2, stage2 + 16384u, 32, qblk * AT_BLK, bh);
        tma_store_commit();
        red_pending = true;
      }
      return true;
    };
    for (int it = 0; it < total && ok; ++it) {
      const int step = it_begin + (it % nsteps);
      const uint32_t ip = (itg + (uint32_t)it) & 1u;
      int kblk;                                               // key block of this step
      float bias_next = 0.f, bias_next2 = 0.f;                // DKV: this thread's raw value(s) for the row two steps ahead
      int bias_bh = 0, bias_step = 0;
      const bool bias_due = MODE == AT_DKV && bias_written == itg + (uint32_t)it + 2u && bias_target(it, bias_bh, bias_step);
      if (MODE == AT_DKV) {
        kblk = blk;
      } else {
        kblk = step;
      }
      const int qb0 = (MODE == AT_DKV ? step : blk) * AT_BLK;  // first query of this step's score tile
      ok = __all_sync(0xFFFFFFFFu, mbar_wait((PP && h) ? b_sdp_full1 : b_sdp_full, ip, abort_flag));
      if (!ok) break;
      tc_fence_after();
      // this thread's 64 scores (and 64 dP values) into registers, then hand the TMEM columns back
      // at once: the next step's S and dP are computed while this step's softmax runs
      uint32_t sv[64], dv[64];
      tmem_ld32_nowait(t_s + lane_off + h * 64, *reinterpret_cast<uint32_t(*)[32]>(&sv[0]));
      tmem_ld32_nowait(t_s + lane_off + h * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[32]));
      if (MODE != AT_FWD) {
        tmem_ld32_nowait(t_dp + lane_off + h * 64, *reinterpret_cast<uint32_t(*)[32]>(&dv[0]));
        tmem_ld32_nowait(t_dp + lane_off + h * 64 + 32, *reinterpret_cast<uint32_t(*)[32]>(&dv[32]));
      }
      tmem_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive((PP && h) ? b_sdp_free1 : b_sdp_free);
      if (bias_due) {                                         // lands under this step's arithmetic
        bias_next = bias_fetch(bias_bh, bias_step);
        bias_next2 = bias_fetch2(bias_bh, bias_step);
      }

      const int key0 = kblk * AT_BLK + h * 64;
      // masking is needed only on the diagonal block and where the sequence ends inside the block
      const bool edge = (p.causal && kblk * AT_BLK + AT_BLK - 1 > qb0) || (kblk + 1) * AT_BLK > p.S ||
                        qb0 + AT_BLK > p.S;
      float resc = 1.f;                                       // FWD: factor for this half's sums when the shift moves
      if (MODE == AT_FWD && !lse_known) {
        // largest c2 * s over the valid keys of this half (four independent chains; the validity
        // test only where a block needs it, and as a select)
        float mx;
        if (!edge && c2 > 0.f) {
          float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
          for (int j = 0; j < 64; j += 4) {
            m0 = fmaxf(m0, __uint_as_float(sv[j]));
            m1 = fmaxf(m1, __uint_as_float(sv[j + 1]));
            m2 = fmaxf(m2, __uint_as_float(sv[j + 2]));
            m3 = fmaxf(m3, __uint_as_float(sv[j + 3]));
          }
          mx = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3)) * c2;      // c2 > 0: the maximum commutes with the scaling
        } else {
          const bool row_ok = qrow < p.S;
          const int last = p.causal ? (qrow < p.S - 1 ? qrow : p.S - 1) : p.S - 1;   // last valid key of this row
          mx = -INFINITY;
#pragma unroll
          for (int j = 0; j < 64; ++j) {
            const float x = (row_ok && key0 + j <= last) ? __uint_as_float(sv[j]) * c2 : -INFINITY;
            mx = fmaxf(mx, x);
          }
        }
        // The shift follows the maximum lazily: it moves only when the maximum has grown by more than
        // 2^8 (the probabilities of a step then stay below 2^8, harmless in FP32 sums and bf16
        // operands), so the accumulator is rescaled on few steps.  While nothing finite has been seen
        // (a fully masked half) the sums are zero and the shift is simply taken.
        if (run_m == -INFINITY) {
          run_m = mx;
        } else if (mx > run_m + 8.0f) {
          resc = ex2_approx(run_m - mx);
          run_l *= resc;
          run_m = mx;
        }
        lse2 = run_m == -INFINITY ? 0.f : run_m;
      }
      {
        uint32_t pk[32], dk[32];
        // two neighbouring keys: P and dS = P (dP - D) as packed bf16 operands.  FP8-operand mode
        // first rounds P onto the E4M3 grid at p_scale and dS onto the E5M2 grid at ds_scale (the
        // grid values are exact in bf16; the scales come back in the epilogue).
        // a pair of dS values as a packed bf16 operand (FP8-operand mode: on the E5M2 grid at ds_scale)
        auto pack_ds = [&](float s0, float s1) -> uint32_t {
          if (F8K) return f8_encode_rn_pair_inrange<BSP_E5M2>(s0 * p.ds_scale, s1 * p.ds_scale);   // two codes, 16 bits
          if (FP8) return f8_grid_bf16x2<BSP_E5M2>(s0 * p.ds_scale, s1 * p.ds_scale);
          return pack_bf16x2(s0, s1);
        };
        // 32 of this thread's 64 columns of an operand (16 packed pairs) back into tensor memory: two
        // 16-bit elements per column, or (codes) four per column
        auto st_half = [&](uint32_t t_base, int half, const uint32_t (&wv)[16]) {
          if (F8K) {
            uint32_t c8[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) c8[i] = (wv[2 * i] & 0xFFFFu) | (wv[2 * i + 1] << 16);
            tmem_st8(t_base + lane_off + h * 16 + half * 8, c8);
          } else {
            tmem_st16(t_base + lane_off + h * 32 + half * 16, wv);
          }
        };
        auto pack_pair = [&](float p0, float p1, uint32_t dp0, uint32_t dp1, float d0, float d1, uint32_t& po,
                             uint32_t& dso) {
          float s0 = 0.f, s1 = 0.f;
          if (MODE == AT_FWD) run_l += p0 + p1;             // the row's normaliser, from the unrounded values
          if (MODE == AT_DKV && !FP8) {
            // (the accumulators already hold dP - D): both products in one packed instruction
            mul_f32x2(s0, s1, p0, p1, __uint_as_float(dp0), __uint_as_float(dp1));
          } else if (MODE != AT_FWD) {
            float t0, t1;
            fma_f32x2(t0, t1, __uint_as_float(dp0), __uint_as_float(dp1), dp_mul, dp_mul, -d0, -d1);
            mul_f32x2(s0, s1, p0, p1, t0, t1);
          }
          if (FP8 && MODE != AT_FWD) {                      // the forward keeps P unrounded
            if (F8K) {                                      // the codes themselves (two per word for now)
              po = f8_encode_rn_pair_inrange<BSP_E4M3>(p0 * p.p_scale, p1 * p.p_scale);
              dso = f8_encode_rn_pair_inrange<BSP_E5M2>(s0 * p.ds_scale, s1 * p.ds_scale);
              return;
            }
            po = f8_grid_bf16x2<BSP_E4M3>(p0 * p.p_scale, p1 * p.p_scale);
            dso = f8_grid_bf16x2<BSP_E5M2>(s0 * p.ds_scale, s1 * p.ds_scale);
            return;
          }
          po = pack_bf16x2(p0, p1);
          if (MODE != AT_FWD) dso = pack_bf16x2(s0, s1);
        };
        // column j of this thread's row: a query (DKV, the row is a key) or a key (the row is a query)
        const int col0 = (MODE == AT_DKV ? qb0 : kblk * AT_BLK) + h * 64;
        const int myrow = MODE == AT_DKV ? blk * AT_BLK + r : qrow;
        auto valid_at = [&](int j) {
          const int cj = col0 + j;
          const int key = MODE == AT_DKV ? myrow : cj, qy = MODE == AT_DKV ? cj : myrow;
          return key < p.S && qy < p.S && (!p.causal || key <= qy);
        };
        // Two columns per iteration on purpose: wider bodies made the compiler's schedule of the
        // exponentials twice as slow.  `masked` adds the validity test that only the diagonal block
        // and the blocks at the end of the sequence need.
        auto pair_at = [&](int j, bool masked) {
          // DKV: the accumulators already hold s - LSE/c and dP - D (see the X tiles)
          const float l0 = MODE == AT_DKV ? 0.f : lse2, d0 = MODE == AT_DKV ? 0.f : dq;
          const float l1 = l0, d1 = d0;
          float a0, a1;
          if (MODE == AT_DKV) {
            mul_f32x2(a0, a1, __uint_as_float(sv[j]), __uint_as_float(sv[j + 1]), c2, c2);
          } else {
            fma_f32x2(a0, a1, __uint_as_float(sv[j]), __uint_as_float(sv[j + 1]), c2, c2, -l0, -l1);
          }
          if (masked) {
            if (!valid_at(j)) a0 = -INFINITY;
            if (!valid_at(j + 1)) a1 = -INFINITY;
          }
          pack_pair(ex2_approx(a0), ex2_approx(a1), dv[j], dv[j + 1], d0, d1, pk[j >> 1], dk[j >> 1]);
        };
        if (MODE == AT_FWD) {
          if (!edge) {
#pragma unroll
            for (int j = 0; j < 64; j += 2) pair_at(j, false);
          } else {
#pragma unroll
            for (int j = 0; j < 64; j += 2) pair_at(j, true);
          }
          // the P buffer is free once the product of the previous step has read it
          ok = __all_sync(0xFFFFFFFFu, mbar_wait((PP && h) ? b_pds_free1 : b_pds_free, ip ^ 1u, abort_flag));
          if (!ok) break;
          if (__any_sync(0xFFFFFFFFu, resc != 1.f)) {
            // that product was also the last one to add to this half's accumulator: rescale the row
            // (the whole warp takes part in the tensor-memory accesses; rows that keep their shift
            // multiply by one).  Never on an item's first step: resc is 1 until a shift exists.
            tc_fence_after();
            const uint32_t t_mine = (h == 0 ? t_acc0 : t_acc1) + lane_off;
#pragma unroll
            for (int c = 0; c < 2; ++c) {
              uint32_t a[32];
              tmem_ld32(t_mine + c * 32, a);
#pragma unroll
              for (int j = 0; j < 32; ++j) a[j] = __float_as_uint(__uint_as_float(a[j]) * resc);
              tmem_st32(t_mine + c * 32, a);
            }
            tmem_wait_st();
            tc_fence_before();
          }
          // the row's 64 probabilities go back into tensor memory as 32 packed pairs (columns h*32 .. h*32+31
          // of the P operand, which sits where the backward modes keep dP)
          st_half(t_dp, 0, *reinterpret_cast<const uint32_t(*)[16]>(&pk[0]));
          st_half(t_dp, 1, *reinterpret_cast<const uint32_t(*)[16]>(&pk[16]));
          tmem_wait_st();
          tc_fence_before();
        } else if (MODE == AT_DQ && ND == 2) {
          // two draws: one exponential per element, two dS values; 32 columns at a time so that the
          // packed operands of both draws stay within the register budget
          uint32_t da[16], db[16];
          auto pair2_at = [&](int j, bool masked) {
            float a0, a1;
            fma_f32x2(a0, a1, __uint_as_float(sv[j]), __uint_as_float(sv[j + 1]), c2, c2, -lse2, -lse2);
            if (masked) {
              if (!valid_at(j)) a0 = -INFINITY;
              if (!valid_at(j + 1)) a1 = -INFINITY;
            }
            const float p0 = ex2_approx(a0), p1 = ex2_approx(a1);
            float t0, t1, u0, u1, s0, s1, r0, r1;
            fma_f32x2(t0, t1, __uint_as_float(dv[j]), __uint_as_float(dv[j + 1]), dp_mul, dp_mul, -dq, -dq);
            fma_f32x2(u0, u1, __uint_as_float(dv[j]), __uint_as_float(dv[j + 1]), dp_mul, dp_mul, -dq2, -dq2);
            mul_f32x2(s0, s1, p0, p1, t0, t1);
            mul_f32x2(r0, r1, p0, p1, u0, u1);
            da[(j & 31) >> 1] = pack_ds(s0, s1);
            db[(j & 31) >> 1] = pack_ds(r0, r1);
          };
          if (!edge) {
#pragma unroll
            for (int j = 0; j < 32; j += 2) pair2_at(j, false);
          } else {
#pragma unroll
            for (int j = 0; j < 32; j += 2) pair2_at(j, true);
          }
          ok = __all_sync(0xFFFFFFFFu, mbar_wait(b_pds_free, ip ^ 1u, abort_flag));
          if (!ok) break;
          st_half(t_ds, 0, da);
          st_half(t_ds2, 0, db);
          if (!edge) {
#pragma unroll
            for (int j = 32; j < 64; j += 2) pair2_at(j, false);
          } else {
#pragma unroll
            for (int j = 32; j < 64; j += 2) pair2_at(j, true);
          }
          st_half(t_ds, 1, da);
          st_half(t_ds2, 1, db);
          tmem_wait_st();
          tc_fence_before();
        } else if (MODE == AT_DQ) {
          if (!edge) {
#pragma unroll
            for (int j = 0; j < 64; j += 2) pair_at(j, false);
          } else {
#pragma unroll
            for (int j = 0; j < 64; j += 2) pair_at(j, true);
          }
          // the dS operand is free once the product of the previous step has read it; then the row's
          // 64 columns go back into tensor memory as 32 packed pairs (columns h*32 .. h*32+31)
          ok = __all_sync(0xFFFFFFFFu, mbar_wait((PP && h) ? b_pds_free1 : b_pds_free, ip ^ 1u, abort_flag));
          if (!ok) break;
          st_half(t_ds, 0, *reinterpret_cast<const uint32_t(*)[16]>(&dk[0]));
          st_half(t_ds, 1, *reinterpret_cast<const uint32_t(*)[16]>(&dk[16]));
          tmem_wait_st();
          tc_fence_before();
        } else if (MODE == AT_DKV && ND == 2) {
          // dK kernel, two draws: the accumulators hold s - LSE/c and dP - D of the first draw; the
          // second draw's dP - D is that plus delta of the column's query.  32 columns at a time.
          uint32_t da[16], db[16];
          const uint32_t dbase = delta0 + (((itg + (uint32_t)it) % 3u) * 128u + (uint32_t)h * 64u) * 4u;
          auto pair2_at = [&](int j, bool masked) {
            // (scalar arithmetic here: the packed forms cost this variant registers it does not have)
            float a0 = __uint_as_float(sv[j]) * c2, a1 = __uint_as_float(sv[j + 1]) * c2;
            if (masked) {
              if (!valid_at(j)) a0 = -INFINITY;
              if (!valid_at(j + 1)) a1 = -INFINITY;
            }
            const float p0 = ex2_approx(a0), p1 = ex2_approx(a1);
            float e0, e1;
            asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(e0), "=f"(e1) : "r"(dbase + (uint32_t)j * 4u));
            const float x0 = __uint_as_float(dv[j]) * dp_mul, x1 = __uint_as_float(dv[j + 1]) * dp_mul;
            da[(j & 31) >> 1] = pack_ds(p0 * x0, p1 * x1);
            db[(j & 31) >> 1] = pack_ds(p0 * (x0 + e0), p1 * (x1 + e1));
          };
          if (!edge) {
#pragma unroll
            for (int j = 0; j < 32; j += 2) pair2_at(j, false);
          } else {
#pragma unroll
            for (int j = 0; j < 32; j += 2) pair2_at(j, true);
          }
          ok = __all_sync(0xFFFFFFFFu, mbar_wait(b_pds_free, ip ^ 1u, abort_flag));
          if (!ok) break;
          st_half(t_ds, 0, da);
          st_half(t_ds2, 0, db);
          if (!edge) {
#pragma unroll
            for (int j = 32; j < 64; j += 2) pair2_at(j, false);
          } else {
#pragma unroll
            for (int j = 32; j < 64; j += 2) pair2_at(j, true);
          }
          st_half(t_ds, 1, da);
          st_half(t_ds2, 1, db);
          tmem_wait_st();
          tc_fence_before();
        } else {
          // DKV: P and dS go back into tensor memory as 32 packed pairs each (columns h*32 .. h*32+31
          // of the operands), in two halves: the first half is stored while the second is computed,
          // which also halves the registers the packed values hold.  The operands are free once the
          // products of the previous step have read them: that wait sits between the halves, where it
          // has long passed.
          if (!edge) {
#pragma unroll
            for (int j = 0; j < 32; j += 2) pair_at(j, false);
          } else {
#pragma unroll
            for (int j = 0; j < 32; j += 2) pair_at(j, true);
          }
          ok = __all_sync(0xFFFFFFFFu, mbar_wait(b_pds_free, ip ^ 1u, abort_flag));
          if (!ok) break;
          // DQF: 32 of the row's 64 dS^T values (four 16-byte chunks of eight queries) into row r of
          // half h of the shared dS^T buffer, 128-byte swizzle: chunk index t ^ (r & 7)
          auto st_half_smem = [&](int half, const uint32_t (&wv)[16]) {
#pragma unroll
            for (int t = 0; t < 4; ++t) {
              const uint32_t off = (uint32_t)h * 16384u + (uint32_t)r * 128u + ((uint32_t)((half * 4 + t) ^ (r & 7)) << 4);
              asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst_buf + off), "r"(wv[4 * t]), "r"(wv[4 * t + 1]),
                           "r"(wv[4 * t + 2]), "r"(wv[4 * t + 3]) : "memory");
            }
          };
          if (DV) st_half(t_p, 0, *reinterpret_cast<const uint32_t(*)[16]>(&pk[0]));
          if (DQF) st_half_smem(0, *reinterpret_cast<const uint32_t(*)[16]>(&dk[0]));
          else st_half(t_ds, 0, *reinterpret_cast<const uint32_t(*)[16]>(&dk[0]));
          if (!edge) {
#pragma unroll
            for (int j = 32; j < 64; j += 2) pair_at(j, false);
          } else {
#pragma unroll
            for (int j = 32; j < 64; j += 2) pair_at(j, true);
          }
          if (DV) st_half(t_p, 1, *reinterpret_cast<const uint32_t(*)[16]>(&pk[16]));
          if (DQF) st_half_smem(1, *reinterpret_cast<const uint32_t(*)[16]>(&dk[16]));
          else st_half(t_ds, 1, *reinterpret_cast<const uint32_t(*)[16]>(&dk[16]));
          tmem_wait_st();
          tc_fence_before();
        }
      }
      if (DQF) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive((PP && h) ? b_pds_ready1 : b_pds_ready);
      // DQF: the dQ share of the step before, now complete (its products were committed ahead of the
      // operands' release that this step has already waited for), goes out while this step's products run
      if (DQF && it > 0) {
        ok = drain_dq(itg + (uint32_t)it - 1u, it_begin + it - 1);
        if (!ok) break;
      }
      if (it == 0 && warp == kAtSoftWarp0 && lane == 0 && store_pending) {
        // the previous item's output has left its staging buffer by now: hand the resident-tile
        // buffer it used back to the TMA producer
        tma_store_wait_read();
        mbar_arrive(b_res_empty + 8 * (((uint32_t)item & 1u) ^ 1u));
        store_pending = false;
      }
      if (bias_due) {
        // (the empty asm pins the first use of the fetched value here, after the step's arithmetic)
        asm volatile("" : "+f"(bias_next), "+f"(bias_next2));
        bias_put(bias_step, bias_written, bias_next, bias_bh == bh && it + 2 < total ? bias_mul : nx_mul, bias_next2);
        ++bias_written;
      }
    }
    if (DQF && ok) ok = drain_dq(itg + (uint32_t)total - 1u, it_begin + total - 1);   // the last step's share
    itg += (uint32_t)total;
    float fwd_w0 = 1.f, fwd_w1 = 1.f;                         // FWD: weights of the two halves' accumulators
    if (MODE == AT_FWD) {
      // the two column halves of the row meet: common shift m, normaliser l, and the LSE in
      // natural-log units.  A half that saw no valid key has shift -inf, sum 0 and weight 0.
      float* xm = xchg;                                       // [2][128] shifts, then [2][128] sums
      xm[h * 128 + r] = run_m;
      xm[256 + h * 128 + r] = run_l;
      named_bar_sync(1, 256);
      const float m0 = xm[r], m1 = xm[128 + r], l0 = xm[256 + r], l1 = xm[384 + r];
      const float m = fmaxf(m0, m1);
      const float e0 = m0 == -INFINITY ? 0.f : ex2_approx(m0 - m), e1 = m1 == -INFINITY ? 0.f : ex2_approx(m1 - m);
      const float l = l0 * e0 + l1 * e1;
      const float inv_l = __fdividef(1.0f, l);
      fwd_w0 = e0 * inv_l;
      fwd_w1 = e1 * inv_l;
      if (h == 0 && qrow < p.S && p.lse_out) p.lse_out[(size_t)bh * p.S + qrow] = (m + log2f(l)) / kLog2e;
      named_bar_sync(1, 256);                                 // the exchange buffer is written again by the next item
    }
    // ---- epilogue: accumulators to global memory (rows = keys for DKV, queries otherwise), 32 KB at a
    // time through the item's resident-tile buffer (no product reads it any more): every thread puts
    // its row's 32 FP32 values of column half h into the 128-byte-swizzle box that a tiled bulk store
    // then writes (whole 128-byte lines; rows beyond the sequence are clipped by the store).
    constexpr bool mc = MC;
    // Monte-Carlo epilogue: the reference values of the warp's 32 rows x 32 columns, fetched by the
    // warp together (load t: four rows of 128 contiguous bytes, lane -> row 4t + lane / 8, 16-byte
    // chunk lane % 8) and handed to the row-owning threads through the staging buffer further down
    float4 rc[8];
    if (mc) {
#pragma unroll
      for (int t = 0; t < 8; ++t) {
        const int orow = blk * AT_BLK + q4 * 32 + 4 * t + (lane >> 3);
        rc[t] = __ldg(reinterpret_cast<const float4*>(p.mc_ref + ((size_t)bh * p.S + (orow < p.S ? orow : 0)) * AT_D + h * 32) +
                      (lane & 7));
      }
    }
    if (ok) ok = __all_sync(0xFFFFFFFFu, mbar_wait(b_acc + 8 * ab, iph, abort_flag));
    if (ok) {
      tc_fence_after();
      const uint32_t rbi = (uint32_t)item & 1u;
      constexpr int nout = MODE == AT_DKV ? 2 : 1;            // DKV: dV (acc0) and dK (acc1)
      // the stores of the item before have long read their staging buffers; make that certain
      if (warp == kAtSoftWarp0 && lane == 0 && store_pending) {
        tma_store_wait_read();
        mbar_arrive(b_res_empty + 8 * (rbi ^ 1u));
        store_pending = false;
      }
      if (DQF && warp == kAtSoftWarp0 && lane == 0 && red_pending) {
        tma_store_wait_read();                                // the last share's reduce-adds have read the staging buffer
        red_pending = false;
      }
      if (MODE == AT_DKV || mc) named_bar_sync(3, 256);       // ... before anyone writes the second staging buffer again
      float rv[32];                                           // this thread's 32 reference values
      if (mc) {
        // through the warp's own 4 KB of the (now free) second staging buffer: chunk (row, c) sits
        // where the output boxes keep it, so every thread finds its row at its own output slots
#pragma unroll
        for (int t = 0; t < 8; ++t) {
          const uint32_t row = (uint32_t)(q4 * 32 + 4 * t + (lane >> 3));
          const uint32_t off = (uint32_t)h * 16384u + row * 128u + ((((uint32_t)lane & 7u) ^ (row & 7u)) << 4);
          asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(stage2 + off), "f"(rc[t].x), "f"(rc[t].y), "f"(rc[t].z),
                       "f"(rc[t].w) : "memory");
        }
        __syncwarp();
#pragma unroll
        for (int t = 0; t < 8; ++t) {
          const uint32_t off = (uint32_t)h * 16384u + (uint32_t)r * 128u + ((uint32_t)(t ^ (r & 7)) << 4);
          asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                       : "=f"(rv[4 * t]), "=f"(rv[4 * t + 1]), "=f"(rv[4 * t + 2]), "=f"(rv[4 * t + 3]) : "r"(stage2 + off));
        }
        __syncwarp();
      }
#pragma unroll
      for (int o = (MODE == AT_DKV && !DV) ? 1 : 0; o < nout; ++o) {
        const uint32_t stg = o == 0 ? res_base + rbi * 2 * kAtTile : stage2;
        float mul;
        if (MODE == AT_DKV) mul = o == 0 ? (FP8 ? inv_do / p.p_scale : 1.f) : p.c * (FP8 ? inv_q / p.ds_scale : 1.f);
        else if (MODE == AT_DQ) mul = p.c * (FP8 ? inv_k / p.ds_scale : 1.f);
        else mul = inv_v * fwd_w0;
        uint32_t a[32], a2[ND == 2 ? 32 : 1];
        tmem_ld32((o == 0 ? t_acc0 : t_acc1) + lane_off + h * 32, a);
        if (ND == 2) tmem_ld32((o == 0 ? t_acc1 : t_acc0) + lane_off + h * 32, *reinterpret_cast<uint32_t(*)[32]>(&a2[0]));
        if (MODE == AT_FWD) {
          // O = w0 O_0 + w1 O_1: fold the second half's accumulator in here
          uint32_t a1[32];
          tmem_ld32(t_acc1 + lane_off + h * 32, a1);
          const float mul1 = inv_v * fwd_w1;
#pragma unroll
          for (int j = 0; j < 32; ++j) a[j] = __float_as_uint(fmaf(__uint_as_float(a1[j]), mul1, __uint_as_float(a[j]) * mul));
          mul = 1.f;
        }
        if (o == nout - 1) {
          // the accumulators may be overwritten by the next item (FWD: the item after next)
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(b_acc_free + 8 * ab);
        }
        if (mc) {
          // g - ref into this output's staging buffer, its square into the other one
          const uint32_t stg2 = o == 0 ? stage2 : res_base + rbi * 2 * kAtTile;
#pragma unroll
          for (int t = 0; t < 8; ++t) {
            const uint32_t off = (uint32_t)h * 16384u + (uint32_t)r * 128u + ((uint32_t)(t ^ (r & 7)) << 4);
            float d[4], q[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              d[e] = __uint_as_float(a[4 * t + e]) * mul - rv[4 * t + e];
              q[e] = d[e] * d[e];
              if (ND == 2) {                                  // the second draw of this launch joins the first
                const float e2 = __uint_as_float(a2[ND == 2 ? 4 * t + e : 0]) * mul - rv[4 * t + e];
                d[e] += e2;
                q[e] = fmaf(e2, e2, q[e]);
              }
            }
            asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(stg + off), "f"(d[0]), "f"(d[1]), "f"(d[2]), "f"(d[3]) : "memory");
            asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(stg2 + off), "f"(q[0]), "f"(q[1]), "f"(q[2]), "f"(q[3]) : "memory");
          }
        } else {
#pragma unroll
          for (int t = 0; t < 8; ++t) {
            const uint32_t off = (uint32_t)h * 16384u + (uint32_t)r * 128u + ((uint32_t)(t ^ (r & 7)) << 4);
            asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(stg + off), "f"(__uint_as_float(a[4 * t]) * mul),
                         "f"(__uint_as_float(a[4 * t + 1]) * mul), "f"(__uint_as_float(a[4 * t + 2]) * mul),
                         "f"(__uint_as_float(a[4 * t + 3]) * mul) : "memory");
          }
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      named_bar_sync(3, 256);
      if (warp == kAtSoftWarp0 && lane == 0) {
        // issue the stores and go on: their completion is only needed before the staging buffers are
        // written again (next epilogue) or handed back (after the next item's first step)
        if (mc) {
          // S1 += g - ref, S2 += (g - ref)^2: each element of the sums is added to once per launch
          const uint32_t sx = MODE == AT_DKV ? stage2 : res_base + rbi * 2 * kAtTile;
          const uint32_t sy = MODE == AT_DKV ? res_base + rbi * 2 * kAtTile : stage2;
          tma_reduce_add_3d(&tm_o0, sx, 0, blk * AT_BLK, bh);
          tma_reduce_add_3d(&tm_o0, sx + 16384u, 32, blk * AT_BLK, bh);
          tma_reduce_add_3d(&tm_o1, sy, 0, blk * AT_BLK, bh);
          tma_reduce_add_3d(&tm_o1, sy + 16384u, 32, blk * AT_BLK, bh);
        } else {
          if (MODE != AT_DKV || DV) {
            tma_store_3d(&tm_o0, res_base + rbi * 2 * kAtTile, 0, blk * AT_BLK, bh);
            tma_store_3d(&tm_o0, res_base + rbi * 2 * kAtTile + 16384u, 32, blk * AT_BLK, bh);
          }
          if (MODE == AT_DKV) {
            tma_store_3d(&tm_o1, stage2, 0, blk * AT_BLK, bh);
            tma_store_3d(&tm_o1, stage2 + 16384u, 32, blk * AT_BLK, bh);
          }
        }
        tma_store_commit();
        store_pending = true;
      }
    }
    }  // items
    if (warp == kAtSoftWarp0 && lane == 0) tma_store_wait_all();         // the bulk stores of this CTA have landed
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

// ------------------------------------------------------------------------------- D pre-pass

// D[d][row] = sum_j dO[row][j] * O_copy[row][j] for n_draws draws (one for U and R).  Eight lanes per
// row of 64, eight elements each; a thread takes kDtRows rows (32 rows apart) and issues all their
// loads before it uses any.  U reads the FP32 original, R the forward's codes, N a fresh stochastic
// rounding of fl32(O * scale[bh]) keyed by the element's index in the whole tensor.  For N the
// rounding of an element is its round-down value plus, when the generator word is below the
// element's threshold (f8_sr_threshold), one grid step: per element the product of dO with the
// round-down value goes into a sum shared by all draws, and a draw costs one comparison and one
// conditional add of dO * step.
template <int DT, int FMT, int kDtRows>
__global__ void __launch_bounds__(256)
attn_dterm_kernel(const void* __restrict__ dO, const float* __restrict__ o_orig, const uint8_t* __restrict__ o_codes,
                  const float* __restrict__ o_scales, const float* __restrict__ do_scales, int64_t rows, int S,
                  int policy, PhiloxKey key, int draw0, int n_draws, float* __restrict__ D) {
  const int sub = threadIdx.x & 7;
  const int64_t row0 = (int64_t)blockIdx.x * (32 * kDtRows) + (threadIdx.x >> 3);
  float g[kDtRows][8], o[kDtRows][8], scale[kDtRows], inv[kDtRows];
  bool active[kDtRows];
  size_t i0[kDtRows];
#pragma unroll
  for (int m = 0; m < kDtRows; ++m) {
    const int64_t row = row0 + 32 * m;
    active[m] = row < rows;
    i0[m] = (size_t)(active[m] ? row : 0) * AT_D + sub * 8;
    const float4 g0 = load4<DT>(dO, i0[m]), g1 = load4<DT>(dO, i0[m] + 4);
    g[m][0] = g0.x; g[m][1] = g0.y; g[m][2] = g0.z; g[m][3] = g0.w;
    g[m][4] = g1.x; g[m][5] = g1.y; g[m][6] = g1.z; g[m][7] = g1.w;
    if (policy == BSP_READ_FORWARD) {
      const uint2 pk = __ldg(reinterpret_cast<const uint2*>(o_codes + i0[m]));
      float d0[4], d1[4];
      f8_decode4<FMT>(pk.x, d0);
      f8_decode4<FMT>(pk.y, d1);
#pragma unroll
      for (int j = 0; j < 4; ++j) { o[m][j] = d0[j]; o[m][4 + j] = d1[j]; }
    } else {
      const float4 a0 = __ldg(reinterpret_cast<const float4*>(o_orig + i0[m]));
      const float4 a1 = __ldg(reinterpret_cast<const float4*>(o_orig + i0[m] + 4));
      o[m][0] = a0.x; o[m][1] = a0.y; o[m][2] = a0.z; o[m][3] = a0.w;
      o[m][4] = a1.x; o[m][5] = a1.y; o[m][6] = a1.z; o[m][7] = a1.w;
    }
  }
#pragma unroll
  for (int m = 0; m < kDtRows; ++m) {
    const int64_t row = active[m] ? row0 + 32 * m : 0;
    scale[m] = o_scales ? __ldg(o_scales + row / S) : 1.f;
    inv[m] = __fdiv_rn(1.0f, scale[m]);
    if (do_scales) {
      // dO holds decoded FP8 codes: bring back its per-(b,h) scale
      const float inv_do = __fdiv_rn(1.0f, __ldg(do_scales + row / S));
#pragma unroll
      for (int j = 0; j < 8; ++j) g[m][j] *= inv_do;
    }
    if (policy == BSP_READ_FORWARD) {
#pragma unroll
      for (int j = 0; j < 8; ++j) o[m][j] *= inv[m];
    }
  }
  auto reduce_store = [&](int m, int d, float s) {
#pragma unroll
    for (int off = 4; off > 0; off >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, off);
    if (active[m] && sub == 0) D[(size_t)d * rows + row0 + 32 * m] = s;
  };
  if (policy != BSP_READ_FRESH) {
#pragma unroll
    for (int m = 0; m < kDtRows; ++m) {
      const float s = ((g[m][0] * o[m][0] + g[m][1] * o[m][1]) + (g[m][2] * o[m][2] + g[m][3] * o[m][3])) +
                      ((g[m][4] * o[m][4] + g[m][5] * o[m][5]) + (g[m][6] * o[m][6] + g[m][7] * o[m][7]));
      reduce_store(m, 0, s);
    }
    return;
  }
  // fresh read: per element the threshold and dO * step; the draw-independent part summed once
  uint32_t thr[kDtRows][8];
  float base[kDtRows];
#pragma unroll
  for (int m = 0; m < kDtRows; ++m) {
    float bs = 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float v = __fmul_rn(o[m][j], scale[m]);
      const float lo = f8_sr_value<FMT>(v, 0xFFFFFFFFu) * inv[m], hi = f8_sr_value<FMT>(v, 0u) * inv[m];
      thr[m][j] = f8_sr_threshold<FMT>(v);
      bs = fmaf(g[m][j], lo, bs);
      o[m][j] = thr[m][j] ? g[m][j] * (hi - lo) : 0.f;      // reuse: dO * step (a NaN stays in the shared sum)
    }
    base[m] = bs;
  }
  for (int d = 0; d < n_draws; ++d) {
#pragma unroll
    for (int m = 0; m < kDtRows; ++m) {
      const uint4 w0 = philox_block(key, (uint64_t)i0[m] >> 2, (uint32_t)(draw0 + d));
      const uint4 w1 = philox_block(key, ((uint64_t)i0[m] >> 2) + 1, (uint32_t)(draw0 + d));
      float s = base[m];
      s += w0.x < thr[m][0] ? o[m][0] : 0.f; s += w0.y < thr[m][1] ? o[m][1] : 0.f;
      s += w0.z < thr[m][2] ? o[m][2] : 0.f; s += w0.w < thr[m][3] ? o[m][3] : 0.f;
      s += w1.x < thr[m][4] ? o[m][4] : 0.f; s += w1.y < thr[m][5] ? o[m][5] : 0.f;
      s += w1.z < thr[m][6] ? o[m][6] : 0.f; s += w1.w < thr[m][7] ? o[m][7] : 0.f;
      reduce_store(m, d, s);
    }
  }
}

// ------------------------------------------------------------------------------- host side

template <int MODE, bool FP8, bool DV, bool MC = false, int ND = 1, bool DQF = false>
static int launch_attn_mode(const void* q, const void* k, const void* v, const void* dO, AttnParams p, cudaStream_t st) {
  CUtensorMap mq, mk, mv, mdo, mo0, mo1, mo2;
  int rc;
  if (DQF && !p.out2) return BSP_ERR_ARG;
  if ((rc = make_out_map(&mo0, p.out0 ? p.out0 : p.out1, p.BH, p.S)) != BSP_OK) return rc;
  if ((rc = make_out_map(&mo1, p.out1 ? p.out1 : p.out0, p.BH, p.S)) != BSP_OK) return rc;
  if ((rc = make_out_map(&mo2, DQF ? p.out2 : (p.out0 ? p.out0 : p.out1), p.BH, p.S)) != BSP_OK) return rc;
  if (FP8 && MODE != AT_FWD) {
    // the backward of the FP8-operand mode loads the codes
    if (!p.cq || !p.ck || !p.cv || !p.cdo) return BSP_ERR_ARG;
    if (!aligned16(p.cq) || !aligned16(p.ck) || !aligned16(p.cv) || !aligned16(p.cdo)) return BSP_ERR_ALIGN;
    if ((rc = make_head_map_u8(&mq, p.cq, p.BH, p.S)) != BSP_OK) return rc;
    if ((rc = make_head_map_u8(&mk, p.ck, p.BH, p.S)) != BSP_OK) return rc;
    if ((rc = make_head_map_u8(&mv, p.cv, p.BH, p.S)) != BSP_OK) return rc;
    if ((rc = make_head_map_u8(&mdo, p.cdo, p.BH, p.S)) != BSP_OK) return rc;
  } else {
    if ((rc = make_head_map(&mq, q, p.BH, p.S)) != BSP_OK) return rc;
    if ((rc = make_head_map(&mk, k, p.BH, p.S)) != BSP_OK) return rc;
    if ((rc = make_head_map(&mv, v, p.BH, p.S)) != BSP_OK) return rc;
    if ((rc = make_head_map(&mdo, dO ? dO : q, p.BH, p.S)) != BSP_OK) return rc;
  }
  static std::atomic<bool> attr_set_dev[kMaxDevices];       // per kernel instantiation and device
  std::atomic<bool>& attr_set = attr_set_dev[device_slot()];
  if (!attr_set.load(std::memory_order_acquire)) {
    BSP_CHECK_CUDA(cudaFuncSetAttribute(attn_kernel<MODE, FP8, DV, MC, ND, DQF>, cudaFuncAttributeMaxDynamicSharedMemorySize, kAtSmem));
    attr_set.store(true, std::memory_order_release);
  }
  // persistent: one CTA per SM walks the (block, head) items, heaviest first
  int nsm = kNumSMs, dev = 0, sm_count = 0;
  if (cudaGetDevice(&dev) == cudaSuccess &&
      cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sm_count > 0)
    nsm = sm_count;
  const int64_t nitems = (int64_t)p.nblk * p.BH;
  const unsigned grid = (unsigned)(nitems < nsm ? nitems : nsm);
  attn_kernel<MODE, FP8, DV, MC, ND, DQF><<<grid, kAtThreads, kAtSmem, st>>>(mq, mk, mv, mdo, mo0, mo1, mo2, p);
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

template <int MODE>
static int launch_attn(const void* q, const void* k, const void* v, const void* dO, AttnParams p, cudaStream_t st) {
  if (MODE != AT_FWD && p.mc_ref != nullptr) {               // Monte-Carlo epilogue: BF16 operands, no dV
    if (p.fp8) {
      if (p.nd == 2) return launch_attn_mode<MODE, true, MODE != AT_DKV, MODE != AT_FWD, MODE != AT_FWD ? 2 : 1>(q, k, v, dO, p, st);
      return launch_attn_mode<MODE, true, MODE != AT_DKV, MODE != AT_FWD>(q, k, v, dO, p, st);
    }
    if (p.nd == 2) return launch_attn_mode<MODE, false, MODE != AT_DKV, MODE != AT_FWD, MODE != AT_FWD ? 2 : 1>(q, k, v, dO, p, st);
    return launch_attn_mode<MODE, false, MODE != AT_DKV, MODE != AT_FWD>(q, k, v, dO, p, st);
  }
  if (MODE == AT_DKV && p.out0 == nullptr)                   // dK only
    return p.fp8 ? launch_attn_mode<MODE, true, false>(q, k, v, dO, p, st) : launch_attn_mode<MODE, false, false>(q, k, v, dO, p, st);
  return p.fp8 ? launch_attn_mode<MODE, true, true>(q, k, v, dO, p, st) : launch_attn_mode<MODE, false, true>(q, k, v, dO, p, st);
}

static bool valid_enum(int v, int hi) { return v >= 0 && v <= hi; }

static int set_fp8(AttnParams& p, const bsp_attn_fp8_t* f) {
  p.fp8 = f ? 1 : 0;
  p.sc_q = f ? f->q_scale : nullptr; p.sc_k = f ? f->k_scale : nullptr;
  p.sc_v = f ? f->v_scale : nullptr; p.sc_do = f ? f->do_scale : nullptr;
  p.p_scale = f ? f->p_scale : 1.f; p.ds_scale = f ? f->ds_scale : 1.f;
  p.cq = f ? f->q_codes : nullptr; p.ck = f ? f->k_codes : nullptr; p.cv = f ? f->v_codes : nullptr; p.cdo = f ? f->do_codes : nullptr;
  if (f && (!f->q_scale || !f->k_scale || !f->v_scale || !f->do_scale || !(f->p_scale > 0.f) || !(f->ds_scale > 0.f)))
    return BSP_ERR_ARG;
  return BSP_OK;
}

int attn_fwd_impl(int B, int H, int S, int Dh, int causal, float softmax_scale, const void* q, const void* k,
                         const void* v, int dt, const bsp_attn_fp8_t* f, float* o, float* lse, bsp_diag_t* diag,
                         void* stream, const float* lse_known) {
  int rc = check_attn_shape(B, H, S, Dh, dt);
  if (rc != BSP_OK) return rc;
  if (!q || !k || !v || !o || (!lse && !lse_known)) return BSP_ERR_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return BSP_ERR_ALIGN;
  AttnParams p{};
  p.BH = B * H; p.S = S; p.nblk = (S + AT_BLK - 1) / AT_BLK; p.causal = causal ? 1 : 0; p.c = softmax_scale;
  p.lse = lse_known; p.dterm = nullptr; p.out0 = o; p.out1 = nullptr; p.lse_out = lse; p.diag = diag; p.mc_ref = nullptr; p.nd = 1;
  if ((rc = set_fp8(p, f)) != BSP_OK) return rc;
  return launch_attn<AT_FWD>(q, k, v, nullptr, p, (cudaStream_t)stream);
}

int attn_dterm_impl(int B, int H, int S, int Dh, const void* dO, int dt, const float* do_scales,
                           const float* o_orig, const uint8_t* o_codes, const float* o_scales, int o_fmt, int d_read,
                           bsp_key_t key, int draw0, int n_draws, float* d_out, void* stream);
int attn_bwd_dterm_impl(int B, int H, int S, int Dh, int causal, float softmax_scale, const void* q,
                               const void* k, const void* v, const void* dO, int dt, const bsp_attn_fp8_t* f,
                               const float* lse, const float* dterm, float* dq, float* dk, float* dv, bsp_diag_t* diag,
                               void* stream);

}  // namespace bsp

using namespace bsp;

extern "C" {

int bsp_attn_fwd_stats(int B, int H, int S, int Dh, int causal, float softmax_scale, const void* q, const void* k,
                       const void* v, int dt, const bsp_attn_fp8_t* fp8, float* o, float* lse, bsp_diag_t* diag,
                       void* stream) {
  return attn_fwd_impl(B, H, S, Dh, causal, softmax_scale, q, k, v, dt, fp8, o, lse, diag, stream);
}

int bsp_attn_dterm(int B, int H, int S, int Dh, const void* dO, int dt, const float* do_scales, const float* o_orig,
                   const uint8_t* o_codes, const float* o_scales, int o_fmt, int d_read, bsp_key_t key, int draw0,
                   int n_draws, float* d_out, bsp_diag_t* diag, void* stream) {
  (void)diag;
  return attn_dterm_impl(B, H, S, Dh, dO, dt, do_scales, o_orig, o_codes, o_scales, o_fmt, d_read, key, draw0, n_draws,
                         d_out, stream);
}

}  // extern "C"

namespace bsp {

int attn_dterm_impl(int B, int H, int S, int Dh, const void* dO, int dt, const float* do_scales,
                           const float* o_orig, const uint8_t* o_codes, const float* o_scales, int o_fmt, int d_read,
                           bsp_key_t key, int draw0, int n_draws, float* d_out, void* stream) {
  if (B <= 0 || H <= 0 || S <= 0 || !valid_enum(dt, 1) || !valid_enum(o_fmt, 1) || !valid_enum(d_read, 2)) return BSP_ERR_ARG;
  if (Dh != AT_D) return BSP_ERR_UNSUPPORTED;
  if (key.tensor_id >= (1u << 24) || key.stream > 255u || key.reserved != 0 || draw0 < 0 || n_draws < 0) return BSP_ERR_ARG;
  if (n_draws == 0) return BSP_OK;
  if (!dO || !d_out) return BSP_ERR_ARG;
  if (d_read == BSP_READ_FORWARD ? (!o_codes || !o_scales) : !o_orig) return BSP_ERR_ARG;
  if (d_read == BSP_READ_FRESH && !o_scales) return BSP_ERR_ARG;
  if (d_read != BSP_READ_FRESH) n_draws = 1;
  if (!aligned16(dO) || !aligned16(o_orig) || (reinterpret_cast<uintptr_t>(o_codes) & 7u)) return BSP_ERR_ALIGN;
  const int64_t rows = (int64_t)B * H * S;
  constexpr int nr = 2;                              // rows per thread (four measured slower for U and R)
  const unsigned grid = (unsigned)((rows + 32 * nr - 1) / (32 * nr));
  cudaStream_t st = (cudaStream_t)stream;
  const PhiloxKey pk = make_key(key);
#define BSP_DT(DT, FMT)                                                                                          \
  attn_dterm_kernel<DT, FMT, nr><<<grid, 256, 0, st>>>(dO, o_orig, o_codes, o_scales, do_scales, rows, S, d_read, \
                                                       pk, draw0, n_draws, d_out)
  if (dt == BSP_F32 && o_fmt == BSP_E4M3) BSP_DT(BSP_F32, BSP_E4M3);
  else if (dt == BSP_F32) BSP_DT(BSP_F32, BSP_E5M2);
  else if (o_fmt == BSP_E4M3) BSP_DT(BSP_BF16, BSP_E4M3);
  else BSP_DT(BSP_BF16, BSP_E5M2);
#undef BSP_DT
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

int attn_bwd_dterm_impl(int B, int H, int S, int Dh, int causal, float softmax_scale, const void* q,
                               const void* k, const void* v, const void* dO, int dt, const bsp_attn_fp8_t* f,
                               const float* lse, const float* dterm, float* dq, float* dk, float* dv, bsp_diag_t* diag,
                               void* stream) {
  int rc = check_attn_shape(B, H, S, Dh, dt);
  if (rc != BSP_OK) return rc;
  if (!q || !k || !v || !dO || !lse || !dterm) return BSP_ERR_ARG;
  if ((dv && !dk) || (!dq && !dk)) return BSP_ERR_ARG;          // dV comes with dK; dK may come alone
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(dO) || !aligned16(dq) || !aligned16(dk) ||
      !aligned16(dv))
    return BSP_ERR_ALIGN;
  AttnParams p{};
  p.BH = B * H; p.S = S; p.nblk = (S + AT_BLK - 1) / AT_BLK; p.causal = causal ? 1 : 0; p.c = softmax_scale;
  p.lse = lse; p.dterm = dterm; p.lse_out = nullptr; p.diag = diag; p.mc_ref = nullptr; p.nd = 1;
  if ((rc = set_fp8(p, f)) != BSP_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  if (dk) {
    p.out0 = dv; p.out1 = dk;
    if ((rc = launch_attn<AT_DKV>(q, k, v, dO, p, st)) != BSP_OK) return rc;
  }
  if (dq) {
    p.out0 = dq; p.out1 = nullptr;
    if ((rc = launch_attn<AT_DQ>(q, k, v, dO, p, st)) != BSP_OK) return rc;
  }
  return BSP_OK;
}

// The same backward in one kernel: the dK/dV kernel also forms each score tile's share of dQ and adds
// it to dQ in global memory (BF16 operands, all three gradients).  dQ is cleared here first.
int attn_bwd_fused_impl(int B, int H, int S, int Dh, int causal, float softmax_scale, const void* q, const void* k,
                        const void* v, const void* dO, int dt, const float* lse, const float* dterm, float* dq, float* dk,
                        float* dv, bsp_diag_t* diag, void* stream) {
  int rc = check_attn_shape(B, H, S, Dh, dt);
  if (rc != BSP_OK) return rc;
  if (!q || !k || !v || !dO || !lse || !dterm || !dq || !dk || !dv) return BSP_ERR_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(dO) || !aligned16(dq) || !aligned16(dk) ||
      !aligned16(dv))
    return BSP_ERR_ALIGN;
  AttnParams p{};
  p.BH = B * H; p.S = S; p.nblk = (S + AT_BLK - 1) / AT_BLK; p.causal = causal ? 1 : 0; p.c = softmax_scale;
  p.lse = lse; p.dterm = dterm; p.lse_out = nullptr; p.diag = diag; p.mc_ref = nullptr; p.nd = 1;
  if ((rc = set_fp8(p, nullptr)) != BSP_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  BSP_CHECK_CUDA(cudaMemsetAsync(dq, 0, (size_t)B * H * S * AT_D * sizeof(float), st));
  p.out0 = dv; p.out1 = dk; p.out2 = dq;
  return launch_attn_mode<AT_DKV, false, true, false, 1, true>(q, k, v, dO, p, st);
}

// nd (1 or 2) draws of the D use for dQ and dK with the Monte-Carlo epilogue: the kernels add g - ref
// and its square to the running sums of their gradient and write no gradient (dV is not computed).
// dterm holds the draws' correction terms back to back, [nd][B*H*S]; with nd = 2 (BF16-operand mode
// only) both kernels take the two draws in one launch (S, dP and P are formed once per step).  The
// sums must not be touched by anything else while this runs.
int attn_bwd_dterm_mc(int B, int H, int S, int Dh, int causal, float softmax_scale, const void* q, const void* k,
                      const void* v, const void* dO, int dt, const bsp_attn_fp8_t* f, const float* lse,
                      const float* dterm, int nd, const float* ref_dq, float* S1q, float* S2q, const float* ref_dk,
                      float* S1k, float* S2k, bsp_diag_t* diag, void* stream) {
  int rc = check_attn_shape(B, H, S, Dh, dt);
  if (rc != BSP_OK) return rc;
  if (!q || !k || !v || !dO || !lse || !dterm || !ref_dq || !S1q || !S2q || !ref_dk || !S1k || !S2k) return BSP_ERR_ARG;
  if (nd < 1 || nd > 2) return BSP_ERR_ARG;
  if (!aligned16(ref_dq) || !aligned16(ref_dk) || !aligned16(S1q) || !aligned16(S2q) || !aligned16(S1k) || !aligned16(S2k))
    return BSP_ERR_ALIGN;
  AttnParams p{};
  p.BH = B * H; p.S = S; p.nblk = (S + AT_BLK - 1) / AT_BLK; p.causal = causal ? 1 : 0; p.c = softmax_scale;
  p.lse = lse; p.lse_out = nullptr; p.diag = diag;
  if ((rc = set_fp8(p, f)) != BSP_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  p.dterm = dterm; p.nd = nd;
  p.mc_ref = ref_dk; p.out0 = S1k; p.out1 = S2k;
  if ((rc = launch_attn<AT_DKV>(q, k, v, dO, p, st)) != BSP_OK) return rc;
  p.mc_ref = ref_dq; p.out0 = S1q; p.out1 = S2q;
  return launch_attn<AT_DQ>(q, k, v, dO, p, st);
}

// x (bf16 [groups][group_size]) -> nearest FP8 codes at each group's own amax scale -> the decoded
// codes as bf16 (exact), plus the scales.
template <int FMT>
__global__ void __launch_bounds__(256)
quantize_decode_kernel(const uint16_t* __restrict__ x, size_t group_size, const float* __restrict__ scales,
                       uint16_t* __restrict__ out, uint8_t* __restrict__ codes, size_t n8) {
  const size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= n8) return;
  const size_t i0 = t * 8;
  const float s = __ldg(scales + i0 / group_size);
  const uint4 raw = __ldg(reinterpret_cast<const uint4*>(x) + t);
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
  uint32_t o[4], c[4];
  DiagCounters dc;                                          // (non-finite inputs were counted by the amax pass)
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float va = __fmul_rn(bf16_bits_to_float(w[i] & 0xFFFFu), s), vb = __fmul_rn(bf16_bits_to_float(w[i] >> 16), s);
    const float a = f8_rn_value<FMT>(va);
    const float b = f8_rn_value<FMT>(vb);
    o[i] = (__float_as_uint(a) >> 16) | (__float_as_uint(b) & 0xFFFF0000u);     // FP8 values are exact in bf16
    c[i] = f8_encode<FMT, false>(va, 0u, dc) | (f8_encode<FMT, false>(vb, 0u, dc) << 8);
  }
  if (out) reinterpret_cast<uint4*>(out)[t] = make_uint4(o[0], o[1], o[2], o[3]);
  if (codes) reinterpret_cast<uint2*>(codes)[t] = make_uint2(c[0] | (c[1] << 16), c[2] | (c[3] << 16));
}

}  // namespace bsp

extern "C" {

int bsp_attn_bwd_dterm(int B, int H, int S, int Dh, int causal, float softmax_scale, const void* q, const void* k,
                       const void* v, const void* dO, int dt, const bsp_attn_fp8_t* fp8, const float* lse,
                       const float* dterm, float* dq, float* dk, float* dv, bsp_diag_t* diag, void* stream) {
  return attn_bwd_dterm_impl(B, H, S, Dh, causal, softmax_scale, q, k, v, dO, dt, fp8, lse, dterm, dq, dk, dv, diag,
                             stream);
}

int bsp_attn_bwd_dterm_fused(int B, int H, int S, int Dh, int causal, float softmax_scale, const void* q, const void* k,
                             const void* v, const void* dO, int dt, const float* lse, const float* dterm, float* dq,
                             float* dk, float* dv, bsp_diag_t* diag, void* stream) {
  return attn_bwd_fused_impl(B, H, S, Dh, causal, softmax_scale, q, k, v, dO, dt, lse, dterm, dq, dk, dv, diag, stream);
}

int bsp_attn_bwd(int B, int H, int S, int Dh, int causal, float softmax_scale, int fp8_operands, const void* q,
                 const void* k, const void* v, const void* dO, int dt, const bsp_attn_fp8_t* fp8, const float* lse,
                 const float* o_orig, const uint8_t* o_codes, const float* o_scales, int o_fmt, int d_read,
                 bsp_key_t key, float* dq, float* dk, float* dv, float* d_out, bsp_diag_t* diag, void* stream) {
  if ((fp8_operands != 0) != (fp8 != nullptr)) return BSP_ERR_ARG;
  if (!d_out || (fp8 && !fp8->do_scale)) return BSP_ERR_ARG;
  int rc = attn_dterm_impl(B, H, S, Dh, dO, dt, fp8 ? fp8->do_scale : nullptr, o_orig, o_codes, o_scales, o_fmt,
                           d_read, key, (int)key.draw, 1, d_out, stream);
  if (rc != BSP_OK) return rc;
  return attn_bwd_dterm_impl(B, H, S, Dh, causal, softmax_scale, q, k, v, dO, dt, fp8, lse, d_out, dq, dk, dv, diag,
                             stream);
}

int bsp_attn_quantize(const void* x, int n_groups, size_t group_size, int fmt, void* xq, uint8_t* codes, float* amax,
                      float* scales, bsp_diag_t* diag, void* stream) {
  if (!x || (!xq && !codes) || !amax || !scales || n_groups <= 0 || !valid_enum(fmt, 1)) return BSP_ERR_ARG;
  if (group_size == 0 || group_size % 8 != 0) return BSP_ERR_UNSUPPORTED;
  if (!aligned16(x) || !aligned16(xq) || (reinterpret_cast<uintptr_t>(codes) & 7u)) return BSP_ERR_ALIGN;
  int rc = bsp_amax(x, BSP_BF16, (size_t)n_groups, group_size, amax, diag, stream);
  if (rc != BSP_OK) return rc;
  if ((rc = bsp_scale_from_amax(amax, (size_t)n_groups, fmt, scales, stream)) != BSP_OK) return rc;
  const size_t n8 = (size_t)n_groups * group_size / 8;
  const unsigned grid = (unsigned)((n8 + 255) / 256);
  cudaStream_t st = (cudaStream_t)stream;
  if (fmt == BSP_E4M3)
    quantize_decode_kernel<BSP_E4M3><<<grid, 256, 0, st>>>(reinterpret_cast<const uint16_t*>(x), group_size, scales,
                                                           reinterpret_cast<uint16_t*>(xq), codes, n8);
  else
    quantize_decode_kernel<BSP_E5M2><<<grid, 256, 0, st>>>(reinterpret_cast<const uint16_t*>(x), group_size, scales,
                                                           reinterpret_cast<uint16_t*>(xq), codes, n8);
  BSP_LAUNCH_CHECK();
  return BSP_OK;
}

}  // extern "C"
