// Internal interface of the Monte-Carlo statistics pass, shared by the two per-use checks: a check
// launches each of its statistics passes into a slot of block partials as soon as the pass's inputs
// are queued, and brings all slots to the host behind one synchronisation at its end.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "common.cuh"

namespace bsp {

constexpr int kStatBlocks = 592;     // 4 per SM
constexpr int kStatFields = 8;       // err2, ref2, se2, z2, z, max|z|, count(|z|>3), unused
constexpr size_t kStatSlotDoubles = (size_t)kStatBlocks * kStatFields;
constexpr size_t kStatSlotBytes = kStatSlotDoubles * sizeof(double);   // a multiple of 256

// Launches the pass over n elements into one slot; *blocks_out = blocks whose partials the slot holds.
int mc_stats_launch(const float* g_ref, const float* g, const float* S2, int64_t n, int K, int fresh,
                    const bsp_verdict_rule_t* rule, double* partials, cudaStream_t st, int* blocks_out);
// Sums a slot's block partials on the host, in block order, and fills the result of the use; the
// verdict follows `rule` (NULL: the default thresholds, see default_rule()).
void mc_stats_finish(const double* host, int blocks, int64_t n, int K, int fresh, const bsp_verdict_rule_t* rule,
                     bsp_use_result_t* result);
const bsp_verdict_rule_t* default_rule();
// A rule is usable when its thresholds are ordered: hold <= fail for both statistics, nothing negative.
bool rule_valid(const bsp_verdict_rule_t* rule);

constexpr int kMaxPendingStats = 12;
struct PendingStats {
  bsp_use_result_t* result[kMaxPendingStats];
  int blocks[kMaxPendingStats], K[kMaxPendingStats], fresh[kMaxPendingStats];
  int64_t n[kMaxPendingStats];
  int count = 0;
  double* slots = nullptr;           // device: kMaxPendingStats slots of kStatSlotDoubles
  cudaStream_t st = nullptr;
  const bsp_verdict_rule_t* rule = nullptr;

  // A fresh read whose every draw equals the reference (a gradient that does not read the saved
  // tensor): all sums are zero, no pass needed.
  void add_exact_fresh(int64_t n_, int K_, bsp_use_result_t* r) { mc_stats_finish(nullptr, 0, n_, K_, 1, rule, r); }
  int add(const float* g_ref, const float* g, const float* S2, int64_t n_, int K_, int fresh_, bsp_use_result_t* r) {
    if (!fresh_ && g == g_ref) {
      // a read that is the reference itself: its error is exactly zero, no pass needed
      mc_stats_finish(nullptr, 0, n_, K_, 0, rule, r);
      return BSP_OK;
    }
    if (count >= kMaxPendingStats) return BSP_ERR_ARG;
    const int slot = count++;
    result[slot] = r; n[slot] = n_; K[slot] = K_; fresh[slot] = fresh_;
    return mc_stats_launch(g_ref, g, S2, n_, K_, fresh_, rule, slots + (size_t)slot * kStatSlotDoubles, st, &blocks[slot]);
  }
  // One copy, one synchronisation, then the host sums.  The stream is idle when this returns.
  int flush() {
    std::vector<double> host((size_t)(count > 0 ? count : 1) * kStatSlotDoubles);
    if (count > 0) {
      BSP_CHECK_CUDA(cudaMemcpyAsync(host.data(), slots, (size_t)count * kStatSlotBytes, cudaMemcpyDeviceToHost, st));
      count_d2h((size_t)count * kStatSlotBytes);
    }
    BSP_CHECK_CUDA(cudaStreamSynchronize(st));
    for (int i = 0; i < count; ++i)
      mc_stats_finish(host.data() + (size_t)i * kStatSlotDoubles, blocks[i], n[i], K[i], fresh[i], rule, result[i]);
    count = 0;
    return BSP_OK;
  }
};

}  // namespace bsp
