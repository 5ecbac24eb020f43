// Tick scheduler and the fused multi-tensor PipeMare update (declarations).
#pragma once
#include "pm_common.cuh"

namespace pm {

// What the scheduler needs to know about a stage (device table, constant over the run).
struct StageSched {
  int32_t tau_f, gap, depth, xdepth, next_xdepth, gin_depth, prev_gin_depth, gmem_depth;
  int32_t skip_dst_depth, skip_depth;   // slots of the skip buffer this stage writes into / reads from (0: none)
};

// Launches the scheduler for pipeline tick `tick` with `n_fed` microbatches fed so far.
// flat_k >= 0 selects the stand-alone update mode: every stage is at update index flat_k.
cudaError_t launch_schedule(const StageSched* sched, const int64_t* nupd, StageDyn* dyn, HyperDev hp,
                            int64_t tick, int64_t n_fed, int64_t flat_k, cudaStream_t stream);

// Launches the fused update over all stages whose dyn[i].active_update is set.
// begin64/end64: stage bounds in units of 64 elements, ascending; total64 = end64[P-1].
cudaError_t launch_update(ArenasDev a, const uint32_t* begin64, const uint32_t* end64, const StageDyn* dyn,
                          int64_t* nupd, int n_stages, uint64_t total64, int optimizer, float beta1, float beta2,
                          float eps, cudaStream_t stream);

}  // namespace pm
