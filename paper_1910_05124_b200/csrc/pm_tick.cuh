// Per-tick kernel launches of the pipeline (declarations shared by the host code).
#pragma once
#include "pm_common.cuh"

namespace pm {

// Everything a tick kernel needs; passed by value.
struct TickArgs {
  const StageDev* st;
  const StageDyn* dyn;
  ArenasDev a;
  char* ring;
  char* ws;
  int32_t T, P;
  int32_t n_in_first, n_out_last;
  uint64_t yout_off;      // ws: last stage's output [2][T*n_out_last] (activation type)
  uint64_t tgt_off;       // ws: target ring [P+1][T*n_out_last] float
  uint64_t loss_off;      // ws: loss log [loss_cap] float
  uint64_t lossred_off;   // ws: per-block loss partials [64] float + completion counter
  int64_t loss_cap;
  int32_t max_lin;        // largest n_lin over stages
  int32_t max_dim;        // largest n_in / n_out over stages
};

// inputs/targets -> stage 1's input ring slot and the target ring (activation type AT = float | bf16).
cudaError_t launch_ingest(const TickArgs& t, int dtype, const void* inputs, const float* targets, int64_t mb,
                          cudaStream_t stream);
// MSE loss of the microbatch whose backward starts this tick, and dL/dy into the last stage's mailbox.
cudaError_t launch_loss(const TickArgs& t, int dtype, cudaStream_t stream);
// dz = dy * act'(z) and db = column sums, level `lvl` of every stage that runs backward this tick.
cudaError_t launch_actbwd(const TickArgs& t, int dtype, int lvl, cudaStream_t stream);

// fp32 SIMT grouped GEMMs (PM_F32 path).  mode: 0 forward, 1 dgrad (corrected weights), 2 wgrad.
cudaError_t launch_simt_gemm(const TickArgs& t, int dtype, int mode, int lvl, cudaStream_t stream);

}  // namespace pm
