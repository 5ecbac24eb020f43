// Tick scheduler and the fused multi-tensor PipeMare update (declarations).
#pragma once
#include "pm_common.cuh"

namespace pm {

// What the scheduler needs to know about a stage (device table, constant over the run).
struct StageSched {
  int32_t tau_f, gap, depth, xdepth, next_xdepth, gin_depth, prev_gin_depth, gmem_depth;
  int32_t skip_dst_depth, skip_depth;   // slots of the skip buffer this stage writes into / reads from (0: none)
  // version rings (microbatch-major order; vdepth <= 1: none): slots, the stage's element range in the arenas and the
  // byte offset of its operand-type ring in the ring arena
  int32_t vdepth, _pad;
  uint64_t begin, count, v_ring;
};

// Launches the scheduler for pipeline tick `tick` with `n_fed` microbatches fed so far.
// flat_k >= 0 selects the stand-alone update mode: every stage is at update index flat_k.
cudaError_t launch_schedule(const StageSched* sched, const int64_t* nupd, StageDyn* dyn, HyperDev hp,
                            int64_t tick, int64_t n_fed, int64_t flat_k, cudaStream_t stream);
// Microbatch-major order: fills the 2P + 1 tables of microbatch t ([2P + 1][P] entries): table v for the launches of
// sub-tick v (stage i forward at v = i, backward at v = 2P - 1 - i), table 2P for the grouped weight-gradient launch
// and the update.
cudaError_t launch_schedule_mb(const StageSched* sched, StageDyn* tables, HyperDev hp, int64_t t, cudaStream_t stream);

// Launches the fused update over all stages whose dyn[i].active_update is set.
// begin64/end64: stage bounds in units of 64 elements, ascending; total64 = end64[P-1].
cudaError_t launch_update(ArenasDev a, const uint32_t* begin64, const uint32_t* end64, const StageDyn* dyn,
                          int64_t* nupd, int n_stages, uint64_t total64, int optimizer, float beta1, float beta2,
                          float eps, cudaStream_t stream, void* lp_base = nullptr, int lp_elem = 0, uint64_t first64 = 0);
// first64: the walk over the arenas starts at this 64-element group (a launch for one stage starts at that stage's slice).
// lp_base / lp_elem: where the operand-type copy of the new weights goes: by default the bfloat16 arena a.w_lp
// (if there is one); microbatch-major order passes the ring arena and the operand size (2 or 4 bytes), and the
// stages' table entries give the slot (StageDyn::lp_shift).

// One fp32 tensor the forward pass reads (a bias, a LayerNorm gain or bias): `count` elements (a multiple of 64,
// padding included) at arena_off of the master weights; its versions sit at ring_off (bytes, slot 0) of the ring
// arena, slot_stride floats apart.
struct SmallSeg { uint64_t arena_off, ring_off; uint32_t count, slot_stride; int32_t stage, _pad; };
// Copies every segment from the master weights into slot dyn[stage].u_vslot of its ring (slot_override >= 0: that slot).
cudaError_t launch_push_small(const float* w, char* ring, const SmallSeg* segs, int n_segs, const StageDyn* dyn,
                              int slot_override, cudaStream_t stream);

}  // namespace pm
