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
  int32_t tau_r, rdepth;                // PipeMare Recompute: delay of the recomputation's weights, slots of their corrected queue
};

// Launches the scheduler for pipeline tick `tick` with `n_fed` microbatches fed so far.
// flat_k >= 0 selects the stand-alone update mode: every stage is at update index flat_k.
cudaError_t launch_schedule(const StageSched* sched, const int64_t* nupd, StageDyn* dyn, HyperDev hp,
                            int64_t tick, int64_t n_fed, int64_t flat_k, cudaStream_t stream);
// Microbatch-major order: fills the tables of microbatch t ([n_tables][P] entries): table v < 2P for the launches of
// sub-tick v (stage i forward at v = i, backward at v = 2P - 1 - i), table 2P for the grouped weight-gradient launch
// and the update.  With PipeMare Recompute (hp.segment > 0) table 2P + 1 holds every stage's recomputation (its forward
// entry with the recompute weights' slot) and table 2P + 2 + k the backward entries of segment k alone (the grouped
// weight-gradient launch of that segment).
// delays / nupd (stochastic delay model only, else null): the step's per-stage delays and the stages' update counters.
cudaError_t launch_schedule_mb(const StageSched* sched, StageDyn* tables, HyperDev hp, int64_t t, cudaStream_t stream,
                               const int32_t* delays = nullptr, const int64_t* nupd = nullptr);
inline int mb_table_count(int P, int segment) { return 2 * P + 1 + (segment > 0 ? 1 + (P + segment - 1) / segment : 0); }

// Launches the fused update over all stages whose dyn[i].active_update is set.
// begin64/end64: stage bounds in units of 64 elements, ascending; total64 = end64[P-1].
cudaError_t launch_update(ArenasDev a, const uint32_t* begin64, const uint32_t* end64, const StageDyn* dyn,
                          int64_t* nupd, int n_stages, uint64_t total64, int optimizer, float beta1, float beta2,
                          float eps, cudaStream_t stream, void* lp_base = nullptr, int lp_elem = 0, uint64_t first64 = 0,
                          const uint32_t* skip_b64 = nullptr, const uint32_t* skip_e64 = nullptr, const float* gsrc = nullptr);
// gsrc: where the gradients are read (element e of stage i at gsrc[dyn[i].g_shift + e]); null: the grad arena.
// skip_b64 / skip_e64: per stage, a range of 64-element groups this launch leaves alone (device arrays, or null): the
// Linear matrices when the weight-gradient GEMM has applied their update in its epilogue.  The stage's update
// counter is incremented here all the same.
// first64: the walk over the arenas starts at this 64-element group (a launch for one stage starts at that stage's slice).
// lp_base / lp_elem: where the operand-type copy of the new weights goes: by default the bfloat16 arena a.w_lp
// (if there is one); microbatch-major order passes the ring arena and the operand size (2 or 4 bytes), and the
// stages' table entries give the slot (StageDyn::lp_shift).

// One fp32 tensor the forward pass reads (a bias, a LayerNorm gain or bias): `count` elements (a multiple of 64,
// padding included) at arena_off of the master weights; its versions sit at ring_off (bytes, slot 0) of the ring
// arena, slot_stride floats apart.
// rc_base: first slot of the stage's corrected recompute weights (= its vdepth), -1 when it keeps none.
struct SmallSeg { uint64_t arena_off, ring_off; uint32_t count, slot_stride; int32_t stage, rc_base; };
// Copies every segment from the master weights into slot dyn[stage].u_vslot of its ring and, for a stage with a queue of
// corrected recompute weights, w - dyn[stage].rc_gap * delta into slot dyn[stage].rc_uslot.  slot_override >= 0 (the
// initial fill, delta = 0): plain copies into that slot and into rc_base + slot_override.
cudaError_t launch_push_small(const float* w, const float* delta, char* ring, const SmallSeg* segs, int n_segs, const StageDyn* dyn,
                              int slot_override, cudaStream_t stream);

}  // namespace pm
