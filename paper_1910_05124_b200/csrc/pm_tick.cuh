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
  uint64_t yout_off;      // ws: last stage's output [2][T*n_out_last]: activation type (MSE) or fp32 logits (CE)
  uint64_t tgt_off;       // ws: target ring [P+1]: [T*n_out_last] float (MSE) or [T] int32 (CE)
  uint64_t pe_off;        // ws: sinusoidal positions [seq_len][d] float (0 if no embedding stage)
  uint64_t rowloss_off;   // ws: per-token losses [T] float (cross-entropy)
  uint64_t colred_off;    // ws: per-row-chunk partial column sums [P][row_chunks][2*max_dim] float
  int32_t row_chunks;     // ceil(T / chunk_rows)
  int32_t chunk_rows;     // rows of a microbatch one block of a column reduction covers (256, or 32 for short microbatches)
  int32_t loss_kind;      // PM_LOSS_*
  int32_t any_pre, any_ln, any_embed, any_residual;   // which grouped launches this pipeline needs
  int32_t att_S, att_dk, att_blocks;                   // attention: sequence length, head width, (sequences x heads); 0 = none
  int32_t max_vocab, max_embed_dim;
  uint64_t loss_off;      // ws: loss log [loss_cap] float
  uint64_t lossred_off;   // ws: per-block loss partials [64] float + completion counter
  int64_t loss_cap;
  // stage lists of the grouped launches (device, in pipeline order): stages with a pre-op, with LayerNorm, with an
  // embedding, with a residual add; grids have one block row per list entry
  const int32_t* pre_ids; const int32_t* ln_ids; const int32_t* embed_ids; const int32_t* res_ids;
  int32_t n_pre, n_ln, n_embed, n_res;
  uint64_t lnred_off;     // ws: LayerNorm parameter-gradient partials [n_ln][ln_chunks][2*max_ln_dim] float
  int32_t ln_chunks, ln_chunk_rows, max_ln_dim;
  // activation-backward launches: column blocks (256 columns) of Linear `lvl` over all stages, flattened;
  // act_start[lvl * (P + 1) + p] is the first block of stage p, act_blocks[lvl] the total
  const int32_t* act_start;
  int32_t act_blocks[PM_MAX_LINEARS];
  int32_t ln_fused;       // every LayerNorm width is a multiple of 8 and at most 1024: one fused backward kernel
  // encoder memory (ring arena) [mem_depth][T*mem_dim], slot = microbatch % mem_depth, and its gradient
  // (workspace) [gmem_depth][T*mem_dim], slot = microbatch % gmem_depth; mem_dim = 0 when there is none
  uint64_t mem_ring, gmem_off;
  int32_t mem_depth, gmem_depth, mem_dim, n_streams;
  int32_t second_embed_stage;   // the stage that embeds the second token stream (when n_streams == 2)
  int32_t max_lin;        // largest n_lin over stages
  int32_t max_dim;        // largest n_in / n_out over stages
  // microbatch-major order: the forward pass reads its weights from the stages' version rings
  int32_t mb_major;
  // launches restricted to one stage (microbatch-major order runs the stages one after the other): kernels that take
  // the stage from a block coordinate use sel_p instead (-1: all stages, the coordinate); the stage lists above then
  // point at that stage's entry; act_first[lvl] is added to the block index of the activation-backward walk
  int32_t sel_p;
  int32_t sel_tile0;      // GEMM launches of one stage: flattened id of the stage's first tile (set by the launcher)
  int32_t act_first[PM_MAX_LINEARS];
  int32_t res_fused;      // the forward GEMM's epilogue adds the skip tensor (bf16 tensor-core path): no residual kernel
  int32_t dgrad_split_below;   // CTA-pair dgrad: a Linear whose two-row-tile groups number fewer than this takes one row tile per
                               // group (0: always two); launches of one stage need enough groups for the CTA pairs
  float loss_scale;       // factor on dL/dy: 1/N with N microbatches per update (the minibatch loss is their mean), else 1
  int32_t ln_li0;         // first entry of ln_ids a launch covers (its grid counts entries from there)
  int32_t colsum_only;    // activation-backward launch that only sums columns (bias gradients) of Linears WITHOUT activation:
                          // stages with an activation were handled by their own launch (microbatch-major order)
  int32_t defer_finish;   // launches of one stage leave the per-chunk partial sums of bias / LayerNorm gradients in place;
                          // one grouped launch over all stages adds them up at the end of the backward pass
  // weight-gradient launch that applies the PipeMare update to the Linear matrices in its epilogue (bf16 tensor-core
  // path): dW never reaches the grad arena; the stage's step size, T2 decay and bias corrections come from its table
  // entry, the optimiser constants from here, and the operand-type copy of the new weights goes to lp_base
  int32_t fin_deferred;   // bias finishing pass launched once for all stages at the end of a microbatch-major backward pass: the partial
                          // rows were written by launches of one stage (Linears with activation) or by the column-sum-only launch
  int32_t ln_stage;       // LayerNorm backward: a block first brings its rows of x, du and the skip gradient into shared memory
                          // with asynchronous copies (all in flight at once), then works from there (set by the launcher)
  int32_t stash;          // weight stashing (tau_bkwd = tau_fwd for every stage): the backward pass reads the queued version the
                          // microbatch's forward read (weights and LayerNorm gain), not the live weights
  int32_t fuse_upd;       // 0: dW is stored (or added) to the grad arena
  int32_t upd_opt;        // PM_SGDM | PM_ADAM
  float upd_beta1, upd_beta2, upd_eps;
  __nv_bfloat16* upd_lp;  // base of the bfloat16 copy: the w_lp arena (tick-major order) or the ring arena (version queues)
};

// stage of a block in a kernel whose grid has one coordinate per stage
__device__ __forceinline__ int stage_of_block(const TickArgs& t, unsigned coord) { return t.sel_p >= 0 ? t.sel_p : (int)coord; }
// the weights the forward pass reads, in the GEMM operand type WT (float | bf16), at element offset `arena_off` of
// the flat arenas: the live weights (tick-major: the stage holds one version), or the stage's version-ring slot
template <typename WT> __device__ __forceinline__ const WT* fwd_weights(const TickArgs& t, const StageDev& s, const StageDyn& d, uint64_t arena_off) {
  if (!t.mb_major) return (sizeof(WT) == 4 ? reinterpret_cast<const WT*>(t.a.w) : reinterpret_cast<const WT*>(t.a.w_lp)) + arena_off;
  return reinterpret_cast<const WT*>(t.ring + s.v_ring) + (uint64_t)d.f_vslot * (s.end - s.begin) + (arena_off - s.begin);
}
// an fp32 tensor the forward pass reads (bias, LayerNorm gain / bias): arena offset and offset inside a small-ring slot
template <typename AT> __device__ __forceinline__ const float* fwd_small(const TickArgs& t, const StageDev& s, const StageDyn& d, uint64_t arena_off, uint32_t soff) {
  if (!t.mb_major) return t.a.w + arena_off;
  if (sizeof(AT) == 4) return fwd_weights<float>(t, s, d, arena_off);
  return reinterpret_cast<const float*>(t.ring + s.s_ring) + (uint64_t)d.f_vslot * s.small_count + soff;
}

// ---- where things live (shared by every tick kernel) -----------------------------------------------------
template <typename AT> __device__ __forceinline__ AT* ring_at(const TickArgs& t, uint64_t off, int slot, uint64_t slot_elems) {
  return reinterpret_cast<AT*>(t.ring + off) + (uint64_t)slot * slot_elems;
}
template <typename AT> __device__ __forceinline__ AT* ws_at(const TickArgs& t, uint64_t off) {
  return reinterpret_cast<AT*>(t.ws + off);
}
// input activation of Linear `lvl` (forward A operand, wgrad B operand); fwd selects this tick's forward or backward slot
template <typename AT> __device__ __forceinline__ const AT* lin_input(const TickArgs& t, const StageDev& s, const StageDyn& d, int lvl, bool fwd) {
  const uint64_t n = (uint64_t)t.T * s.lin[lvl].n_in;
  if (lvl > 0) return ring_at<AT>(t, s.lin[lvl - 1].h_ring, fwd ? d.f_slot : d.b_slot, n);
  if (s.pre != PRE_NONE) return ring_at<AT>(t, s.u_ring, fwd ? d.f_slot : d.b_slot, n);
  return ring_at<AT>(t, s.x_ring, fwd ? d.f_xslot : d.b_xslot, n);
}
// slot of a stage's gradient mailbox that holds what was written during the previous tick
__device__ __forceinline__ int gin_slot_read(const StageDev& s, const StageDyn& d) { (void)s; return d.gin_rslot; }
// slot of the dz operand of a stage's last Linear when that operand is the incoming gradient itself (no activation,
// no attention): the rotating mailbox slot written during the previous tick, or the memory-gradient ring slot of the
// microbatch for the stage that emits the memory
__device__ __forceinline__ int dz_mailbox_slot(const TickArgs& t, const StageDev& s, const StageDyn& d) {
  (void)t; return s.emit_memory ? d.gmem_slot : d.gin_rslot;
}
// gradient of the memory for the microbatch in backward at a stage
template <typename AT> __device__ __forceinline__ AT* gmem_at(const TickArgs& t, const StageDyn& d) {
  return ws_at<AT>(t, t.gmem_off) + (uint64_t)d.gmem_slot * ((uint64_t)t.T * t.mem_dim);
}
// gradient w.r.t. this stage's main output: written by the next stage during the previous tick; the stage that
// emits the memory receives the sum the cross-attention stages left in the memory-gradient ring
template <typename AT> __device__ __forceinline__ AT* gin_read(const TickArgs& t, const StageDev& s, const StageDyn& d) {
  if (s.emit_memory) return gmem_at<AT>(t, d);
  return ws_at<AT>(t, s.gin) + (uint64_t)gin_slot_read(s, d) * ((uint64_t)t.T * s.d_out_main);
}
// where stage p writes the gradient w.r.t. its main input (= stage p-1's main output)
template <typename AT> __device__ __forceinline__ AT* gin_write_prev(const TickArgs& t, int p, const StageDyn& d) {
  const StageDev& sp = t.st[p - 1];
  return ws_at<AT>(t, sp.gin) + (uint64_t)d.prev_wslot * ((uint64_t)t.T * sp.d_out_main);
}
// gradient w.r.t. the skip tensor stage p emitted: it equals the gradient the receiving (residual) stage took in
// skip_hop ticks ago for the same microbatch, i.e. what the stage after that one wrote skip_hop + 1 ticks ago
template <typename AT> __device__ __forceinline__ const AT* gskip_read(const TickArgs& t, int p, const StageDyn& d) {
  const StageDev& sn = t.st[p + t.st[p].skip_hop];
  if (sn.emit_memory) return gmem_at<AT>(t, d);
  const int slot = (int)((d.tick + 2 * sn.gin_depth - t.st[p].skip_hop - 1) % sn.gin_depth);
  return ws_at<AT>(t, sn.gin) + (uint64_t)slot * ((uint64_t)t.T * sn.d_out_main);
}
// does stage p emit a skip tensor
__device__ __forceinline__ bool emits_skip(const StageDev& s) { return s.skip_hop > 0; }
// the memory of the microbatch a stage processes (forward or backward)
template <typename AT> __device__ __forceinline__ AT* mem_at(const TickArgs& t, int64_t mb) {
  return ring_at<AT>(t, t.mem_ring, (int)(mb % t.mem_depth), (uint64_t)t.T * t.mem_dim);
}
// dz = dy * act'(z) of Linear lvl as the wgrad / dgrad operand: without an activation it IS the incoming gradient
template <typename AT> __device__ __forceinline__ const AT* dz_src(const TickArgs& t, const StageDev& s, const StageDyn& d, int lvl) {
  if (bwd_act(s.lin[lvl]) != PM_ACT_NONE) return ws_at<AT>(t, s.dz);
  if (lvl < s.n_lin - 1) return ws_at<AT>(t, s.dh);
  if (feeds_attention(s.post)) return ws_at<AT>(t, s.dy);
  return gin_read<AT>(t, s, d);
}
// destination of Linear lvl's activation y in the forward pass (nullptr: not written)
template <typename AT> __device__ __forceinline__ AT* y_dest(const TickArgs& t, int p, const StageDev& s, const StageDyn& d, int lvl) {
  const LinDev& L = s.lin[lvl];
  if (!(L.flags & LF_WRITE_Y)) return nullptr;
  const uint64_t n = (uint64_t)t.T * L.n_out;
  if (lvl < s.n_lin - 1) return ring_at<AT>(t, L.h_ring, d.f_slot, n);
  if (s.post == POST_RESIDUAL) return ws_at<AT>(t, s.ytmp);
  if (p < t.P - 1) return ring_at<AT>(t, t.st[p + 1].x_ring, d.f_next_xslot, n);
  return ws_at<AT>(t, t.yout_off) + (uint64_t)(d.tick & 1) * n;
}

// inputs/targets -> stage 1's input ring slot and the target ring (activation type AT = float | bf16).
cudaError_t launch_ingest(const TickArgs& t, int dtype, const void* inputs, const float* targets, int64_t mb,
                          cudaStream_t stream);
// MSE loss of the microbatch whose backward starts this tick, and dL/dy into the last stage's mailbox.
cudaError_t launch_loss(const TickArgs& t, int dtype, cudaStream_t stream);
// dz = dy * act'(z) and db = column sums, level `lvl` of every stage that runs backward this tick.
cudaError_t launch_actbwd(const TickArgs& t, int dtype, int lvl, cudaStream_t stream);
int actbwd_launches(const TickArgs& t);
// the finishing passes that launches with defer_finish left out, grouped over all stages (bias column sums, LayerNorm
// parameter gradients)
cudaError_t launch_deferred_finish(const TickArgs& t, int dtype, cudaStream_t stream);
int deferred_finish_launches(const TickArgs& t);
cudaError_t launch_ln_finish(const TickArgs& t, cudaStream_t stream);      // pm_xfmr.cu
int ln_finish_launches(const TickArgs& t);

// Transformer pieces (all grouped over the stages that carry the op this tick).
cudaError_t launch_pre_fwd(const TickArgs& t, int dtype, cudaStream_t stream);        // embedding / LayerNorm forward (+ skip hand-over)
cudaError_t launch_post_fwd(const TickArgs& t, int dtype, cudaStream_t stream, bool skip_attention);   // attention forward (SIMT), residual add
cudaError_t launch_post_bwd(const TickArgs& t, int dtype, cudaStream_t stream);       // attention backward
// tensor-core attention (bf16, sequences of 128, heads of 64)
struct AttnPlan;
uint64_t attn_workspace_bytes(int n_stages);
bool attn_tc_supported(int dtype, int S, int dk);
cudaError_t attn_tc_launch(AttnPlan* plan, const TickArgs& t, bool forward, cudaStream_t stream);
void attn_plan_destroy(AttnPlan* plan);
int* attn_status_word(AttnPlan* plan);
cudaError_t launch_pre_bwd(const TickArgs& t, int dtype, cudaStream_t stream);        // LayerNorm / embedding backward
int pre_bwd_launches(const TickArgs& t);
size_t attention_smem_bytes(int S, int dk, int dtype);
cudaError_t attention_set_smem_limits(int S, int dk, int dtype);

// fp32 SIMT grouped GEMMs (PM_F32 path).  mode: 0 forward, 1 dgrad (corrected weights), 2 wgrad.
cudaError_t launch_simt_gemm(const TickArgs& t, int dtype, int mode, int lvl, cudaStream_t stream);

}  // namespace pm
