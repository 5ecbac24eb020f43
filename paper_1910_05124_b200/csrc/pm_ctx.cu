// Host side of the C ABI: layout arithmetic, context set-up, and the launch sequence of a tick.
#include <functional>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <string>
#include <vector>

#include "pm_tick.cuh"
#include "pm_update.cuh"
#include "pm_umma.cuh"

namespace pm {
pm_status attn_plan_create(AttnPlan** out, const TickArgs& t, const std::vector<StageDev>& st, void* ws_region, cudaStream_t stream, std::string& err);
}

using namespace pm;

namespace {

thread_local std::string g_error = "";

inline uint64_t align_up(uint64_t v, uint64_t a) { return (v + a - 1) / a * a; }

struct Layout {
  std::vector<StageDev> st;
  std::vector<StageSched> sched;
  std::vector<uint32_t> begin64, end64;
  std::vector<uint32_t> skip_b64, skip_e64;   // per stage, the Linear matrix's range in 64-element groups (fused update), else empty
  uint64_t off_skb = 0, off_ske = 0;
  int32_t fuse = 0;                     // the weight-gradient GEMM applies the update of the Linear matrices in its epilogue
  int32_t stash = 0;                    // weight stashing: every stage has tau_bkwd = tau_fwd (microbatch-major order)
  int32_t materialize = 0;              // the corrected backward weights are written by the update into a slot of the version queue
  int32_t stochastic = 0;               // stage-wise stochastic delays (Appendix E): slots of the gradient ring (tau_max + 1), 0: off
  uint64_t g_ring = 0, off_delays = 0;  // ring: [stochastic][total] float gradients of the last microbatches; ws: the step's delays [P]
  uint64_t ring_bytes = 0, ws_bytes = 0, total = 0;
  // workspace offsets
  uint64_t off_st = 0, off_sched = 0, off_dyn = 0, off_nupd = 0, off_b64 = 0, off_e64 = 0, off_alpha = 0;
  uint64_t off_loss = 0, off_tgt = 0, off_yout = 0, off_umma = 0, off_lossred = 0, off_pe = 0, off_rowloss = 0, off_attn = 0, off_colred = 0;
  uint64_t off_ids = 0, off_lnred = 0, mem_ring = 0, off_gmem = 0;
  int32_t mem_stage = -1, last_mem_reader = -1, mem_dim = 0, mem_depth = 0, gmem_depth = 0, n_streams = 1;
  bool att_plain = true;
  std::vector<int32_t> ids;             // [pre | ln | embed | residual] stage lists, P entries each; then act_start[PM_MAX_LINEARS][P+1]
  int32_t act_blocks[PM_MAX_LINEARS] = {};
  int32_t n_pre = 0, n_ln = 0, n_embed = 0, n_res = 0, ln_chunks = 0, ln_chunk_rows = 0, max_ln_dim = 0, ln_fused = 1;
  int32_t row_chunks = 1, chunk_rows = 256;
  bool att_tc = false;
  int32_t any_pre = 0, any_ln = 0, any_embed = 0, any_residual = 0, att_S = 0, att_dk = 0, att_blocks = 0, max_vocab = 0;
  int32_t pe_seq = 0, pe_d = 0;
  int64_t loss_cap = 0;
  int32_t max_lin = 0, max_dim = 0, n_in_first = 0, n_out_last = 0;
  // microbatch-major order
  bool mb = false;
  bool queue = false;                   // the forward pass reads its weights from per-stage version queues (mb, or entry period > 1)
  int32_t E = 1;                        // tick-major order: ticks between two entering microbatches
  int32_t n_tables = 1;                 // per-tick tables: 1, or 2P + 1 (one per sub-tick and one for the grouped launches),
                                        // with PipeMare Recompute one more for the recomputation and one per segment
  int32_t segment = 0;                  // PipeMare Recompute: stages per segment (0: none)
  std::vector<SmallSeg> segs;           // fp32 tensors the forward pass reads, per version ring slot (bf16 operands)
  uint64_t off_segs = 0;
  std::vector<int32_t> pre_idx, ln_idx, embed_idx, res_idx;   // position of a stage in the stage lists (-1: not in it)
};

pm_status fail(pm_ctx* ctx, pm_status s, const std::string& msg);

// Parameter tensors of an op: count (0, 1 or 2) and their sizes.
static int op_params(const pm_op_desc& op, uint64_t* n0, uint64_t* n1) {
  switch (op.kind) {
    case PM_OP_LINEAR: *n0 = (uint64_t)op.n_in * op.n_out; *n1 = (uint64_t)op.n_out; return 2;
    case PM_OP_LAYERNORM: *n0 = (uint64_t)op.n_in; *n1 = (uint64_t)op.n_in; return 2;
    case PM_OP_EMBED: *n0 = (uint64_t)op.n_in * op.n_out; *n1 = 0; return 1;
    default: *n0 = *n1 = 0; return 0;
  }
}

pm_status build_layout(const pm_config* cfg, const pm_stage_desc* stages, Layout& L, std::string& err) {
  if (!cfg || !stages) { err = "null config or stage list"; return PM_ERR_INVALID_ARG; }
  const int P = cfg->n_stages;
  if (P < 1 || P > PM_MAX_STAGES) { err = "n_stages must be in [1, " + std::to_string(PM_MAX_STAGES) + "]"; return PM_ERR_INVALID_ARG; }
  if (cfg->microbatch < 1) { err = "microbatch must be positive"; return PM_ERR_INVALID_ARG; }
  if (cfg->compute_dtype != PM_F32 && cfg->compute_dtype != PM_BF16) { err = "unknown compute_dtype"; return PM_ERR_INVALID_ARG; }
  if (cfg->optimizer != PM_SGDM && cfg->optimizer != PM_ADAM) { err = "unknown optimizer"; return PM_ERR_INVALID_ARG; }
  if (cfg->loss != PM_LOSS_MSE && cfg->loss != PM_LOSS_CE) { err = "unknown loss"; return PM_ERR_INVALID_ARG; }
  if (cfg->t1_enable && cfg->t1_K < 1) { err = "t1_K must be >= 1"; return PM_ERR_INVALID_ARG; }
  if (cfg->loop_order != PM_TICK_MAJOR && cfg->loop_order != PM_MB_MAJOR) { err = "unknown loop_order"; return PM_ERR_INVALID_ARG; }
  const bool mb = cfg->loop_order == PM_MB_MAJOR;
  if (cfg->n_micro < 0) { err = "n_micro must be >= 0"; return PM_ERR_INVALID_ARG; }
  if (cfg->n_micro > 1 && !mb) {
    // in a running pipeline the version a forward pass reads depends on the microbatch's position inside its minibatch
    // (floor((a - tau)/N) updates have landed), not on the fixed delay ceil(tau/N) of Table 1; the queue of weight
    // versions realises Table 1's model exactly
    err = "n_micro > 1 (several microbatches per update) is built for PM_MB_MAJOR order";
    return PM_ERR_UNSUPPORTED;
  }
  L.mb = mb;
  if (cfg->recompute_segment < 0) { err = "recompute_segment must be >= 0"; return PM_ERR_INVALID_ARG; }
  if (cfg->recompute_segment > 0 && !mb) {
    // the recomputation reads weights of its own delay tau_recomp: a third version per stage and microbatch, which the
    // queue of weight versions has and a tick schedule with one live version does not
    err = "recompute_segment > 0 (PipeMare Recompute) is built for PM_MB_MAJOR order";
    return PM_ERR_UNSUPPORTED;
  }
  const int S = cfg->recompute_segment >= P ? 0 : cfg->recompute_segment;    // one segment covering everything: the forward pass itself
  L.segment = S;
  if (cfg->stochastic_tau_max < 0) { err = "stochastic_tau_max must be >= 0"; return PM_ERR_INVALID_ARG; }
  const bool stoch = cfg->stochastic_tau_max > 0;
  if (stoch) {
    const char* why = nullptr;
    if (!mb) why = "PM_MB_MAJOR order (every microbatch is differentiated on one consistent set of weights)";
    else if (cfg->n_micro > 1) why = "one microbatch per update";
    else if (S > 0) why = "no recomputation";
    else if (cfg->fuse_update) why = "the separate update kernel (gradients wait in a ring before they are applied)";
    if (why) { err = std::string("stochastic_tau_max > 0 is built for ") + why; return PM_ERR_UNSUPPORTED; }
  }
  L.stochastic = stoch ? cfg->stochastic_tau_max + 1 : 0;
  const bool mat = cfg->materialize_backward != 0;
  if (mat && (!mb || S > 0 || stoch || cfg->fuse_update)) {
    err = "materialize_backward is built for PM_MB_MAJOR order without recompute_segment, stochastic_tau_max or fuse_update";
    return PM_ERR_UNSUPPORTED;
  }
  L.materialize = mat ? 1 : 0;
  if (cfg->entry_period < 0 || cfg->entry_period > 2 * P) { err = "entry_period must be in [0, 2 * n_stages]"; return PM_ERR_INVALID_ARG; }
  const int E = (!mb && cfg->entry_period > 1) ? cfg->entry_period : 1;
  const bool queue = mb || E > 1;
  L.E = E; L.queue = queue;
  L.n_tables = mb ? mb_table_count(P, S) : 1;
  const uint64_t esz = cfg->compute_dtype == PM_F32 ? 4 : 2;
  const uint64_t T = (uint64_t)cfg->microbatch;
  const bool ce = cfg->loss == PM_LOSS_CE;
  L.st.assign(P, StageDev{});
  L.sched.assign(P, StageSched{});
  L.begin64.assign(P, 0);
  L.end64.assign(P, 0);
  uint64_t ring = 0;
  uint64_t prev_end = 0;
  bool any_stash = false, any_plain = false;                 // stages with tau_bkwd = tau_fwd > 0 / with tau_bkwd = 0 < tau_fwd
  auto stage_err = [&](int p, const std::string& m) { err = "stage " + std::to_string(p) + ": " + m; };
  for (int p = 0; p < P; ++p) {
    const pm_stage_desc& sd = stages[p];
    StageDev& s = L.st[p];
    if (sd.n_ops < 1 || sd.n_ops > PM_MAX_LINEARS + 2 || !sd.ops) { stage_err(p, "bad op count"); return PM_ERR_INVALID_ARG; }
    if (!mb && (sd.tau_bkwd != 0 || sd.tau_fwd != 2 * (P - (p + 1)) + 1)) {
      stage_err(p, "the tick schedule realises tau_fwd = 2(P-i)+1, tau_bkwd = 0 only");
      return PM_ERR_UNSUPPORTED;
    }
    if (mb && sd.tau_fwd >= 0 && sd.tau_bkwd == sd.tau_fwd && sd.tau_fwd > 0) any_stash = true;     // weight stashing (Section 2.2)
    else if (mb && sd.tau_fwd > 0) any_plain = true;
    if (mb && ((sd.tau_bkwd != 0 && sd.tau_bkwd != sd.tau_fwd) || sd.tau_fwd < 0 || (any_stash && any_plain))) {
      stage_err(p, "microbatch-major order takes tau_fwd >= 0 with tau_bkwd = 0, or tau_bkwd = tau_fwd for every stage (weight stashing)");
      return sd.tau_fwd < 0 || sd.tau_bkwd < 0 ? PM_ERR_INVALID_ARG : PM_ERR_UNSUPPORTED;
    }
    if (sd.param_offset % PM_ALIGN_ELEMS || sd.param_count % PM_ALIGN_ELEMS) { stage_err(p, "param_offset/param_count must be multiples of 64"); return PM_ERR_INVALID_ARG; }
    if (sd.param_offset < prev_end) { err = "stage slices must ascend without overlap"; return PM_ERR_INVALID_ARG; }
    uint64_t need = 0;
    pm_status ps = pm_stage_param_count(sd.ops, sd.n_ops, &need);
    if (ps != PM_OK) { stage_err(p, "bad op list"); return ps; }
    if (sd.param_count < need) { stage_err(p, "param_count smaller than its ops need"); return PM_ERR_INVALID_ARG; }
    s.tau_f = sd.tau_fwd; s.gap = sd.tau_fwd - sd.tau_bkwd;
    if (stoch) s.gap = 0;                                    // forward and backward read the same weights: nothing for T2 to correct
    s.depth = s.tau_f + 1; s.xdepth = s.tau_f + 2;
    // the previous stage takes its ReLU mask from this stage's stashed input, one tick after this stage's own
    // backward: one more slot keeps it until then
    if (p > 0 && (L.st[p - 1].lin[L.st[p - 1].n_lin - 1].flags & LF_ACT_FROM_Y)) s.xdepth = s.tau_f + 3;
    // microbatch-major order: one microbatch in flight, so every activation ring has one slot; what grows with
    // the delay is the queue of weight versions
    s.vdepth = 1;
    if (mb) { s.depth = 1; s.xdepth = 1; s.vdepth = stoch ? 1 : s.tau_f + 1; }   // stochastic delays: the live weights only
    // PipeMare Recompute (Appendix A.2): inside a segment the recomputation runs ahead of the backward pass like the
    // forward pass of a pipeline of that many stages, tau_recomp = ceil((2(S - j) + 1) / N) for the j-th stage of a
    // segment of S, never above tau_fwd; the last segment's backward follows its forward at that very distance, so
    // nothing is recomputed there.  With T2 a stage whose recomputation is younger than its forward keeps a queue of
    // tau_recomp + 1 corrected versions (Appendix D) behind its version slots.
    s.tau_r = s.tau_f; s.rdepth = 0;
    if (S > 0) {
      const int seg_end = std::min(P, (p / S + 1) * S);
      const int nm = cfg->n_micro > 1 ? cfg->n_micro : 1;
      if (seg_end < P) s.tau_r = std::min(s.tau_f, (2 * (seg_end - 1 - p) + 1 + nm - 1) / nm);
      if (cfg->t2_enable && s.tau_r < s.tau_f) s.rdepth = s.tau_r + 1;
    }
    // materialize_backward: the same mechanism with delay 0: one slot holding w_v - (tau_fwd - 0) delta_v of the live version,
    // which is exactly the T2-corrected operand of the next backward pass
    if (mat && cfg->t2_enable && s.gap > 0) { s.tau_r = 0; s.rdepth = 1; }
    if (E > 1) {
      // a microbatch every E ticks: a stash written at tick mE + i is read at tick mE + i + tau, so floor(tau / E) + 1
      // microbatches are alive in a stage; the input ring keeps one more (it is also the forward mailbox) and another
      // when the previous stage takes its ReLU mask from it a tick after this stage's backward
      const int extra = s.xdepth - (s.tau_f + 1);
      s.depth = s.tau_f / E + 1; s.xdepth = s.depth + extra; s.vdepth = s.tau_f + 1;
    }
    s.begin = sd.param_offset; s.end = sd.param_offset + sd.param_count;
    prev_end = s.end;
    L.begin64[p] = (uint32_t)(s.begin / 64); L.end64[p] = (uint32_t)(s.end / 64);
    // ---- parse [pre] LINEAR+ [post]
    int idx = 0;
    s.pre = PRE_NONE; s.post = POST_NONE; s.n_lin = 0;
    auto offsets = [&](int op, uint64_t* a, uint64_t* b) { pm_op_param_offsets(sd.ops, sd.n_ops, op, a, b); *a += s.begin; *b += s.begin; };
    if (sd.ops[0].kind == PM_OP_EMBED) {
      const pm_op_desc& op = sd.ops[0];
      const bool second = (op.flags & PM_OPF_SECOND_STREAM) != 0;
      if ((p == 0) == second) { stage_err(p, "EMBED belongs to the first stage (first stream) or, with PM_OPF_SECOND_STREAM, to a later one"); return PM_ERR_UNSUPPORTED; }
      if (second && !L.st[p - 1].emit_memory) { stage_err(p, "a second-stream EMBED must follow the stage that emits the memory"); return PM_ERR_UNSUPPORTED; }
      if (L.pe_seq > 0 && (L.pe_seq != op.seq_len || L.pe_d != op.n_out)) { stage_err(p, "all EMBED ops share seq_len and width"); return PM_ERR_UNSUPPORTED; }
      s.ids_stream = second ? 1 : 0;
      s.ids_depth = mb ? 1 : (E > 1 ? (2 * P - p) / E + 2 : 2 * P - p);
      if (second) L.n_streams = 2;
      if (op.n_in < 1 || op.n_out < 4 || (op.n_out & 3) || op.seq_len < 1 || T % op.seq_len) { stage_err(p, "bad EMBED description (width a multiple of four, seq_len dividing the microbatch)"); return PM_ERR_INVALID_ARG; }
      s.pre = PRE_EMBED; s.vocab = op.n_in; s.seq_len = op.seq_len;
      uint64_t dummy; offsets(0, &s.tab_off, &dummy);
      L.pe_seq = op.seq_len; L.pe_d = op.n_out;
      idx = 1;
    } else if (sd.ops[0].kind == PM_OP_LAYERNORM) {
      if (sd.ops[0].n_in < 1 || sd.ops[0].n_in != sd.ops[0].n_out) { stage_err(p, "LAYERNORM needs n_in = n_out"); return PM_ERR_INVALID_ARG; }
      s.pre = PRE_LN;
      s.from_memory = (sd.ops[0].flags & PM_OPF_FROM_MEMORY) ? 1 : 0;
      offsets(0, &s.g_off, &s.beta_off);
      idx = 1;
    }
    const int pre_width = idx == 1 ? sd.ops[0].n_out : -1;
    s.max_dim = 0;
    int max_out = 0, max_in = 0;
    while (idx < sd.n_ops && sd.ops[idx].kind == PM_OP_LINEAR) {
      if (s.n_lin == PM_MAX_LINEARS) { stage_err(p, "too many Linear ops"); return PM_ERR_INVALID_ARG; }
      const pm_op_desc& op = sd.ops[idx];
      if (op.n_in < 1 || op.n_out < 1 || op.act < PM_ACT_NONE || op.act > PM_ACT_GELU) { stage_err(p, "bad Linear description"); return PM_ERR_INVALID_ARG; }
      if (cfg->compute_dtype == PM_BF16 && (op.n_in % 8 || op.n_out % 8)) { err = "PM_BF16 needs Linear dimensions that are multiples of 8"; return PM_ERR_SHAPE; }
      LinDev& ld = s.lin[s.n_lin];
      ld.n_in = op.n_in; ld.n_out = op.n_out; ld.act = op.act;
      offsets(idx, &ld.w_off, &ld.b_off);
      if (s.n_lin > 0 && op.n_in != s.lin[s.n_lin - 1].n_out) { stage_err(p, "Linear n_in does not match the previous n_out"); return PM_ERR_SHAPE; }
      max_out = std::max(max_out, op.n_out); max_in = std::max(max_in, op.n_in);
      ++s.n_lin; ++idx;
    }
    if (s.n_lin < 1) { stage_err(p, "a stage needs at least one LINEAR"); return PM_ERR_INVALID_ARG; }
    if (pre_width >= 0 && pre_width != s.lin[0].n_in) { stage_err(p, "pre-op width does not match the Linear's n_in"); return PM_ERR_SHAPE; }
    if (idx < sd.n_ops) {
      const pm_op_desc& op = sd.ops[idx];
      if (op.kind == PM_OP_ATTENTION) {
        const int n_out = s.lin[s.n_lin - 1].n_out;
        if (n_out % 3 || op.n_heads < 1 || (n_out / 3) % op.n_heads || op.seq_len < 1 || T % op.seq_len) { stage_err(p, "bad ATTENTION description"); return PM_ERR_INVALID_ARG; }
        if (op.seq_len > 128 && !attn_tc_supported(cfg->compute_dtype, op.seq_len, (n_out / 3) / op.n_heads)) { stage_err(p, "ATTENTION beyond 128 tokens is built for 256 tokens, bf16 and heads of width 64"); return PM_ERR_UNSUPPORTED; }
        s.post = POST_ATTENTION; s.n_heads = op.n_heads; s.seq_len = op.seq_len;
        s.causal = (op.flags & PM_OPF_CAUSAL) ? 1 : 0;
        s.skip_hop = 1;
      } else if (op.kind == PM_OP_CROSS_ATTENTION) {
        const int n_out = s.lin[s.n_lin - 1].n_out;
        if (n_out % 2 || op.n_heads < 1 || (n_out / 2) % op.n_heads || op.seq_len < 1 || T % op.seq_len) { stage_err(p, "bad CROSS_ATTENTION description"); return PM_ERR_INVALID_ARG; }
        if (op.seq_len > 128 && !attn_tc_supported(cfg->compute_dtype, op.seq_len, (n_out / 2) / op.n_heads)) { stage_err(p, "attention beyond 128 tokens is built for 256 tokens, bf16 and heads of width 64"); return PM_ERR_UNSUPPORTED; }
        if (!s.from_memory || n_out / 2 != s.lin[0].n_in) { stage_err(p, "CROSS_ATTENTION needs LAYERNORM | PM_OPF_FROM_MEMORY and a memory as wide as the queries"); return PM_ERR_UNSUPPORTED; }
        s.post = POST_CROSS_ATTENTION; s.n_heads = op.n_heads; s.seq_len = op.seq_len;
      } else if (op.kind == PM_OP_SKIP_OUT) { s.post = POST_SKIP_OUT; s.skip_hop = (op.flags & PM_OPF_SKIP_TWO) ? 2 : 1; }
      else if (op.kind == PM_OP_RESIDUAL) { s.post = POST_RESIDUAL; s.emit_memory = (op.flags & PM_OPF_EMIT_MEMORY) ? 1 : 0; }
      else { stage_err(p, "unexpected op after the Linear ops"); return PM_ERR_INVALID_ARG; }
      ++idx;
    }
    if (idx != sd.n_ops) { stage_err(p, "ops must follow [EMBED|LAYERNORM] LINEAR+ [ATTENTION|SKIP_OUT|RESIDUAL]"); return PM_ERR_INVALID_ARG; }
    if ((s.pre != PRE_NONE || s.post != POST_NONE) && s.n_lin != 1) { stage_err(p, "a stage with a pre- or post-op holds exactly one LINEAR"); return PM_ERR_UNSUPPORTED; }
    s.d_in = s.lin[0].n_in;
    const int n_out_last = s.lin[s.n_lin - 1].n_out;
    s.d_out_main = s.post == POST_ATTENTION ? n_out_last / 3 : (s.post == POST_CROSS_ATTENTION ? n_out_last / 2 : n_out_last);
    s.gin_depth = 3;
    if (s.from_memory && s.post != POST_CROSS_ATTENTION) { stage_err(p, "PM_OPF_FROM_MEMORY belongs to a stage ending in CROSS_ATTENTION"); return PM_ERR_UNSUPPORTED; }
    if (s.emit_memory) {
      if (L.mem_stage >= 0) { stage_err(p, "one stage emits the memory"); return PM_ERR_UNSUPPORTED; }
      L.mem_stage = p; L.mem_dim = n_out_last;
    }
    if (s.from_memory) {
      if (L.mem_stage < 0 || L.mem_dim != s.lin[0].n_in) { stage_err(p, "no memory of this width was emitted before this stage"); return PM_ERR_UNSUPPORTED; }
      L.last_mem_reader = p;
    }
    s.max_dim = std::max(std::max(max_in, max_out), s.d_in);
    // ---- chaining
    if (p > 0) {
      const StageDev& q = L.st[p - 1];
      const int main_in = s.post == POST_CROSS_ATTENTION ? s.d_out_main : s.d_in;        // width of the main input
      if (s.pre != PRE_EMBED && main_in != q.d_out_main) { stage_err(p, "input width does not match the previous stage's output"); return PM_ERR_SHAPE; }
      if (q.emit_memory && s.pre != PRE_EMBED) { stage_err(p, "the stage after the one that emits the memory starts with a second-stream EMBED"); return PM_ERR_UNSUPPORTED; }
      // skip tensors: an emitter hop positions back must exist for a RESIDUAL, and only then
      int src = -1;
      if (q.skip_hop == 1) src = p - 1;
      if (p >= 2 && L.st[p - 2].skip_hop == 2) { if (src >= 0 || q.post != POST_CROSS_ATTENTION) { stage_err(p, "a skip over two stages passes over a CROSS_ATTENTION stage only"); return PM_ERR_UNSUPPORTED; } src = p - 2; }
      if ((src >= 0) != (s.post == POST_RESIDUAL)) { stage_err(p, "RESIDUAL must follow the stage that sends it a skip tensor, and only then"); return PM_ERR_UNSUPPORTED; }
      if (s.post == POST_RESIDUAL) {
        if (L.st[src].d_in != n_out_last) { stage_err(p, "skip tensor width does not match the Linear's output"); return PM_ERR_SHAPE; }
        s.skip_depth = (p - src) + 1;
        s.gin_depth = (p - src) + 2;
      }
    } else if (s.post == POST_RESIDUAL) { stage_err(p, "the first stage has no skip tensor to add"); return PM_ERR_UNSUPPORTED; }
    if (p + s.skip_hop > P - 1 && s.skip_hop > 0) { stage_err(p, "a skip tensor needs its RESIDUAL stage"); return PM_ERR_UNSUPPORTED; }
    if (p == P - 1 && ce && (s.n_lin != 1 || s.post != POST_NONE || s.lin[0].act != PM_ACT_NONE)) { stage_err(p, "PM_LOSS_CE needs a last stage of one Linear without activation or post-op"); return PM_ERR_UNSUPPORTED; }
    // ---- what each Linear's forward writes
    for (int l = 0; l < s.n_lin; ++l) {
      LinDev& ld = s.lin[l];
      const bool last = l == s.n_lin - 1;
      const bool logits = last && p == P - 1 && ce;
      ld.flags = 0;
      const bool to_attention = last && (s.post == POST_ATTENTION || s.post == POST_CROSS_ATTENTION);   // q, k, v stash
      // a ReLU needs no stash of its own when its output is stashed anyway: between two Linears of a stage, or as
      // the main input of the next stage (not when a RESIDUAL adds to it first or the next stage embeds tokens)
      const bool next_takes_y = p + 1 < P && !(stages[p + 1].n_ops > 0 && stages[p + 1].ops[0].kind == PM_OP_EMBED) &&
                                (s.post == POST_NONE || s.post == POST_SKIP_OUT);
      if (ld.act == PM_ACT_RELU && (!last || next_takes_y)) ld.flags |= LF_ACT_FROM_Y;
      if ((ld.act != PM_ACT_NONE && !(ld.flags & LF_ACT_FROM_Y)) || to_attention) ld.flags |= LF_WRITE_Z;
      if (!to_attention && !logits) ld.flags |= LF_WRITE_Y;
      if (logits) ld.flags |= LF_OUT_F32;
      // The ReLU's backward can be applied by the next stage's dgrad epilogue when that stage takes y as its plain input
      // (tensor-core path).  Off unless PM_RELU_FUSE=1 is in the environment: the mask costs the dgrad epilogue, which is on
      // that kernel's critical path (single-buffered accumulators), more than the separate pass costs (measured: config 4
      // dgrad 0.215 -> 0.290 ms per tick against 0.014 ms saved in the activation-backward pass).
      const char* fuse_env = getenv("PM_RELU_FUSE");
      const bool fuse_ok = fuse_env && fuse_env[0] == '1';
      // (never with weight stashing, whose plain dgrad epilogue applies no mask: a stage with tau_bkwd = tau_fwd > 0)
      if (fuse_ok && cfg->compute_dtype == PM_BF16 && last && (ld.flags & LF_ACT_FROM_Y) && next_takes_y &&
          stages[p + 1].ops[0].kind == PM_OP_LINEAR && !(sd.tau_fwd > 0 && sd.tau_bkwd == sd.tau_fwd) &&
          !(stages[p + 1].tau_fwd > 0 && stages[p + 1].tau_bkwd == stages[p + 1].tau_fwd))
        ld.flags |= LF_DZ_FUSED;
    }
    if (p > 0 && (L.st[p - 1].lin[L.st[p - 1].n_lin - 1].flags & LF_DZ_FUSED)) s.mask_dx = 1;
    // ---- rings
    if (s.pre != PRE_EMBED) { s.x_ring = ring; ring = align_up(ring + (uint64_t)s.xdepth * T * s.d_in * esz, 256); }
    if (s.pre != PRE_NONE) { s.u_ring = ring; ring = align_up(ring + (uint64_t)s.depth * T * s.d_in * esz, 256); }
    if (s.pre == PRE_LN) { s.stat_ring = ring; ring = align_up(ring + (uint64_t)s.depth * T * 2 * 4, 256); }
    if (s.pre == PRE_EMBED) { s.ids_ring = ring; ring = align_up(ring + (uint64_t)s.ids_depth * T * 4, 256); }
    for (int l = 0; l < s.n_lin; ++l) {
      if (s.lin[l].flags & LF_WRITE_Z) { s.lin[l].z_ring = ring; ring = align_up(ring + (uint64_t)s.depth * T * s.lin[l].n_out * esz, 256); }
      if (l < s.n_lin - 1) { s.lin[l].h_ring = ring; ring = align_up(ring + (uint64_t)s.depth * T * s.lin[l].n_out * esz, 256); }
    }
    if (queue) {
      // queue of weight versions: the whole slice in the operand type, and (bf16 operands) the fp32 tensors the forward
      // pass reads -- LayerNorm gain and bias, Linear biases -- packed into slots of small_count floats
      s.v_ring = ring; ring = align_up(ring + (uint64_t)(s.vdepth + s.rdepth) * (s.end - s.begin) * esz, 256);
      uint32_t so = 0;
      auto seg = [&](uint64_t arena_off, uint64_t n, uint32_t* soff) {
        *soff = so;
        const uint32_t padded = (uint32_t)align_up(n, PM_ALIGN_ELEMS);
        for (uint32_t o = 0; o < padded; o += 2048) {                           // pieces of at most 2048 floats: one block copies a piece
          const uint32_t cnt = std::min<uint32_t>(2048, padded - o);
          L.segs.push_back(SmallSeg{arena_off + o, 0, cnt, 0, p, (int32_t)(so + o)});   // ring_off, slot_stride, rc_base filled below
        }
        so += padded;
      };
      if (esz == 2) {
        if (s.pre == PRE_LN) { seg(s.g_off, (uint64_t)s.d_in, &s.g_soff); seg(s.beta_off, (uint64_t)s.d_in, &s.beta_soff); }
        for (int l = 0; l < s.n_lin; ++l) seg(s.lin[l].b_off, (uint64_t)s.lin[l].n_out, &s.lin[l].b_soff);
        s.small_count = so;
        s.s_ring = ring; ring = align_up(ring + (uint64_t)(s.vdepth + s.rdepth) * so * 4, 256);
        for (auto& g : L.segs) if (g.stage == p) { g.ring_off = s.s_ring + 4ull * (uint32_t)g.rc_base; g.slot_stride = so; g.rc_base = s.rdepth > 0 ? s.vdepth : -1; }
      }
    }
    L.max_lin = std::max(L.max_lin, s.n_lin);
    L.max_dim = std::max(L.max_dim, s.max_dim);
    if (s.pre != PRE_NONE) L.any_pre = 1;
    if (s.pre == PRE_LN) L.any_ln = 1;
    if (s.pre == PRE_EMBED) { L.any_embed = 1; L.max_vocab = std::max(L.max_vocab, s.vocab); }
    if (s.post == POST_RESIDUAL) L.any_residual = 1;
    if (s.post == POST_ATTENTION || s.post == POST_CROSS_ATTENTION) {
      if (s.causal || s.post == POST_CROSS_ATTENTION) L.att_plain = false;
      const int dk = s.d_out_main / s.n_heads;
      L.att_S = std::max(L.att_S, s.seq_len); L.att_dk = std::max(L.att_dk, dk);
      L.att_blocks = std::max(L.att_blocks, (int)(T / s.seq_len) * s.n_heads);
    }
    L.sched[p].tau_f = s.tau_f; L.sched[p].gap = s.gap; L.sched[p].depth = s.depth; L.sched[p].xdepth = s.xdepth;
    L.sched[p].vdepth = s.vdepth; L.sched[p].begin = s.begin; L.sched[p].count = s.end - s.begin; L.sched[p].v_ring = s.v_ring;
    L.sched[p].tau_r = s.tau_r; L.sched[p].rdepth = s.rdepth;
  }
  // Weight stashing (Section 2.2, tau_bkwd = tau_fwd): the backward pass of a microbatch reads the queued version its forward
  // read, in the operand type (the copy the forward used), so dgrad is a plain GEMM and T2 has nothing to correct.
  L.stash = any_stash ? 1 : 0;
  if (L.stash && (S > 0 || stoch || cfg->fuse_update || mat)) {
    err = "weight stashing (tau_bkwd = tau_fwd) is not combined with recompute_segment, stochastic_tau_max, fuse_update or materialize_backward";
    return PM_ERR_UNSUPPORTED;
  }
  // Fused update (pm_config.fuse_update): the weight-gradient GEMM's epilogue updates the Linear matrices, the update
  // kernel the rest of every stage (biases, LayerNorm parameters, embedding tables, padding).
  L.fuse = 0;
  L.skip_b64.assign(P, 0); L.skip_e64.assign(P, 0);
  if (cfg->fuse_update) {
    const char* why = nullptr;
    if (cfg->compute_dtype != PM_BF16) why = "the tensor-core (PM_BF16) path";
    else if (L.max_lin != 1) why = "one Linear per stage";
    else if (cfg->n_micro > 1) why = "one microbatch per update (the gradients of a minibatch are summed in the grad arena)";
    else if (S > 0) why = "no recomputation (a segment's stashes are overwritten before the update phase)";
    else if (E > 1) why = "an entry period of one tick";
    if (why) { err = std::string("fuse_update is built for ") + why; return PM_ERR_UNSUPPORTED; }
    L.fuse = 1;
    for (int p = 0; p < P; ++p) {
      const LinDev& l0 = L.st[p].lin[0];
      L.skip_b64[p] = (uint32_t)(l0.w_off / 64);
      L.skip_e64[p] = (uint32_t)((l0.w_off + (uint64_t)l0.n_out * l0.n_in) / 64);     // dimensions are multiples of 8: whole groups
    }
  }
  for (int p = 0; p < P; ++p) {
    L.sched[p].next_xdepth = p + 1 < P ? L.st[p + 1].xdepth : 0;
    L.sched[p].gin_depth = L.st[p].gin_depth;
    L.sched[p].prev_gin_depth = p > 0 ? L.st[p - 1].gin_depth : 0;
    L.sched[p].skip_dst_depth = L.st[p].skip_hop > 0 ? L.st[p + L.st[p].skip_hop].skip_depth : 0;
    L.sched[p].skip_depth = L.st[p].skip_depth;
  }
  if (L.mem_stage >= 0) {
    if (L.last_mem_reader < 0) { err = "a memory is emitted but no CROSS_ATTENTION stage reads it"; return PM_ERR_UNSUPPORTED; }
    L.st[L.last_mem_reader].mem_first = 1;
    L.mem_depth = mb ? 1 : (E > 1 ? (2 * P - 2 * L.mem_stage) / E + 2 : 2 * P - 2 * L.mem_stage);
    L.gmem_depth = mb ? 1 : (E > 1 ? (P - L.mem_stage + 2) / E + 2 : P - L.mem_stage + 2);
    for (int p = 0; p < P; ++p) L.sched[p].gmem_depth = L.gmem_depth;
    L.mem_ring = ring; ring = align_up(ring + (uint64_t)L.mem_depth * T * L.mem_dim * esz, 256);
  }
  L.att_tc = L.att_blocks > 0;
  for (int p = 0; p < P; ++p)
    if (feeds_attention(L.st[p].post) && (L.st[p].seq_len != L.att_S || !attn_tc_supported(cfg->compute_dtype, L.st[p].seq_len, L.st[p].d_out_main / L.st[p].n_heads))) L.att_tc = false;
  if (L.att_blocks > 0 && !L.att_tc && attention_smem_bytes(L.att_S, L.att_dk, cfg->compute_dtype) > 227 * 1024) { err = "attention tile (seq_len x head width) does not fit in shared memory"; return PM_ERR_UNSUPPORTED; }
  L.total = L.st[P - 1].end;
  if (L.stochastic > 0) { L.g_ring = ring; ring = align_up(ring + (uint64_t)L.stochastic * L.total * 4, 256); }   // gradients of the last tau_max + 1 microbatches
  L.ring_bytes = ring;
  L.n_in_first = L.st[0].pre == PRE_EMBED ? 0 : L.st[0].lin[0].n_in;
  L.n_out_last = L.st[P - 1].lin[L.st[P - 1].n_lin - 1].n_out;
  L.loss_cap = cfg->loss_log_capacity > 0 ? cfg->loss_log_capacity : 4096;
  // workspace
  uint64_t w = 0;
  L.off_st = w; w = align_up(w + sizeof(StageDev) * P, 256);
  L.off_sched = w; w = align_up(w + sizeof(StageSched) * P, 256);
  L.off_dyn = w; w = align_up(w + sizeof(StageDyn) * P * (uint64_t)L.n_tables, 256);
  L.off_nupd = w; w = align_up(w + sizeof(int64_t) * P, 256);
  L.off_b64 = w; w = align_up(w + sizeof(uint32_t) * P, 256);
  L.off_e64 = w; w = align_up(w + sizeof(uint32_t) * P, 256);
  L.off_delays = w; w = align_up(w + sizeof(int32_t) * P, 256);
  L.off_skb = w; w = align_up(w + sizeof(uint32_t) * P, 256);
  L.off_ske = w; w = align_up(w + sizeof(uint32_t) * P, 256);
  L.off_alpha = w; w = align_up(w + sizeof(double) * (cfg->alpha_by_step ? (uint64_t)cfg->alpha_len : 0), 256);
  L.off_loss = w; w = align_up(w + sizeof(float) * (uint64_t)L.loss_cap, 256);
  L.off_lossred = w; w = align_up(w + 512, 256);
  L.off_rowloss = w; w = align_up(w + (ce ? T * 4 : 0), 256);
  // short microbatches: more, smaller blocks (the reductions are latency-bound); so do the one-stage launches of
  // microbatch-major order, whose grids cover a single stage
  L.chunk_rows = T > 512 ? (mb ? 64 : 256) : 32;
  L.row_chunks = (int32_t)((T + L.chunk_rows - 1) / L.chunk_rows);
  L.off_colred = w; w = align_up(w + (L.row_chunks > 1 ? (uint64_t)P * L.row_chunks * 2 * L.max_dim * 4 : 0), 256);
  L.off_pe = w; w = align_up(w + (uint64_t)L.pe_seq * L.pe_d * 4, 256);
  L.ids.assign((size_t)4 * P, 0);
  L.pre_idx.assign(P, -1); L.ln_idx.assign(P, -1); L.embed_idx.assign(P, -1); L.res_idx.assign(P, -1);
  for (int p = 0; p < P; ++p) {
    const StageDev& s = L.st[p];
    if (s.pre != PRE_NONE) { L.pre_idx[p] = L.n_pre; L.ids[(size_t)0 * P + L.n_pre++] = p; }
    if (s.pre == PRE_LN) {
      L.ln_idx[p] = L.n_ln;
      L.ids[(size_t)1 * P + L.n_ln++] = p; L.max_ln_dim = std::max(L.max_ln_dim, s.d_in);
      if ((s.d_in & 7) != 0 || s.d_in > 1024) L.ln_fused = 0;
    }
    if (s.pre == PRE_EMBED) { L.embed_idx[p] = L.n_embed; L.ids[(size_t)2 * P + L.n_embed++] = p; }
    if (s.post == POST_RESIDUAL) { L.res_idx[p] = L.n_res; L.ids[(size_t)3 * P + L.n_res++] = p; }
  }
  for (int l = 0; l < PM_MAX_LINEARS; ++l) {
    int32_t acc = 0;
    for (int p = 0; p < P; ++p) {
      L.ids.push_back(acc);
      if (l < L.st[p].n_lin) acc += (L.st[p].lin[l].n_out + 255) / 256;
    }
    L.ids.push_back(acc);
    L.act_blocks[l] = acc;
  }
  L.off_ids = w; w = align_up(w + sizeof(int32_t) * L.ids.size(), 256);
  L.off_segs = w; w = align_up(w + sizeof(SmallSeg) * L.segs.size(), 256);
  if (L.mem_stage >= 0 && !L.ln_fused) { err = "stages that read the memory need LayerNorm widths that are multiples of 8 and at most 1024"; return PM_ERR_UNSUPPORTED; }
  L.ln_chunk_rows = mb ? 16 : 64;
  L.ln_chunks = (int32_t)((T + L.ln_chunk_rows - 1) / L.ln_chunk_rows);
  L.off_lnred = w; w = align_up(w + (uint64_t)L.n_ln * L.ln_chunks * 2 * L.max_ln_dim * 4, 256);
  L.off_tgt = w; w = align_up(w + (uint64_t)(P + 1) * T * (ce ? 4 : (uint64_t)L.n_out_last * 4), 256);
  L.off_yout = w; w = align_up(w + 2 * T * L.n_out_last * (ce ? 4 : esz), 256);
  L.off_umma = w; w = align_up(w + (cfg->compute_dtype == PM_BF16 ? umma_workspace_bytes((int)T, L.st, 0) : 0), 256);
  L.off_attn = w; w = align_up(w + (L.att_tc ? attn_workspace_bytes(P) : 0), 256);
  L.off_gmem = w; w = align_up(w + (uint64_t)L.gmem_depth * T * L.mem_dim * esz, 256);
  for (int p = 0; p < P; ++p) {
    StageDev& s = L.st[p];
    const uint64_t n_out_last = s.lin[s.n_lin - 1].n_out;
    uint64_t mo = 0, mi = 0;
    for (int l = 0; l < s.n_lin; ++l) { mo = std::max<uint64_t>(mo, s.lin[l].n_out); mi = std::max<uint64_t>(mi, s.lin[l].n_in); }
    s.gin = w; w = align_up(w + (uint64_t)s.gin_depth * T * s.d_out_main * esz, 256);
    if (s.post == POST_RESIDUAL) {
      s.skip_in = w; w = align_up(w + (uint64_t)s.skip_depth * T * n_out_last * esz, 256);
      s.ytmp = w; w = align_up(w + T * n_out_last * esz, 256);
    }
    if (s.post == POST_ATTENTION || s.post == POST_CROSS_ATTENTION) { s.dy = w; w = align_up(w + T * n_out_last * esz, 256); }
    s.dz = w; w = align_up(w + T * mo * esz, 256);
    s.dh = w; w = align_up(w + T * mi * esz, 256);
  }
  L.ws_bytes = w;
  return PM_OK;
}

}  // namespace

struct pm_ctx {
  pm_config cfg;
  Layout L;
  TickArgs ta;
  HyperDev hp;
  ArenasDev a;
  cudaStream_t stream;
  char* ws;
  int64_t tick = 0, n_fed = 0;
  int phase = 0;           // 0: expects forward, 1: expects backward, 2: expects update
  bool draining = false;
  std::string err;
  UmmaPlan* umma = nullptr;
  AttnPlan* attn = nullptr;
  uint64_t launches = 0;
  // The kernel sequence of a phase is the same in every steady-state tick (what differs sits in the device-side
  // schedule table), so each phase is captured once into a CUDA graph and replayed: one launch instead of up to a
  // dozen.  Captured on a private stream (the caller's may be the legacy default stream, which cannot capture),
  // replayed on the caller's.  PM_CUDA_GRAPHS=0 in the environment, profiling, or a failed capture keep the
  // phase on plain launches.
  struct PhaseGraph { cudaGraphExec_t exec = nullptr; int eager_runs = 0; uint64_t launches = 0; bool failed = false; };
  PhaseGraph g_fwd, g_bwd, g_upd;
  // Tick-major order with an entry period E > 1 ("sparse ticks"): a tick's launches cover only the stages whose turn it
  // is (those at distance = tick mod E from a microbatch's entry), one graph per phase and residue; the forward stages
  // run on a stream of their own, next to the backward and update of the same tick (see sparse_forward).
  std::vector<PhaseGraph> gs_fwd, gs_bwd, gs_upd;
  cudaStream_t fwd_stream = nullptr;
  cudaEvent_t ev_sched = nullptr, ev_fwd = nullptr;
  bool fwd_pending = false;             // work of the last tick's forward may still be running on fwd_stream
  std::vector<int> seg_first, seg_count;   // small-tensor segments of a stage: [seg_first[p], + seg_count[p])
  std::vector<int32_t> h_delays;           // stochastic delay model: host copy of the delays in force
  bool graphs = true;
  cudaStream_t cap_stream = nullptr;
  cudaStream_t ls = nullptr;            // the stream the phase bodies launch on: `stream`, or `cap_stream` while capturing
  ~pm_ctx() {
    for (PhaseGraph* g : {&g_fwd, &g_bwd, &g_upd}) if (g->exec) cudaGraphExecDestroy(g->exec);
    for (auto* v : {&gs_fwd, &gs_bwd, &gs_upd}) for (auto& g : *v) if (g.exec) cudaGraphExecDestroy(g.exec);
    if (fwd_stream) cudaStreamDestroy(fwd_stream);
    if (ev_sched) cudaEventDestroy(ev_sched);
    if (ev_fwd) cudaEventDestroy(ev_fwd);
    if (cap_stream) cudaStreamDestroy(cap_stream);
  }
  // optional per-kernel-class timing with CUDA events on the context's stream
  bool prof_on = false;
  int prof_cls = 0;
  std::vector<cudaEvent_t> prof_ev;          // pairs: start, stop
  std::vector<int> prof_pair_cls;
  size_t prof_used = 0;   // kernels enqueued by this context so far
};

namespace {
pm_status fail(pm_ctx* ctx, pm_status s, const std::string& msg) {
  if (ctx) ctx->err = msg;
  g_error = msg;
  return s;
}
pm_status cuda_fail(pm_ctx* ctx, cudaError_t e, const char* what) {
  return fail(ctx, PM_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}
}  // namespace

extern "C" {

const char* pm_status_string(pm_status s) {
  switch (s) {
    case PM_OK: return "PM_OK";
    case PM_ERR_INVALID_ARG: return "PM_ERR_INVALID_ARG";
    case PM_ERR_SHAPE: return "PM_ERR_SHAPE";
    case PM_ERR_STATE: return "PM_ERR_STATE";
    case PM_ERR_NOMEM: return "PM_ERR_NOMEM";
    case PM_ERR_UNSUPPORTED: return "PM_ERR_UNSUPPORTED";
    case PM_ERR_CUDA: return "PM_ERR_CUDA";
    case PM_ERR_TIMEOUT: return "PM_ERR_TIMEOUT";
  }
  return "PM_ERR_?";
}

pm_status pm_stage_param_count(const pm_op_desc* ops, int32_t n_ops, uint64_t* count) {
  if (!ops || !count || n_ops < 1) return PM_ERR_INVALID_ARG;
  uint64_t c = 0;
  for (int l = 0; l < n_ops; ++l) {
    if (ops[l].kind < PM_OP_LINEAR || ops[l].kind > PM_OP_CROSS_ATTENTION) return PM_ERR_INVALID_ARG;
    if (ops[l].kind <= PM_OP_LAYERNORM && (ops[l].n_in < 1 || ops[l].n_out < 1)) return PM_ERR_INVALID_ARG;
    uint64_t n0, n1;
    const int k = op_params(ops[l], &n0, &n1);
    if (k >= 1) c = align_up(c + n0, PM_ALIGN_ELEMS);
    if (k >= 2) c = align_up(c + n1, PM_ALIGN_ELEMS);
  }
  *count = c;
  return PM_OK;
}

pm_status pm_op_param_offsets(const pm_op_desc* ops, int32_t n_ops, int32_t op, uint64_t* w_off, uint64_t* b_off) {
  if (!ops || op < 0 || op >= n_ops) return PM_ERR_INVALID_ARG;
  uint64_t c = 0;
  for (int l = 0; l <= op; ++l) {
    uint64_t n0, n1;
    const int k = op_params(ops[l], &n0, &n1);
    const uint64_t o0 = c;
    if (k >= 1) c = align_up(c + n0, PM_ALIGN_ELEMS);
    const uint64_t o1 = c;
    if (k >= 2) c = align_up(c + n1, PM_ALIGN_ELEMS);
    if (l == op) {
      if (k == 0) return PM_ERR_INVALID_ARG;
      if (w_off) *w_off = o0;
      if (b_off) *b_off = o1;
    }
  }
  return PM_OK;
}

pm_status pm_query_bytes(const pm_config* cfg, const pm_stage_desc* stages, uint64_t* state_bytes,
                         uint64_t* ring_bytes, uint64_t* workspace_bytes) {
  Layout L;
  std::string err;
  pm_status s = build_layout(cfg, stages, L, err);
  if (s != PM_OK) return fail(nullptr, s, err);
  // fp32 copies: w, m, delta, grad (+ s for Adam); plus the bf16 copy of w for PM_BF16
  uint64_t copies = cfg->optimizer == PM_ADAM ? 5 : 4;
  if (state_bytes) *state_bytes = L.total * 4 * copies + (cfg->compute_dtype == PM_BF16 ? L.total * 2 : 0);
  if (ring_bytes) *ring_bytes = L.ring_bytes;
  if (workspace_bytes) *workspace_bytes = L.ws_bytes;
  return PM_OK;
}

pm_status pm_init_stages(pm_ctx** out, const pm_config* cfg, const pm_stage_desc* stages, const pm_arenas* arenas,
                         void* ring, uint64_t ring_bytes, void* workspace, uint64_t workspace_bytes, void* stream) {
  if (!out) return fail(nullptr, PM_ERR_INVALID_ARG, "null output pointer");
  *out = nullptr;
  if (!arenas) return fail(nullptr, PM_ERR_INVALID_ARG, "null arenas");
  Layout L;
  std::string err;
  pm_status s = build_layout(cfg, stages, L, err);
  if (s != PM_OK) return fail(nullptr, s, err);
  if (!arenas->w || !arenas->m || !arenas->delta || !arenas->grad) return fail(nullptr, PM_ERR_INVALID_ARG, "w, m, delta and grad arenas are required");
  if (cfg->optimizer == PM_ADAM && !arenas->s) return fail(nullptr, PM_ERR_INVALID_ARG, "Adam needs the s arena");
  if (cfg->compute_dtype == PM_BF16 && !arenas->w_lp) return fail(nullptr, PM_ERR_INVALID_ARG, "PM_BF16 needs the w_lp arena");
  if (arenas->count < L.total) return fail(nullptr, PM_ERR_NOMEM, "arenas hold " + std::to_string(arenas->count) + " elements, stages need " + std::to_string(L.total));
  if (ring_bytes < L.ring_bytes || (!ring && L.ring_bytes)) return fail(nullptr, PM_ERR_NOMEM, "ring buffer too small: need " + std::to_string(L.ring_bytes) + " bytes");
  if (workspace_bytes < L.ws_bytes || !workspace) return fail(nullptr, PM_ERR_NOMEM, "workspace too small: need " + std::to_string(L.ws_bytes) + " bytes");
  if (((uintptr_t)ring | (uintptr_t)workspace | (uintptr_t)arenas->w | (uintptr_t)arenas->m | (uintptr_t)arenas->delta |
       (uintptr_t)arenas->grad | (uintptr_t)arenas->s | (uintptr_t)arenas->w_lp) & 255)
    return fail(nullptr, PM_ERR_INVALID_ARG, "device buffers must be 256-byte aligned");

  pm_ctx* c = new pm_ctx();
  c->cfg = *cfg;
  c->cfg.alpha_by_step = nullptr;
  c->L = L;
  c->stream = (cudaStream_t)stream;
  c->ls = c->stream;
  { const char* v = getenv("PM_CUDA_GRAPHS"); c->graphs = !(v && v[0] == '0'); }
  if (c->graphs && cudaStreamCreateWithFlags(&c->cap_stream, cudaStreamNonBlocking) != cudaSuccess) { cudaGetLastError(); c->cap_stream = nullptr; }
  c->ws = (char*)workspace;
  const int P = cfg->n_stages;
  c->a = ArenasDev{arenas->w, arenas->m, arenas->s, arenas->delta, arenas->grad, (__nv_bfloat16*)arenas->w_lp, arenas->count};
  cudaError_t e;
#define UP(off, vec) \
  if ((e = cudaMemcpyAsync(c->ws + (off), (vec).data(), sizeof((vec)[0]) * (vec).size(), cudaMemcpyHostToDevice, c->stream)) != cudaSuccess) { \
    pm_status r = cuda_fail(nullptr, e, "table upload"); delete c; return r; }
  UP(L.off_st, c->L.st);
  UP(L.off_sched, c->L.sched);
  UP(L.off_b64, c->L.begin64);
  UP(L.off_e64, c->L.end64);
  UP(L.off_skb, c->L.skip_b64);
  UP(L.off_ske, c->L.skip_e64);
  UP(L.off_ids, c->L.ids);
  if (!c->L.segs.empty()) { UP(L.off_segs, c->L.segs); }
#undef UP
  if (cfg->alpha_by_step) {
    if (cfg->alpha_len < 1) { delete c; return fail(nullptr, PM_ERR_INVALID_ARG, "alpha_len must be >= 1 with alpha_by_step"); }
    e = cudaMemcpyAsync(c->ws + L.off_alpha, cfg->alpha_by_step, sizeof(double) * cfg->alpha_len, cudaMemcpyHostToDevice, c->stream);
    if (e != cudaSuccess) { pm_status r = cuda_fail(nullptr, e, "alpha table upload"); delete c; return r; }
  }
  e = cudaMemsetAsync(c->ws + L.off_nupd, 0, sizeof(int64_t) * P, c->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(c->ws + L.off_dyn, 0, sizeof(StageDyn) * P * (uint64_t)L.n_tables, c->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(c->ws + L.off_delays, 0, sizeof(int32_t) * P, c->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(c->ws + L.off_lossred, 0, 512, c->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);   // host tables may go out of scope after this
  if (e != cudaSuccess) { pm_status r = cuda_fail(nullptr, e, "context set-up"); delete c; return r; }

  c->hp = HyperDev{};
  c->hp.optimizer = cfg->optimizer; c->hp.t1 = cfg->t1_enable; c->hp.t2 = cfg->t2_enable; c->hp.n_stages = P;
  c->hp.K = cfg->t1_K > 0 ? cfg->t1_K : 1; c->hp.D = cfg->t2_D; c->hp.alpha_const = cfg->alpha_const;
  c->hp.alpha_tab = cfg->alpha_by_step ? (const double*)(c->ws + L.off_alpha) : nullptr;
  c->hp.alpha_len = cfg->alpha_len;
  c->hp.beta1 = cfg->beta1; c->hp.beta2 = cfg->beta2; c->hp.eps = cfg->eps;
  c->hp.warm = 0; c->hp.period = 2 * (int64_t)cfg->n_stages;
  c->hp.entry_period = L.E;
  c->hp.mb_major = L.queue ? 1 : 0; c->hp.lp_elem = cfg->compute_dtype == PM_F32 ? 4 : 2;
  c->hp.n_micro = cfg->n_micro > 1 ? cfg->n_micro : 1;
  c->hp.segment = L.segment;
  c->hp.stochastic = L.stochastic; c->hp.total = L.total;
  c->hp.materialize = L.materialize;

  TickArgs& t = c->ta;
  t.st = (const StageDev*)(c->ws + L.off_st);
  t.dyn = (const StageDyn*)(c->ws + L.off_dyn);
  t.a = c->a; t.ring = (char*)ring; t.ws = c->ws; t.T = cfg->microbatch; t.P = P;
  t.n_in_first = L.n_in_first; t.n_out_last = L.n_out_last;
  t.yout_off = L.off_yout; t.tgt_off = L.off_tgt; t.loss_off = L.off_loss; t.loss_cap = L.loss_cap; t.lossred_off = L.off_lossred;
  t.max_lin = L.max_lin; t.max_dim = L.max_dim;
  t.mb_major = L.queue ? 1 : 0; t.sel_p = -1; t.sel_tile0 = 0;
  t.res_fused = cfg->compute_dtype == PM_BF16 ? 1 : 0;
  t.ln_li0 = 0; t.defer_finish = 0; t.colsum_only = 0; t.ln_stage = 0; t.fin_deferred = 0;
  t.dgrad_split_below = 0;
  t.loss_scale = 1.0f / (float)(cfg->n_micro > 1 ? cfg->n_micro : 1);
  t.stash = (L.stash || L.materialize) ? 1 : 0;     // the backward pass reads its table entry's version slot
  t.fuse_upd = 0; t.upd_opt = cfg->optimizer; t.upd_beta1 = cfg->beta1; t.upd_beta2 = cfg->beta2; t.upd_eps = cfg->eps;
  t.upd_lp = L.queue ? reinterpret_cast<__nv_bfloat16*>(t.ring) : c->a.w_lp;
  for (int l = 0; l < PM_MAX_LINEARS; ++l) t.act_first[l] = 0;
  t.pe_off = L.off_pe; t.rowloss_off = L.off_rowloss; t.loss_kind = cfg->loss;
  t.colred_off = L.off_colred; t.row_chunks = L.row_chunks; t.chunk_rows = L.chunk_rows;
  t.any_pre = L.any_pre; t.any_ln = L.any_ln; t.any_embed = L.any_embed; t.any_residual = L.any_residual;
  t.att_S = L.att_S; t.att_dk = L.att_dk; t.att_blocks = L.att_blocks; t.max_vocab = L.max_vocab; t.max_embed_dim = L.pe_d;
  {
    const int32_t* ids = (const int32_t*)(c->ws + L.off_ids);
    t.pre_ids = ids; t.ln_ids = ids + P; t.embed_ids = ids + 2 * P; t.res_ids = ids + 3 * P;
    t.n_pre = L.n_pre; t.n_ln = L.n_ln; t.n_embed = L.n_embed; t.n_res = L.n_res;
    t.lnred_off = L.off_lnred; t.ln_chunks = L.ln_chunks; t.ln_chunk_rows = L.ln_chunk_rows; t.max_ln_dim = L.max_ln_dim;
    t.ln_fused = L.ln_fused;
    t.act_start = ids + 4 * P;
    t.mem_ring = L.mem_ring; t.gmem_off = L.off_gmem; t.mem_depth = L.mem_depth; t.gmem_depth = L.gmem_depth;
    t.mem_dim = L.mem_dim; t.n_streams = L.n_streams;
    t.second_embed_stage = 0;
    for (int p = 0; p < P; ++p) if (L.st[p].pre == PRE_EMBED && L.st[p].ids_stream == 1) t.second_embed_stage = p;
    for (int l = 0; l < PM_MAX_LINEARS; ++l) t.act_blocks[l] = L.act_blocks[l];
  }
  if (L.pe_seq > 0) {
    // sinusoidal positions: PE[pos, 2i] = sin(pos / 10000^(2i/d)), PE[pos, 2i+1] = cos(same); double, rounded once to float
    std::vector<float> pe((size_t)L.pe_seq * L.pe_d);
    for (int pos = 0; pos < L.pe_seq; ++pos)
      for (int i = 0; i < L.pe_d / 2; ++i) {
        const double ang = (double)pos / std::pow(10000.0, 2.0 * i / (double)L.pe_d);
        pe[(size_t)pos * L.pe_d + 2 * i] = (float)std::sin(ang);
        pe[(size_t)pos * L.pe_d + 2 * i + 1] = (float)std::cos(ang);
      }
    e = cudaMemcpyAsync(c->ws + L.off_pe, pe.data(), pe.size() * sizeof(float), cudaMemcpyHostToDevice, c->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
    if (e != cudaSuccess) { pm_status r = cuda_fail(nullptr, e, "position table upload"); delete c; return r; }
  }
  if (L.att_tc) {
    std::string aerr;
    pm_status as = attn_plan_create(&c->attn, t, c->L.st, c->ws + L.off_attn, c->stream, aerr);
    if (as != PM_OK) { delete c; return fail(nullptr, as, aerr); }
  } else if (L.att_blocks > 0) {
    e = attention_set_smem_limits(L.att_S, L.att_dk, cfg->compute_dtype);
    if (e != cudaSuccess) { pm_status r = cuda_fail(nullptr, e, "attention shared-memory limit"); delete c; return r; }
  }

  if (cfg->compute_dtype == PM_BF16) {
    std::string uerr;
    pm_status us = umma_plan_create(&c->umma, t, c->L.st, c->ws + L.off_umma, c->stream, uerr);
    if (us != PM_OK) { delete c; return fail(nullptr, us, uerr); }
  }
  if (L.E > 1) {
    const char* v = getenv("PM_SPARSE_TICKS");           // PM_SPARSE_TICKS=0: every tick launches grids over all stages (for comparisons)
    if (!(v && v[0] == '0')) {
      c->gs_fwd.assign((size_t)L.E, pm_ctx::PhaseGraph{}); c->gs_bwd.assign((size_t)L.E, pm_ctx::PhaseGraph{}); c->gs_upd.assign((size_t)L.E, pm_ctx::PhaseGraph{});
      const char* v2 = getenv("PM_FWD_STREAM");          // PM_FWD_STREAM=0: forward and backward of a tick on one stream
      if (!(v2 && v2[0] == '0')) {
        if (cudaStreamCreateWithFlags(&c->fwd_stream, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->ev_sched, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->ev_fwd, cudaEventDisableTiming) != cudaSuccess) { cudaGetLastError(); c->fwd_stream = nullptr; }
      }
    }
    c->seg_first.assign(P, 0); c->seg_count.assign(P, 0);
    for (size_t k = 0; k < c->L.segs.size(); ++k) {
      const int p = c->L.segs[k].stage;
      if (c->seg_count[p] == 0) c->seg_first[p] = (int)k;
      c->seg_count[p] += 1;
    }
  }
  if (L.queue) {
    // version 0 of every stage's queue: the initial weights in the operand type, and the small fp32 tensors
    const bool f32 = cfg->compute_dtype == PM_F32;
    for (int p = 0; p < P && e == cudaSuccess; ++p) {
      const StageDev& s = c->L.st[p];
      const void* src = f32 ? (const void*)(arenas->w + s.begin) : (const void*)(arenas->w_lp + s.begin);
      const uint64_t bytes = (s.end - s.begin) * (f32 ? 4 : 2);
      e = cudaMemcpyAsync(t.ring + s.v_ring, src, bytes, cudaMemcpyDeviceToDevice, c->stream);
      // corrected recompute weights of version 0: delta_0 = 0, so the initial weights themselves
      if (e == cudaSuccess && s.rdepth > 0) e = cudaMemcpyAsync(t.ring + s.v_ring + (uint64_t)s.vdepth * bytes, src, bytes, cudaMemcpyDeviceToDevice, c->stream);
    }
    if (e == cudaSuccess) e = launch_push_small(c->a.w, c->a.delta, t.ring, (const SmallSeg*)(c->ws + L.off_segs), (int)c->L.segs.size(), t.dyn, 0, c->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
    if (e != cudaSuccess) { pm_status r = cuda_fail(nullptr, e, "weight-version queue set-up"); pm_destroy(c); return r; }
  }
  *out = c;
  return PM_OK;
}

// every call checked here enqueued `kernels` kernels
static pm_status check(pm_ctx* ctx, cudaError_t e, const char* what, int kernels = 1) {
  ctx->launches += kernels;
  if (ctx->prof_on && ctx->prof_cls >= 0 && ctx->prof_used < ctx->prof_pair_cls.size()) {
    cudaEventRecord(ctx->prof_ev[2 * ctx->prof_used + 1], ctx->stream);
    ctx->prof_pair_cls[ctx->prof_used] = ctx->prof_cls;
    ctx->prof_used += 1;
    ctx->prof_cls = -1;
  }
  return e == cudaSuccess ? PM_OK : cuda_fail(ctx, e, what);
}
// marks the start of a timed launch of class `cls`; the matching stop is recorded by check()
static inline void prof_begin(pm_ctx* ctx, int cls) {
  if (!ctx->prof_on || ctx->prof_used >= ctx->prof_pair_cls.size()) { ctx->prof_cls = -1; return; }
  ctx->prof_cls = cls;
  cudaEventRecord(ctx->prof_ev[2 * ctx->prof_used], ctx->stream);
}
#define TIMED(cls, call) (prof_begin(ctx, cls), call)

// Runs the kernel launches of one phase (`body` launches on ctx->ls): plainly the first times and whenever graphs
// are off, then once under stream capture to build the phase's graph, then by replaying that graph.
static pm_status run_phase(pm_ctx* ctx, pm_ctx::PhaseGraph& g, const std::function<pm_status()>& body, cudaStream_t run_on = nullptr) {
  if (!run_on) run_on = ctx->stream;
  ctx->ls = run_on;
  if (!ctx->graphs || ctx->prof_on || g.failed || !ctx->cap_stream) return body();
  if (g.exec) {
    ctx->launches += g.launches;
    cudaError_t e = cudaGraphLaunch(g.exec, run_on);
    return e == cudaSuccess ? PM_OK : cuda_fail(ctx, e, "graph launch");
  }
  if (g.eager_runs < 2) { ++g.eager_runs; return body(); }      // modules loaded, function attributes set
  const uint64_t l0 = ctx->launches;
  if (cudaStreamBeginCapture(ctx->cap_stream, cudaStreamCaptureModeRelaxed) != cudaSuccess) { cudaGetLastError(); g.failed = true; return body(); }
  ctx->ls = ctx->cap_stream;
  const pm_status sb = body();
  ctx->ls = run_on;
  cudaGraph_t graph = nullptr;
  cudaError_t e = cudaStreamEndCapture(ctx->cap_stream, &graph);
  if (sb == PM_OK && e == cudaSuccess && graph) {
    g.launches = ctx->launches - l0;
    e = cudaGraphInstantiate(&g.exec, graph, 0);
  } else if (e == cudaSuccess) e = cudaErrorUnknown;
  if (graph) cudaGraphDestroy(graph);
  if (e != cudaSuccess) {                                        // nothing has run yet: do the phase with plain launches
    cudaGetLastError();
    g.failed = true; g.exec = nullptr;
    ctx->launches = l0;
    return body();
  }
  e = cudaGraphLaunch(g.exec, run_on);
  return e == cudaSuccess ? PM_OK : cuda_fail(ctx, e, "graph launch");
}

// is a microbatch in flight at any of the stages whose distance from the entry tick lies in [lo, hi]?
static bool any_stage_active(const pm_ctx* ctx, int64_t lo, int64_t hi) {
  if (ctx->hp.warm == 0 && ctx->hp.entry_period <= 1) return ctx->tick - lo >= 0 && ctx->tick - hi < ctx->n_fed;
  for (int64_t off = lo; off <= hi; ++off) {
    const int64_t m = mb_at_tick(ctx->tick - off, ctx->hp.warm, ctx->hp.period, ctx->hp.entry_period);
    if (m >= 0 && m < ctx->n_fed) return true;
  }
  return false;
}

pm_status pm_set_warmup(pm_ctx* ctx, int64_t n_microbatches) {
  if (!ctx || n_microbatches < 0) return fail(ctx, PM_ERR_INVALID_ARG, "bad argument");
  if (ctx->tick != 0 || ctx->phase != 0) return fail(ctx, PM_ERR_STATE, "the warm-up length is set before the first tick");
  if (ctx->hp.entry_period > 1 && n_microbatches > 0) return fail(ctx, PM_ERR_UNSUPPORTED, "warm-up epochs are not combined with an entry period");
  if (ctx->hp.n_micro > 1 && n_microbatches > 0) return fail(ctx, PM_ERR_UNSUPPORTED, "warm-up epochs are built for one microbatch per update");
  ctx->hp.warm = n_microbatches;
  return PM_OK;
}


// ---- microbatch-major order -------------------------------------------------------------------------------------
// One microbatch at a time: stages 1..P forward (stage i reads weight version max(0, t - tau_fwd,i) from its queue),
// the loss, stages P..1 backward against the live weights, the weight gradients, then the update of every stage,
// which also writes version t + 1 into the queues.  The kernels are those of the tick schedule: sub-tick v of
// microbatch t is virtual tick 2P t + v with exactly one stage in forward (v = i) or backward (v = 2P - 1 - i), so
// mailboxes and skip buffers are addressed as in a pipeline tick; each launch is restricted to its stage.

// Launch arguments of sub-tick table `v`, restricted to stage p (p < 0: all stages).
static TickArgs mb_args(const pm_ctx* ctx, int v, int p) {
  TickArgs t = ctx->ta;
  const Layout& L = ctx->L;
  const int P = ctx->cfg.n_stages;
  t.dyn = (const StageDyn*)(ctx->ws + L.off_dyn) + (size_t)v * P;
  if (p < 0) return t;
  const StageDev& s = L.st[p];
  const int32_t* ids = (const int32_t*)(ctx->ws + L.off_ids);
  t.sel_p = p;
  t.n_pre = L.pre_idx[p] >= 0 ? 1 : 0;      t.pre_ids = ids + (L.pre_idx[p] >= 0 ? L.pre_idx[p] : 0);
  t.n_ln = L.ln_idx[p] >= 0 ? 1 : 0;        t.ln_li0 = L.ln_idx[p] >= 0 ? L.ln_idx[p] : 0;      // the list itself stays whole: partial sums are kept per entry
  t.n_embed = L.embed_idx[p] >= 0 ? 1 : 0;  t.embed_ids = ids + 2 * P + (L.embed_idx[p] >= 0 ? L.embed_idx[p] : 0);
  t.n_res = L.res_idx[p] >= 0 ? 1 : 0;      t.res_ids = ids + 3 * P + (L.res_idx[p] >= 0 ? L.res_idx[p] : 0);
  t.any_pre = t.n_pre; t.any_ln = t.n_ln; t.any_embed = t.n_embed; t.any_residual = t.n_res;
  if (!feeds_attention(s.post)) t.att_blocks = 0;
  for (int l = 0; l < PM_MAX_LINEARS; ++l) {
    const int32_t* start = L.ids.data() + (size_t)4 * P + (size_t)l * (P + 1);
    t.act_first[l] = start[p];
    t.act_blocks[l] = start[p + 1] - start[p];
  }
  return t;
}

// The launches of ONE stage's forward pass (ta restricted to it).
static pm_status stage_forward(pm_ctx* ctx, const TickArgs& ta, int p) {
  const int dt = ctx->cfg.compute_dtype;
  const StageDev& sd = ctx->L.st[p];
  pm_status s;
  if (sd.pre != PRE_NONE && (s = TIMED(PM_PROF_PRE_FWD, check(ctx, launch_pre_fwd(ta, dt, ctx->ls), "embedding / LayerNorm forward"))) != PM_OK) return s;
  for (int l = 0; l < sd.n_lin; ++l) {
    prof_begin(ctx, PM_PROF_GEMM_FWD);
    cudaError_t e = dt == PM_F32 ? launch_simt_gemm(ta, dt, 0, l, ctx->ls) : umma_launch(ctx->umma, ta, 0, l, ctx->ls);
    if ((s = check(ctx, e, "forward GEMM")) != PM_OK) return s;
  }
  const bool att = feeds_attention(sd.post);
  if (att && ctx->attn && (s = TIMED(PM_PROF_ATTN_FWD, check(ctx, attn_tc_launch(ctx->attn, ta, true, ctx->ls), "attention forward"))) != PM_OK) return s;
  const int n_post = ((att && !ctx->attn) ? 1 : 0) + ((sd.post == POST_RESIDUAL && !ctx->ta.res_fused) ? 1 : 0);
  if (n_post && (s = TIMED(PM_PROF_POST_FWD, check(ctx, launch_post_fwd(ta, dt, ctx->ls, ctx->attn != nullptr), "attention / residual forward", n_post))) != PM_OK) return s;
  return PM_OK;
}

// The launches of ONE stage's backward pass (ta restricted to it).  grouped: the weight gradient, the bias column sums of
// Linears without activation and the finishing passes are left to grouped launches over all stages (ta.defer_finish set).
static pm_status stage_backward(pm_ctx* ctx, const TickArgs& ta, int p, bool grouped) {
  const int dt = ctx->cfg.compute_dtype;
  const int P = ctx->cfg.n_stages;
  const StageDev& sd = ctx->L.st[p];
  pm_status s;
  if (p == P - 1 && (s = TIMED(PM_PROF_LOSS, check(ctx, launch_loss(ta, dt, ctx->ls), "loss"))) != PM_OK) return s;
  if (feeds_attention(sd.post)) {
    if (ctx->attn) { if ((s = TIMED(PM_PROF_ATTN_BWD, check(ctx, attn_tc_launch(ctx->attn, ta, false, ctx->ls), "attention backward"))) != PM_OK) return s; }
    else if ((s = TIMED(PM_PROF_ATTN_BWD, check(ctx, launch_post_bwd(ta, dt, ctx->ls), "attention backward"))) != PM_OK) return s;
  }
  for (int l = sd.n_lin - 1; l >= 0; --l) {
    // dz = dy * act'(z) must exist before this stage's dgrad; a Linear without activation needs only the column sums
    // of its incoming gradient (the bias gradient), which can wait for one grouped launch
    if ((!grouped || bwd_act(sd.lin[l]) != PM_ACT_NONE) &&
        (s = TIMED(PM_PROF_ACT_BWD, check(ctx, launch_actbwd(ta, dt, l, ctx->ls), "activation backward", actbwd_launches(ta)))) != PM_OK) return s;
    cudaError_t e;
    if (!grouped) {
      prof_begin(ctx, PM_PROF_WGRAD);
      e = dt == PM_F32 ? launch_simt_gemm(ta, dt, 2, l, ctx->ls) : umma_launch(ctx->umma, ta, 2, l, ctx->ls);
      if ((s = check(ctx, e, "wgrad GEMM")) != PM_OK) return s;
    }
    if (p == 0 && l == 0 && sd.pre != PRE_EMBED) continue;          // raw network inputs need no gradient
    prof_begin(ctx, PM_PROF_DGRAD);
    e = dt == PM_F32 ? launch_simt_gemm(ta, dt, 1, l, ctx->ls) : umma_launch(ctx->umma, ta, (ctx->L.stash || ctx->L.materialize) ? 4 : 1, l, ctx->ls);
    if ((s = check(ctx, e, "dgrad GEMM")) != PM_OK) return s;
  }
  const int n_pre = sd.pre != PRE_NONE ? pre_bwd_launches(ta) : 0;
  if (n_pre && (s = TIMED(PM_PROF_PRE_BWD, check(ctx, launch_pre_bwd(ta, dt, ctx->ls), "LayerNorm / embedding backward", n_pre))) != PM_OK) return s;
  return PM_OK;
}

static pm_status mb_forward(pm_ctx* ctx, const void* inputs, const void* targets) {
  if (!inputs || !targets) return fail(ctx, PM_ERR_INVALID_ARG, "microbatch-major order takes a microbatch at every step (there is nothing to drain)");
  const int dt = ctx->cfg.compute_dtype;
  const int P = ctx->cfg.n_stages;
  const int64_t mb = ctx->n_fed;
  pm_status s;
  const bool stoch = ctx->L.stochastic > 0;
  s = TIMED(PM_PROF_SCHEDULE, check(ctx, launch_schedule_mb((const StageSched*)(ctx->ws + ctx->L.off_sched), (StageDyn*)(ctx->ws + ctx->L.off_dyn),
                                                            ctx->hp, mb, ctx->stream,
                                                            stoch ? (const int32_t*)(ctx->ws + ctx->L.off_delays) : nullptr,
                                                            stoch ? (const int64_t*)(ctx->ws + ctx->L.off_nupd) : nullptr), "schedule"));
  if (s != PM_OK) return s;
  s = TIMED(PM_PROF_INGEST, check(ctx, launch_ingest(ctx->ta, dt, inputs, (const float*)targets, mb, ctx->stream), "ingest"));
  if (s != PM_OK) return s;
  s = run_phase(ctx, ctx->g_fwd, [&]() -> pm_status {
    pm_status s;
    for (int p = 0; p < P; ++p)
      if ((s = stage_forward(ctx, mb_args(ctx, p, p), p)) != PM_OK) return s;
    return PM_OK;
  });
  if (s != PM_OK) return s;
  ctx->n_fed = mb + 1;
  ctx->phase = 1;
  return PM_OK;
}

// The grouped launches that close a backward pass over the stages table `table` marks (all of them, or one recompute
// segment): the weight gradients as one launch.
static pm_status grouped_wgrad(pm_ctx* ctx, int table, bool fused = false) {
  const int dt = ctx->cfg.compute_dtype;
  TickArgs ta = mb_args(ctx, table, -1);
  ta.fuse_upd = fused ? 1 : 0;
  prof_begin(ctx, PM_PROF_WGRAD);
  cudaError_t e = dt == PM_F32 ? launch_simt_gemm(ta, dt, 2, 0, ctx->ls) : umma_launch(ctx->umma, ta, 2, 0, ctx->ls);
  return check(ctx, e, "wgrad GEMM");
}

static pm_status mb_backward(pm_ctx* ctx) {
  const int dt = ctx->cfg.compute_dtype;
  const int P = ctx->cfg.n_stages;
  // With one Linear per stage nothing overwrites a stage's dz before the end of the backward chain, so the weight
  // gradients of all stages run as ONE grouped launch (the tick schedule's launch, which fills the GPU); stages
  // with several Linears reuse their dz scratch from level to level and form each weight gradient on the spot.
  const bool grouped = ctx->L.max_lin == 1;
  // PipeMare Recompute (Appendix A.2): segments from the last to the first; before a segment's backward its stages run
  // forward again from the input the forward pass left at the segment's first stage, with the recompute weights
  // (table 2P + 1), overwriting every stash the backward reads.  The last segment's backward follows its forward
  // directly: nothing to recompute.  A segment's weight gradients are formed before the next (earlier) segment is
  // recomputed, because that recomputation overwrites the input of this segment's first stage.
  const int S = ctx->L.segment;
  const int n_seg = S > 0 ? (P + S - 1) / S : 1;
  pm_status s = run_phase(ctx, ctx->g_bwd, [&]() -> pm_status {
    pm_status s;
    for (int k = n_seg - 1; k >= 0; --k) {
      const int lo = S > 0 ? k * S : 0, hi = S > 0 ? std::min(P, lo + S) : P;
      if (S > 0 && k < n_seg - 1)
        for (int p = lo; p < hi; ++p)
          if ((s = stage_forward(ctx, mb_args(ctx, 2 * P + 1, p), p)) != PM_OK) return s;
      for (int p = hi - 1; p >= lo; --p) {
        TickArgs ta = mb_args(ctx, 2 * P - 1 - p, p);
        ta.defer_finish = grouped ? 1 : 0;      // the partial sums of bias and LayerNorm gradients are added up once, below
        if ((s = stage_backward(ctx, ta, p, grouped)) != PM_OK) return s;
      }
      if (grouped && S > 0 && (s = grouped_wgrad(ctx, 2 * P + 2 + k)) != PM_OK) return s;
    }
    if (grouped) {
      TickArgs ta = mb_args(ctx, 2 * P, -1);
      ta.colsum_only = 1; ta.defer_finish = 1;                  // bias gradients of the Linears without activation, all stages at once
      if ((s = TIMED(PM_PROF_ACT_BWD, check(ctx, launch_actbwd(ta, dt, 0, ctx->ls), "bias gradient column sums", actbwd_launches(ta)))) != PM_OK) return s;
      ta.colsum_only = 0; ta.defer_finish = 0;
      if (S == 0 && !ctx->L.fuse && (s = grouped_wgrad(ctx, 2 * P)) != PM_OK) return s;   // fused update: formed in the update phase
      const int n_fin = deferred_finish_launches(ta);
      if (n_fin && (s = TIMED(PM_PROF_PRE_BWD, check(ctx, launch_deferred_finish(ta, dt, ctx->ls), "bias / LayerNorm gradient sums", n_fin))) != PM_OK) return s;
    }
    return PM_OK;
  });
  if (s != PM_OK) return s;
  ctx->phase = 2;
  return PM_OK;
}

static pm_status mb_update(pm_ctx* ctx) {
  const int P = ctx->cfg.n_stages;
  if (ctx->n_fed % ctx->hp.n_micro != 0) {          // inside a minibatch: the gradients stay in the arena and the next microbatch adds to them
    ctx->tick += 1;
    ctx->phase = 0;
    return PM_OK;
  }
  const StageDyn* dyn_all = (const StageDyn*)(ctx->ws + ctx->L.off_dyn) + (size_t)2 * P * P;
  const float* gsrc = nullptr;
  if (ctx->L.stochastic > 0) {
    // stochastic delays (Appendix E): this microbatch's gradients join the ring of the last tau_max + 1; every stage's update
    // reads the slot its table entry names (the slot changes from step to step, so the copy stays outside the graph)
    float* gq = reinterpret_cast<float*>(ctx->ta.ring + ctx->L.g_ring);
    const int64_t mb = ctx->n_fed - 1;
    cudaError_t ce = cudaMemcpyAsync(gq + (uint64_t)(mb % ctx->L.stochastic) * ctx->L.total, ctx->a.grad, ctx->L.total * sizeof(float),
                                     cudaMemcpyDeviceToDevice, ctx->stream);
    if (ce != cudaSuccess) return cuda_fail(ctx, ce, "gradient ring copy");
    gsrc = gq;
  }
  pm_status s = run_phase(ctx, ctx->g_upd, [&]() -> pm_status {
    // fused update: the weight gradients of all stages as one launch whose epilogue updates the Linear matrices
    if (ctx->L.fuse) { pm_status fs = grouped_wgrad(ctx, 2 * P, true); if (fs != PM_OK) return fs; }
    prof_begin(ctx, PM_PROF_UPDATE);
    cudaError_t e = launch_update(ctx->a, (const uint32_t*)(ctx->ws + ctx->L.off_b64), (const uint32_t*)(ctx->ws + ctx->L.off_e64), dyn_all,
                                  (int64_t*)(ctx->ws + ctx->L.off_nupd), P, ctx->L.total / 64, ctx->cfg.optimizer, ctx->cfg.beta1,
                                  ctx->cfg.beta2, ctx->cfg.eps, ctx->ls, ctx->ta.ring, ctx->hp.lp_elem, 0,
                                  ctx->L.fuse ? (const uint32_t*)(ctx->ws + ctx->L.off_skb) : nullptr,
                                  ctx->L.fuse ? (const uint32_t*)(ctx->ws + ctx->L.off_ske) : nullptr, gsrc);
    pm_status s = check(ctx, e, "update");
    if (s != PM_OK || ctx->L.segs.empty()) return s;
    prof_begin(ctx, PM_PROF_UPDATE);
    e = launch_push_small(ctx->a.w, ctx->a.delta, ctx->ta.ring, (const SmallSeg*)(ctx->ws + ctx->L.off_segs), (int)ctx->L.segs.size(), dyn_all, -1, ctx->ls);
    return check(ctx, e, "weight-version push");
  });
  if (s != PM_OK) return s;
  ctx->tick += 1;
  ctx->phase = 0;
  return PM_OK;
}

// ---- sparse ticks (tick-major order with an entry period E > 1) ----------------------------------------------------
// Only the stages at distance = tick mod E from a microbatch's entry can hold a microbatch in a given tick, so a
// tick's launches are restricted to them (each stage's kernels as in microbatch-major order), with one CUDA graph per
// phase and residue.  A tick's forward stages depend on nothing its backward stages or updates produce (their
// weights come from the version queues, their inputs from the previous tick's forward; the ring depths keep the two
// apart), so they run on a stream of their own next to the backward and update of the same tick; the tick's
// schedule waits for the previous tick's forward, and the forward waits for the schedule, which follows the previous
// tick's update.
static bool sparse_ticks(const pm_ctx* ctx) { return ctx->L.E > 1 && !ctx->gs_fwd.empty(); }

static void sparse_stages(const pm_ctx* ctx, bool fwd, std::vector<int>& out) {
  const int P = ctx->cfg.n_stages, E = ctx->L.E;
  out.clear();
  for (int p = 0; p < P; ++p) {
    const int64_t off = fwd ? p : 2 * (int64_t)P - 1 - p;
    if ((((ctx->tick - off) % E) + E) % E == 0) out.push_back(p);   // whether a microbatch IS there the kernels read from the schedule table
  }
}

static pm_status sparse_forward_phase(pm_ctx* ctx) {
  const bool side = ctx->fwd_stream && !ctx->prof_on;
  if (side) {
    cudaError_t e = cudaEventRecord(ctx->ev_sched, ctx->stream);                 // schedule table and inputs of this tick are in place
    if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->fwd_stream, ctx->ev_sched, 0);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "forward stream");
  }
  std::vector<int> st;
  sparse_stages(ctx, true, st);
  pm_status s = run_phase(ctx, ctx->gs_fwd[(size_t)(ctx->tick % ctx->L.E)], [&]() -> pm_status {
    for (int p : st) { pm_status s = stage_forward(ctx, mb_args(ctx, 0, p), p); if (s != PM_OK) return s; }
    return PM_OK;
  }, side ? ctx->fwd_stream : nullptr);
  if (s != PM_OK) return s;
  if (side) {
    cudaError_t e = cudaEventRecord(ctx->ev_fwd, ctx->fwd_stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "forward stream");
    ctx->fwd_pending = true;
  }
  return PM_OK;
}

static pm_status sparse_backward_phase(pm_ctx* ctx) {
  std::vector<int> st;
  sparse_stages(ctx, false, st);
  return run_phase(ctx, ctx->gs_bwd[(size_t)(ctx->tick % ctx->L.E)], [&]() -> pm_status {
    for (auto it = st.rbegin(); it != st.rend(); ++it) {                           // later stages first, as everywhere
      pm_status s = stage_backward(ctx, mb_args(ctx, 0, *it), *it, false);
      if (s != PM_OK) return s;
    }
    return PM_OK;
  });
}

static pm_status sparse_update_phase(pm_ctx* ctx) {
  std::vector<int> st;
  sparse_stages(ctx, false, st);
  return run_phase(ctx, ctx->gs_upd[(size_t)(ctx->tick % ctx->L.E)], [&]() -> pm_status {
    for (int p : st) {
      prof_begin(ctx, PM_PROF_UPDATE);
      cudaError_t e = launch_update(ctx->a, (const uint32_t*)(ctx->ws + ctx->L.off_b64) + p, (const uint32_t*)(ctx->ws + ctx->L.off_e64) + p,
                                    (const StageDyn*)(ctx->ws + ctx->L.off_dyn) + p, (int64_t*)(ctx->ws + ctx->L.off_nupd) + p, 1,
                                    ctx->L.end64[p], ctx->cfg.optimizer, ctx->cfg.beta1, ctx->cfg.beta2, ctx->cfg.eps, ctx->ls,
                                    (void*)ctx->ta.ring, ctx->hp.lp_elem, ctx->L.begin64[p]);
      pm_status s = check(ctx, e, "update");
      if (s != PM_OK) return s;
      if (ctx->seg_count[p] > 0) {
        prof_begin(ctx, PM_PROF_UPDATE);
        // the segments name their stage by its index in the whole table: hand the kernel the table's base
        e = launch_push_small(ctx->a.w, ctx->a.delta, ctx->ta.ring, (const SmallSeg*)(ctx->ws + ctx->L.off_segs) + ctx->seg_first[p], ctx->seg_count[p],
                              (const StageDyn*)(ctx->ws + ctx->L.off_dyn), -1, ctx->ls);
        if ((s = check(ctx, e, "weight-version push")) != PM_OK) return s;
      }
    }
    return PM_OK;
  });
}

pm_status pm_forward(pm_ctx* ctx, const void* inputs, const void* targets) {
  if (!ctx) return fail(nullptr, PM_ERR_INVALID_ARG, "null context");
  if (ctx->phase != 0) return fail(ctx, PM_ERR_STATE, "pm_forward called out of order (expected pm_backward or pm_update)");
  if (ctx->L.mb) return mb_forward(ctx, inputs, targets);
  if ((inputs == nullptr) != (targets == nullptr)) return fail(ctx, PM_ERR_INVALID_ARG, "inputs and targets must both be given or both be NULL");
  if (inputs && ctx->draining) return fail(ctx, PM_ERR_STATE, "microbatches must be fed on consecutive ticks; the pipeline is already draining");
  const int64_t mb = mb_at_tick(ctx->tick, ctx->hp.warm, ctx->hp.period, ctx->hp.entry_period);   // the microbatch that may enter now, or -1
  if (inputs && mb < 0) return fail(ctx, PM_ERR_STATE, ctx->hp.entry_period > 1 ? "a microbatch enters every entry_period ticks; this tick takes none"
                                                                               : "during the synchronous warm-up a microbatch enters every 2 * n_stages ticks; this tick takes none");
  const int dt = ctx->cfg.compute_dtype;
  pm_status s;
  if (inputs) ctx->n_fed = mb + 1; else if (mb >= 0) ctx->draining = true;   // an empty tick between two warm-up microbatches ends nothing
  if (ctx->fwd_pending) {                          // sparse ticks: the previous tick's forward still reads the schedule table
    cudaError_t ew = cudaStreamWaitEvent(ctx->stream, ctx->ev_fwd, 0);
    if (ew != cudaSuccess) return cuda_fail(ctx, ew, "forward stream");
    ctx->fwd_pending = false;
  }
  s = TIMED(PM_PROF_SCHEDULE, check(ctx, launch_schedule((const StageSched*)(ctx->ws + ctx->L.off_sched), (const int64_t*)(ctx->ws + ctx->L.off_nupd),
                                 (StageDyn*)(ctx->ws + ctx->L.off_dyn), ctx->hp, ctx->tick, ctx->n_fed, -1, ctx->stream), "schedule"));
  if (s != PM_OK) return s;
  if (inputs) {
    s = TIMED(PM_PROF_INGEST, check(ctx, launch_ingest(ctx->ta, dt, inputs, (const float*)targets, mb, ctx->stream), "ingest"));
    if (s != PM_OK) return s;
  }
  if (sparse_ticks(ctx)) {
    if (any_stage_active(ctx, 0, ctx->cfg.n_stages - 1) && (s = sparse_forward_phase(ctx)) != PM_OK) return s;
    ctx->phase = 1;
    return PM_OK;
  }
  // forward of every stage whose microbatch exists
  if (any_stage_active(ctx, 0, ctx->cfg.n_stages - 1)) {
    s = run_phase(ctx, ctx->g_fwd, [&]() -> pm_status {
      pm_status s;
      if (ctx->L.any_pre && (s = TIMED(PM_PROF_PRE_FWD, check(ctx, launch_pre_fwd(ctx->ta, dt, ctx->ls), "embedding / LayerNorm forward"))) != PM_OK) return s;
      for (int l = 0; l < ctx->L.max_lin; ++l) {
        prof_begin(ctx, PM_PROF_GEMM_FWD);
        cudaError_t e = dt == PM_F32 ? launch_simt_gemm(ctx->ta, dt, 0, l, ctx->ls)
                                     : umma_launch(ctx->umma, ctx->ta, 0, l, ctx->ls);
        if ((s = check(ctx, e, "forward GEMM")) != PM_OK) return s;
      }
      if (ctx->attn && (s = TIMED(PM_PROF_ATTN_FWD, check(ctx, attn_tc_launch(ctx->attn, ctx->ta, true, ctx->ls), "attention forward"))) != PM_OK) return s;
      const int n_post = ((ctx->L.att_blocks > 0 && !ctx->attn) ? 1 : 0) + ((ctx->L.any_residual && !ctx->ta.res_fused) ? 1 : 0);
      if (n_post && (s = TIMED(PM_PROF_POST_FWD, check(ctx, launch_post_fwd(ctx->ta, dt, ctx->ls, ctx->attn != nullptr), "attention / residual forward", n_post))) != PM_OK) return s;
      return PM_OK;
    });
    if (s != PM_OK) return s;
  }
  ctx->phase = 1;
  return PM_OK;
}

pm_status pm_backward(pm_ctx* ctx) {
  if (!ctx) return fail(nullptr, PM_ERR_INVALID_ARG, "null context");
  if (ctx->phase != 1) return fail(ctx, PM_ERR_STATE, "pm_backward must follow pm_forward");
  if (ctx->L.mb) return mb_backward(ctx);
  const int dt = ctx->cfg.compute_dtype;
  const int P = ctx->cfg.n_stages;
  pm_status s;
  // any backward this tick?  stage P runs the microbatch that entered P ticks ago, stage 1 the one from 2P-1 ticks ago
  const bool any = any_stage_active(ctx, P, 2 * P - 1);
  if (any && sparse_ticks(ctx)) {
    if ((s = sparse_backward_phase(ctx)) != PM_OK) return s;
  } else if (any) {
    s = run_phase(ctx, ctx->g_bwd, [&]() -> pm_status {
      pm_status s;
      if ((s = TIMED(PM_PROF_LOSS, check(ctx, launch_loss(ctx->ta, dt, ctx->ls), "loss"))) != PM_OK) return s;
      if (ctx->attn) { if ((s = TIMED(PM_PROF_ATTN_BWD, check(ctx, attn_tc_launch(ctx->attn, ctx->ta, false, ctx->ls), "attention backward"))) != PM_OK) return s; }
      else if (ctx->L.att_blocks > 0 && (s = TIMED(PM_PROF_ATTN_BWD, check(ctx, launch_post_bwd(ctx->ta, dt, ctx->ls), "attention backward"))) != PM_OK) return s;
      for (int l = ctx->L.max_lin - 1; l >= 0; --l) {
        if ((s = TIMED(PM_PROF_ACT_BWD, check(ctx, launch_actbwd(ctx->ta, dt, l, ctx->ls), "activation backward", actbwd_launches(ctx->ta)))) != PM_OK) return s;
        cudaError_t e = cudaSuccess;
        if (!ctx->L.fuse) {                                           // fused update: formed in the update phase
          prof_begin(ctx, PM_PROF_WGRAD);
          e = dt == PM_F32 ? launch_simt_gemm(ctx->ta, dt, 2, l, ctx->ls)
                           : umma_launch(ctx->umma, ctx->ta, 2, l, ctx->ls);
          if ((s = check(ctx, e, "wgrad GEMM")) != PM_OK) return s;
        }
        prof_begin(ctx, PM_PROF_DGRAD);
        e = dt == PM_F32 ? launch_simt_gemm(ctx->ta, dt, 1, l, ctx->ls)
                         : umma_launch(ctx->umma, ctx->ta, 1, l, ctx->ls);
        if ((s = check(ctx, e, "dgrad GEMM")) != PM_OK) return s;
      }
      const int n_pre = pre_bwd_launches(ctx->ta);
      if (n_pre && (s = TIMED(PM_PROF_PRE_BWD, check(ctx, launch_pre_bwd(ctx->ta, dt, ctx->ls), "LayerNorm / embedding backward", n_pre))) != PM_OK) return s;
      return PM_OK;
    });
    if (s != PM_OK) return s;
  }
  ctx->phase = 2;
  return PM_OK;
}

pm_status pm_update(pm_ctx* ctx) {
  if (!ctx) return fail(nullptr, PM_ERR_INVALID_ARG, "null context");
  if (ctx->phase != 2) return fail(ctx, PM_ERR_STATE, "pm_update must follow pm_backward");
  if (ctx->L.mb) return mb_update(ctx);
  const int P = ctx->cfg.n_stages;
  const bool any = any_stage_active(ctx, P, 2 * P - 1);
  if (any && sparse_ticks(ctx)) {
    pm_status s = sparse_update_phase(ctx);
    if (s != PM_OK) return s;
  } else if (any) {
    pm_status s = run_phase(ctx, ctx->g_upd, [&]() -> pm_status {
      cudaError_t e;
      if (ctx->L.fuse) {
        // the weight gradients of the stages in backward, with the update of their Linear matrices in the epilogue
        TickArgs ta = ctx->ta;
        ta.fuse_upd = 1;
        prof_begin(ctx, PM_PROF_WGRAD);
        e = umma_launch(ctx->umma, ta, 2, 0, ctx->ls);
        pm_status fs = check(ctx, e, "wgrad GEMM with fused update");
        if (fs != PM_OK) return fs;
      }
      prof_begin(ctx, PM_PROF_UPDATE);
      e = launch_update(ctx->a, (const uint32_t*)(ctx->ws + ctx->L.off_b64), (const uint32_t*)(ctx->ws + ctx->L.off_e64),
                        (const StageDyn*)(ctx->ws + ctx->L.off_dyn), (int64_t*)(ctx->ws + ctx->L.off_nupd), P,
                        ctx->L.total / 64, ctx->cfg.optimizer, ctx->cfg.beta1, ctx->cfg.beta2, ctx->cfg.eps, ctx->ls,
                        ctx->L.queue ? (void*)ctx->ta.ring : nullptr, ctx->hp.lp_elem, 0,
                        ctx->L.fuse ? (const uint32_t*)(ctx->ws + ctx->L.off_skb) : nullptr,
                        ctx->L.fuse ? (const uint32_t*)(ctx->ws + ctx->L.off_ske) : nullptr);
      pm_status s = check(ctx, e, "update");
      if (s != PM_OK || !ctx->L.queue || ctx->L.segs.empty()) return s;
      prof_begin(ctx, PM_PROF_UPDATE);                                 // fp32 copies of the updated stages' small tensors into their queues
      e = launch_push_small(ctx->a.w, ctx->a.delta, ctx->ta.ring, (const SmallSeg*)(ctx->ws + ctx->L.off_segs), (int)ctx->L.segs.size(),
                            (const StageDyn*)(ctx->ws + ctx->L.off_dyn), -1, ctx->ls);
      return check(ctx, e, "weight-version push");
    });
    if (s != PM_OK) return s;
  }
  ctx->tick += 1;
  ctx->phase = 0;
  return PM_OK;
}

pm_status pm_step(pm_ctx* ctx, const void* inputs, const void* targets) {
  pm_status s = pm_forward(ctx, inputs, targets);
  if (s != PM_OK) return s;
  if ((s = pm_backward(ctx)) != PM_OK) return s;
  return pm_update(ctx);
}

// After a synchronisation: did any CTA give up on a bounded wait?
static pm_status check_device_status(pm_ctx* ctx) {
  int* words[2] = {umma_status_word(ctx->umma), attn_status_word(ctx->attn)};
  for (int* w : words) {
    if (!w) continue;
    int code = 0;
    cudaError_t e = cudaMemcpy(&code, w, sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "status read-back");
    if (code != 0) return fail(ctx, PM_ERR_TIMEOUT, "a bounded device-side wait expired in a tensor-core kernel (role code " + std::to_string(code) + ")");
  }
  return PM_OK;
}

pm_status pm_set_delays(pm_ctx* ctx, const int32_t* delays) {
  if (!ctx || !delays) return fail(ctx, PM_ERR_INVALID_ARG, "null argument");
  if (ctx->L.stochastic == 0) return fail(ctx, PM_ERR_STATE, "pm_set_delays belongs to the stochastic delay model (pm_config.stochastic_tau_max > 0)");
  if (ctx->phase != 0) return fail(ctx, PM_ERR_STATE, "pm_set_delays between steps only");
  const int P = ctx->cfg.n_stages;
  for (int p = 0; p < P; ++p)
    if (delays[p] < 0 || delays[p] >= ctx->L.stochastic) return fail(ctx, PM_ERR_INVALID_ARG, "delay of stage " + std::to_string(p) + " outside [0, stochastic_tau_max]");
  ctx->h_delays.assign(delays, delays + P);
  // ordered on the context's stream behind the previous step's schedule kernel, which read the old values
  cudaError_t e = cudaMemcpyAsync(ctx->ws + ctx->L.off_delays, ctx->h_delays.data(), sizeof(int32_t) * P, cudaMemcpyHostToDevice, ctx->stream);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "delay upload");
  return PM_OK;
}

pm_status pm_get_bookkeeping(pm_ctx* ctx, int32_t stage, int64_t* out8) {
  if (!ctx || !out8) return fail(ctx, PM_ERR_INVALID_ARG, "null argument");
  if (stage < 0 || stage >= ctx->cfg.n_stages) return fail(ctx, PM_ERR_INVALID_ARG, "stage out of range");
  StageDyn d;
  int64_t n = 0;
  cudaError_t e = cudaStreamSynchronize(ctx->stream);
  if (e == cudaSuccess && ctx->fwd_stream) e = cudaStreamSynchronize(ctx->fwd_stream);
  if (ctx->L.mb) {
    // the stage's forward ran in sub-tick `stage`, its backward in sub-tick 2P - 1 - stage of the last microbatch
    const int P = ctx->cfg.n_stages;
    StageDyn df, db;
    const char* tab = ctx->ws + ctx->L.off_dyn;
    if (e == cudaSuccess) e = cudaMemcpy(&df, tab + sizeof(StageDyn) * ((size_t)stage * P + stage), sizeof(StageDyn), cudaMemcpyDeviceToHost);
    if (e == cudaSuccess) e = cudaMemcpy(&db, tab + sizeof(StageDyn) * ((size_t)(2 * P - 1 - stage) * P + stage), sizeof(StageDyn), cudaMemcpyDeviceToHost);
    if (e == cudaSuccess) e = cudaMemcpy(&n, ctx->ws + ctx->L.off_nupd + sizeof(int64_t) * stage, sizeof(int64_t), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "bookkeeping read-back");
    if (pm_status ds = check_device_status(ctx)) return ds;
    out8[0] = df.f_mb; out8[1] = df.f_ver; out8[2] = db.b_mb; out8[3] = db.b_ver; out8[4] = n;
    out8[5] = df.f_vslot; out8[6] = ctx->L.segment > 0 ? db.r_ver : (int64_t)db.b_slot; out8[7] = ctx->n_fed - 1;
    if (ctx->L.stochastic > 0) {                                  // the update table's entry names the microbatch whose gradient was applied
      StageDyn du;
      e = cudaMemcpy(&du, tab + sizeof(StageDyn) * ((size_t)(2 * P) * P + stage), sizeof(StageDyn), cudaMemcpyDeviceToHost);
      if (e != cudaSuccess) return cuda_fail(ctx, e, "bookkeeping read-back");
      out8[6] = du.r_ver;
    }
    return PM_OK;
  }
  if (e == cudaSuccess) e = cudaMemcpy(&d, ctx->ws + ctx->L.off_dyn + sizeof(StageDyn) * stage, sizeof(StageDyn), cudaMemcpyDeviceToHost);
  if (e == cudaSuccess) e = cudaMemcpy(&n, ctx->ws + ctx->L.off_nupd + sizeof(int64_t) * stage, sizeof(int64_t), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "bookkeeping read-back");
  if (pm_status ds = check_device_status(ctx)) return ds;
  out8[0] = d.f_mb; out8[1] = d.f_ver; out8[2] = d.b_mb; out8[3] = d.b_ver; out8[4] = n;
  out8[5] = d.f_slot; out8[6] = d.b_slot; out8[7] = d.tick;
  return PM_OK;
}

pm_status pm_get_losses(pm_ctx* ctx, float* host_out, int64_t first_mb, int64_t n) {
  if (!ctx || !host_out || first_mb < 0 || n < 0) return fail(ctx, PM_ERR_INVALID_ARG, "bad argument");
  const int P = ctx->cfg.n_stages;
  // a microbatch's loss is computed P ticks after it entered; ticks completed so far = ctx->tick
  const int64_t last = ctx->tick - P - 1, t0 = ctx->hp.warm * ctx->hp.period;   // latest entry tick whose loss exists
  const int64_t entered = last < 0 ? 0 : (ctx->hp.entry_period > 1 ? last / ctx->hp.entry_period + 1
                                          : (last < t0 ? last / ctx->hp.period + 1 : ctx->hp.warm + (last - t0) + 1));
  const int64_t done = ctx->L.mb ? ctx->n_fed - (ctx->phase == 1 ? 1 : 0) : std::min<int64_t>(ctx->n_fed, entered);
  if (first_mb + n > done) return fail(ctx, PM_ERR_INVALID_ARG, "loss of a microbatch that has not finished was requested");
  if (done - first_mb > ctx->L.loss_cap) return fail(ctx, PM_ERR_INVALID_ARG, "requested losses have left the device log");
  cudaError_t e = cudaStreamSynchronize(ctx->stream);
  if (e == cudaSuccess && ctx->fwd_stream) e = cudaStreamSynchronize(ctx->fwd_stream);
  for (int64_t i = 0; i < n && e == cudaSuccess; ++i)
    e = cudaMemcpy(host_out + i, ctx->ws + ctx->L.off_loss + sizeof(float) * ((first_mb + i) % ctx->L.loss_cap), sizeof(float), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "loss read-back");
  if (pm_status ds = check_device_status(ctx)) return ds;
  return PM_OK;
}

uint64_t pm_launch_count(pm_ctx* ctx) { return ctx ? ctx->launches : 0; }

pm_status pm_selftest_wait_timeout(pm_ctx* ctx, int64_t limit_cycles) {
  if (!ctx || limit_cycles < 1) return fail(ctx, PM_ERR_INVALID_ARG, "bad argument");
  if (!ctx->umma) return fail(ctx, PM_ERR_UNSUPPORTED, "the bounded waits belong to the tensor-core kernels (PM_BF16 contexts)");
  int* d_ret = reinterpret_cast<int*>(ctx->ws + ctx->L.off_lossred) + 100;      // a spare word of the loss-reduction block
  cudaError_t e = cudaMemsetAsync(d_ret, 0, sizeof(int), ctx->stream);
  if (e == cudaSuccess) e = umma_wait_timeout_probe(ctx->umma, (long long)limit_cycles, d_ret, ctx->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
  int ret = 0;
  if (e == cudaSuccess) e = cudaMemcpy(&ret, d_ret, sizeof(int), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "wait self-test");
  if (ret != 2) return fail(ctx, PM_ERR_STATE, "the probe's wait did not give up (code " + std::to_string(ret) + ")");
  const pm_status st = check_device_status(ctx);        // what any synchronising call reports after an expiry
  e = umma_clear_status(ctx->umma, ctx->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "wait self-test");
  return st;
}

pm_status pm_profile_enable(pm_ctx* ctx, int32_t on) {
  if (!ctx) return fail(nullptr, PM_ERR_INVALID_ARG, "null context");
  if (on && ctx->prof_ev.empty()) {
    const size_t pairs = 8192;
    ctx->prof_ev.resize(2 * pairs);
    for (auto& ev : ctx->prof_ev)
      if (cudaEventCreate(&ev) != cudaSuccess) { ctx->prof_ev.clear(); return fail(ctx, PM_ERR_CUDA, "cudaEventCreate failed"); }
    ctx->prof_pair_cls.assign(pairs, 0);
  }
  ctx->prof_on = on != 0;
  ctx->prof_used = 0;
  ctx->prof_cls = -1;
  return PM_OK;
}

pm_status pm_profile_read(pm_ctx* ctx, float* ms_by_class, int64_t* launches_by_class) {
  if (!ctx || !ms_by_class || !launches_by_class) return fail(ctx, PM_ERR_INVALID_ARG, "null argument");
  cudaError_t e = cudaStreamSynchronize(ctx->stream);
  if (e == cudaSuccess && ctx->fwd_stream) e = cudaStreamSynchronize(ctx->fwd_stream);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "profile read");
  for (int i = 0; i < PM_PROF_CLASSES; ++i) { ms_by_class[i] = 0.f; launches_by_class[i] = 0; }
  for (size_t i = 0; i < ctx->prof_used; ++i) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, ctx->prof_ev[2 * i], ctx->prof_ev[2 * i + 1]) == cudaSuccess) {
      ms_by_class[ctx->prof_pair_cls[i]] += ms;
      launches_by_class[ctx->prof_pair_cls[i]] += 1;
    }
  }
  ctx->prof_used = 0;
  return PM_OK;
}

const char* pm_last_error(pm_ctx* ctx) { return ctx ? ctx->err.c_str() : g_error.c_str(); }

void pm_destroy(pm_ctx* ctx) {
  if (!ctx) return;
  if (ctx->fwd_stream) cudaStreamSynchronize(ctx->fwd_stream);
  umma_plan_destroy(ctx->umma);
  attn_plan_destroy(ctx->attn);
  for (auto& ev : ctx->prof_ev) cudaEventDestroy(ev);
  delete ctx;
}

// ---- stand-alone fused update -------------------------------------------------------------------

uint64_t pm_update_flat_workspace_bytes(int32_t n_stages) {
  if (n_stages < 1) return 0;
  uint64_t P = (uint64_t)n_stages, w = 0;
  w = align_up(w + sizeof(StageSched) * P, 256);
  w = align_up(w + sizeof(StageDyn) * P, 256);
  w = align_up(w + sizeof(int64_t) * P, 256);
  w = align_up(w + sizeof(uint32_t) * P, 256);
  w = align_up(w + sizeof(uint32_t) * P, 256);
  return w;
}

pm_status pm_update_flat(const pm_arenas* arenas, const uint64_t* stage_offsets, const uint64_t* stage_counts,
                         const int32_t* tau_fwd, const int32_t* tau_bkwd, int32_t n_stages, const pm_config* cfg,
                         int64_t k, void* workspace, uint64_t workspace_bytes, void* stream) {
  if (!arenas || !stage_offsets || !stage_counts || !tau_fwd || !tau_bkwd || !cfg) return fail(nullptr, PM_ERR_INVALID_ARG, "null argument");
  if (n_stages < 1 || n_stages > PM_MAX_STAGES) return fail(nullptr, PM_ERR_INVALID_ARG, "n_stages out of range");
  if (k < 0) return fail(nullptr, PM_ERR_INVALID_ARG, "k must be >= 0");
  if (cfg->optimizer != PM_SGDM && cfg->optimizer != PM_ADAM) return fail(nullptr, PM_ERR_INVALID_ARG, "unknown optimizer");
  if (!arenas->w || !arenas->m || !arenas->delta || !arenas->grad || (cfg->optimizer == PM_ADAM && !arenas->s))
    return fail(nullptr, PM_ERR_INVALID_ARG, "missing arena");
  if (cfg->alpha_by_step && cfg->alpha_len < 1) return fail(nullptr, PM_ERR_INVALID_ARG, "alpha_len must be >= 1 with alpha_by_step");
  const uint64_t need = pm_update_flat_workspace_bytes(n_stages);
  if (!workspace || workspace_bytes < need) return fail(nullptr, PM_ERR_NOMEM, "workspace too small: need " + std::to_string(need) + " bytes");
  const uint64_t P = (uint64_t)n_stages;
  thread_local std::vector<char> host;             // staging for the stage table: no allocation after the first call of a thread
  host.assign(need, 0);
  uint64_t off_sched = 0, off_dyn = align_up(sizeof(StageSched) * P, 256);
  uint64_t off_nupd = align_up(off_dyn + sizeof(StageDyn) * P, 256);
  uint64_t off_b = align_up(off_nupd + sizeof(int64_t) * P, 256);
  uint64_t off_e = align_up(off_b + sizeof(uint32_t) * P, 256);
  StageSched* sc = (StageSched*)(host.data() + off_sched);
  uint32_t* b64 = (uint32_t*)(host.data() + off_b);
  uint32_t* e64 = (uint32_t*)(host.data() + off_e);
  uint64_t prev_end = 0;
  for (int i = 0; i < n_stages; ++i) {
    if (stage_offsets[i] % PM_ALIGN_ELEMS) return fail(nullptr, PM_ERR_INVALID_ARG, "stage offsets must be multiples of 64 elements");
    if (stage_offsets[i] < prev_end) return fail(nullptr, PM_ERR_INVALID_ARG, "stage slices must ascend without overlap");
    if (tau_fwd[i] < 0 || tau_bkwd[i] < 0 || tau_bkwd[i] > tau_fwd[i]) return fail(nullptr, PM_ERR_INVALID_ARG, "need 0 <= tau_bkwd <= tau_fwd");
    if (stage_counts[i] > arenas->count || stage_offsets[i] > arenas->count - stage_counts[i])      // also catches a sum that would wrap
      return fail(nullptr, PM_ERR_NOMEM, "stage slice exceeds the arenas");
    uint64_t end = align_up(stage_offsets[i] + stage_counts[i], PM_ALIGN_ELEMS);
    if (end > arenas->count) return fail(nullptr, PM_ERR_NOMEM, "stage slice exceeds the arenas");
    prev_end = end;
    sc[i] = StageSched{tau_fwd[i], tau_fwd[i] - tau_bkwd[i], 1, 1, 0, 0};
    b64[i] = (uint32_t)(stage_offsets[i] / 64);
    e64[i] = (uint32_t)(end / 64);
  }
  cudaStream_t st = (cudaStream_t)stream;
  char* ws = (char*)workspace;
  cudaError_t e = cudaMemcpyAsync(ws, host.data(), need, cudaMemcpyHostToDevice, st);   // pageable source: staged before the call returns
  if (e != cudaSuccess) return cuda_fail(nullptr, e, "stage table upload");
  HyperDev hp{};
  hp.optimizer = cfg->optimizer; hp.t1 = cfg->t1_enable; hp.t2 = cfg->t2_enable; hp.n_stages = n_stages;
  hp.K = cfg->t1_K > 0 ? cfg->t1_K : 1; hp.D = cfg->t2_D;
  hp.alpha_const = cfg->alpha_by_step ? cfg->alpha_by_step[k < cfg->alpha_len ? k : cfg->alpha_len - 1] : cfg->alpha_const;
  hp.alpha_tab = nullptr; hp.alpha_len = 0;
  hp.beta1 = cfg->beta1; hp.beta2 = cfg->beta2; hp.eps = cfg->eps;
  hp.warm = 0; hp.period = 1;
  e = launch_schedule((const StageSched*)(ws + off_sched), (const int64_t*)(ws + off_nupd), (StageDyn*)(ws + off_dyn), hp, 0, 0, k, st);
  if (e != cudaSuccess) return cuda_fail(nullptr, e, "schedule");
  ArenasDev a{arenas->w, arenas->m, arenas->s, arenas->delta, arenas->grad, (__nv_bfloat16*)arenas->w_lp, arenas->count};
  e = launch_update(a, (const uint32_t*)(ws + off_b), (const uint32_t*)(ws + off_e), (const StageDyn*)(ws + off_dyn),
                    (int64_t*)(ws + off_nupd), n_stages, e64[n_stages - 1], cfg->optimizer, cfg->beta1, cfg->beta2, cfg->eps, st);
  if (e != cudaSuccess) return cuda_fail(nullptr, e, "update");
  return PM_OK;
}

}  // extern "C"
