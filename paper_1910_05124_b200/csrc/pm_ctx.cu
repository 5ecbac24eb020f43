// Host side of the C ABI: layout arithmetic, context set-up, and the launch sequence of a tick.
#include <cstdio>
#include <cstring>
#include <string>
#include <vector>

#include "pm_tick.cuh"
#include "pm_update.cuh"
#include "pm_umma.cuh"

using namespace pm;

namespace {

thread_local std::string g_error = "";

inline uint64_t align_up(uint64_t v, uint64_t a) { return (v + a - 1) / a * a; }

struct Layout {
  std::vector<StageDev> st;
  std::vector<StageSched> sched;
  std::vector<uint32_t> begin64, end64;
  uint64_t ring_bytes = 0, ws_bytes = 0, total = 0;
  // workspace offsets
  uint64_t off_st = 0, off_sched = 0, off_dyn = 0, off_nupd = 0, off_b64 = 0, off_e64 = 0, off_alpha = 0;
  uint64_t off_loss = 0, off_tgt = 0, off_yout = 0, off_umma = 0, off_lossred = 0;
  int64_t loss_cap = 0;
  int32_t max_lin = 0, max_dim = 0, n_in_first = 0, n_out_last = 0;
};

pm_status fail(pm_ctx* ctx, pm_status s, const std::string& msg);

pm_status build_layout(const pm_config* cfg, const pm_stage_desc* stages, Layout& L, std::string& err) {
  if (!cfg || !stages) { err = "null config or stage list"; return PM_ERR_INVALID_ARG; }
  const int P = cfg->n_stages;
  if (P < 1 || P > PM_MAX_STAGES) { err = "n_stages must be in [1, " + std::to_string(PM_MAX_STAGES) + "]"; return PM_ERR_INVALID_ARG; }
  if (cfg->microbatch < 1) { err = "microbatch must be positive"; return PM_ERR_INVALID_ARG; }
  if (cfg->compute_dtype != PM_F32 && cfg->compute_dtype != PM_BF16) { err = "unknown compute_dtype"; return PM_ERR_INVALID_ARG; }
  if (cfg->optimizer != PM_SGDM && cfg->optimizer != PM_ADAM) { err = "unknown optimizer"; return PM_ERR_INVALID_ARG; }
  if (cfg->loss != PM_LOSS_MSE) { err = "only PM_LOSS_MSE is built"; return PM_ERR_UNSUPPORTED; }
  if (cfg->t1_enable && cfg->t1_K < 1) { err = "t1_K must be >= 1"; return PM_ERR_INVALID_ARG; }
  const uint64_t esz = cfg->compute_dtype == PM_F32 ? 4 : 2;
  const uint64_t T = (uint64_t)cfg->microbatch;
  L.st.assign(P, StageDev{});
  L.sched.assign(P, StageSched{});
  L.begin64.assign(P, 0);
  L.end64.assign(P, 0);
  uint64_t ring = 0;
  int prev_out = -1;
  uint64_t prev_end = 0;
  for (int p = 0; p < P; ++p) {
    const pm_stage_desc& sd = stages[p];
    StageDev& s = L.st[p];
    if (sd.n_ops < 1 || sd.n_ops > PM_MAX_LINEARS || !sd.ops) { err = "stage " + std::to_string(p) + ": n_ops must be in [1, " + std::to_string(PM_MAX_LINEARS) + "]"; return PM_ERR_INVALID_ARG; }
    if (sd.tau_bkwd != 0 || sd.tau_fwd != 2 * (P - (p + 1)) + 1) {
      err = "stage " + std::to_string(p) + ": the tick schedule realises tau_fwd = 2(P-i)+1, tau_bkwd = 0 only";
      return PM_ERR_UNSUPPORTED;
    }
    if (sd.param_offset % PM_ALIGN_ELEMS || sd.param_count % PM_ALIGN_ELEMS) { err = "stage " + std::to_string(p) + ": param_offset/param_count must be multiples of 64"; return PM_ERR_INVALID_ARG; }
    if (sd.param_offset < prev_end) { err = "stage slices must ascend without overlap"; return PM_ERR_INVALID_ARG; }
    uint64_t need = 0;
    pm_status ps = pm_stage_param_count(sd.ops, sd.n_ops, &need);
    if (ps != PM_OK) { err = "stage " + std::to_string(p) + ": bad op list"; return ps; }
    if (sd.param_count < need) { err = "stage " + std::to_string(p) + ": param_count smaller than its ops need"; return PM_ERR_INVALID_ARG; }
    s.tau_f = sd.tau_fwd; s.gap = sd.tau_fwd - sd.tau_bkwd; s.n_lin = sd.n_ops;
    s.depth = s.tau_f + 1; s.xdepth = s.tau_f + 2;
    s.begin = sd.param_offset; s.end = sd.param_offset + sd.param_count;
    prev_end = s.end;
    L.begin64[p] = (uint32_t)(s.begin / 64); L.end64[p] = (uint32_t)(s.end / 64);
    s.max_dim = 0;
    for (int l = 0; l < sd.n_ops; ++l) {
      const pm_op_desc& op = sd.ops[l];
      if (op.kind != PM_OP_LINEAR) { err = "only PM_OP_LINEAR is built"; return PM_ERR_UNSUPPORTED; }
      if (op.n_in < 1 || op.n_out < 1 || op.act < PM_ACT_NONE || op.act > PM_ACT_GELU) { err = "bad Linear description"; return PM_ERR_INVALID_ARG; }
      if (cfg->compute_dtype == PM_BF16 && (op.n_in % 8 || op.n_out % 8)) { err = "PM_BF16 needs Linear dimensions that are multiples of 8"; return PM_ERR_SHAPE; }
      if (prev_out >= 0 && op.n_in != prev_out) { err = "stage " + std::to_string(p) + " op " + std::to_string(l) + ": n_in does not match the previous n_out"; return PM_ERR_SHAPE; }
      prev_out = op.n_out;
      LinDev& ld = s.lin[l];
      ld.n_in = op.n_in; ld.n_out = op.n_out; ld.act = op.act;
      uint64_t wo, bo;
      pm_op_param_offsets(sd.ops, sd.n_ops, l, &wo, &bo);
      ld.w_off = s.begin + wo; ld.b_off = s.begin + bo;
      s.max_dim = std::max(s.max_dim, std::max(op.n_in, op.n_out));
    }
    // rings
    s.x_ring = ring; ring = align_up(ring + (uint64_t)s.xdepth * T * s.lin[0].n_in * esz, 256);
    for (int l = 0; l < s.n_lin; ++l) {
      s.lin[l].z_ring = ring; ring = align_up(ring + (uint64_t)s.depth * T * s.lin[l].n_out * esz, 256);
      if (l < s.n_lin - 1) { s.lin[l].h_ring = ring; ring = align_up(ring + (uint64_t)s.depth * T * s.lin[l].n_out * esz, 256); }
    }
    L.max_lin = std::max(L.max_lin, s.n_lin);
    L.max_dim = std::max(L.max_dim, s.max_dim);
    L.sched[p].tau_f = s.tau_f; L.sched[p].gap = s.gap; L.sched[p].depth = s.depth; L.sched[p].xdepth = s.xdepth;
  }
  for (int p = 0; p < P; ++p) L.sched[p].next_xdepth = p + 1 < P ? L.st[p + 1].xdepth : 0;
  L.ring_bytes = ring;
  L.total = L.st[P - 1].end;
  L.n_in_first = L.st[0].lin[0].n_in;
  L.n_out_last = L.st[P - 1].lin[L.st[P - 1].n_lin - 1].n_out;
  L.loss_cap = cfg->loss_log_capacity > 0 ? cfg->loss_log_capacity : 4096;
  // workspace
  uint64_t w = 0;
  L.off_st = w; w = align_up(w + sizeof(StageDev) * P, 256);
  L.off_sched = w; w = align_up(w + sizeof(StageSched) * P, 256);
  L.off_dyn = w; w = align_up(w + sizeof(StageDyn) * P, 256);
  L.off_nupd = w; w = align_up(w + sizeof(int64_t) * P, 256);
  L.off_b64 = w; w = align_up(w + sizeof(uint32_t) * P, 256);
  L.off_e64 = w; w = align_up(w + sizeof(uint32_t) * P, 256);
  L.off_alpha = w; w = align_up(w + sizeof(double) * (cfg->alpha_by_step ? (uint64_t)cfg->alpha_len : 0), 256);
  L.off_loss = w; w = align_up(w + sizeof(float) * (uint64_t)L.loss_cap, 256);
  L.off_lossred = w; w = align_up(w + 512, 256);
  L.off_tgt = w; w = align_up(w + sizeof(float) * (uint64_t)(P + 1) * T * L.n_out_last, 256);
  L.off_yout = w; w = align_up(w + 2 * T * L.n_out_last * esz, 256);
  L.off_umma = w; w = align_up(w + (cfg->compute_dtype == PM_BF16 ? umma_workspace_bytes(P) : 0), 256);
  for (int p = 0; p < P; ++p) {
    StageDev& s = L.st[p];
    const int n_out_last = s.lin[s.n_lin - 1].n_out;
    s.gin = w; w = align_up(w + 2 * T * n_out_last * esz, 256);
    s.dz = w; w = align_up(w + T * s.max_dim * esz, 256);
    s.dh = w; w = align_up(w + T * s.max_dim * esz, 256);
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
  uint64_t launches = 0;   // kernels enqueued by this context so far
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
    if (ops[l].n_in < 1 || ops[l].n_out < 1) return PM_ERR_INVALID_ARG;
    c = align_up(c + (uint64_t)ops[l].n_in * ops[l].n_out, PM_ALIGN_ELEMS);
    c = align_up(c + (uint64_t)ops[l].n_out, PM_ALIGN_ELEMS);
  }
  *count = c;
  return PM_OK;
}

pm_status pm_op_param_offsets(const pm_op_desc* ops, int32_t n_ops, int32_t op, uint64_t* w_off, uint64_t* b_off) {
  if (!ops || op < 0 || op >= n_ops) return PM_ERR_INVALID_ARG;
  uint64_t c = 0;
  for (int l = 0; l <= op; ++l) {
    uint64_t wo = c;
    c = align_up(c + (uint64_t)ops[l].n_in * ops[l].n_out, PM_ALIGN_ELEMS);
    uint64_t bo = c;
    c = align_up(c + (uint64_t)ops[l].n_out, PM_ALIGN_ELEMS);
    if (l == op) { if (w_off) *w_off = wo; if (b_off) *b_off = bo; }
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
#undef UP
  if (cfg->alpha_by_step) {
    if (cfg->alpha_len < 1) { delete c; return fail(nullptr, PM_ERR_INVALID_ARG, "alpha_len must be >= 1 with alpha_by_step"); }
    e = cudaMemcpyAsync(c->ws + L.off_alpha, cfg->alpha_by_step, sizeof(double) * cfg->alpha_len, cudaMemcpyHostToDevice, c->stream);
    if (e != cudaSuccess) { pm_status r = cuda_fail(nullptr, e, "alpha table upload"); delete c; return r; }
  }
  e = cudaMemsetAsync(c->ws + L.off_nupd, 0, sizeof(int64_t) * P, c->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(c->ws + L.off_dyn, 0, sizeof(StageDyn) * P, c->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(c->ws + L.off_lossred, 0, 512, c->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);   // host tables may go out of scope after this
  if (e != cudaSuccess) { pm_status r = cuda_fail(nullptr, e, "context set-up"); delete c; return r; }

  c->hp = HyperDev{};
  c->hp.optimizer = cfg->optimizer; c->hp.t1 = cfg->t1_enable; c->hp.t2 = cfg->t2_enable; c->hp.n_stages = P;
  c->hp.K = cfg->t1_K > 0 ? cfg->t1_K : 1; c->hp.D = cfg->t2_D; c->hp.alpha_const = cfg->alpha_const;
  c->hp.alpha_tab = cfg->alpha_by_step ? (const double*)(c->ws + L.off_alpha) : nullptr;
  c->hp.alpha_len = cfg->alpha_len;
  c->hp.beta1 = cfg->beta1; c->hp.beta2 = cfg->beta2; c->hp.eps = cfg->eps;

  TickArgs& t = c->ta;
  t.st = (const StageDev*)(c->ws + L.off_st);
  t.dyn = (const StageDyn*)(c->ws + L.off_dyn);
  t.a = c->a; t.ring = (char*)ring; t.ws = c->ws; t.T = cfg->microbatch; t.P = P;
  t.n_in_first = L.n_in_first; t.n_out_last = L.n_out_last;
  t.yout_off = L.off_yout; t.tgt_off = L.off_tgt; t.loss_off = L.off_loss; t.loss_cap = L.loss_cap; t.lossred_off = L.off_lossred;
  t.max_lin = L.max_lin; t.max_dim = L.max_dim;

  if (cfg->compute_dtype == PM_BF16) {
    std::string uerr;
    pm_status us = umma_plan_create(&c->umma, t, c->L.st, c->ws + L.off_umma, c->stream, uerr);
    if (us != PM_OK) { delete c; return fail(nullptr, us, uerr); }
  }
  *out = c;
  return PM_OK;
}

// every call checked here enqueued exactly one kernel
static pm_status check(pm_ctx* ctx, cudaError_t e, const char* what) {
  ctx->launches += 1;
  return e == cudaSuccess ? PM_OK : cuda_fail(ctx, e, what);
}

pm_status pm_forward(pm_ctx* ctx, const void* inputs, const void* targets) {
  if (!ctx) return fail(nullptr, PM_ERR_INVALID_ARG, "null context");
  if (ctx->phase != 0) return fail(ctx, PM_ERR_STATE, "pm_forward called out of order (expected pm_backward or pm_update)");
  if ((inputs == nullptr) != (targets == nullptr)) return fail(ctx, PM_ERR_INVALID_ARG, "inputs and targets must both be given or both be NULL");
  if (inputs && ctx->draining) return fail(ctx, PM_ERR_STATE, "microbatches must be fed on consecutive ticks; the pipeline is already draining");
  const int dt = ctx->cfg.compute_dtype;
  pm_status s;
  if (inputs) ctx->n_fed = ctx->tick + 1; else ctx->draining = true;
  s = check(ctx, launch_schedule((const StageSched*)(ctx->ws + ctx->L.off_sched), (const int64_t*)(ctx->ws + ctx->L.off_nupd),
                                 (StageDyn*)(ctx->ws + ctx->L.off_dyn), ctx->hp, ctx->tick, ctx->n_fed, -1, ctx->stream), "schedule");
  if (s != PM_OK) return s;
  if (inputs) {
    s = check(ctx, launch_ingest(ctx->ta, dt, inputs, (const float*)targets, ctx->tick, ctx->stream), "ingest");
    if (s != PM_OK) return s;
  }
  // forward of every stage whose microbatch exists: s - (i-1) in [0, n_fed)
  if (ctx->tick - (ctx->cfg.n_stages - 1) < ctx->n_fed) {
    for (int l = 0; l < ctx->L.max_lin; ++l) {
      cudaError_t e = dt == PM_F32 ? launch_simt_gemm(ctx->ta, dt, 0, l, ctx->stream)
                                   : umma_launch(ctx->umma, ctx->ta, 0, l, ctx->stream);
      if ((s = check(ctx, e, "forward GEMM")) != PM_OK) return s;
    }
  }
  ctx->phase = 1;
  return PM_OK;
}

pm_status pm_backward(pm_ctx* ctx) {
  if (!ctx) return fail(nullptr, PM_ERR_INVALID_ARG, "null context");
  if (ctx->phase != 1) return fail(ctx, PM_ERR_STATE, "pm_backward must follow pm_forward");
  const int dt = ctx->cfg.compute_dtype;
  const int P = ctx->cfg.n_stages;
  pm_status s;
  // any backward this tick?  stage P runs microbatch tick-P, stage 1 runs tick-(2P-1)
  const bool any = ctx->tick - P >= 0 && ctx->tick - (2 * (int64_t)P - 1) < ctx->n_fed;
  if (any) {
    if ((s = check(ctx, launch_loss(ctx->ta, dt, ctx->stream), "loss")) != PM_OK) return s;
    for (int l = ctx->L.max_lin - 1; l >= 0; --l) {
      if ((s = check(ctx, launch_actbwd(ctx->ta, dt, l, ctx->stream), "activation backward")) != PM_OK) return s;
      cudaError_t e = dt == PM_F32 ? launch_simt_gemm(ctx->ta, dt, 2, l, ctx->stream)
                                   : umma_launch(ctx->umma, ctx->ta, 2, l, ctx->stream);
      if ((s = check(ctx, e, "wgrad GEMM")) != PM_OK) return s;
      e = dt == PM_F32 ? launch_simt_gemm(ctx->ta, dt, 1, l, ctx->stream)
                       : umma_launch(ctx->umma, ctx->ta, 1, l, ctx->stream);
      if ((s = check(ctx, e, "dgrad GEMM")) != PM_OK) return s;
    }
  }
  ctx->phase = 2;
  return PM_OK;
}

pm_status pm_update(pm_ctx* ctx) {
  if (!ctx) return fail(nullptr, PM_ERR_INVALID_ARG, "null context");
  if (ctx->phase != 2) return fail(ctx, PM_ERR_STATE, "pm_update must follow pm_backward");
  const int P = ctx->cfg.n_stages;
  const bool any = ctx->tick - P >= 0 && ctx->tick - (2 * (int64_t)P - 1) < ctx->n_fed;
  if (any) {
    cudaError_t e = launch_update(ctx->a, (const uint32_t*)(ctx->ws + ctx->L.off_b64), (const uint32_t*)(ctx->ws + ctx->L.off_e64),
                                  (const StageDyn*)(ctx->ws + ctx->L.off_dyn), (int64_t*)(ctx->ws + ctx->L.off_nupd), P,
                                  ctx->L.total / 64, ctx->cfg.optimizer, ctx->cfg.beta1, ctx->cfg.beta2, ctx->cfg.eps, ctx->stream);
    pm_status s = check(ctx, e, "update");
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
  int* w = umma_status_word(ctx->umma);
  if (!w) return PM_OK;
  int code = 0;
  cudaError_t e = cudaMemcpy(&code, w, sizeof(int), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "status read-back");
  if (code != 0) return fail(ctx, PM_ERR_TIMEOUT, "a bounded device-side wait expired in a GEMM kernel (role code " + std::to_string(code) + ")");
  return PM_OK;
}

pm_status pm_get_bookkeeping(pm_ctx* ctx, int32_t stage, int64_t* out8) {
  if (!ctx || !out8) return fail(ctx, PM_ERR_INVALID_ARG, "null argument");
  if (stage < 0 || stage >= ctx->cfg.n_stages) return fail(ctx, PM_ERR_INVALID_ARG, "stage out of range");
  StageDyn d;
  int64_t n = 0;
  cudaError_t e = cudaStreamSynchronize(ctx->stream);
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
  // microbatch t's loss is computed in tick t+P; ticks completed so far = ctx->tick
  const int64_t done = std::min<int64_t>(ctx->n_fed, ctx->tick - P);
  if (first_mb + n > done) return fail(ctx, PM_ERR_INVALID_ARG, "loss of a microbatch that has not finished was requested");
  if (done - first_mb > ctx->L.loss_cap) return fail(ctx, PM_ERR_INVALID_ARG, "requested losses have left the device log");
  cudaError_t e = cudaStreamSynchronize(ctx->stream);
  for (int64_t i = 0; i < n && e == cudaSuccess; ++i)
    e = cudaMemcpy(host_out + i, ctx->ws + ctx->L.off_loss + sizeof(float) * ((first_mb + i) % ctx->L.loss_cap), sizeof(float), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "loss read-back");
  if (pm_status ds = check_device_status(ctx)) return ds;
  return PM_OK;
}

uint64_t pm_launch_count(pm_ctx* ctx) { return ctx ? ctx->launches : 0; }

const char* pm_last_error(pm_ctx* ctx) { return ctx ? ctx->err.c_str() : g_error.c_str(); }

void pm_destroy(pm_ctx* ctx) {
  if (!ctx) return;
  umma_plan_destroy(ctx->umma);
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
  const uint64_t need = pm_update_flat_workspace_bytes(n_stages);
  if (!workspace || workspace_bytes < need) return fail(nullptr, PM_ERR_NOMEM, "workspace too small: need " + std::to_string(need) + " bytes");
  const uint64_t P = (uint64_t)n_stages;
  std::vector<char> host(need, 0);
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
    uint64_t end = align_up(stage_offsets[i] + stage_counts[i], PM_ALIGN_ELEMS);
    if (end > arenas->count) return fail(nullptr, PM_ERR_NOMEM, "stage slice exceeds the arenas");
    prev_end = end;
    sc[i] = StageSched{tau_fwd[i], tau_fwd[i] - tau_bkwd[i], 1, 1, 0, 0};
    b64[i] = (uint32_t)(stage_offsets[i] / 64);
    e64[i] = (uint32_t)(end / 64);
  }
  cudaStream_t st = (cudaStream_t)stream;
  char* ws = (char*)workspace;
  cudaError_t e = cudaMemcpyAsync(ws, host.data(), need, cudaMemcpyHostToDevice, st);
  if (e != cudaSuccess) return cuda_fail(nullptr, e, "stage table upload");
  HyperDev hp{};
  hp.optimizer = cfg->optimizer; hp.t1 = cfg->t1_enable; hp.t2 = cfg->t2_enable; hp.n_stages = n_stages;
  hp.K = cfg->t1_K > 0 ? cfg->t1_K : 1; hp.D = cfg->t2_D;
  hp.alpha_const = cfg->alpha_by_step ? cfg->alpha_by_step[k < cfg->alpha_len ? k : cfg->alpha_len - 1] : cfg->alpha_const;
  hp.alpha_tab = nullptr; hp.alpha_len = 0;
  hp.beta1 = cfg->beta1; hp.beta2 = cfg->beta2; hp.eps = cfg->eps;
  e = launch_schedule((const StageSched*)(ws + off_sched), (const int64_t*)(ws + off_nupd), (StageDyn*)(ws + off_dyn), hp, 0, 0, k, st);
  if (e != cudaSuccess) return cuda_fail(nullptr, e, "schedule");
  ArenasDev a{arenas->w, arenas->m, arenas->s, arenas->delta, arenas->grad, (__nv_bfloat16*)arenas->w_lp, arenas->count};
  e = launch_update(a, (const uint32_t*)(ws + off_b), (const uint32_t*)(ws + off_e), (const StageDyn*)(ws + off_dyn),
                    (int64_t*)(ws + off_nupd), n_stages, e64[n_stages - 1], cfg->optimizer, cfg->beta1, cfg->beta2, cfg->eps, st);
  if (e != cudaSuccess) return cuda_fail(nullptr, e, "update");
  return PM_OK;
}

}  // extern "C"
