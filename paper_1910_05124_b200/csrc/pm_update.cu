// Tick scheduler and the fused multi-tensor PipeMare update.
//
// The update is a pure HBM stream: per parameter it reads g, w, m, delta (and s for
// Adam) and writes w, m, delta (and s) in fp32 plus a bfloat16 copy of w: 30 bytes per
// parameter for momentum SGD, 38 for Adam.  One launch covers every stage; the stage
// that owns a 64-element group is found by binary search in shared memory, and that
// stage's scalars (T1 step size, T2 decay, Adam bias corrections) come from the table
// the scheduler wrote for this tick.
//
// Arithmetic order (each operation rounded once in fp32, no fused multiply-add, so that
// results can be reproduced bit for bit by any IEEE implementation):
//   SGD-m (Appendix B.3):  v' = beta*v - alpha*g ;  w' = w + v'
//   Adam:  m' = b1*m + (1-b1)*g ;  s' = b2*s + (1-b2)*(g*g) ;
//          w' = w - (alpha*(m'/bc1)) / (sqrt(s'/bc2) + eps)
//   T2 (Section 3.2):      delta' = gamma*delta + (1-gamma)*(w' - w)
#include "pm_update.cuh"
#include "pm_update_math.cuh"

namespace pm {

// ---- scheduler -------------------------------------------------------------------------------
//
// Tick s, stage i (1-based): forward of the microbatch that entered at tick s-(i-1); backward and update of
// the one that entered at tick s-(2P-i) (microbatch = entry tick, except during a synchronous warm-up).  T1 (Eq. 2): alpha_i = alpha_base(k) / tau_i^p, p = 1 - min(k/K, 1).
// T2: gamma_i = D^(1/(tau_fwd,i - tau_bkwd,i)).  Scalars are evaluated in double and rounded to
// float once.
// Per-stage state of one tick: forward microbatch a and backward microbatch b (-1: idle), `ver` updates applied to the
// stage so far, the version `fver` its forward reads; k >= 0 activates the update with that index.
__device__ StageDyn make_dyn(const StageSched& s, const HyperDev& hp, int64_t tick, int64_t a, int64_t b, int64_t k,
                             int64_t ver, int64_t fver, bool slots, int64_t kb = -2) {
  StageDyn d;
  d.tick = tick;
  d.accum = 0; d._pad2 = 0;
  d.rc_uslot = -1; d.rc_shift = 0; d.r_ver = fver; d.rc_gap = 0.f; d.g_shift = 0;
  if (kb == -2) kb = b;                               // update index the microbatch in backward belongs to (N = 1: itself)
  const bool fa = a >= 0, ba = b >= 0;
  d.f_mb = a; d.b_mb = b; d.k = k;
  d.f_slot = (fa && slots) ? (int32_t)(a % s.depth) : 0;
  d.f_xslot = (fa && slots) ? (int32_t)(a % s.xdepth) : 0;
  d.f_next_xslot = (fa && slots && s.next_xdepth > 0) ? (int32_t)(a % s.next_xdepth) : 0;
  d.b_slot = (ba && slots) ? (int32_t)(b % s.depth) : 0;
  d.b_xslot = (ba && slots) ? (int32_t)(b % s.xdepth) : 0;
  d.gin_rslot = s.gin_depth > 0 ? (int32_t)((tick + s.gin_depth - 1) % s.gin_depth) : 0;
  d.prev_wslot = s.prev_gin_depth > 0 ? (int32_t)(tick % s.prev_gin_depth) : 0;
  d.gmem_slot = (s.gmem_depth > 0 && ba) ? (int32_t)(b % s.gmem_depth) : 0;
  d.skip_wslot = s.skip_dst_depth > 0 ? (int32_t)(tick % s.skip_dst_depth) : 0;
  d.skip_rslot = s.skip_depth > 0 ? (int32_t)((tick + 1) % s.skip_depth) : 0;
  d.b_next_xslot = (ba && slots && s.next_xdepth > 0) ? (int32_t)(b % s.next_xdepth) : 0;
  d.f_ver = fver;
  d.b_ver = ver;
  // version rings (microbatch-major order): version v sits in slot v % vdepth
  d.f_vslot = s.vdepth > 1 ? (int32_t)(fver % s.vdepth) : 0;
  d.u_vslot = s.vdepth > 1 ? (int32_t)((ver + 1) % s.vdepth) : 0;
  d.lp_shift = hp.mb_major ? (int64_t)(s.v_ring / (uint64_t)hp.lp_elem) + (int64_t)d.u_vslot * (int64_t)s.count - (int64_t)s.begin : 0;
  if (hp.mb_major && s.rdepth > 0) {
    // corrected recompute weights of version ver + 1: slot vdepth + (ver + 1) % rdepth of the same rings
    d.rc_uslot = s.vdepth + (int32_t)((ver + 1) % s.rdepth);
    d.rc_shift = (int64_t)(s.v_ring / (uint64_t)hp.lp_elem) + (int64_t)d.rc_uslot * (int64_t)s.count - (int64_t)s.begin;
    d.rc_gap = (float)(s.tau_f - s.tau_r);
  }
  d.active_update = k >= 0 ? 1 : 0;
  d.alpha = 0.f; d.gamma = 0.f; d.one_minus_gamma = 1.f; d.bc1 = 1.f; d.bc2 = 1.f; d.use_delta = 0;
  const int64_t kk = k >= 0 ? k : kb;                 // the update index of the microbatch in backward
  if (kk >= 0) {
    double base = hp.alpha_const;
    if (hp.alpha_tab != nullptr) base = hp.alpha_tab[kk < hp.alpha_len ? kk : hp.alpha_len - 1];
    double alpha = base;
    // warm-up microbatches (Section 4) are synchronous: standard step size, no correction, delta left alone; the T1
    // annealing counts from the first PipeMare step
    const bool sync = kk < hp.warm;
    if (hp.t1 && !sync) {
      double r = (double)(kk - hp.warm) / (double)hp.K;
      double p = 1.0 - (r < 1.0 ? r : 1.0);
      int tau = s.tau_f > 1 ? s.tau_f : 1;
      alpha = base / pow((double)tau, p);
    }
    d.alpha = (float)alpha;
    if (hp.t2 && s.gap > 0 && !sync) {
      d.gamma = (float)pow(hp.D, 1.0 / (double)s.gap);
      d.one_minus_gamma = 1.0f - d.gamma;
      d.use_delta = 1;
    }
    if (hp.optimizer == PM_ADAM) {
      d.bc1 = (float)(1.0 - pow((double)hp.beta1, (double)(kk + 1)));
      d.bc2 = (float)(1.0 - pow((double)hp.beta2, (double)(kk + 1)));
    }
  }
  return d;
}

__global__ void schedule_kernel(const StageSched* __restrict__ sched, const int64_t* __restrict__ nupd,
                                StageDyn* __restrict__ dyn, HyperDev hp, int64_t tick, int64_t n_fed,
                                int64_t flat_k) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= hp.n_stages) return;
  const StageSched s = sched[i];
  const int P = hp.n_stages;
  const int64_t ver = nupd[i];
  if (flat_k >= 0) { dyn[i] = make_dyn(s, hp, tick, -1, -1, flat_k, ver, ver, false); return; }
  int64_t a = mb_at_tick(tick - i, hp.warm, hp.period, hp.entry_period);
  int64_t b = mb_at_tick(tick - (2 * (int64_t)P - (i + 1)), hp.warm, hp.period, hp.entry_period);
  if (!(a >= 0 && a < n_fed)) a = -1;
  if (!(b >= 0 && b < n_fed)) b = -1;
  // One microbatch per tick: the weights a stage holds ARE version max(0, a - tau).  With a microbatch only every E
  // ticks more updates have landed by the time a forward runs, and the forward takes the version Table 1's delay
  // names from the stage's queue.
  int64_t fver = ver;
  if (hp.entry_period > 1 && a >= 0) { fver = a - s.tau_f; if (fver < 0) fver = 0; }
  dyn[i] = make_dyn(s, hp, tick, a, b, b, ver, fver, true);
}

cudaError_t launch_schedule(const StageSched* sched, const int64_t* nupd, StageDyn* dyn, HyperDev hp,
                            int64_t tick, int64_t n_fed, int64_t flat_k, cudaStream_t stream) {
  int threads = 128;
  int blocks = (hp.n_stages + threads - 1) / threads;
  schedule_kernel<<<blocks, threads, 0, stream>>>(sched, nupd, dyn, hp, tick, n_fed, flat_k);
  return cudaGetLastError();
}

// Microbatch-major order (the paper's own statement of the method, Section 2.1: a queue of weight versions per
// stage).  Microbatch t runs alone: stage i's forward in sub-tick i, its backward in sub-tick 2P-1-i, on the same
// mailbox-slot arithmetic as a pipeline tick (virtual tick = 2P t + sub-tick).  The forward reads version
// max(0, t - tau_fwd,i) from the stage's version ring (during a synchronous warm-up version t, afterwards nothing
// older than the end of the warm-up), the backward the live weights (version t).  Table v in 0..2P-1 serves the
// launches of sub-tick v; table 2P marks every stage in backward with its own backward sub-tick's slots and an
// active update: it serves the grouped weight-gradient launch and the fused update.
__global__ void schedule_mb_kernel(const StageSched* __restrict__ sched, StageDyn* __restrict__ tables, HyperDev hp, int64_t t,
                                   const int32_t* __restrict__ delays, const int64_t* __restrict__ nupd) {
  const int P = hp.n_stages;
  const int i = blockIdx.x * blockDim.x + threadIdx.x, v = blockIdx.y;
  if (i >= P) return;
  const StageSched s = sched[i];
  const int64_t base = 2 * (int64_t)P * t;
  // N microbatches per update (Section 2.1): versions, delays and step indices count updates; microbatch t belongs to
  // update u = t / N, every microbatch of a minibatch reads the same versions, the update follows the N-th
  const int64_t N = hp.n_micro > 1 ? hp.n_micro : 1;
  const int64_t u = t / N;
  int64_t fver = u - s.tau_f;
  if (u < hp.warm) fver = u; else if (fver < hp.warm) fver = hp.warm;
  if (fver < 0) fver = 0;
  StageDyn d;
  if (hp.stochastic > 0) {
    // Stage-wise stochastic delays (Appendix E): forward and backward of microbatch t on the stage's current weights
    // (version = updates it has applied); the update table activates the stage when the gradient of microbatch
    // t - delay exists, points it at that microbatch's slot of the gradient ring and indexes its step-size schedule,
    // T1 annealing and bias corrections by the stage's own update count
    const int64_t ver = nupd[i];
    const int64_t src = t - (int64_t)delays[i];
    if (v < 2 * P) d = make_dyn(s, hp, base + v, v == i ? t : -1, v == 2 * P - 1 - i ? t : -1, -1, ver, ver, true, ver);
    else {
      d = make_dyn(s, hp, base + 2 * P - 1 - i, -1, t, src >= 0 ? ver : -1, ver, ver, true, ver);
      d.g_shift = src >= 0 ? (src % hp.stochastic) * (int64_t)hp.total : 0;
    }
    d.r_ver = src >= 0 ? src : -1;
    tables[(size_t)v * P + i] = d;
    return;
  }
  // PipeMare Recompute (Appendix A.2, Appendix D): the version the recomputation reads, clamped like the forward's
  int64_t rver = u - s.tau_r;
  if (u < hp.warm) rver = u; else if (rver < hp.warm) rver = hp.warm;
  if (rver < 0) rver = 0;
  const int seg = hp.segment > 0 ? i / hp.segment : 0;
  if (v < 2 * P) d = make_dyn(s, hp, base + v, v == i ? t : -1, v == 2 * P - 1 - i ? t : -1, -1, u, fver, true, u);
  else if (v == 2 * P) d = make_dyn(s, hp, base + 2 * P - 1 - i, -1, t, (t % N == N - 1) ? u : -1, u, fver, true, u);
  else if (v == 2 * P + 1) {
    // the stage's forward entry again (same virtual tick, so the same mailbox and skip slots), reading the recompute
    // weights: the corrected queue behind the version slots when the stage keeps one, else the plain version
    d = make_dyn(s, hp, base + i, t, -1, -1, u, fver, true, u);
    d.f_vslot = s.rdepth > 0 ? s.vdepth + (int32_t)(rver % s.rdepth) : (s.vdepth > 1 ? (int32_t)(rver % s.vdepth) : 0);
  } else {
    // backward entries of one segment alone: the grouped weight-gradient launch that follows the segment's backward
    const bool mine = seg == v - (2 * P + 2);
    d = make_dyn(s, hp, base + 2 * P - 1 - i, -1, mine ? t : -1, -1, u, fver, true, u);
  }
  d.r_ver = rver;
  if (hp.materialize && (v >= 2 * P || v == 2 * P - 1 - i)) {
    // a backward entry: its version slot is the one the update filled with w - tau delta of the live version (stages that
    // keep none -- no gap, or T2 off -- read the live version itself)
    d.f_vslot = s.rdepth > 0 ? s.vdepth : (s.vdepth > 1 ? (int32_t)(u % s.vdepth) : 0);
  }
  d.accum = (t % N != 0) ? 1 : 0;
  tables[(size_t)v * P + i] = d;
}

cudaError_t launch_schedule_mb(const StageSched* sched, StageDyn* tables, HyperDev hp, int64_t t, cudaStream_t stream,
                               const int32_t* delays, const int64_t* nupd) {
  const int threads = 128;
  dim3 grid((hp.n_stages + threads - 1) / threads, mb_table_count(hp.n_stages, hp.segment));
  schedule_mb_kernel<<<grid, threads, 0, stream>>>(sched, tables, hp, t, delays, nupd);
  return cudaGetLastError();
}

// ---- fused update ------------------------------------------------------------------------------

__device__ __forceinline__ float4 ld_stream(const float* p) { return __ldcs(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ void st_stream(float* p, float4 v) { __stcs(reinterpret_cast<float4*>(p), v); }

constexpr int kUpdThreads = 256;
constexpr int kUpdUnroll = 2;      // float4 groups per thread per array in flight

// LP: operand-type copy of the new weights: 0 none, 1 bfloat16, 2 float (a version-ring slot of fp32 operands);
// element e of the arenas goes to lp_base[lp_shift + e], lp_shift from the stage's table entry (0: the w_lp arena)
template <int OPT, int LP>
__global__ void __launch_bounds__(kUpdThreads, 3)
update_kernel(ArenasDev a, void* __restrict__ lp_base, const uint32_t* __restrict__ begin64, const uint32_t* __restrict__ end64,
              const StageDyn* __restrict__ dyn, int64_t* __restrict__ nupd, int n_stages, uint64_t total_vec4,
              float beta1, float beta2, float eps, uint64_t first_vec4, const uint32_t* __restrict__ skip_b64, const uint32_t* __restrict__ skip_e64,
              const float* __restrict__ gsrc) {
  extern __shared__ uint32_t sm_bounds[];           // [n_stages] begins, then [n_stages] ends, then the skipped ranges' begins and ends
  uint32_t* sb = sm_bounds;
  uint32_t* se = sm_bounds + n_stages;
  // ranges (one per stage, in 64-element groups) that another kernel has updated already: the Linear matrices, when the
  // weight-gradient GEMM applies the update in its epilogue
  uint32_t* kb = sm_bounds + 2 * n_stages;
  uint32_t* ke = sm_bounds + 3 * n_stages;
  const bool skip = skip_b64 != nullptr;
  for (int i = threadIdx.x; i < n_stages; i += blockDim.x) {
    sb[i] = begin64[i]; se[i] = end64[i];
    kb[i] = skip ? skip_b64[i] : 0u; ke[i] = skip ? skip_e64[i] : 0u;
  }
  __syncthreads();
  const float omb1 = __fsub_rn(1.0f, beta1), omb2 = __fsub_rn(1.0f, beta2);
  const uint64_t stride = (uint64_t)gridDim.x * kUpdThreads * kUpdUnroll;
  for (uint64_t base = first_vec4 + (uint64_t)blockIdx.x * kUpdThreads * kUpdUnroll; base < total_vec4; base += stride) {
    if (skip) {
      // the whole span of this block lies inside a skipped range (and past the stage's first group): nothing to do
      const uint32_t g0 = (uint32_t)(base >> 4), g1 = (uint32_t)((base + (uint64_t)kUpdThreads * kUpdUnroll - 1) >> 4);
      int lo = 0, hi = n_stages - 1;
      while (lo < hi) { int mid = (lo + hi + 1) >> 1; if (sb[mid] <= g0) lo = mid; else hi = mid - 1; }
      if (kb[lo] <= g0 && g1 < ke[lo] && g0 > sb[lo]) continue;
    }
    uint64_t v[kUpdUnroll];
    int stage[kUpdUnroll];
    UpdScalars sc[kUpdUnroll];
    float4 g[kUpdUnroll], w[kUpdUnroll], m[kUpdUnroll], dl[kUpdUnroll], s[kUpdUnroll];
#pragma unroll
    for (int u = 0; u < kUpdUnroll; ++u) {
      v[u] = base + (uint64_t)u * kUpdThreads + threadIdx.x;
      stage[u] = -1;
      if (v[u] < total_vec4) {
        uint32_t e64 = (uint32_t)(v[u] >> 4);
        int lo = 0, hi = n_stages - 1;               // largest i with sb[i] <= e64
        while (lo < hi) { int mid = (lo + hi + 1) >> 1; if (sb[mid] <= e64) lo = mid; else hi = mid - 1; }
        if (sb[lo] <= e64 && e64 < se[lo] && dyn[lo].active_update) {
          if (skip && kb[lo] <= e64 && e64 < ke[lo]) {                     // updated elsewhere; the stage's counter is still kept here
            if (e64 == sb[lo] && (v[u] & 15) == 0) nupd[lo] += 1;
          } else stage[u] = lo;
        }
      }
      if (stage[u] >= 0) {
        const uint64_t e = v[u] * 4;
        const StageDyn& d = dyn[stage[u]];
        g[u] = ld_stream(gsrc + (d.g_shift + (int64_t)e));
        w[u] = ld_stream(a.w + e);
        m[u] = ld_stream(a.m + e);
        sc[u].alpha = d.alpha; sc[u].gamma = d.gamma; sc[u].omg = d.one_minus_gamma;
        sc[u].bc1 = d.bc1; sc[u].bc2 = d.bc2; sc[u].use_delta = d.use_delta;
        if (LP != 0) { sc[u].lp_shift = d.lp_shift; sc[u].rc_shift = d.rc_uslot >= 0 ? d.rc_shift : -1; sc[u].rc_gap = d.rc_gap; }
        if (sc[u].use_delta || (LP != 0 && sc[u].rc_shift >= 0)) dl[u] = ld_stream(a.delta + e);
        if (OPT == PM_ADAM) s[u] = ld_stream(a.s + e);
      }
    }
#pragma unroll
    for (int u = 0; u < kUpdUnroll; ++u) {
      if (stage[u] < 0) continue;
      const uint64_t e = v[u] * 4;
      float4 wn;
      wn.x = upd_one<OPT>(g[u].x, w[u].x, m[u].x, s[u].x, dl[u].x, sc[u], beta1, beta2, omb1, omb2, eps);
      wn.y = upd_one<OPT>(g[u].y, w[u].y, m[u].y, s[u].y, dl[u].y, sc[u], beta1, beta2, omb1, omb2, eps);
      wn.z = upd_one<OPT>(g[u].z, w[u].z, m[u].z, s[u].z, dl[u].z, sc[u], beta1, beta2, omb1, omb2, eps);
      wn.w = upd_one<OPT>(g[u].w, w[u].w, m[u].w, s[u].w, dl[u].w, sc[u], beta1, beta2, omb1, omb2, eps);
      st_stream(a.w + e, wn);
      st_stream(a.m + e, m[u]);
      if (OPT == PM_ADAM) st_stream(a.s + e, s[u]);
      if (sc[u].use_delta) st_stream(a.delta + e, dl[u]);
      if (LP == 1) {
        __nv_bfloat162 lo2 = __floats2bfloat162_rn(wn.x, wn.y);
        __nv_bfloat162 hi2 = __floats2bfloat162_rn(wn.z, wn.w);
        uint2 packed;
        packed.x = *reinterpret_cast<uint32_t*>(&lo2);
        packed.y = *reinterpret_cast<uint32_t*>(&hi2);
        *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(lp_base) + (sc[u].lp_shift + (int64_t)e)) = packed;   // re-read by a later forward: default caching
      } else if (LP == 2) {
        *reinterpret_cast<float4*>(reinterpret_cast<float*>(lp_base) + (sc[u].lp_shift + (int64_t)e)) = wn;
      }
      if (LP != 0 && sc[u].rc_shift >= 0) {
        // T2 for recompute (Appendix D): the weights a recomputation tau_recomp updates from now reads, corrected with the
        // accumulator as it stands with this version: w' - (tau_fwd - tau_recomp) * delta'
        const float gp = sc[u].rc_gap;
        float4 r;
        r.x = __fsub_rn(wn.x, __fmul_rn(gp, dl[u].x)); r.y = __fsub_rn(wn.y, __fmul_rn(gp, dl[u].y));
        r.z = __fsub_rn(wn.z, __fmul_rn(gp, dl[u].z)); r.w = __fsub_rn(wn.w, __fmul_rn(gp, dl[u].w));
        if (LP == 1) {
          __nv_bfloat162 lo2 = __floats2bfloat162_rn(r.x, r.y);
          __nv_bfloat162 hi2 = __floats2bfloat162_rn(r.z, r.w);
          uint2 packed;
          packed.x = *reinterpret_cast<uint32_t*>(&lo2);
          packed.y = *reinterpret_cast<uint32_t*>(&hi2);
          *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(lp_base) + (sc[u].rc_shift + (int64_t)e)) = packed;
        } else {
          *reinterpret_cast<float4*>(reinterpret_cast<float*>(lp_base) + (sc[u].rc_shift + (int64_t)e)) = r;
        }
      }
      if ((uint32_t)(v[u] >> 4) == sb[stage[u]] && (v[u] & 15) == 0) nupd[stage[u]] += 1;
    }
  }
}

cudaError_t launch_update(ArenasDev a, const uint32_t* begin64, const uint32_t* end64, const StageDyn* dyn,
                          int64_t* nupd, int n_stages, uint64_t total64, int optimizer, float beta1, float beta2,
                          float eps, cudaStream_t stream, void* lp_base, int lp_elem, uint64_t first64,
                          const uint32_t* skip_b64, const uint32_t* skip_e64, const float* gsrc) {
  if (total64 == 0 || n_stages == 0 || first64 >= total64) return cudaSuccess;
  uint64_t total_vec4 = total64 * 16;
  const uint64_t first_vec4 = first64 * 16;
  uint64_t per_block = (uint64_t)kUpdThreads * kUpdUnroll;
  uint64_t need = (total_vec4 - first_vec4 + per_block - 1) / per_block;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  uint64_t cap = (uint64_t)sms * 8;                 // whole waves of resident blocks
  int blocks = (int)(need < cap ? need : cap);
  size_t smem = sizeof(uint32_t) * 4 * (size_t)n_stages;
  // the operand-type copy: the w_lp arena (bfloat16) unless the caller names a version ring and its element size
  if (lp_base == nullptr) { lp_base = a.w_lp; lp_elem = 2; }
  if (gsrc == nullptr) gsrc = a.grad;
  const int lp = lp_base == nullptr ? 0 : (lp_elem == 4 ? 2 : 1);
#define PM_UPD(OPT, LP) update_kernel<OPT, LP><<<blocks, kUpdThreads, smem, stream>>>(a, lp_base, begin64, end64, dyn, nupd, n_stages, total_vec4, beta1, beta2, eps, first_vec4, skip_b64, skip_e64, gsrc)
  if (optimizer == PM_SGDM) { if (lp == 0) PM_UPD(PM_SGDM, 0); else if (lp == 1) PM_UPD(PM_SGDM, 1); else PM_UPD(PM_SGDM, 2); }
  else { if (lp == 0) PM_UPD(PM_ADAM, 0); else if (lp == 1) PM_UPD(PM_ADAM, 1); else PM_UPD(PM_ADAM, 2); }
#undef PM_UPD
  return cudaGetLastError();
}

// ---- fp32 copies of the small forward-read tensors into the version rings -------------------------------------
// With bfloat16 operands the forward pass still reads biases and LayerNorm parameters in fp32; in microbatch-major
// order their versions sit in a ring of their own, filled here from the master weights after every update.
__global__ void __launch_bounds__(128) push_small_kernel(const float* __restrict__ w, const float* __restrict__ delta, char* __restrict__ ring,
                                                         const SmallSeg* __restrict__ segs, int n_segs, const StageDyn* __restrict__ dyn, int slot_override) {
  for (int sg = blockIdx.x; sg < n_segs; sg += gridDim.x) {
    const SmallSeg g = segs[sg];
    if (slot_override < 0 && !dyn[g.stage].active_update) continue;          // the stage was not updated this tick
    const int slot = slot_override >= 0 ? slot_override : dyn[g.stage].u_vslot;
    float* base = reinterpret_cast<float*>(ring + g.ring_off);
    float* dst = base + (uint64_t)slot * g.slot_stride;
    const float* src = w + g.arena_off;
    // corrected recompute weights of the same version (T2 for recompute, Appendix D): w - (tau_fwd - tau_recomp) * delta
    const int rslot = g.rc_base < 0 ? -1 : (slot_override >= 0 ? g.rc_base + slot_override : dyn[g.stage].rc_uslot);
    float* rdst = rslot >= 0 ? base + (uint64_t)rslot * g.slot_stride : nullptr;
    const float gap = (rslot >= 0 && slot_override < 0) ? dyn[g.stage].rc_gap : 0.f;
    const float* dl = delta + g.arena_off;
    for (uint32_t i = threadIdx.x * 4; i < g.count; i += blockDim.x * 4) {
      const float4 v = *reinterpret_cast<const float4*>(src + i);
      *reinterpret_cast<float4*>(dst + i) = v;
      if (rdst) {
        float4 r = v;
        if (slot_override < 0) {
          const float4 d4 = *reinterpret_cast<const float4*>(dl + i);
          r.x = __fsub_rn(v.x, __fmul_rn(gap, d4.x)); r.y = __fsub_rn(v.y, __fmul_rn(gap, d4.y));
          r.z = __fsub_rn(v.z, __fmul_rn(gap, d4.z)); r.w = __fsub_rn(v.w, __fmul_rn(gap, d4.w));
        }
        *reinterpret_cast<float4*>(rdst + i) = r;
      }
    }
  }
}

cudaError_t launch_push_small(const float* w, const float* delta, char* ring, const SmallSeg* segs, int n_segs, const StageDyn* dyn,
                              int slot_override, cudaStream_t stream) {
  if (n_segs == 0) return cudaSuccess;
  push_small_kernel<<<n_segs < 1184 ? n_segs : 1184, 128, 0, stream>>>(w, delta, ring, segs, n_segs, dyn, slot_override);
  return cudaGetLastError();
}

}  // namespace pm
