// Shared device-side tables and small helpers of the PipeMare library.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "pipemare.h"

namespace pm {

enum { PRE_NONE = 0, PRE_EMBED = 1, PRE_LN = 2 };
enum { POST_NONE = 0, POST_ATTENTION = 1, POST_SKIP_OUT = 2, POST_RESIDUAL = 3, POST_CROSS_ATTENTION = 4 };
// LF_ACT_FROM_Y: a ReLU whose pre-activation is not stashed: the backward takes the mask from the stashed output
// (y > 0 exactly where z > 0), which the next Linear keeps for its weight gradient anyway
// LF_DZ_FUSED: a ReLU at the end of a stage whose output is the next stage's stashed input (bf16 tensor-core path): the
// next stage's dgrad epilogue applies the mask (its own stashed input > 0) to the gradient it sends back, so this
// Linear receives dz itself and its backward pass treats it as a Linear without activation
enum { LF_WRITE_Z = 1, LF_WRITE_Y = 2, LF_OUT_F32 = 4, LF_ACT_FROM_Y = 8, LF_DZ_FUSED = 16 };

// Static description of one Linear inside a stage (device copy).
struct LinDev {
  int32_t n_in, n_out, act;
  int32_t flags;              // LF_*: which of z (pre-activation stash), y (activation) the forward writes; fp32 logits
  uint64_t w_off, b_off;      // element offsets into the flat arenas
  uint64_t z_ring;            // byte offset in the ring arena of z[depth][T*n_out] (pre-activation / q,k,v stash)
  uint64_t h_ring;            // byte offset of this Linear's output stash h[depth][T*n_out] (unused for the last Linear)
  uint32_t b_soff;            // offset of the bias inside a slot of the stage's small-tensor version ring
  uint32_t _pad;
};

// Static description of one stage (device copy).  A stage is [pre-op] Linear{1..4} [post-op]:
//   pre : embedding (+ positions) | LayerNorm | none        post: attention | skip_out | residual | none
struct StageDev {
  int32_t tau_f, gap;         // tau_fwd, tau_fwd - tau_bkwd
  int32_t n_lin;
  int32_t depth;              // slots of the stash rings = tau_f + 1
  int32_t xdepth;             // slots of the main-input ring = tau_f + 2 (it doubles as the forward mailbox)
  int32_t max_dim;
  int32_t pre, post;
  int32_t n_heads, seq_len, vocab;
  int32_t d_in;               // width of the main input (= width of u, the first Linear's input)
  int32_t d_out_main;         // width of the main output handed to the next stage
  int32_t causal;             // attention: keys after the query are masked
  int32_t skip_hop;           // emitting stage: the skip tensor goes to stage p + skip_hop (0: emits none)
  int32_t skip_depth;         // receiving stage: slots of skip_in = hop + 1, slot = writer's tick % skip_depth
  int32_t gin_depth;          // slots of gin: 3, or 4 when a stage two positions back reads it as its skip gradient
  int32_t from_memory;        // LayerNorm input (and its backward output) is the memory, not the main stream
  int32_t emit_memory;        // residual stage whose output is the memory; its incoming gradient is the memory gradient
  int32_t mem_first;          // from_memory stage that runs its backward first (the last one): it stores, the others add
  int32_t ids_stream;         // embedding: which input stream (0, 1)
  int32_t ids_depth;          // embedding: slots of ids_ring, slot = microbatch % ids_depth
  int32_t mask_dx;            // the gradient this stage's first Linear sends to the previous stage is masked with (own input > 0):
                              // the previous stage ends in a ReLU whose backward is fused here (LF_DZ_FUSED)
  int32_t vdepth;             // weight versions the forward pass can reach: 1 (the live weights, tick-major) or tau_f + 1
  uint32_t small_count;       // fp32 elements of a slot of s_ring (biases, LayerNorm gain and bias), a multiple of 64
  uint32_t g_soff, beta_soff; // offsets of LayerNorm gain / bias inside a slot of s_ring
  int32_t tau_r;              // PipeMare Recompute: delay of the weights the recomputation reads (= tau_f: nothing is recomputed)
  int32_t rdepth;             // slots of the queue of T2-corrected recompute weights behind the vdepth version slots (0: none;
                              // the recomputation then reads plain versions)
  int32_t _pad;
  uint64_t begin, end;        // padded element range of the stage's parameters in the arenas
  // Queue of weight versions (Section 2.1: the forward pass of microbatch t reads the weights after t - tau_fwd
  // updates), microbatch-major order only.  v_ring: [vdepth][end - begin] copies of the stage's slice in the GEMM
  // operand type (what the forward GEMM and the embedding read); s_ring: [vdepth][small_count] fp32 copies of the
  // tensors the forward pass reads in fp32 (bf16 operands only; with fp32 operands v_ring holds them).  Version v
  // sits in slot v % vdepth; the update writes version k + 1 there.  With PipeMare Recompute and T2 (Appendix D) each
  // ring has rdepth = tau_r + 1 more slots behind those: slot vdepth + v % rdepth holds w_v - (tau_f - tau_r) delta_v,
  // what the recomputation of microbatch v + tau_r reads, formed by the update that produced version v.
  uint64_t v_ring, s_ring;
  uint64_t tab_off, g_off, beta_off;   // arena offsets: embedding table / LayerNorm gain / LayerNorm bias
  uint64_t x_ring;            // ring: x[xdepth][T*d_in] main input (not used by an embedding stage)
  uint64_t u_ring;            // ring: u[depth][T*d_in] first Linear's input when a pre-op produces it
  uint64_t stat_ring;         // ring: LayerNorm mean, rstd [depth][T*2] float
  uint64_t ids_ring;          // ring: token ids [depth][T] int32 (embedding stage)
  uint64_t skip_in;           // ws: incoming skip tensor [2][T*n_out] (residual stage), slot = tick parity of its writer
  uint64_t ytmp;              // ws: Linear output awaiting the residual add [T*n_out]
  uint64_t gin;               // ws: incoming gradient w.r.t. the main output [3][T*d_out_main], slot = writer's tick % 3
  uint64_t dy;                // ws: gradient w.r.t. the Linear output when a post-op produces it [T*n_out] (attention)
  uint64_t dz;                // ws: dz scratch [T*max_dim]
  uint64_t dh;                // ws: dgrad output scratch [T*max_dim] (du of the first Linear, dh between Linears)
  LinDev lin[PM_MAX_LINEARS];
};

// Per-tick state of one stage, written by the schedule kernel, read by every other kernel.
struct StageDyn {
  int64_t f_mb, b_mb;         // microbatch in forward / backward this tick (-1: idle)
  int64_t f_ver, b_ver;       // weight version (= updates applied) those passes read
  int64_t k;                  // update index applied this tick (= b_mb), -1 if idle
  int64_t tick;
  int32_t f_slot, f_xslot;    // ring slots written by the forward (z/h rings, x ring)
  int32_t f_next_xslot;       // slot of the NEXT stage's x ring that receives this forward's output
  int32_t b_slot, b_xslot;    // ring slots read by the backward
  int32_t active_update;
  float alpha, gamma, one_minus_gamma, bc1, bc2;
  int32_t use_delta;          // T2 on and gap > 0
  int32_t gin_rslot;          // slot of this stage's gradient mailbox written during the previous tick
  int32_t prev_wslot;         // slot of the previous stage's gradient mailbox this tick's backward writes
  int32_t gmem_slot;          // slot of the memory-gradient ring of the microbatch in backward
  int32_t skip_wslot;         // emitting stage: slot of the receiving stage's skip buffer this tick's forward writes
  int32_t skip_rslot;         // receiving stage: slot of its skip buffer this tick's forward reads
  int32_t b_next_xslot;       // slot of the NEXT stage's x ring that holds the output of the microbatch in backward
  int32_t f_vslot;            // slot of the version rings the forward reads (0 in tick-major order)
  int32_t u_vslot;            // slot of the version rings the update fills with the new weights
  int64_t lp_shift;           // the update writes the operand-type copy of element e to lp_base[lp_shift + e]
  int32_t accum;              // parameter gradients of this backward are ADDED to what the grad arena holds (the second to
                              // N-th microbatch of a minibatch, Section 2.1); 0: they overwrite it
  int32_t rc_uslot;           // slot of the version rings that takes the corrected recompute weights of the new version (-1: none)
  int64_t rc_shift;           // their operand-type copy of element e goes to lp_base[rc_shift + e]
  int64_t r_ver;              // weight version the recomputation of the microbatch in backward reads (PipeMare Recompute)
  float rc_gap;               // tau_fwd - tau_recomp
  int32_t _pad2;
  int64_t g_shift;            // the update reads the gradient of element e at gsrc[g_shift + e] (0: the grad arena itself; stochastic
                              // delays: the slot of the gradient ring that holds the microbatch this stage applies)
};

// Hyper-parameters the schedule kernel needs.
struct HyperDev {
  int32_t optimizer, t1, t2, n_stages;
  int64_t K;
  double D;
  double alpha_const;
  const double* alpha_tab;    // device, may be null
  int64_t alpha_len;
  float beta1, beta2, eps;
  int64_t warm, period;       // synchronous warm-up (Section 4): the first `warm` microbatches enter `period` = 2P ticks apart
  int32_t mb_major;           // microbatch-major order: one microbatch in flight, forward weights from the version rings
  int32_t lp_elem;            // bytes of an element of the version rings' operand copy (2 or 4)
  int32_t n_micro;            // N: microbatches per update (microbatch-major order; 1 elsewhere)
  int32_t entry_period;       // tick-major order: a microbatch enters every entry_period ticks (1: every tick)
  int32_t segment;            // PipeMare Recompute: stages per segment (0: no recomputation)
  int32_t stochastic;         // stage-wise stochastic delays (Appendix E): slots of the gradient ring, tau_max + 1 (0: off)
  uint64_t total;             // elements of the arenas (one slot of the gradient ring)
  int32_t materialize;        // backward entries point at the slot that holds the materialised corrected weights (or the live version)
  int32_t _pad3;
};

// The microbatch that enters the first stage at tick a, or -1: during the warm-up one microbatch every `period` ticks
// (the pipeline holds one microbatch at a time, which is synchronous training), afterwards one per tick.
__host__ __device__ inline int64_t mb_at_tick(int64_t a, int64_t warm, int64_t period, int64_t entry_period = 1) {
  if (a < 0) return -1;
  if (entry_period > 1) return (a % entry_period == 0) ? a / entry_period : -1;   // a sparser pipeline: one microbatch every E ticks
  const int64_t t0 = warm * period;
  if (a < t0) return (a % period == 0) ? a / period : -1;
  return warm + (a - t0);
}

struct ArenasDev {
  float* w; float* m; float* s; float* delta; float* grad; __nv_bfloat16* w_lp;
  uint64_t count;
};

__device__ __forceinline__ float act_fwd(float z, int act) {
  if (act == PM_ACT_RELU) return fmaxf(z, 0.0f);
  if (act == PM_ACT_GELU) return 0.5f * z * (1.0f + erff(z * 0.70710678118654752440f));
  return z;
}
__device__ __forceinline__ float act_grad(float z, int act) {
  if (act == PM_ACT_RELU) return z > 0.0f ? 1.0f : 0.0f;
  if (act == PM_ACT_GELU)
    return 0.5f * (1.0f + erff(z * 0.70710678118654752440f)) + z * expf(-0.5f * z * z) * 0.39894228040143267794f;
  return 1.0f;
}

// the activation as the backward pass sees it (a fused ReLU has been applied upstream already)
__host__ __device__ __forceinline__ int bwd_act(const LinDev& L) { return (L.flags & LF_DZ_FUSED) ? PM_ACT_NONE : L.act; }
// the stage's last Linear feeds an attention op (its output is the q, k, v stash; its gradient comes from s.dy)
__host__ __device__ __forceinline__ bool feeds_attention(int post) { return post == POST_ATTENTION || post == POST_CROSS_ATTENTION; }

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }
// eight consecutive elements (16-byte aligned for bf16, 32-byte for float) to / from fp32 registers
template <typename T> __device__ __forceinline__ void load8(const T* p, float (&v)[8]);
template <> __device__ __forceinline__ void load8<float>(const float* p, float (&v)[8]) {
  const float4 a = *reinterpret_cast<const float4*>(p), b = *reinterpret_cast<const float4*>(p + 4);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
template <> __device__ __forceinline__ void load8<__nv_bfloat16>(const __nv_bfloat16* p, float (&v)[8]) {
  const uint4 q = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w[i]));
    v[2 * i] = f.x; v[2 * i + 1] = f.y;
  }
}
template <typename T> __device__ __forceinline__ void store8(T* p, const float (&v)[8]);
template <> __device__ __forceinline__ void store8<float>(float* p, const float (&v)[8]) {
  *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
  *reinterpret_cast<float4*>(p + 4) = make_float4(v[4], v[5], v[6], v[7]);
}
template <> __device__ __forceinline__ void store8<__nv_bfloat16>(__nv_bfloat16* p, const float (&v)[8]) {
  uint32_t w[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
    w[i] = *reinterpret_cast<uint32_t*>(&h);
  }
  *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
}

// value as the GEMM operand type would hold it
template <typename T> __device__ __forceinline__ float round_as(float v) { return to_f<T>(from_f<T>(v)); }

}  // namespace pm
