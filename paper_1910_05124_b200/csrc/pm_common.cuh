// Shared device-side tables and small helpers of the PipeMare library.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "pipemare.h"

namespace pm {

// Static description of one Linear inside a stage (device copy).
struct LinDev {
  int32_t n_in, n_out, act, _pad;
  uint64_t w_off, b_off;      // element offsets into the flat arenas
  uint64_t z_ring;            // byte offset in the ring arena of z[depth][T*n_out] (pre-activation stash)
  uint64_t h_ring;            // byte offset of this Linear's output stash h[depth][T*n_out] (unused for the last Linear)
};

// Static description of one stage (device copy).
struct StageDev {
  int32_t tau_f, gap;         // tau_fwd, tau_fwd - tau_bkwd
  int32_t n_lin;
  int32_t depth;              // slots of z / h rings  = tau_f + 1
  int32_t xdepth;             // slots of the input ring = tau_f + 2 (it doubles as the forward mailbox)
  int32_t max_dim;
  uint64_t begin, end;        // padded element range of the stage's parameters in the arenas
  uint64_t x_ring;            // byte offset of x[xdepth][T*n_in0]
  uint64_t gin;               // workspace byte offset: incoming gradient mailbox [2][T*n_out_last]
  uint64_t dz;                // workspace byte offset: dz scratch [T*max_dim]
  uint64_t dh;                // workspace byte offset: dh scratch [T*max_dim]
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
};

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

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }
// value as the GEMM operand type would hold it
template <typename T> __device__ __forceinline__ float round_as(float v) { return to_f<T>(from_f<T>(v)); }

}  // namespace pm
