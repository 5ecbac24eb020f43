// The arithmetic of one PipeMare update of one parameter, shared by the fused update kernel and by the weight-gradient
// GEMM's epilogue when the update is applied there.  Each operation is rounded once in fp32 in the written order, no
// fused multiply-add, so that any IEEE implementation reproduces the bits:
//   SGD-m (Appendix B.3):  v' = beta*v - alpha*g ;  w' = w + v'
//   Adam:  m' = b1*m + (1-b1)*g ;  s' = b2*s + (1-b2)*(g*g) ;  w' = w - (alpha*(m'/bc1)) / (sqrt(s'/bc2) + eps)
//   T2 (Section 3.2):      delta' = gamma*delta + (1-gamma)*(w' - w)
#pragma once
#include "pm_common.cuh"

namespace pm {

struct UpdScalars {
  float alpha, gamma, omg, bc1, bc2;
  int use_delta;
  int64_t lp_shift;
  int64_t rc_shift;     // element shift of the corrected recompute copy of the new weights, -1: none
  float rc_gap;         // tau_fwd - tau_recomp
};


template <int OPT>
__device__ __forceinline__ float upd_one(float g, float w, float& m, float& s, float& dl, const UpdScalars& c,
                                         float beta1, float beta2, float omb1, float omb2, float eps) {
  float wn;
  if (OPT == PM_SGDM) {
    m = __fsub_rn(__fmul_rn(beta1, m), __fmul_rn(c.alpha, g));
    wn = __fadd_rn(w, m);
  } else {
    m = __fadd_rn(__fmul_rn(beta1, m), __fmul_rn(omb1, g));
    s = __fadd_rn(__fmul_rn(beta2, s), __fmul_rn(omb2, __fmul_rn(g, g)));
    // Correctly rounded division and square root leave their short instruction sequence for a subroutine when an
    // operand is zero (parameters whose gradient has been zero so far: untouched embedding rows).  Those lanes
    // divide 1 instead and keep the zero, which is what the operation returns for them (0 / b = 0 with the sign
    // of the zero for b > 0, sqrt(+-0) = +-0), so the results are the same bits.
    const bool mz = m == 0.f, sz = s == 0.f;
    const float mq = __fdiv_rn(mz ? 1.f : m, c.bc1), sq = __fdiv_rn(sz ? 1.f : s, c.bc2);
    const float mh = mz ? m : mq, sh = sz ? s : sq;
    const float rt = __fsqrt_rn(sh == 0.f ? 1.f : sh);
    const float den = __fadd_rn(sh == 0.f ? sh : rt, eps);
    const float num = __fmul_rn(c.alpha, mh);
    const bool nz = num == 0.f && den > 0.f;
    const float q = __fdiv_rn(nz ? 1.f : num, den);
    wn = __fsub_rn(w, nz ? num : q);
  }
  if (c.use_delta) dl = __fadd_rn(__fmul_rn(c.gamma, dl), __fmul_rn(c.omg, __fsub_rn(wn, w)));
  return wn;
}

}  // namespace pm
