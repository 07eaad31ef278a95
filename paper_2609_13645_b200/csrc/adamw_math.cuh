// The AdamW update of one element (Section "Sources of the Speedup" and the optimizer-tail listing of the appendix
// "Why the Engine Is Faster, Mechanism by Mechanism": fused clip + Adam + bf16 write-back), written with explicit
// round-to-nearest intrinsics so that every kernel that applies it (the multi-tensor pass, the weight-gradient GEMM
// epilogue, the split-K reduction) produces the same bits from the same inputs: no compiler-chosen contraction.
#pragma once
#include <cuda_runtime.h>

namespace fs {

struct AdamCoef {
  float lr, beta1, beta2, omb1, omb2, eps;  // omb = 1 - beta
  float rbc1, rbc2;                         // 1 / (1 - beta^t): reciprocals of the bias corrections, rounded once
};

__device__ __forceinline__ AdamCoef make_adam_coef(float lr, float beta1, float beta2, float eps, float bc1, float bc2) {
  AdamCoef c;
  c.lr = lr; c.beta1 = beta1; c.beta2 = beta2; c.omb1 = 1.0f - beta1; c.omb2 = 1.0f - beta2; c.eps = eps;
  c.rbc1 = __frcp_rn(bc1); c.rbc2 = __frcp_rn(bc2);
  return c;
}

// g: gradient (already multiplied by the clip coefficient); wd: weight decay of this tensor
__device__ __forceinline__ void adamw_elem(float g, float wd, const AdamCoef& c, float& p, float& m, float& v) {
  m = __fmaf_rn(c.beta1, m, __fmul_rn(c.omb1, g));
  v = __fmaf_rn(c.beta2, v, __fmul_rn(__fmul_rn(c.omb2, g), g));
  const float mhat = __fmul_rn(m, c.rbc1);
  const float vhat = __fmul_rn(v, c.rbc2);
  // square root and quotient on the special-function unit (each within 2 ulp): the update term is lr * 1e-3 of the
  // parameter's magnitude, so this is invisible next to the fp32 rounding of p itself, and it halves the epilogue's
  // instruction count
  float root, quot;
  asm("sqrt.approx.f32 %0, %1;" : "=f"(root) : "f"(vhat));
  const float den = __fadd_rn(root, c.eps);
  asm("div.approx.f32 %0, %1, %2;" : "=f"(quot) : "f"(mhat), "f"(den));
  const float upd = __fmaf_rn(wd, p, quot);
  p = __fmaf_rn(-c.lr, upd, p);
}

}  // namespace fs
