// Per-element arithmetic shared by every kernel that folds or applies (device code only), so
// that all entry points give the same bits for the same inputs.
#pragma once

#include "adama_internal.h"

namespace adama {

// Algorithm 2, inner loop body:  m += (1-beta1) g/N,  v += (1-beta2) (g/N)^2,
// with a = (1-beta1)/N and b = (1-beta2)/N^2 formed on the host.
__device__ __forceinline__ void fold1(float g, float &m, float &v, float a, float b) {
    m = fmaf(a, g, m);
    v = fmaf(b * g, g, v);
}

__device__ __forceinline__ float sqrt_fast(float x) {
    float r;
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ float rcp_fast(float x) {
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

// Algorithm 2, "Update", plus the decay of the next mini-batch:
//   w -= step * m / (sqrt(v*inv_bc2) + eps);  m *= beta1;  v *= beta2
// (step = lr/(1-beta1^t), inv_bc2 = 1/(1-beta2^t), optional decoupled decay in w_keep).
// Square root and reciprocal are the 1-ulp hardware approximations: the IEEE-rounded forms
// branch into slow paths for zero and denormal operands (exactly-zero m or v, common in
// padding and unused embedding rows, made a 335 M-element apply 1.6-1.9x slower), while the
// update term is <= ~1e-1 of |w|, so 2-3 ulp there is < 1e-7 on w.
// beta = hi + lo: the small product is rounded first (its error is ~1e-15 relative to the
// result), then one fma rounds x*hi + x*lo once; the other order would round x*hi first and
// lose the sub-ulp correction every time.
__device__ __forceinline__ void apply1(float &w, float &m, float &v, const ApplyConstants &c) {
    const float denom = sqrt_fast(v * c.inv_bc2) + c.eps;
    w = fmaf(-c.step, m * rcp_fast(denom), w * c.w_keep);
    m = fmaf(m, c.beta1_hi, m * c.beta1_lo);
    v = fmaf(v, c.beta2_hi, v * c.beta2_lo);
}

}  // namespace adama
