// One AdamW element update, shared by the table-driven kernel and the fused weight-row kernel, so that
// both produce the same bits.  The bias corrections enter as the per-step scalars lr/bc1 and
// 1/sqrt(bc2) (same update algebraically); square root and quotient use the hardware's approximate
// instructions (about 2 ulp each), far inside what the float32 moments themselves carry.
#pragma once
#include "kernels.h"

namespace mrem {

__device__ __forceinline__ float sqrt_approx(float x) {
  float y;
  asm("sqrt.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// p <- max(p * (1 - lr*wd) - lr * (m/bc1) / (sqrt(v/bc2) + eps), min_value); m, v updated in place.
__device__ __forceinline__ float adam_one(float p, float g, float& m, float& v, const OptimScalars& o, float wd_on,
                                          float min_value) {
  m = __fmaf_rn(o.beta1, m, __fmul_rn(__fsub_rn(1.f, o.beta1), g));
  v = __fmaf_rn(o.beta2, v, __fmul_rn(__fmul_rn(__fsub_rn(1.f, o.beta2), g), g));
  const float decay = __fsub_rn(1.f, __fmul_rn(__fmul_rn(o.lr, wd_on), o.weight_decay));
  const float denom = __fmaf_rn(sqrt_approx(v), o.rsqrt_bc2, o.eps);
  const float upd = __fdividef(__fmul_rn(o.lr_bc1, m), denom);
  return fmaxf(__fsub_rn(__fmul_rn(p, decay), upd), min_value);
}

// Straight-through factors of the weight quantizer at z = w / s: whether the gradient passes to w,
// and the level d w_hat / d s is measured from (code on the integer grid, k + 0.5 on the half-integer one).
// Round to nearest even without the conversion unit: adding and subtracting 1.5 * 2^23 leaves rint(x) for
// |x| < 2^22 (codes are at most 127 in magnitude); the sum's low mantissa bits are the integer itself.
constexpr float RINT_MAGIC = 12582912.f;
__device__ __forceinline__ float rint_small(float x) { return __fsub_rn(__fadd_rn(x, RINT_MAGIC), RINT_MAGIC); }

__device__ __forceinline__ void weight_ste(float z, float qmax, int grid, bool& in, float& level) {
  if (grid == 0) {
    in = z >= -qmax && z <= qmax;
    level = rint_small(fminf(fmaxf(z, -qmax), qmax));
  } else {
    in = z >= -2.f && z < 2.f;
    level = fminf(fmaxf(floorf(z), -2.f), 1.f) + 0.5f;
  }
}

// Adds one element's contribution to d loss / d step; single-rounding operations only, so every
// kernel that walks a row in the same order gets the same bits.
__device__ __forceinline__ float step_grad_acc(float acc, float w, float d, float s, float r_s, float qmax, int grid,
                                               bool& in) {
  const float z = quotient(w, s, r_s);
  float level;
  weight_ste(z, qmax, grid, in, level);
  return __fmaf_rn(d, __fsub_rn(level, in ? z : 0.f), acc);
}

}  // namespace mrem
