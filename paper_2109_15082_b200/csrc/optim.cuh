// One AdamW element update, shared by the table-driven kernel and the fused weight-row kernel.
// Written with explicit single-rounding intrinsics so that both kernels produce the same bits.
#pragma once
#include "kernels.h"

namespace mrem {

// p <- max(p * (1 - lr*wd) - lr * (m/bc1) / (sqrt(v/bc2) + eps), min_value); m, v updated in place.
__device__ __forceinline__ float adam_one(float p, float g, float& m, float& v, const OptimScalars& o, float wd_on,
                                          float min_value) {
  m = __fadd_rn(__fmul_rn(o.beta1, m), __fmul_rn(__fsub_rn(1.f, o.beta1), g));
  v = __fadd_rn(__fmul_rn(o.beta2, v), __fmul_rn(__fmul_rn(__fsub_rn(1.f, o.beta2), g), g));
  const float decay = __fsub_rn(1.f, __fmul_rn(__fmul_rn(o.lr, wd_on), o.weight_decay));
  const float denom = __fadd_rn(__fsqrt_rn(__fdiv_rn(v, o.bc2)), o.eps);
  const float upd = __fdiv_rn(__fmul_rn(o.lr, __fdiv_rn(m, o.bc1)), denom);
  return fmaxf(__fsub_rn(__fmul_rn(p, decay), upd), min_value);
}

// Straight-through factors of the weight quantizer at z = w / s: whether the gradient passes to w,
// and the level d w_hat / d s is measured from (code on the integer grid, k + 0.5 on the half-integer one).
__device__ __forceinline__ void weight_ste(float z, float qmax, int grid, bool& in, float& level) {
  if (grid == 0) {
    in = z >= -qmax && z <= qmax;
    level = (float)__float2int_rn(fminf(fmaxf(z, -qmax), qmax));
  } else {
    in = z >= -2.f && z < 2.f;
    level = fminf(fmaxf(floorf(z), -2.f), 1.f) + 0.5f;
  }
}

// Adds one element's contribution to d loss / d step; single-rounding operations only, so every
// kernel that walks a row in the same order gets the same bits.
__device__ __forceinline__ float step_grad_acc(float acc, float w, float d, float s, float qmax, int grid, bool& in) {
  const float z = __fdiv_rn(w, s);
  float level;
  weight_ste(z, qmax, grid, in, level);
  return __fmaf_rn(d, __fsub_rn(level, in ? z : 0.f), acc);
}

}  // namespace mrem
