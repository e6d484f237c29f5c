// Shared device/host helpers of the MREM reconstruction-step kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace mrem {

typedef __nv_bfloat16 bf16;

// ---------------------------------------------------------------- status word (device, sticky)
enum DeviceStatus : int {
  DEV_OK = 0,
  DEV_TIMEOUT_TMA = 1,      // a wait on a TMA-filled stage ran out
  DEV_TIMEOUT_MMA = 2,      // a wait on a tensor-core commit ran out
  DEV_TIMEOUT_EPI = 3,      // a wait on an accumulator hand-over ran out
  DEV_NONFINITE = 4,        // the loss kernel met a non-finite value
  DEV_BAD_INDEX = 5,        // an embedding index outside its table (clamped)
};

// ---------------------------------------------------------------- programmatic dependent launch
// Every kernel of the library is launched so that it may start while its predecessor in the stream is
// still draining: it announces itself (pdl_trigger) and then waits (pdl_wait) until everything the
// predecessor wrote is visible, before it touches global memory.  What runs before the wait (barrier
// and TMEM set-up in the tensor-core kernels) and the launch latency itself overlap the predecessor's tail.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

extern unsigned long long g_wait_limit_ns;   // limit of every device-side wait, copied into each launch's parameters
extern int g_programmatic_launch;      // 1: launch with programmatic stream serialization (default)
// Set to 1 to make the NEXT launch a plain stream-ordered one (consumed by that launch): such a kernel starts only after
// everything enqueued before it on its stream has completed, and no later kernel can start before it does.  The first
// kernel of every forward pass is launched this way, so that whatever an earlier pass or update wrote (weight codes,
// dequantized weights) is complete for every kernel of the pass, also before its own dependency wait.
extern thread_local int g_plain_next_launch;

template <typename... KArgs, typename... Args>
inline cudaError_t launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = (g_programmatic_launch && !g_plain_next_launch) ? 1 : 0;
  g_plain_next_launch = 0;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---------------------------------------------------------------- storage-type access
template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<bf16>(bf16 v) { return __bfloat162float(v); }

template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16_rn(v); }

// value of v after a round trip through storage type T
template <typename T> __device__ __forceinline__ float stored(float v) { return to_f<T>(from_f<T>(v)); }

// ---------------------------------------------------------------- reductions
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ int warp_sum_i(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Block-wide sum in a fixed order (warp shuffles, then warp 0 over the per-warp values).
// `sh` must hold 32 floats.  Every thread gets the result.
__device__ __forceinline__ float block_sum(float v, float* sh) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) sh[w] = v;
  __syncthreads();
  float r = (lane < nw) ? sh[lane] : 0.f;
  r = warp_sum(r);
  return r;
}
__device__ __forceinline__ float block_max(float v, float* sh) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_max(v);
  __syncthreads();
  if (lane == 0) sh[w] = v;
  __syncthreads();
  float r = (lane < nw) ? sh[lane] : -INFINITY;
  r = warp_max(r);
  return r;
}

// ---------------------------------------------------------------- math
// 2^x by the special-function unit alone (x <= 0 here: scores minus their maximum); about 2 ulp, flushes to zero below 2^-126
__device__ __forceinline__ float exp2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float rcp_approx(float x) {
  float y;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// x / s from r_s = RN(1/s): one product, the exact residual by FMA, one correction.  Equals the correctly
// rounded quotient except where x/s lies within ~2^-48 (relative) of the midpoint of two floats; a value
// sitting exactly on a clipping boundary gets the same side as the quantizer's IEEE division.  For
// bfloat16-valued x (8 significant bits) it IS the correctly rounded quotient for every float32 s:
// checked over all 128 x 2^23 significand pairs (the exponents do not enter while x/s, 1/s and the
// residual stay in the normal range, which holds for activations and steps by many orders of magnitude).
// Used for the straight-through factors (a surrogate gradient) and, in the fused attention kernel, for the
// codes of bfloat16-stored tensors; every other code is produced with the division instruction.
__device__ __forceinline__ float quotient(float x, float s, float r_s) {
  const float z0 = __fmul_rn(x, r_s);
  return __fmaf_rn(__fmaf_rn(-z0, s, x), r_s, z0);
}

// Nearest integer (ties to even) of a float with |z| < 2^22 by adding and subtracting 1.5 * 2^23: two additions on the
// ordinary pipes instead of two conversions.  `bits` receives the bit pattern of z + 1.5 * 2^23, whose low mantissa bits are
// the integer in two's complement (its low byte IS the 8-bit code).
constexpr float ROUND_MAGIC = 12582912.f;
__device__ __forceinline__ float rne_magic(float z, uint32_t& bits) {
  const float t = __fadd_rn(z, ROUND_MAGIC);
  bits = __float_as_uint(t);
  return __fsub_rn(t, ROUND_MAGIC);
}
__device__ __forceinline__ float rne_magic(float z) { uint32_t b; return rne_magic(z, b); }

// The integer code of Eq. 1, nearest integer (ties to even) of clip(n / s, lo, hi), bit for bit what the IEEE division
// gives, at a fraction of its instructions; returned as a float, with the bit pattern that carries its low byte.
// r_s = RN(1 / s).  The three-instruction quotient is within one ulp of the correctly rounded one (1.5e-5 at |z| <= 255),
// so the two can round to different integers only when the quotient lies that close to a half-integer: any value within
// 2^-10 of one is decided by the division instruction instead (about one element in a thousand).  A quotient beyond the
// range is clipped to the same bound by both.  EXACT_QUOTIENT: the numerator is a bfloat16 value, for which the quotient
// IS the correctly rounded one (see quotient()) and no second look is needed.
template <bool EXACT_QUOTIENT>
__device__ __forceinline__ float code_f(float n, float s, float r_s, float lo, float hi, uint32_t& bits) {
  // (the first product is kept inside [lo - 1, hi + 1]: unchanged wherever the code is not simply a bound, and a
  //  numerator so large that n * r_s overflows then still ends on the bound of its sign instead of a NaN)
  const float z0 = fminf(fmaxf(__fmul_rn(n, r_s), lo - 1.f), hi + 1.f);
  float zc = fminf(fmaxf(__fmaf_rn(__fmaf_rn(-z0, s, n), r_s, z0), lo), hi);
  float q = rne_magic(zc, bits);
  if constexpr (!EXACT_QUOTIENT) {
    if (fabsf(fabsf(zc - q) - 0.5f) < 9.765625e-4f) {
      zc = fminf(fmaxf(__fdiv_rn(n, s), lo), hi);
      q = rne_magic(zc, bits);
    }
  }
  return q;
}
__device__ __forceinline__ int code_of(float n, float s, float r_s, float lo, float hi) {
  uint32_t b;
  return (int)code_f<false>(n, s, r_s, lo, hi, b);
}
// low bytes of four words -> one word (byte i from b_i)
__device__ __forceinline__ uint32_t pack_low_bytes(uint32_t b0, uint32_t b1, uint32_t b2, uint32_t b3) {
  return __byte_perm(__byte_perm(b0, b1, 0x0040), __byte_perm(b2, b3, 0x0040), 0x5410);
}

// GELU(u) = u * Phi(u) with the erf form.  erf(x) = 1 - (a1 t + ... + a5 t^5) exp(-x^2), t = 1/(1 + p x), x >= 0
// (Abramowitz & Stegun 7.1.26, |error| <= 1.5e-7, below half a float32 ulp of 1 + erf for u > 0): one
// exponential serves both erf and the density needed by the derivative.
//   tail = (1 - erf(|u| / sqrt 2)) / 2 = Phi(-|u|)   (the coefficients below are a_i / 2),   ex = exp(-u^2 / 2)
__device__ __forceinline__ void gelu_parts(float u, float& tail, float& ex) {
  const float au = fabsf(u);
  ex = exp2_approx(u * u * -0.72134752044448170f);          // -log2(e) / 2
  const float t = rcp_approx(fmaf(0.23164189f, au, 1.f));    // p / sqrt 2
  float poly = fmaf(0.5307027145f, t, -0.7265760135f);
  poly = fmaf(poly, t, 0.7107068705f);
  poly = fmaf(poly, t, -0.142248368f);
  poly = fmaf(poly, t, 0.127414796f);
  tail = poly * t * ex;
}
// u * Phi(u) = max(u, 0) - |u| * Phi(-|u|): the value both the forward pass and the backward pass (which re-forms it
// for the quantizer's mask) compute, bit for bit
__device__ __forceinline__ float gelu_from_tail(float u, float tail) { return fmaf(-fabsf(u), tail, fmaxf(u, 0.f)); }
__device__ __forceinline__ float gelu_erf(float u) {
  float tail, ex;
  gelu_parts(u, tail, ex);
  return gelu_from_tail(u, tail);
}
// d/du (u Phi(u)) = Phi(u) + u phi(u)
__device__ __forceinline__ float gelu_grad_from_parts(float u, float tail, float ex) {
  const float cdf = u >= 0.f ? 1.f - tail : tail;
  return fmaf(u, ex * 0.39894228040143268f, cdf);             // exp(-u^2/2) / sqrt(2 pi)
}
__device__ __forceinline__ float gelu_erf_grad(float u) {
  float tail, ex;
  gelu_parts(u, tail, ex);
  return gelu_grad_from_parts(u, tail, ex);
}

// ---------------------------------------------------------------- GEMM interface (both back ends)
enum OutKind : int { OUT_F32 = 0, OUT_BF16 = 1, OUT_I32 = 2 };

// out[b][m][n] = act( alpha * col_scale[n] * acc + col_bias[n] + row_bias[m] + residual[b][m][n] )
// alpha = alpha_const * (*alpha_p0) * (*alpha_p1)   (null pointers count as 1)
struct Epilogue {
  void* out;
  const void* residual;        // same kind and strides as out, or null
  long long ldc, c_b0, c_b1;   // element strides of out/residual: row, batch0, batch1
  int out_kind;                // OutKind
  int act;                     // 0 none, 1 erf-GELU
  float alpha_const;
  const float* alpha_p0;
  const float* alpha_p1;
  const float* col_scale;      // [N] or null
  const float* col_bias;       // [N] or null
  const float* row_bias;       // [M] or null
};

// One operand of C[m,n] = sum_k A[m,k] * B[n,k].  `mn_contig` = 1 when the operand is
// stored with its M (or N) index contiguous and k strided, 0 when k is contiguous.
struct OperandDesc {
  const void* ptr;
  long long ld;                // element stride of the non-contiguous index
  long long s_b0, s_b1;        // element strides of the batch indices
  int mn_contig;
  int is_static;               // 1: nothing the stream's preceding kernel writes (a weight matrix, codes of the last update):
                               //    its first tiles may be fetched while that kernel is still finishing (B operand only)
};

struct GemmShape { int M, N, K, nb0, nb1; };

}  // namespace mrem
