// Weight codes whose scale is recomputed from the weights instead of learnt (Sec. 5.1 names one such rule for 2-bit
// and one for 4-bit weights), one block per output row.
//
// Ternary rule (2-bit):  delta = 0.7 * mean|w|,  t = sign(w) * 1[|w| > delta],  alpha = mean of |w| over the kept
// entries (0 when none is kept),  w_hat = alpha * t.  Nothing is learnt about the scale: the update is
// AdamW on the latent weights with the gradient of w_hat passed through unchanged, followed by the same
// rule on the new weights.  Both means are accumulated in float64 in a fixed order and the comparison
// |w| > delta is made in float32 on float32(delta), so the codes are a function of the stored weights
// alone.  Two kernels share the row routine: the stand-alone quantizer and the fused update.
//
// Refitted scale (b-bit, the loss-aware rule read with unit curvature weights): minimise ||w - alpha q||^2 over
// alpha and q in Omega(b)^n by alternating the two exact half-steps  q = Pi_Omega(b)(w / alpha)  (Eq. 1, float32
// division)  and  alpha = <q, w> / <q, q>  (float64 sums in a fixed order, alpha rounded to float32), LAQ_ROUNDS
// times from alpha_0 = min(3 mean|w|, max|w|) / qmax; a row of zeros keeps alpha = 0 and codes 0.
#include "optim.cuh"

namespace mrem {

namespace {

// Threads per row (NT) and float4 vectors per thread kept in registers (MAXV): a block of 256 threads with 4 vectors
// each holds rows up to 4096 wide; the alternating rule, whose 16 rounds are a dependent chain per thread, takes 128
// threads with 2 vectors each for rows up to 1024 wide (measured against 32 x 8 and 256 x 1).
constexpr int TW_THREADS = 256;
constexpr int TW_MAXV = 4;
constexpr int TW_NARROW_THREADS = 128;   // rows up to 1024 wide under the alternating rule: 2 vectors per thread
constexpr int TW_NARROW_MAXV = 2;

__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ double block_sum_d(double v, double* sh) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_sum_d(v);
  __syncthreads();
  if (lane == 0) sh[w] = v;
  __syncthreads();
  double r = (lane < nw) ? sh[lane] : 0.0;
  return warp_sum_d(r);
}
__device__ __forceinline__ int block_sum_i(int v, int* sh) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_sum_i(v);
  __syncthreads();
  if (lane == 0) sh[w] = v;
  __syncthreads();
  int r = (lane < nw) ? sh[lane] : 0;
  return warp_sum_i(r);
}

template <typename T>
__device__ __forceinline__ void store4(T* p, float a, float b, float c, float d);
template <>
__device__ __forceinline__ void store4<float>(float* p, float a, float b, float c, float d) {
  *reinterpret_cast<float4*>(p) = make_float4(a, b, c, d);
}
template <>
__device__ __forceinline__ void store4<bf16>(bf16* p, float a, float b, float c, float d) {
  uint2 t;
  __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&t);
  h[0] = __floats2bfloat162_rn(a, b);
  h[1] = __floats2bfloat162_rn(c, d);
  *reinterpret_cast<uint2*>(p) = t;
}

__device__ __forceinline__ int tern(float w, float delta) { return fabsf(w) > delta ? (w > 0.f ? 1 : -1) : 0; }

// The rule on one row.  `cached`: the row sits in wr[] (vector c = threadIdx.x + i * NT), else it is re-read
// from w_row.  Writes codes, row sum, scale and the dequantized row.
template <typename T, int NT, int MAXV>
__device__ __forceinline__ void ternary_row(const float4* wr, bool cached, const float* w_row, int cols, int row,
                                            int8_t* codes_row, int32_t* rowsum, float* scale, T* what_row,
                                            double* shd, int* shi) {
  const int nvec = cols / 4;
  double s = 0.0;
  if (cached) {
#pragma unroll
    for (int i = 0; i < MAXV; ++i) {
      const int c = threadIdx.x + i * NT;
      if (c < nvec) s += (double)fabsf(wr[i].x) + (double)fabsf(wr[i].y) + (double)fabsf(wr[i].z) + (double)fabsf(wr[i].w);
    }
  } else {
    for (int c = threadIdx.x; c < nvec; c += NT) {
      const float4 v = reinterpret_cast<const float4*>(w_row)[c];
      s += (double)fabsf(v.x) + (double)fabsf(v.y) + (double)fabsf(v.z) + (double)fabsf(v.w);
    }
  }
  s = block_sum_d(s, shd);
  const float delta = (float)(0.7 * (s / (double)cols));
  double ks = 0.0;
  int cnt = 0;
  auto acc = [&](float4 v) {
    if (fabsf(v.x) > delta) { ks += (double)fabsf(v.x); ++cnt; }
    if (fabsf(v.y) > delta) { ks += (double)fabsf(v.y); ++cnt; }
    if (fabsf(v.z) > delta) { ks += (double)fabsf(v.z); ++cnt; }
    if (fabsf(v.w) > delta) { ks += (double)fabsf(v.w); ++cnt; }
  };
  if (cached) {
#pragma unroll
    for (int i = 0; i < MAXV; ++i) {
      const int c = threadIdx.x + i * NT;
      if (c < nvec) acc(wr[i]);
    }
  } else {
    for (int c = threadIdx.x; c < nvec; c += NT) acc(reinterpret_cast<const float4*>(w_row)[c]);
  }
  ks = block_sum_d(ks, shd);
  cnt = block_sum_i(cnt, shi);
  const float alpha = (float)(ks / (double)(cnt > 0 ? cnt : 1));
  int sum = 0;
  auto emit = [&](int c, float4 v) {
    const int q0 = tern(v.x, delta), q1 = tern(v.y, delta), q2 = tern(v.z, delta), q3 = tern(v.w, delta);
    *reinterpret_cast<uint32_t*>(codes_row + 4 * c) =
        (uint32_t)(q0 & 0xff) | ((uint32_t)(q1 & 0xff) << 8) | ((uint32_t)(q2 & 0xff) << 16) | ((uint32_t)(q3 & 0xff) << 24);
    if (what_row) store4<T>(what_row + 4 * c, alpha * (float)q0, alpha * (float)q1, alpha * (float)q2, alpha * (float)q3);
    sum += q0 + q1 + q2 + q3;
  };
  if (cached) {
#pragma unroll
    for (int i = 0; i < MAXV; ++i) {
      const int c = threadIdx.x + i * NT;
      if (c < nvec) emit(c, wr[i]);
    }
  } else {
    for (int c = threadIdx.x; c < nvec; c += NT) emit(c, reinterpret_cast<const float4*>(w_row)[c]);
  }
  sum = block_sum_i(sum, shi);
  if (threadIdx.x == 0) {
    rowsum[row] = sum;
    scale[row] = alpha;
  }
}

constexpr int LAQ_ROUNDS = 16;

__device__ __forceinline__ int laq_code(float w, float alpha, float qmax) {
  return __float2int_rn(fminf(fmaxf(__fdiv_rn(w, alpha), -qmax), qmax));
}
// The same code from RN(1 / alpha): quotient() differs from the division only where w / alpha lies within 2^-48
// (relative) of the midpoint of two floats, and the code differs only if that quotient is also next to a half-integer.
// Used in the rounds that only feed the two sums; the codes that are written out come from the division.
__device__ __forceinline__ int laq_code_fast(float w, float alpha, float r_alpha, float qmax) {
  return __float2int_rn(fminf(fmaxf(quotient(w, alpha, r_alpha), -qmax), qmax));
}
// (double)q for |q| < 2^31 without the conversion unit: 2^52 + 2^31 + q is exact in the low word of a double.
__device__ __forceinline__ double int_as_double(int q) {
  return __hiloint2double(0x43300000, (int)(0x80000000u ^ (unsigned)q)) - 4503601774854144.0;
}

// Block-wide sum of a double and of an int in one pass.  Every thread gets the results.
__device__ __forceinline__ void block_sum_di(double& a, int& n, double* shd, int* shi) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  a = warp_sum_d(a);
  n = __reduce_add_sync(0xffffffffu, n);
  __syncthreads();
  if (lane == 0) { shd[w] = a; shi[w] = n; }
  __syncthreads();
  a = warp_sum_d(lane < nw ? shd[lane] : 0.0);
  n = __reduce_add_sync(0xffffffffu, lane < nw ? shi[lane] : 0);
}

// The alternating rule on one row (same conventions as ternary_row).
template <typename T, int NT, int MAXV>
__device__ __forceinline__ void laq_row(const float4* wr, bool cached, const float* w_row, int cols, int row, int bits,
                                        int8_t* codes_row, int32_t* rowsum, float* scale, T* what_row, double* shd,
                                        int* shi, float* shf) {
  const int nvec = cols / 4;
  const float qmax = (float)((1 << (bits - 1)) - 1);
  auto for_row = [&](auto&& f) {
    if (cached) {
#pragma unroll
      for (int i = 0; i < MAXV; ++i) {
        const int c = threadIdx.x + i * NT;
        if (c < nvec) f(c, wr[i]);
      }
    } else {
      for (int c = threadIdx.x; c < nvec; c += NT) f(c, reinterpret_cast<const float4*>(w_row)[c]);
    }
  };
  double s = 0.0;
  float mx = 0.f;
  for_row([&](int, float4 v) {
    s += (double)fabsf(v.x) + (double)fabsf(v.y) + (double)fabsf(v.z) + (double)fabsf(v.w);
    mx = fmaxf(fmaxf(mx, fmaxf(fabsf(v.x), fabsf(v.y))), fmaxf(fabsf(v.z), fabsf(v.w)));
  });
  s = block_sum_d(s, shd);
  mx = block_max(mx, shf);
  float alpha = (float)(fmin(3.0 * (s / (double)cols), (double)mx) / (double)qmax);
  for (int r = 0; r + 1 < LAQ_ROUNDS; ++r) {
    double qw = 0.0, qw1 = 0.0, qw2 = 0.0, qw3 = 0.0;
    int qq = 0;
    auto sums = [&](auto code) {
      if (cached) {
#pragma unroll
        for (int i = 0; i < MAXV; ++i) {
          if (threadIdx.x + i * NT < nvec) {
            const int q0 = code(wr[i].x), q1 = code(wr[i].y), q2 = code(wr[i].z), q3 = code(wr[i].w);
            qw = fma(int_as_double(q0), (double)wr[i].x, qw);        // four independent chains
            qw1 = fma(int_as_double(q1), (double)wr[i].y, qw1);
            qw2 = fma(int_as_double(q2), (double)wr[i].z, qw2);
            qw3 = fma(int_as_double(q3), (double)wr[i].w, qw3);
            qq += q0 * q0 + q1 * q1 + q2 * q2 + q3 * q3;
          }
        }
      } else {
        for (int c = threadIdx.x; c < nvec; c += NT) {
          const float4 v = reinterpret_cast<const float4*>(w_row)[c];
          const int q0 = code(v.x), q1 = code(v.y), q2 = code(v.z), q3 = code(v.w);
          qw = fma(int_as_double(q0), (double)v.x, qw);
          qw1 = fma(int_as_double(q1), (double)v.y, qw1);
          qw2 = fma(int_as_double(q2), (double)v.z, qw2);
          qw3 = fma(int_as_double(q3), (double)v.w, qw3);
          qq += q0 * q0 + q1 * q1 + q2 * q2 + q3 * q3;
        }
      }
    };
    if (alpha > 1e-30f) {                                  // 1 / alpha and the residual stay in the normal range
      const float r_alpha = __frcp_rn(alpha);
      sums([&](float w) { return laq_code_fast(w, alpha, r_alpha, qmax); });
    } else if (alpha > 0.f) {
      sums([&](float w) { return laq_code(w, alpha, qmax); });
    }
    qw = (qw + qw1) + (qw2 + qw3);
    block_sum_di(qw, qq, shd, shi);
    alpha = qq > 0 ? (float)(qw / (double)qq) : 0.f;
  }
  // last round: the codes of this alpha (by the division of Eq. 1) go out with the scale refitted to them
  double qw = 0.0;
  int qq = 0, sum = 0;
  for_row([&](int c, float4 v) {
    int q0 = 0, q1 = 0, q2 = 0, q3 = 0;
    if (alpha > 0.f) {
      q0 = laq_code(v.x, alpha, qmax); q1 = laq_code(v.y, alpha, qmax);
      q2 = laq_code(v.z, alpha, qmax); q3 = laq_code(v.w, alpha, qmax);
    }
    qw += (double)q0 * (double)v.x + (double)q1 * (double)v.y + (double)q2 * (double)v.z + (double)q3 * (double)v.w;
    qq += q0 * q0 + q1 * q1 + q2 * q2 + q3 * q3;
    sum += q0 + q1 + q2 + q3;
    *reinterpret_cast<uint32_t*>(codes_row + 4 * c) =
        (uint32_t)(q0 & 0xff) | ((uint32_t)(q1 & 0xff) << 8) | ((uint32_t)(q2 & 0xff) << 16) | ((uint32_t)(q3 & 0xff) << 24);
  });
  block_sum_di(qw, qq, shd, shi);
  const float next = qq > 0 ? (float)(qw / (double)qq) : 0.f;
  if (what_row) {
    auto unpack = [](uint32_t pk, int j) { return (float)(int)(int8_t)(pk >> (8 * j)); };
    for (int c = threadIdx.x; c < nvec; c += NT) {        // this thread's own codes, written above
      const uint32_t pk = *reinterpret_cast<const uint32_t*>(codes_row + 4 * c);
      store4<T>(what_row + 4 * c, next * unpack(pk, 0), next * unpack(pk, 1), next * unpack(pk, 2), next * unpack(pk, 3));
    }
  }
  sum = block_sum_i(sum, shi);
  if (threadIdx.x == 0) {
    rowsum[row] = sum;
    scale[row] = next;
  }
}

template <typename T, int RULE, int NT, int MAXV>
__device__ __forceinline__ void closed_form_row(const float4* wr, bool cached, const float* w_row, int cols,
                                                int row, int bits, int8_t* codes_row, int32_t* rowsum, float* scale,
                                                T* what_row, double* shd, int* shi, float* shf) {
  if (RULE == 3) laq_row<T, NT, MAXV>(wr, cached, w_row, cols, row, bits, codes_row, rowsum, scale, what_row, shd, shi, shf);
  else ternary_row<T, NT, MAXV>(wr, cached, w_row, cols, row, codes_row, rowsum, scale, what_row, shd, shi);
}

template <typename T, int RULE, int NT, int MAXV>
__global__ void __launch_bounds__(NT, NT == TW_NARROW_THREADS ? 8 : (RULE == 2 ? 5 : 4)) closed_form_quantize_kernel(const float* __restrict__ w, int cols,
                                                                      int bits,
                                                                      int8_t* __restrict__ codes,
                                                                      int32_t* __restrict__ rowsum,
                                                                      float* __restrict__ scale, T* __restrict__ what) {
  pdl_trigger();
  pdl_wait();
  __shared__ double shd[64];
  __shared__ int shi[32];
  __shared__ float shf[32];
  const int row = blockIdx.x;
  const long long base = (long long)row * cols;
  const int nvec = cols / 4;
  const bool cached = nvec <= MAXV * NT;
  float4 wr[MAXV];
  if (cached) {
#pragma unroll
    for (int i = 0; i < MAXV; ++i) {
      const int c = threadIdx.x + i * NT;
      if (c < nvec) wr[i] = reinterpret_cast<const float4*>(w + base)[c];
    }
  }
  closed_form_row<T, RULE, NT, MAXV>(wr, cached, w + base, cols, row, bits, codes + base, rowsum, scale,
                     what ? what + base : nullptr, shd, shi, shf);
}

// AdamW on the row (gradient of w_hat passed through unchanged), then the rule on the new weights.
template <typename T, int RULE, int NT, int MAXV>
__global__ void __launch_bounds__(NT, NT == TW_NARROW_THREADS ? 8 : (RULE == 2 ? 5 : 4)) closed_form_update_kernel(float* __restrict__ w, const float* __restrict__ g,
                                                                    float* __restrict__ m, float* __restrict__ v,
                                                                    const OptimScalars* __restrict__ sc, int cols,
                                                                    int train_w, int bits,
                                                                    int8_t* __restrict__ codes,
                                                                    int32_t* __restrict__ rowsum,
                                                                    float* __restrict__ scale, T* __restrict__ what) {
  pdl_trigger();
  pdl_wait();
  __shared__ double shd[64];
  __shared__ int shi[32];
  __shared__ float shf[32];
  const int row = blockIdx.x;
  const OptimScalars o = *sc;
  const long long base = (long long)row * cols;
  const int nvec = cols / 4;
  const bool cached = nvec <= MAXV * NT;
  float4* w4 = reinterpret_cast<float4*>(w + base);
  const float4* g4 = reinterpret_cast<const float4*>(g + base);
  float4* m4 = reinterpret_cast<float4*>(m + base);
  float4* v4 = reinterpret_cast<float4*>(v + base);
  float4 wr[MAXV];
  auto upd = [&](int c) {
    float4 wv = w4[c];
    if (train_w) {
      const float4 d = g4[c];
      float4 mm = m4[c], vv = v4[c];
      wv.x = adam_one(wv.x, d.x, mm.x, vv.x, o, 1.f, -INFINITY);
      wv.y = adam_one(wv.y, d.y, mm.y, vv.y, o, 1.f, -INFINITY);
      wv.z = adam_one(wv.z, d.z, mm.z, vv.z, o, 1.f, -INFINITY);
      wv.w = adam_one(wv.w, d.w, mm.w, vv.w, o, 1.f, -INFINITY);
      w4[c] = wv;
      m4[c] = mm;
      v4[c] = vv;
    }
    return wv;
  };
  if (cached) {
#pragma unroll
    for (int i = 0; i < MAXV; ++i) {
      const int c = threadIdx.x + i * NT;
      if (c < nvec) wr[i] = upd(c);
    }
  } else {
    for (int c = threadIdx.x; c < nvec; c += NT) upd(c);
    __syncthreads();                     // the row is re-read below by other threads of the block
  }
  closed_form_row<T, RULE, NT, MAXV>(wr, cached, w + base, cols, row, bits, codes + base, rowsum, scale,
                     what ? what + base : nullptr, shd, shi, shf);
}

}  // namespace

void launch_closed_form_quantize(const float* w, int rows, int cols, int rule, int bits, int8_t* codes, int32_t* rowsum,
                                 float* scale, void* what, int dt, cudaStream_t st) {
  Scope sc("quantize_weight", (double)rows * cols * (5.0 + (what ? (dt == 1 ? 2.0 : 4.0) : 0.0)) + rows * 8.0, 0, st);
  auto go = [&](auto kernel, int nt, auto* out) { launch_k(kernel, rows, nt, 0, st, w, cols, bits, codes, rowsum, scale, out); };
  const bool narrow = rule == 3 && cols <= TW_NARROW_THREADS * 4 * TW_NARROW_MAXV;
  if (dt == 1) {
    if (narrow) go(closed_form_quantize_kernel<bf16, 3, TW_NARROW_THREADS, TW_NARROW_MAXV>, TW_NARROW_THREADS, (bf16*)what);
    else if (rule == 3) go(closed_form_quantize_kernel<bf16, 3, TW_THREADS, TW_MAXV>, TW_THREADS, (bf16*)what);
    else go(closed_form_quantize_kernel<bf16, 2, TW_THREADS, TW_MAXV>, TW_THREADS, (bf16*)what);
  } else {
    if (narrow) go(closed_form_quantize_kernel<float, 3, TW_NARROW_THREADS, TW_NARROW_MAXV>, TW_NARROW_THREADS, (float*)what);
    else if (rule == 3) go(closed_form_quantize_kernel<float, 3, TW_THREADS, TW_MAXV>, TW_THREADS, (float*)what);
    else go(closed_form_quantize_kernel<float, 2, TW_THREADS, TW_MAXV>, TW_THREADS, (float*)what);
  }
}

void launch_closed_form_update(float* w, const float* g, float* m, float* v, const OptimScalars* sc, int rows, int cols,
                               int train_w, int rule, int bits, int8_t* codes, int32_t* rowsum, float* scale, void* what,
                               int dt, cudaStream_t st) {
  Scope scope("fused_weight_update", (double)rows * cols * (29.0 + (what ? (dt == 1 ? 2.0 : 4.0) : 0.0)), 0, st);
  auto go = [&](auto kernel, int nt, auto* out) {
    launch_k(kernel, rows, nt, 0, st, w, g, m, v, sc, cols, train_w, bits, codes, rowsum, scale, out);
  };
  const bool narrow = rule == 3 && cols <= TW_NARROW_THREADS * 4 * TW_NARROW_MAXV;
  if (dt == 1) {
    if (narrow) go(closed_form_update_kernel<bf16, 3, TW_NARROW_THREADS, TW_NARROW_MAXV>, TW_NARROW_THREADS, (bf16*)what);
    else if (rule == 3) go(closed_form_update_kernel<bf16, 3, TW_THREADS, TW_MAXV>, TW_THREADS, (bf16*)what);
    else go(closed_form_update_kernel<bf16, 2, TW_THREADS, TW_MAXV>, TW_THREADS, (bf16*)what);
  } else {
    if (narrow) go(closed_form_update_kernel<float, 3, TW_NARROW_THREADS, TW_NARROW_MAXV>, TW_NARROW_THREADS, (float*)what);
    else if (rule == 3) go(closed_form_update_kernel<float, 3, TW_THREADS, TW_MAXV>, TW_THREADS, (float*)what);
    else go(closed_form_update_kernel<float, 2, TW_THREADS, TW_MAXV>, TW_THREADS, (float*)what);
  }
}

}  // namespace mrem
