// Quantizer kernels (Eq. 1 of the paper) and step-size initialisation.  HBM-bound:
// 16-byte vector loads/stores, one pass over each tensor, warp-shuffle reductions.
#include "kernels.h"
#include "vec.cuh"

namespace mrem {

namespace {

// ------------------------------------------------------------------ weight quantizer
// One block per output row.  grid 0: q = rne(clip(w/s, -qmax, qmax)); grid 1 (2-bit,
// levels (k+0.5)s): c = 2*clip(floor(w/s), -2, 1) + 1 with scale s/2.
template <typename T>
__global__ void __launch_bounds__(256) quantize_weight_kernel(const float* __restrict__ w, int cols,
                                                              const float* __restrict__ steps, int per_row, int bits,
                                                              int grid, int8_t* __restrict__ codes,
                                                              int32_t* __restrict__ rowsum, float* __restrict__ scale,
                                                              T* __restrict__ what) {
  pdl_trigger();
  pdl_wait();
  __shared__ int sh[32];
  const int row = blockIdx.x;
  const float s = steps[per_row ? row : 0];
  const float sc = grid == 0 ? s : 0.5f * s;
  const float qmax = (float)((1 << (bits - 1)) - 1);
  const float* wr = w + (long long)row * cols;
  int8_t* cr = codes + (long long)row * cols;
  T* hr = what ? what + (long long)row * cols : nullptr;
  int sum = 0;
  for (int c = threadIdx.x; c < cols; c += blockDim.x) {
    const float z = __fdiv_rn(wr[c], s);
    int q;
    if (grid == 0) q = __float2int_rn(fminf(fmaxf(z, -qmax), qmax));
    else q = 2 * (int)fminf(fmaxf(floorf(z), -2.f), 1.f) + 1;
    cr[c] = (int8_t)q;
    if (hr) hr[c] = from_f<T>(sc * (float)q);
    sum += q;
  }
  sum = warp_sum_i(sum);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = sum;
  __syncthreads();
  if (threadIdx.x < 32) {
    int v = threadIdx.x < (blockDim.x >> 5) ? sh[threadIdx.x] : 0;
    v = warp_sum_i(v);
    if (threadIdx.x == 0) {
      rowsum[row] = v;
      scale[row] = sc;
    }
  }
}

// ------------------------------------------------------------------ activation quantizer
__device__ __forceinline__ int act_code(float x, float s, float r_s, float off, bool has_off, float lo, float hi) {
  return code_of(has_off ? __fsub_rn(x, off) : x, s, r_s, lo, hi);
}

template <typename T, int V>
__global__ void __launch_bounds__(256) quantize_act_kernel(const T* __restrict__ x, long long rows, int cols,
                                                           long long ld_x, const float* __restrict__ step,
                                                           const float* __restrict__ offset, float lo, float hi,
                                                           int8_t* __restrict__ q8, long long ld_q8,
                                                           T* __restrict__ qt, long long ld_qt, int seg_cols,
                                                           const float* __restrict__ step1,
                                                           const float* __restrict__ step2) {
  pdl_trigger();
  pdl_wait();
  // seg_cols > 0: three column segments of that width (a multiple of V), each with its own step
  const float s0 = *step, s1 = seg_cols ? *step1 : s0, s2 = seg_cols ? *step2 : s0;
  const float r0 = __frcp_rn(s0), r1 = __frcp_rn(s1), r2 = __frcp_rn(s2);
  const bool has_off = offset != nullptr;
  const float off = has_off ? *offset : 0.f;
  const int vcols = cols / V;
  const long long total = rows * vcols;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const long long r = i / vcols;
    const int c = (int)(i - r * vcols) * V;
    float v[V];
    load_vec<T, V>(x + r * ld_x + c, v);
    const int seg = !seg_cols || c < seg_cols ? 0 : (c < 2 * seg_cols ? 1 : 2);
    const float s = seg == 0 ? s0 : (seg == 1 ? s1 : s2), r_s = seg == 0 ? r0 : (seg == 1 ? r1 : r2);
    int q[V];
#pragma unroll
    for (int j = 0; j < V; ++j) q[j] = act_code(v[j], s, r_s, off, has_off, lo, hi);
    if (q8) store_codes<V>(q8 + r * ld_q8 + c, q);
    if (qt) {
#pragma unroll
      for (int j = 0; j < V; ++j) v[j] = (float)q[j];
      store_vec<T, V>(qt + r * ld_qt + c, v);
    }
  }
}

// The vector form: TPR threads walk one row's 16-byte vectors (TPR divides the vector count of a row where possible),
// 256 / TPR rows per block round; no index divisions, codes by code_f, packed stores.
template <typename T, int V, int TPR>
__global__ void __launch_bounds__(256) quantize_act_rows_kernel(const T* __restrict__ x, long long rows, int cols,
                                                                long long ld_x, const float* __restrict__ step,
                                                                const float* __restrict__ offset, float lo, float hi,
                                                                int8_t* __restrict__ q8, long long ld_q8,
                                                                T* __restrict__ qt, long long ld_qt, int seg_cols,
                                                                const float* __restrict__ step1,
                                                                const float* __restrict__ step2) {
  pdl_trigger();
  pdl_wait();
  const float s0 = *step, s1 = seg_cols ? *step1 : s0, s2 = seg_cols ? *step2 : s0;
  const float r0 = __frcp_rn(s0), r1 = __frcp_rn(s1), r2 = __frcp_rn(s2);
  const bool has_off = offset != nullptr;
  const float off = has_off ? *offset : 0.f;
  constexpr int RPB = 256 / TPR;
  const int tr = threadIdx.x / TPR, tc = threadIdx.x % TPR, vcols = cols / V;
  for (long long r = blockIdx.x * (long long)RPB + tr; r < rows; r += (long long)gridDim.x * RPB) {
    const T* xr = x + r * ld_x;
#pragma unroll 2
    for (int cv = tc; cv < vcols; cv += TPR) {
      const int c = cv * V;
      float v[V];
      load_vec<T, V>(xr + c, v);
      const int seg = !seg_cols || c < seg_cols ? 0 : (c < 2 * seg_cols ? 1 : 2);
      const float s = seg == 0 ? s0 : (seg == 1 ? s1 : s2), r_s = seg == 0 ? r0 : (seg == 1 ? r1 : r2);
      uint32_t b[V];
      if (sizeof(T) == 2 && !has_off) {                    // bfloat16 numerators: the quotient is the exact one
#pragma unroll
        for (int j = 0; j < V; ++j) v[j] = code_f<true>(v[j], s, r_s, lo, hi, b[j]);
      } else {
#pragma unroll
        for (int j = 0; j < V; ++j) v[j] = code_f<false>(has_off ? __fsub_rn(v[j], off) : v[j], s, r_s, lo, hi, b[j]);
      }
      if (q8) store_code_bytes<V>(q8 + r * ld_q8 + c, b);
      if (qt) store_vec<T, V>(qt + r * ld_qt + c, v);
    }
  }
}

template <typename T, int V>
__global__ void __launch_bounds__(256) mix_kernel(const T* __restrict__ f, const T* __restrict__ fh, float lam,
                                                  T* __restrict__ out, long long n) {
  pdl_trigger();
  pdl_wait();
  for (long long i = (blockIdx.x * (long long)blockDim.x + threadIdx.x) * V; i < n; i += (long long)gridDim.x * blockDim.x * V) {
    float a[V], b[V];
    load_vec<T, V>(f + i, a);
    load_vec<T, V>(fh + i, b);
#pragma unroll
    for (int j = 0; j < V; ++j) a[j] = lam * a[j] + (1.f - lam) * b[j];
    store_vec<T, V>(out + i, a);
  }
}

// g = stored(gelu(u)), then the quantizer of the GELU site.
template <typename T, int V>
__global__ void __launch_bounds__(256) gelu_quant_kernel(const T* __restrict__ u, long long n,
                                                         const float* __restrict__ step,
                                                         const float* __restrict__ offset, float lo, float hi,
                                                         int8_t* __restrict__ q8, T* __restrict__ qt) {
  pdl_trigger();
  pdl_wait();
  const float s = *step, r_s = __frcp_rn(s);
  const bool has_off = offset != nullptr;
  const float off = has_off ? *offset : 0.f;
  for (long long i = (blockIdx.x * (long long)blockDim.x + threadIdx.x) * V; i < n; i += (long long)gridDim.x * blockDim.x * V) {
    float v[V];
    load_vec<T, V>(u + i, v);
    uint32_t b[V];
    if (sizeof(T) == 2 && !has_off) {
#pragma unroll
      for (int j = 0; j < V; ++j) v[j] = code_f<true>(stored<T>(gelu_erf(v[j])), s, r_s, lo, hi, b[j]);
    } else {
#pragma unroll
      for (int j = 0; j < V; ++j) {
        const float g = stored<T>(gelu_erf(v[j]));
        v[j] = code_f<false>(has_off ? __fsub_rn(g, off) : g, s, r_s, lo, hi, b[j]);
      }
    }
    if (q8) store_code_bytes<V>(q8 + i, b);
    if (qt) store_vec<T, V>(qt + i, v);
  }
}

// ------------------------------------------------------------------ step initialisation
// stat[row] = max|w| (rule 0) or mean|w| (rule 1) of one row; per_row: steps[row] = stat/qmax | stat.
__global__ void __launch_bounds__(256) weight_row_stat_kernel(const float* __restrict__ w, int cols, int rule,
                                                              float* __restrict__ stat) {
  pdl_trigger();
  pdl_wait();
  __shared__ float sh[32];
  const float* wr = w + (long long)blockIdx.x * cols;
  float acc = 0.f;
  for (int c = threadIdx.x; c < cols; c += blockDim.x) {
    const float a = fabsf(wr[c]);
    acc = rule == 0 ? fmaxf(acc, a) : acc + a;
  }
  acc = rule == 0 ? block_max(acc, sh) : block_sum(acc, sh);
  if (threadIdx.x == 0) stat[blockIdx.x] = acc;
}
__global__ void weight_steps_from_stat_kernel(const float* __restrict__ stat, int rows, int cols, int per_row,
                                              int rule, float qmax, float* __restrict__ steps) {
  pdl_trigger();
  pdl_wait();
  if (per_row) {
    for (int r = blockIdx.x * blockDim.x + threadIdx.x; r < rows; r += gridDim.x * blockDim.x) {
      const float v = rule == 0 ? __fdiv_rn(stat[r], qmax) : __fdiv_rn(stat[r], (float)cols);
      steps[r] = fmaxf(v, 1e-8f);
    }
  } else if (blockIdx.x == 0 && threadIdx.x == 0) {
    float acc = 0.f;
    for (int r = 0; r < rows; ++r) acc = rule == 0 ? fmaxf(acc, stat[r]) : acc + stat[r];
    const float v = rule == 0 ? __fdiv_rn(acc, qmax) : __fdiv_rn(acc, (float)rows * (float)cols);
    steps[0] = fmaxf(v, 1e-8f);
  }
}

template <typename T>
__global__ void __launch_bounds__(256) minmax_kernel(const T* __restrict__ x, long long ld, long long rows, int cols,
                                                     float* __restrict__ part) {
  pdl_trigger();
  pdl_wait();
  __shared__ float sh[32];
  float lo = INFINITY, hi = -INFINITY;
  const long long total = rows * cols;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const long long r = i / cols;
    const float v = to_f<T>(x[r * ld + (i - r * cols)]);
    lo = fminf(lo, v);
    hi = fmaxf(hi, v);
  }
  hi = block_max(hi, sh);
  lo = -block_max(-lo, sh);
  if (threadIdx.x == 0) {
    part[blockIdx.x] = lo;
    part[gridDim.x + blockIdx.x] = hi;
  }
}
__global__ void minmax_final_kernel(const float* __restrict__ part, int n, float* __restrict__ out) {
  pdl_trigger();
  pdl_wait();
  if (threadIdx.x == 0 && blockIdx.x == 0) {
    float lo = INFINITY, hi = -INFINITY;
    for (int i = 0; i < n; ++i) {
      lo = fminf(lo, part[i]);
      hi = fmaxf(hi, part[n + i]);
    }
    out[0] = lo;
    out[1] = hi;
  }
}
__global__ void step_from_minmax_kernel(const float* __restrict__ mm, int mode, float qmax, float* step, float* offset) {
  pdl_trigger();
  pdl_wait();
  if (threadIdx.x == 0 && blockIdx.x == 0) {
    float s, o = 0.f;
    if (mode == 0) s = __fdiv_rn(fmaxf(fabsf(mm[0]), fabsf(mm[1])), qmax);
    else if (mode == 1) s = __fdiv_rn(mm[1], qmax);
    else { s = __fdiv_rn(__fsub_rn(mm[1], mm[0]), qmax); o = mm[0]; }
    *step = fmaxf(s, 1e-8f);
    if (offset) *offset = o;
  }
}

__global__ void __launch_bounds__(256) gather_rows_kernel(const uint4* __restrict__ src, const int* __restrict__ idx,
                                                          long long row_vecs, uint4* __restrict__ out) {
  pdl_trigger();
  pdl_wait();
  const uint4* s = src + (long long)idx[blockIdx.y] * row_vecs;
  uint4* o = out + (long long)blockIdx.y * row_vecs;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < row_vecs; i += (long long)gridDim.x * blockDim.x)
    o[i] = s[i];
}

__global__ void __launch_bounds__(256) widen_bf16_kernel(const bf16* __restrict__ src, float* __restrict__ dst, long long n) {
  pdl_trigger();
  pdl_wait();
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
    dst[i] = __bfloat162float(src[i]);
}

template <typename T>
__global__ void __launch_bounds__(256) narrow_kernel(const float* __restrict__ src, T* __restrict__ dst, long long n) {
  pdl_trigger();
  pdl_wait();
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
    dst[i] = from_f<T>(src[i]);
}

inline int grid_for(long long work_items, int threads = 256, int cap = 148 * 8) {
  long long b = (work_items + threads - 1) / threads;
  if (b < 1) b = 1;
  return (int)(b < cap ? b : cap);
}

template <typename T>
bool vec_ok(const void* p, long long ld, int cols) {
  constexpr int V = 16 / (int)sizeof(T);
  return p == nullptr || ((reinterpret_cast<uintptr_t>(p) & 15) == 0 && ld % V == 0 && cols % V == 0);
}

}  // namespace

void launch_quantize_weight(const float* w, int rows, int cols, const float* steps, int per_row, int bits, int grid,
                            int8_t* codes, int32_t* rowsum, float* scale, void* what, int dt, cudaStream_t st) {
  Scope sc("quantize_weight", (double)rows * cols * (5.0 + (what ? (dt == 1 ? 2.0 : 4.0) : 0.0)) + rows * 8.0, 0, st);
  if (dt == 1)
    launch_k(quantize_weight_kernel<bf16>, rows, 256, 0, st, w, cols, steps, per_row, bits, grid, codes, rowsum, scale, (bf16*)what);
  else
    launch_k(quantize_weight_kernel<float>, rows, 256, 0, st, w, cols, steps, per_row, bits, grid, codes, rowsum, scale, (float*)what);
}

template <typename T>
static void quantize_act_t(const T* x, long long rows, int cols, long long ld_x, const float* step, const float* offset,
                           int lo, int hi, int8_t* q8, long long ld_q8, T* qt, long long ld_qt, int seg_cols,
                           const float* step1, const float* step2, cudaStream_t st) {
  constexpr int V = 16 / (int)sizeof(T);
  const bool v = vec_ok<T>(x, ld_x, cols) && vec_ok<T>(qt, ld_qt, cols) && seg_cols % V == 0 &&
                 (q8 == nullptr || ((reinterpret_cast<uintptr_t>(q8) % V) == 0 && ld_q8 % V == 0));
  if (v) {
    const int vcols = cols / V;
#define MREM_QROWS(TPR) do { const long long want = (rows + 256 / TPR - 1) / (256 / TPR); \
      launch_k(quantize_act_rows_kernel<T, V, TPR>, (int)(want < RED_BLOCKS ? want : RED_BLOCKS), 256, 0, st, x, rows, cols, ld_x, step, offset, (float)lo, (float)hi, q8, ld_q8, qt, ld_qt, seg_cols, step1, step2); } while (0)
    if (vcols % 128 == 0) MREM_QROWS(128);
    else if (vcols % 64 == 0) MREM_QROWS(64);
    else if (vcols >= 128) MREM_QROWS(128);
    else MREM_QROWS(32);
#undef MREM_QROWS
  } else
    launch_k(quantize_act_kernel<T, 1>, grid_for(rows * cols), 256, 0, st, x, rows, cols, ld_x, step, offset, (float)lo, (float)hi, q8, ld_q8, qt, ld_qt, seg_cols, step1, step2);
}

void launch_quantize_act(const void* x, int dt, long long rows, int cols, long long ld_x, const float* step,
                         const float* offset, int lo, int hi, int8_t* q8, long long ld_q8, void* qt,
                         long long ld_qt, cudaStream_t st) {
  if (rows <= 0 || cols <= 0) return;
  Scope sc("quantize_act", (double)rows * cols * ((dt == 1 ? 2.0 : 4.0) * (qt ? 2 : 1) + (q8 ? 1 : 0)), 0, st);
  if (dt == 1) quantize_act_t<bf16>((const bf16*)x, rows, cols, ld_x, step, offset, lo, hi, q8, ld_q8, (bf16*)qt, ld_qt, 0, nullptr, nullptr, st);
  else quantize_act_t<float>((const float*)x, rows, cols, ld_x, step, offset, lo, hi, q8, ld_q8, (float*)qt, ld_qt, 0, nullptr, nullptr, st);
}

void launch_quantize_act3(const void* x, int dt, long long rows, int seg_cols, long long ld_x, const float* step0,
                          const float* step1, const float* step2, int lo, int hi, void* qt, long long ld_qt,
                          cudaStream_t st) {
  if (rows <= 0 || seg_cols <= 0) return;
  Scope sc("quantize_act", (double)rows * 3 * seg_cols * (dt == 1 ? 2.0 : 4.0) * 2, 0, st);
  if (dt == 1) quantize_act_t<bf16>((const bf16*)x, rows, 3 * seg_cols, ld_x, step0, nullptr, lo, hi, nullptr, 0, (bf16*)qt, ld_qt, seg_cols, step1, step2, st);
  else quantize_act_t<float>((const float*)x, rows, 3 * seg_cols, ld_x, step0, nullptr, lo, hi, nullptr, 0, (float*)qt, ld_qt, seg_cols, step1, step2, st);
}

void launch_widen_bf16(const void* src, float* dst, long long n, cudaStream_t st) {
  if (n > 0) launch_k(widen_bf16_kernel, grid_for(n), 256, 0, st, (const bf16*)src, dst, n);
}

void launch_narrow(const float* src, void* dst, long long n, int dt, cudaStream_t st) {
  if (n <= 0) return;
  if (dt == 1) launch_k(narrow_kernel<bf16>, grid_for(n), 256, 0, st, src, (bf16*)dst, n);
  else launch_k(narrow_kernel<float>, grid_for(n), 256, 0, st, src, (float*)dst, n);
}

void launch_mix(const void* f, const void* f_hat, float lam, void* out, long long n, int dt, cudaStream_t st) {
  if (n <= 0) return;
  Scope sc("teacher_forcing_mix", (double)n * 3 * (dt == 1 ? 2.0 : 4.0), 0, st);
  if (dt == 1) {
    if (n % 8 == 0 && vec_ok<bf16>(f, 8, 8) && vec_ok<bf16>(f_hat, 8, 8) && vec_ok<bf16>(out, 8, 8))
      launch_k(mix_kernel<bf16, 8>, grid_for(n / 8), 256, 0, st, (const bf16*)f, (const bf16*)f_hat, lam, (bf16*)out, n);
    else
      launch_k(mix_kernel<bf16, 1>, grid_for(n), 256, 0, st, (const bf16*)f, (const bf16*)f_hat, lam, (bf16*)out, n);
  } else {
    if (n % 4 == 0 && vec_ok<float>(f, 4, 4) && vec_ok<float>(f_hat, 4, 4) && vec_ok<float>(out, 4, 4))
      launch_k(mix_kernel<float, 4>, grid_for(n / 4), 256, 0, st, (const float*)f, (const float*)f_hat, lam, (float*)out, n);
    else
      launch_k(mix_kernel<float, 1>, grid_for(n), 256, 0, st, (const float*)f, (const float*)f_hat, lam, (float*)out, n);
  }
}

void launch_gelu_quant(const void* u, long long n, const float* step, const float* offset, int lo, int hi,
                       int8_t* q8, void* qt, int dt, cudaStream_t st) {
  if (n <= 0) return;
  Scope sc("gelu_quant", (double)n * ((dt == 1 ? 2.0 : 4.0) * (qt ? 2 : 1) + (q8 ? 1 : 0)), 0, st);
  if (dt == 1) {
    const bool v = n % 8 == 0 && vec_ok<bf16>(u, 8, 8) && vec_ok<bf16>(qt, 8, 8) && (reinterpret_cast<uintptr_t>(q8) % 8) == 0;
    if (v) launch_k(gelu_quant_kernel<bf16, 8>, grid_for(n / 8), 256, 0, st, (const bf16*)u, n, step, offset, (float)lo, (float)hi, q8, (bf16*)qt);
    else launch_k(gelu_quant_kernel<bf16, 1>, grid_for(n), 256, 0, st, (const bf16*)u, n, step, offset, (float)lo, (float)hi, q8, (bf16*)qt);
  } else {
    const bool v = n % 4 == 0 && vec_ok<float>(u, 4, 4) && vec_ok<float>(qt, 4, 4) && (reinterpret_cast<uintptr_t>(q8) % 4) == 0;
    if (v) launch_k(gelu_quant_kernel<float, 4>, grid_for(n / 4), 256, 0, st, (const float*)u, n, step, offset, (float)lo, (float)hi, q8, (float*)qt);
    else launch_k(gelu_quant_kernel<float, 1>, grid_for(n), 256, 0, st, (const float*)u, n, step, offset, (float)lo, (float)hi, q8, (float*)qt);
  }
}

void launch_init_weight_steps(const float* w, int rows, int cols, int per_row, int rule, float qmax, float* steps,
                              float* scratch, cudaStream_t st) {
  launch_k(weight_row_stat_kernel, rows, 256, 0, st, w, cols, rule, scratch);
  launch_k(weight_steps_from_stat_kernel, per_row ? (rows + 255) / 256 : 1, 256, 0, st, scratch, rows, cols, per_row, rule, qmax, steps);
}

void launch_minmax(const void* x, long long ld, long long rows, int cols, float* out, float* scratch, int dt,
                   cudaStream_t st) {
  if (dt == 1) launch_k(minmax_kernel<bf16>, RED_BLOCKS, 256, 0, st, (const bf16*)x, ld, rows, cols, scratch);
  else launch_k(minmax_kernel<float>, RED_BLOCKS, 256, 0, st, (const float*)x, ld, rows, cols, scratch);
  launch_k(minmax_final_kernel, 1, 32, 0, st, scratch, RED_BLOCKS, out);
}

void launch_step_from_minmax(const float* minmax, int mode, float qmax, float* step, float* offset, cudaStream_t st) {
  launch_k(step_from_minmax_kernel, 1, 32, 0, st, minmax, mode, qmax, step, offset);
}

void launch_gather_rows(const void* src, const int* d_idx, int n_rows, long long row_bytes, void* out,
                        cudaStream_t st) {
  const long long row_vecs = row_bytes / 16;
  Scope sc("gather_rows", 2.0 * n_rows * (double)row_bytes, 0, st);
  dim3 grid(grid_for(row_vecs, 256, 64), n_rows);
  launch_k(gather_rows_kernel, grid, 256, 0, st, (const uint4*)src, d_idx, row_vecs, (uint4*)out);
}

}  // namespace mrem
