// Row-wise kernels: LayerNorm forward/backward, attention softmax forward/backward (with the
// quantizer of the probabilities), and column sums over rows (bias / LayerNorm-parameter
// gradients).  One warp owns one row and keeps it in registers (one read of each input,
// 8- or 16-byte vector accesses, warp-shuffle reductions); a slower re-reading form covers
// rows too long for the register cache or views that are not vector aligned.
#include "kernels.h"
#include "vec.cuh"

namespace mrem {

namespace {

constexpr int MAXNV = 4;     // vectors per lane held in registers

__device__ __forceinline__ float qz(float x, float s, float off, bool has_off) {
  return __fdiv_rn(has_off ? __fsub_rn(x, off) : x, s);
}
__device__ __forceinline__ int qcode(float z, float lo, float hi) { return __float2int_rn(fminf(fmaxf(z, lo), hi)); }

// 4 consecutive values
template <typename T> __device__ __forceinline__ void load4(const T* p, float* v);
template <> __device__ __forceinline__ void load4<float>(const float* p, float* v) {
  const float4 t = *reinterpret_cast<const float4*>(p);
  v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
}
template <> __device__ __forceinline__ void load4<bf16>(const bf16* p, float* v) {
  const uint2 t = *reinterpret_cast<const uint2*>(p);
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&t);
  const float2 a = __bfloat1622float2(h[0]), b = __bfloat1622float2(h[1]);
  v[0] = a.x; v[1] = a.y; v[2] = b.x; v[3] = b.y;
}
template <typename T> __device__ __forceinline__ void store4(T* p, const float* v);
template <> __device__ __forceinline__ void store4<float>(float* p, const float* v) {
  *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
}
template <> __device__ __forceinline__ void store4<bf16>(bf16* p, const float* v) {
  uint2 t;
  __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&t);
  h[0] = __floats2bfloat162_rn(v[0], v[1]);
  h[1] = __floats2bfloat162_rn(v[2], v[3]);
  *reinterpret_cast<uint2*>(p) = t;
}

// V consecutive floats of a per-column vector (16-byte aligned when V % 4 == 0: the vector paths guarantee it)
template <int V>
__device__ __forceinline__ void load_cols(const float* __restrict__ p, float* v) {
  if constexpr (V % 4 == 0) {
#pragma unroll
    for (int j = 0; j < V; j += 4) {
      const float4 t = __ldg(reinterpret_cast<const float4*>(p + j));
      v[j] = t.x; v[j + 1] = t.y; v[j + 2] = t.z; v[j + 3] = t.w;
    }
  } else {
#pragma unroll
    for (int j = 0; j < V; ++j) v[j] = p[j];
  }
}

// ------------------------------------------------------------------ LayerNorm forward
// CACHED: the row sits in registers (cols <= 32 * V * MAXNV, cols % V == 0); else V == 1 and
// the row is re-read from L1/L2 in each of the three passes.
template <typename T, int V, bool CACHED>
__global__ void __launch_bounds__(128) ln_fwd_kernel(const T* __restrict__ y, const float* __restrict__ gamma,
                                                     const float* __restrict__ beta, float eps, long long rows,
                                                     int cols, T* __restrict__ out, float* __restrict__ mean,
                                                     float* __restrict__ rstd, const float* __restrict__ step,
                                                     float qmax, int8_t* __restrict__ q8, T* __restrict__ qt) {
  pdl_trigger();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const long long row = blockIdx.x * 4ll + (threadIdx.x >> 5);
  if (row >= rows) return;
  const T* yr = y + row * cols;
  float v[CACHED ? MAXNV : 1][V];
  float sum = 0.f;
  if constexpr (CACHED) {
#pragma unroll
    for (int i = 0; i < MAXNV; ++i) {
      const int c = (lane + 32 * i) * V;
      if (c < cols) {
        load_vec<T, V>(yr + c, v[i]);
#pragma unroll
        for (int j = 0; j < V; ++j) sum += v[i][j];
      }
    }
  } else {
    for (int c = lane; c < cols; c += 32) sum += to_f<T>(yr[c]);
  }
  const float mu = warp_sum(sum) / (float)cols;
  float sq = 0.f;
  if constexpr (CACHED) {
#pragma unroll
    for (int i = 0; i < MAXNV; ++i)
      if ((lane + 32 * i) * V < cols) {
#pragma unroll
        for (int j = 0; j < V; ++j) sq += (v[i][j] - mu) * (v[i][j] - mu);
      }
  } else {
    for (int c = lane; c < cols; c += 32) { const float d = to_f<T>(yr[c]) - mu; sq += d * d; }
  }
  const float rs = 1.f / sqrtf(warp_sum(sq) / (float)cols + eps);
  if (lane == 0) {
    if (mean) mean[row] = mu;
    if (rstd) rstd[row] = rs;
  }
  const float s = step ? *step : 1.f, r_s = __frcp_rn(s);
  auto emit = [&](int c, float* o) {
    float gm[V], bt[V];
    load_cols<V>(gamma + c, gm);
    load_cols<V>(beta + c, bt);
#pragma unroll
    for (int j = 0; j < V; ++j) o[j] = (o[j] - mu) * rs * gm[j] + bt[j];
    store_vec<T, V>(out + row * cols + c, o);
    if (step) {
      uint32_t b[V];
#pragma unroll
      for (int j = 0; j < V; ++j) o[j] = code_f<sizeof(T) == 2>(stored<T>(o[j]), s, r_s, -qmax, qmax, b[j]);   // bfloat16-valued numerators are exact
      if (q8) store_code_bytes<V>(q8 + row * cols + c, b);
      if (qt) store_vec<T, V>(qt + row * cols + c, o);
    }
  };
  if constexpr (CACHED) {
#pragma unroll
    for (int i = 0; i < MAXNV; ++i) {
      const int c = (lane + 32 * i) * V;
      if (c < cols) emit(c, v[i]);
    }
  } else {
    for (int c = lane; c < cols; c += 32) {
      float o[V];
      o[0] = to_f<T>(yr[c]);
      emit(c, o);
    }
  }
}

// ------------------------------------------------------------------ LayerNorm backward
template <typename T, int V, bool CACHED>
__global__ void __launch_bounds__(128) ln_bwd_kernel(const T* __restrict__ dout, const T* __restrict__ dout2,
                                                     const T* __restrict__ y, const float* __restrict__ mean,
                                                     const float* __restrict__ rstd, const float* __restrict__ gamma,
                                                     long long rows, int cols, T* __restrict__ dy,
                                                     T* __restrict__ dsum) {
  pdl_trigger();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const long long row = blockIdx.x * 4ll + (threadIdx.x >> 5);
  if (row >= rows) return;
  const float mu = mean[row], rs = rstd[row];
  const long long base = row * cols;
  float d[CACHED ? MAXNV : 1][V], xn[CACHED ? MAXNV : 1][V];
  float s1 = 0.f, s2 = 0.f;
  // total incoming gradient of one vector; written to dsum (rounded to storage) when requested
  auto fetch = [&](int c, float* dv, float* xv) {
    load_vec<T, V>(dout + base + c, dv);
    if (dout2) {
      float e[V];
      load_vec<T, V>(dout2 + base + c, e);
#pragma unroll
      for (int j = 0; j < V; ++j) dv[j] += e[j];
      if (dsum) {
        store_vec<T, V>(dsum + base + c, dv);
#pragma unroll
        for (int j = 0; j < V; ++j) dv[j] = stored<T>(dv[j]);
      }
    }
    load_vec<T, V>(y + base + c, xv);
    float gm[V];
    load_cols<V>(gamma + c, gm);
#pragma unroll
    for (int j = 0; j < V; ++j) {
      xv[j] = (xv[j] - mu) * rs;
      dv[j] *= gm[j];
    }
  };
  if constexpr (CACHED) {
#pragma unroll
    for (int i = 0; i < MAXNV; ++i) {
      const int c = (lane + 32 * i) * V;
      if (c < cols) {
        fetch(c, d[i], xn[i]);
#pragma unroll
        for (int j = 0; j < V; ++j) { s1 += d[i][j]; s2 += d[i][j] * xn[i][j]; }
      }
    }
  } else {
    for (int c = lane; c < cols; c += 32) {
      fetch(c, d[0], xn[0]);
      s1 += d[0][0];
      s2 += d[0][0] * xn[0][0];
    }
  }
  s1 = warp_sum(s1) / (float)cols;
  s2 = warp_sum(s2) / (float)cols;
  if constexpr (CACHED) {
#pragma unroll
    for (int i = 0; i < MAXNV; ++i) {
      const int c = (lane + 32 * i) * V;
      if (c < cols) {
#pragma unroll
        for (int j = 0; j < V; ++j) d[i][j] = rs * (d[i][j] - s1 - xn[i][j] * s2);
        store_vec<T, V>(dy + base + c, d[i]);
      }
    }
  } else {
    const T* dsrc = (dout2 && dsum) ? dsum : dout;
    for (int c = lane; c < cols; c += 32) {
      float dv = to_f<T>(dsrc[base + c]);
      if (dout2 && !dsum) dv += to_f<T>(dout2[base + c]);
      const float x = (to_f<T>(y[base + c]) - mu) * rs;
      dy[base + c] = from_f<T>(rs * (dv * gamma[c] - s1 - x * s2));
    }
  }
}

// ------------------------------------------------------------------ LayerNorm backward fed by a straight-through mask
// The gradient that enters the LayerNorm is assembled on the fly:
//   dv = dout (when given) + 1[lo <= x / step <= hi] * dxhat + add,
// i.e. the straight-through pass of the activation quantizer that saw x (Sec. 3.1.1) followed by the skip
// connection, which the separate kernels write to memory and read back.  dv goes to dsum (the column
// reductions read it) and, rounded as stored, into the LayerNorm backward.  The quantizer's step-size
// gradient leaves as one partial sum per block (fixed order; slots beyond the grid are zeroed).
// Rows up to 32 * V * MAXNV wide, one warp per row, warps stride over the rows.
template <typename T, int V>
__global__ void __launch_bounds__(128, 7) ln_bwd_ste_kernel(const T* __restrict__ dout, const T* __restrict__ x,
                                                         const T* __restrict__ dxhat, const T* __restrict__ add,
                                                         const float* __restrict__ step, float lo, float hi,
                                                         const T* __restrict__ y, const float* __restrict__ mean,
                                                         const float* __restrict__ rstd, const float* __restrict__ gamma,
                                                         long long rows, int cols, T* __restrict__ dy,
                                                         T* __restrict__ dsum, float* __restrict__ part_s, int n_slots) {
  pdl_trigger();
  pdl_wait();
  __shared__ float sh[4];
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const float s = *step, r_s = __frcp_rn(s);
  float ds = 0.f;
  for (long long row = blockIdx.x * 4ll + wid; row < rows; row += gridDim.x * 4ll) {
    const float mu = mean[row], rs = rstd[row];
    const long long base = row * cols;
    float d[MAXNV][V], xn[MAXNV][V];
    float s1 = 0.f, s2 = 0.f;
#pragma unroll
    for (int i = 0; i < MAXNV; ++i) {
      const int c = (lane + 32 * i) * V;
      if (c < cols) {
        float xv[V], e[V];
        load_vec<T, V>(x + base + c, xv);
        load_vec<T, V>(dxhat + base + c, d[i]);
        load_vec<T, V>(add + base + c, e);
#pragma unroll
        for (int j = 0; j < V; ++j) {
          const float z = quotient(xv[j], s, r_s);
          const bool in = z >= lo && z <= hi;
          ds += d[i][j] * (rne_magic(fminf(fmaxf(z, lo), hi)) - (in ? z : 0.f));
          d[i][j] = (in ? d[i][j] : 0.f) + e[j];
        }
        if (dout) {
          load_vec<T, V>(dout + base + c, e);
#pragma unroll
          for (int j = 0; j < V; ++j) d[i][j] += e[j];
        }
        store_vec<T, V>(dsum + base + c, d[i]);
        load_vec<T, V>(y + base + c, xn[i]);
        float gm[V];
        load_cols<V>(gamma + c, gm);
#pragma unroll
        for (int j = 0; j < V; ++j) {
          xn[i][j] = (xn[i][j] - mu) * rs;
          d[i][j] = stored<T>(d[i][j]) * gm[j];
          s1 += d[i][j];
          s2 += d[i][j] * xn[i][j];
        }
      }
    }
    s1 = warp_sum(s1) / (float)cols;
    s2 = warp_sum(s2) / (float)cols;
#pragma unroll
    for (int i = 0; i < MAXNV; ++i) {
      const int c = (lane + 32 * i) * V;
      if (c < cols) {
#pragma unroll
        for (int j = 0; j < V; ++j) d[i][j] = rs * (d[i][j] - s1 - xn[i][j] * s2);
        store_vec<T, V>(dy + base + c, d[i]);
      }
    }
  }
  ds = warp_sum(ds);
  if (lane == 0) sh[wid] = ds;
  __syncthreads();
  if (threadIdx.x == 0) part_s[blockIdx.x] = (sh[0] + sh[1]) + (sh[2] + sh[3]);
  if (blockIdx.x == 0)
    for (int i = gridDim.x + threadIdx.x; i < n_slots; i += blockDim.x) part_s[i] = 0.f;
}

// ------------------------------------------------------------------ column sums over rows
// out0[c] = sum_r a[r,c];  out1[c] = sum_r a[r,c] * (y[r,c] - mean[r]) * rstd[r] (when y);  out2[c] = sum_r a2[r,c]
// (when a2).  A block of 8 x 32 threads owns 8*V columns (one 128-byte line per row for 16-byte vectors) of
// one chunk of rows (gridDim.y chunks): a thread keeps four rows' loads in flight and adds them in row
// order, the block adds its 32 row groups in index order; the last block to finish a column group (ticket
// counter) adds the chunks' partials in index order, so the result does not depend on scheduling.
constexpr int COLRED_CT = 8, COLRED_RT = 32;
template <typename T, int V>
__global__ void __launch_bounds__(256, 2) col_reduce_kernel(const T* __restrict__ a, long long ld_a,
                                                            const T* __restrict__ y, const float* __restrict__ mean,
                                                            const float* __restrict__ rstd, const T* __restrict__ a2,
                                                            long long ld_a2, long long rows, int cols,
                                                            float* __restrict__ out0, float* __restrict__ out1,
                                                            float* __restrict__ out2, float* __restrict__ scratch,
                                                            long long plane, int* __restrict__ counters) {
  pdl_trigger();
  pdl_wait();
  constexpr int BC = COLRED_CT * V;                        // columns per block
  __shared__ float sh[3][COLRED_RT][BC + 1];
  __shared__ int is_last;
  const int tx = threadIdx.x % COLRED_CT, ty = threadIdx.x / COLRED_CT;
  const int c = blockIdx.x * BC + tx * V;
  const int chunks = gridDim.y;
  const long long per = (rows + chunks - 1) / chunks;
  const long long r0 = blockIdx.y * per, r1 = r0 + per < rows ? r0 + per : rows;
  float a0[V], a1[V], a2s[V];
#pragma unroll
  for (int j = 0; j < V; ++j) a0[j] = a1[j] = a2s[j] = 0.f;
  if (c < cols) {
    constexpr int RW = RawWords<T, V>::N;
    for (long long rb = r0 + ty; rb < r1; rb += 4 * COLRED_RT) {
      uint32_t v[4][RW], w[4][RW], u[4][RW];
      float mu[4], rs[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {                       // all loads of four rows first (raw words: few registers)
        const long long r = rb + COLRED_RT * k;
        if (r < r1) {
          load_raw<T, V>(a + r * ld_a + c, v[k]);
          if (y) { load_raw<T, V>(y + r * cols + c, w[k]); mu[k] = mean[r]; rs[k] = rstd[r]; }
          if (a2) load_raw<T, V>(a2 + r * ld_a2 + c, u[k]);
        }
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if (rb + COLRED_RT * k < r1) {
          float fv[V], fw[V];
          widen_raw<T, V>(v[k], fv);
#pragma unroll
          for (int j = 0; j < V; ++j) a0[j] += fv[j];
          if (y) {
            widen_raw<T, V>(w[k], fw);
#pragma unroll
            for (int j = 0; j < V; ++j) a1[j] += fv[j] * (fw[j] - mu[k]) * rs[k];
          }
          if (a2) {
            widen_raw<T, V>(u[k], fw);
#pragma unroll
            for (int j = 0; j < V; ++j) a2s[j] += fw[j];
          }
        }
      }
    }
  }
#pragma unroll
  for (int j = 0; j < V; ++j) { sh[0][ty][tx * V + j] = a0[j]; sh[1][ty][tx * V + j] = a1[j]; sh[2][ty][tx * V + j] = a2s[j]; }
  __syncthreads();
  const int n_planes = a2 ? 3 : (y ? 2 : 1);
  for (int i = threadIdx.x; i < n_planes * BC; i += 256) {
    const int pl = i / BC, col = i - pl * BC, cc = blockIdx.x * BC + col;
    if (cc >= cols || (pl == 1 && !y)) continue;
    float t = 0.f;
#pragma unroll
    for (int k = 0; k < COLRED_RT; ++k) t += sh[pl][k][col];
    scratch[pl * plane + (long long)blockIdx.y * cols + cc] = t;
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) is_last = atomicAdd(&counters[blockIdx.x], 1) == chunks - 1;
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  for (int i = threadIdx.x; i < n_planes * BC; i += 256) {
    const int pl = i / BC, col = i - pl * BC, cc = blockIdx.x * BC + col;
    if (cc >= cols || (pl == 1 && !y)) continue;
    const float* src = scratch + pl * plane + cc;
    float t = 0.f;
    for (int k0 = 0; k0 < chunks; k0 += 8) {               // eight loads in flight, added in index order
      float q[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) q[k] = k0 + k < chunks ? src[(long long)(k0 + k) * cols] : 0.f;
#pragma unroll
      for (int k = 0; k < 8; ++k) t += q[k];
    }
    float* out = pl == 0 ? out0 : (pl == 1 ? out1 : out2);
    out[cc] = t;
  }
  if (threadIdx.x == 0) counters[blockIdx.x] = 0;         // ready for the next launch on this stream
}

// ------------------------------------------------------------------ softmax forward
// CACHED: S % 4 == 0 and S <= 128 * MAXNV; the row of scores stays in registers.
template <typename T, bool CACHED>
__global__ void __launch_bounds__(128) softmax_fwd_kernel(const float* __restrict__ scores,
                                                          const int* __restrict__ valid_len, int h, int S,
                                                          long long rows, T* __restrict__ P,
                                                          const float* __restrict__ step,
                                                          const float* __restrict__ offset, float lo, float hi,
                                                          T* __restrict__ qt) {
  pdl_trigger();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const long long row = blockIdx.x * 4ll + (threadIdx.x >> 5);
  if (row >= rows) return;
  const int b = (int)(row / ((long long)h * S));
  int len = valid_len ? valid_len[b] : S;
  len = len < 1 ? 1 : (len > S ? S : len);
  const float* sr = scores + row * S;
  const float s = step ? *step : 1.f;
  const bool has_off = offset != nullptr;
  const float off = has_off ? *offset : 0.f;
  if constexpr (CACHED) {
    float e[MAXNV][4];
    float mx = -INFINITY;
#pragma unroll
    for (int i = 0; i < MAXNV; ++i) {
      const int c = (lane + 32 * i) * 4;
      if (c < S) {
        load4<float>(sr + c, e[i]);
#pragma unroll
        for (int j = 0; j < 4; ++j) if (c + j < len) mx = fmaxf(mx, e[i][j]);
      }
    }
    mx = warp_max(mx);
    float sum = 0.f;
#pragma unroll
    for (int i = 0; i < MAXNV; ++i) {
      const int c = (lane + 32 * i) * 4;
      if (c < S) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          e[i][j] = c + j < len ? expf(e[i][j] - mx) : 0.f;
          sum += e[i][j];
        }
      }
    }
    sum = warp_sum(sum);
#pragma unroll
    for (int i = 0; i < MAXNV; ++i) {
      const int c = (lane + 32 * i) * 4;
      if (c < S) {
#pragma unroll
        for (int j = 0; j < 4; ++j) e[i][j] = __fdiv_rn(e[i][j], sum);
        store4<T>(P + row * S + c, e[i]);
        if (qt) {
#pragma unroll
          for (int j = 0; j < 4; ++j) e[i][j] = (float)qcode(qz(stored<T>(e[i][j]), s, off, has_off), lo, hi);
          store4<T>(qt + row * S + c, e[i]);
        }
      }
    }
  } else {
    float mx = -INFINITY;
    for (int j = lane; j < len; j += 32) mx = fmaxf(mx, sr[j]);
    mx = warp_max(mx);
    float sum = 0.f;
    for (int j = lane; j < len; j += 32) sum += expf(sr[j] - mx);
    sum = warp_sum(sum);
    for (int j = lane; j < S; j += 32) {
      const float p = j < len ? __fdiv_rn(expf(sr[j] - mx), sum) : 0.f;
      P[row * S + j] = from_f<T>(p);
      if (qt) qt[row * S + j] = from_f<T>((float)qcode(qz(stored<T>(p), s, off, has_off), lo, hi));
    }
  }
}

// ------------------------------------------------------------------ softmax backward with the STE of the P quantizer
template <typename T, bool CACHED>
__global__ void __launch_bounds__(256) softmax_bwd_kernel(const T* __restrict__ P, const T* __restrict__ dphat,
                                                          T* __restrict__ dS, long long rows, int S,
                                                          const float* __restrict__ step, float lo, float hi,
                                                          int quantized, float* __restrict__ part_s) {
  pdl_trigger();
  pdl_wait();
  __shared__ float sh[32];
  const int lane = threadIdx.x & 31;
  const long long warp0 = blockIdx.x * 8ll + (threadIdx.x >> 5), nwarps = gridDim.x * 8ll;
  const float s = quantized ? *step : 1.f, r_s = __frcp_rn(s);
  float ds = 0.f;
  for (long long row = warp0; row < rows; row += nwarps) {
    const long long base = row * S;
    if constexpr (CACHED) {
      float p[MAXNV][4], d[MAXNV][4];
      float dot = 0.f;
#pragma unroll
      for (int i = 0; i < MAXNV; ++i) {
        const int c = (lane + 32 * i) * 4;
        if (c < S) {
          load4<T>(P + base + c, p[i]);
          load4<T>(dphat + base + c, d[i]);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            if (quantized) {
              const float z = quotient(p[i][j], s, r_s);
              const bool in = z >= lo && z <= hi;
              ds += d[i][j] * ((float)qcode(z, lo, hi) - (in ? z : 0.f));
              d[i][j] = in ? d[i][j] : 0.f;
            }
            dot += d[i][j] * p[i][j];
          }
        }
      }
      dot = warp_sum(dot);
#pragma unroll
      for (int i = 0; i < MAXNV; ++i) {
        const int c = (lane + 32 * i) * 4;
        if (c < S) {
#pragma unroll
          for (int j = 0; j < 4; ++j) d[i][j] = p[i][j] * (d[i][j] - dot);
          store4<T>(dS + base + c, d[i]);
        }
      }
    } else {
      float dot = 0.f;
      for (int j = lane; j < S; j += 32) {
        const float p = to_f<T>(P[base + j]);
        float d = to_f<T>(dphat[base + j]);
        if (quantized) {
          const float z = quotient(p, s, r_s);
          const bool in = z >= lo && z <= hi;
          ds += d * ((float)qcode(z, lo, hi) - (in ? z : 0.f));
          d = in ? d : 0.f;
        }
        dot += d * p;
      }
      dot = warp_sum(dot);
      for (int j = lane; j < S; j += 32) {
        const float p = to_f<T>(P[base + j]);
        float d = to_f<T>(dphat[base + j]);
        if (quantized) {
          const float z = quotient(p, s, r_s);
          d = (z >= lo && z <= hi) ? d : 0.f;
        }
        dS[base + j] = from_f<T>(p * (d - dot));
      }
    }
  }
  ds = block_sum(ds, sh);
  if (threadIdx.x == 0 && part_s) part_s[blockIdx.x] = ds;
}

inline bool al16(const void* p) { return p == nullptr || (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

}  // namespace

#define MREM_DT(dt, T, ...)            \
  do {                                 \
    if ((dt) == 1) { using T = bf16; __VA_ARGS__; } else { using T = float; __VA_ARGS__; } \
  } while (0)

void launch_layernorm_fwd(const void* y, const float* gamma, const float* beta, float eps, long long rows, int cols,
                          void* out, float* mean, float* rstd, const float* step, int qmax, int8_t* q8, void* qt,
                          int dt, cudaStream_t st) {
  if (rows <= 0) return;
  Scope sc("layernorm_fwd", (double)rows * cols * ((dt == 1 ? 2.0 : 4.0) * (qt ? 3 : 2) + (q8 ? 1 : 0)), 0, st);
  const int grid = (int)((rows + 3) / 4);
  MREM_DT(dt, T, {
    constexpr int V = 16 / (int)sizeof(T);
    const bool v = cols % V == 0 && cols <= 32 * V * MAXNV && al16(y) && al16(out) && al16(qt) && al16(gamma) && al16(beta) &&
                   (reinterpret_cast<uintptr_t>(q8) % V) == 0;
    if (v) launch_k(ln_fwd_kernel<T, V, true>, grid, 128, 0, st, (const T*)y, gamma, beta, eps, rows, cols, (T*)out, mean, rstd, step, (float)qmax, q8, (T*)qt);
    else launch_k(ln_fwd_kernel<T, 1, false>, grid, 128, 0, st, (const T*)y, gamma, beta, eps, rows, cols, (T*)out, mean, rstd, step, (float)qmax, q8, (T*)qt);
  });
}

void launch_layernorm_bwd(const void* dout, const void* dout2, const void* y, const float* mean, const float* rstd,
                          const float* gamma, long long rows, int cols, void* dy, void* dsum, int dt,
                          cudaStream_t st) {
  if (rows <= 0) return;
  Scope sc("layernorm_bwd", (double)rows * cols * (dt == 1 ? 2.0 : 4.0) * (3 + (dout2 ? 1 : 0) + (dsum ? 1 : 0)), 0, st);
  const int grid = (int)((rows + 3) / 4);
  MREM_DT(dt, T, {
    constexpr int V = 16 / (int)sizeof(T);
    const bool v = cols % V == 0 && cols <= 32 * V * MAXNV && al16(dout) && al16(dout2) && al16(y) && al16(dy) && al16(dsum) && al16(gamma);
    if (v) launch_k(ln_bwd_kernel<T, V, true>, grid, 128, 0, st, (const T*)dout, (const T*)dout2, (const T*)y, mean, rstd, gamma, rows, cols, (T*)dy, (T*)dsum);
    else launch_k(ln_bwd_kernel<T, 1, false>, grid, 128, 0, st, (const T*)dout, (const T*)dout2, (const T*)y, mean, rstd, gamma, rows, cols, (T*)dy, (T*)dsum);
  });
}

bool layernorm_bwd_ste_supported(int cols, int dt) {
  const int V = dt == 1 ? 8 : 4;
  return cols % V == 0 && cols <= 32 * V * MAXNV;
}

bool launch_layernorm_bwd_ste(const void* dout, const void* x, const void* dxhat, const void* add, const float* step,
                              int lo, int hi, const void* y, const float* mean, const float* rstd, const float* gamma,
                              long long rows, int cols, void* dy, void* dsum, float* part_s, int dt, cudaStream_t st) {
  if (rows <= 0) return false;
  bool done = false;
  MREM_DT(dt, T, {
    constexpr int V = 16 / (int)sizeof(T);
    const bool v = cols % V == 0 && cols <= 32 * V * MAXNV && al16(dout) && al16(x) && al16(dxhat) && al16(add) && al16(y) &&
                   al16(dy) && al16(dsum) && al16(gamma);
    if (v) {
      Scope sc("layernorm_bwd_ste", (double)rows * cols * (dt == 1 ? 2.0 : 4.0) * (6 + (dout ? 1 : 0)), 0, st);
      const long long want = (rows + 3) / 4;
      const int grid = (int)(want < RED_BLOCKS ? want : RED_BLOCKS);
      launch_k(ln_bwd_ste_kernel<T, V>, grid, 128, 0, st, (const T*)dout, (const T*)x, (const T*)dxhat, (const T*)add, step,
               (float)lo, (float)hi, (const T*)y, mean, rstd, gamma, rows, cols, (T*)dy, (T*)dsum, part_s, RED_BLOCKS);
      done = true;
    }
  });
  return done;
}

void launch_col_reduce(const void* a, long long ld_a, const void* y, const float* mean, const float* rstd,
                       const void* a2, long long ld_a2, long long rows, int cols, float* out0, float* out1,
                       float* out2, float* scratch, long long plane_floats, int* counters, int dt, cudaStream_t st) {
  Scope sc("col_reduce", (double)rows * cols * (dt == 1 ? 2.0 : 4.0) * (1 + (y ? 1 : 0) + (a2 ? 1 : 0)), 0, st);
  // as many row chunks as one plane of the scratch holds, up to two blocks per SM (one wave) and 128 rows per chunk
#define MREM_COLRED(T, V) do { const int col_blocks = (cols + COLRED_CT * V - 1) / (COLRED_CT * V); \
    long long chunks = plane_floats / cols; \
    if (chunks > 288 / col_blocks) chunks = 288 / col_blocks; \
    if (chunks > (rows + 4 * COLRED_RT - 1) / (4 * COLRED_RT)) chunks = (rows + 4 * COLRED_RT - 1) / (4 * COLRED_RT); \
    if (chunks < 1) chunks = 1; \
    dim3 grid(col_blocks, (unsigned)chunks); \
    launch_k(col_reduce_kernel<T, V>, grid, 256, 0, st, (const T*)a, ld_a, (const T*)y, mean, rstd, (const T*)a2, ld_a2, rows, cols, out0, out1, out2, scratch, plane_floats, counters); } while (0)
  const bool vec_ok = cols % 8 == 0 && ld_a % 8 == 0 && ld_a2 % 8 == 0 && al16(a) && al16(y) && al16(a2);
  if (dt == 1) { if (vec_ok) MREM_COLRED(bf16, 8); else MREM_COLRED(bf16, 1); }
  else { if (vec_ok) MREM_COLRED(float, 4); else MREM_COLRED(float, 1); }
#undef MREM_COLRED
}

void launch_softmax_fwd(const float* scores, const int* valid_len, int B, int h, int S, void* P, const float* step,
                        const float* offset, int lo, int hi, void* qt, int dt, cudaStream_t st) {
  const long long rows = (long long)B * h * S;
  if (rows <= 0) return;
  Scope sc("softmax_fwd", (double)rows * S * (4.0 + (dt == 1 ? 2.0 : 4.0) * (qt ? 2 : 1)), 0, st);
  const int grid = (int)((rows + 3) / 4);
  const bool cached = S % 4 == 0 && S <= 128 * MAXNV && al16(scores) && al16(P) && al16(qt);
  MREM_DT(dt, T, {
    if (cached) launch_k(softmax_fwd_kernel<T, true>, grid, 128, 0, st, scores, valid_len, h, S, rows, (T*)P, step, offset, (float)lo, (float)hi, (T*)qt);
    else launch_k(softmax_fwd_kernel<T, false>, grid, 128, 0, st, scores, valid_len, h, S, rows, (T*)P, step, offset, (float)lo, (float)hi, (T*)qt);
  });
}

void launch_softmax_bwd(const void* P, const void* dphat, void* dS, long long rows, int S, const float* step,
                        int lo, int hi, int quantized, float* part_s, int dt, cudaStream_t st) {
  Scope sc("softmax_bwd", (double)rows * S * 3 * (dt == 1 ? 2.0 : 4.0), 0, st);
  const bool cached = S % 4 == 0 && S <= 128 * MAXNV && al16(P) && al16(dphat) && al16(dS);
  MREM_DT(dt, T, {
    if (cached) launch_k(softmax_bwd_kernel<T, true>, RED_BLOCKS, 256, 0, st, (const T*)P, (const T*)dphat, (T*)dS, rows, S, step, (float)lo, (float)hi, quantized, part_s);
    else launch_k(softmax_bwd_kernel<T, false>, RED_BLOCKS, 256, 0, st, (const T*)P, (const T*)dphat, (T*)dS, rows, S, step, (float)lo, (float)hi, quantized, part_s);
  });
}

}  // namespace mrem
