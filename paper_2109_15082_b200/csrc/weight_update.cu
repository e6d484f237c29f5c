// Fused update of one weight matrix and its per-row quantization steps (Algorithm 2:
// Update(w), Update(s)), one block per output row and ONE pass over the row's state:
//   1. straight-through factors of the weight quantizer at the old (w, s): the step
//      gradient ds = sum_k dW_hat * d w_hat / d s (fixed-order block sum),
//   2. AdamW on the row's step (clamped to stay positive),
//   3. AdamW on the latent weights with the masked gradient dW = dW_hat * 1[inside],
//   4. Eq. 1 on the new weights with the new step: int8 codes, row sum, dequantization
//      scale and the dequantized row for the next step's products.
// The row's weights and gradients are read once with 16-byte loads and held in registers
// (rows up to 4096 wide; longer rows are re-read).  Traffic per weight: read w, g, m, v
// (16 B), write w, m, v (12 B), codes (1 B) and the dequantized value (2 or 4 B); the separate
// passes it replaces move about twice that.
#include "optim.cuh"

namespace mrem {

namespace {


// Code of Eq. 1 and the same value as a float.  Integer grid: the sum with 1.5 * 2^23 holds the code in its
// low mantissa bits (two's complement), so neither direction goes through the conversion unit.
__device__ __forceinline__ int weight_code(float w, float s, float r_s, float qmax, int grid, float& qf) {
  if (grid == 0) {      // the exact code without the division instruction (code_f); r_s = RN(1 / s)
    uint32_t bits;
    qf = code_f<false>(w, s, r_s, -qmax, qmax, bits);
    return (int)(int8_t)(bits & 0xffu);
  }
  const float z = __fdiv_rn(w, s);
  const int q = 2 * (int)fminf(fmaxf(floorf(z), -2.f), 1.f) + 1;
  qf = (float)q;
  return q;
}

template <typename T>
__device__ __forceinline__ void store_what4(T* p, float a, float b, float c, float d);
template <>
__device__ __forceinline__ void store_what4<float>(float* p, float a, float b, float c, float d) {
  *reinterpret_cast<float4*>(p) = make_float4(a, b, c, d);
}
template <>
__device__ __forceinline__ void store_what4<bf16>(bf16* p, float a, float b, float c, float d) {
  uint2 t;
  __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&t);
  h[0] = __floats2bfloat162_rn(a, b);
  h[1] = __floats2bfloat162_rn(c, d);
  *reinterpret_cast<uint2*>(p) = t;
}

// NT threads per row, NV float4 vectors per thread kept in registers: (256, 1) for rows up to 1024 wide,
// (512, 2) up to 4096; wider rows are re-read.
// GRID (the weight grid, 0: Eq. 1's integers, 1: half-integer 2-bit levels) is a template parameter: the per-weight code
// then holds one of the two rules, not both under predicates.
template <typename T, int NV, int NT, int GRID>
__global__ void __launch_bounds__(NT, NT == 256 ? 6 : 2) fused_weight_update_kernel(
    float* __restrict__ w, const float* __restrict__ g, float* __restrict__ m, float* __restrict__ v,
    float* __restrict__ steps, const float* __restrict__ ds_in, float* __restrict__ m_s, float* __restrict__ v_s,
    const OptimScalars* __restrict__ sc, int cols, int bits, int train_w, int train_s,
    int8_t* __restrict__ codes, int32_t* __restrict__ rowsum, float* __restrict__ scale, T* __restrict__ what) {
  pdl_trigger();
  pdl_wait();
  constexpr int grid = GRID;
  __shared__ float sh[32];
  __shared__ int shi[32];
  __shared__ float s_new_sh;
  const int row = blockIdx.x;
  const OptimScalars o = *sc;
  const float s_old = steps[row];
  const float r_old = __frcp_rn(s_old);
  float ms_pre = 0.f, vs_pre = 0.f;
  if (threadIdx.x == 0 && train_s) { ms_pre = m_s[row]; vs_pre = v_s[row]; }
  const float qmax = (float)((1 << (bits - 1)) - 1);
  const long long base = (long long)row * cols;
  const int nvec = cols / 4;                                   // cols is a multiple of 16
  const bool cached = nvec <= NV * NT;
  const float4* w4 = reinterpret_cast<const float4*>(w + base);
  const float4* g4 = reinterpret_cast<const float4*>(g + base);
  float4 wr[NV], gr[NV], mr[NV], vr[NV];
  const float4* m4c = reinterpret_cast<const float4*>(m + base);
  const float4* v4c = reinterpret_cast<const float4*>(v + base);
  // 1. step gradient of this row; the masked gradient is kept for step 3.  The moments are fetched now
  //    as well, so that their latency hides behind the reduction and the step's own update.
  float ds = 0.f;
  if (cached) {
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const int c = threadIdx.x + i * NT;
      if (c < nvec) {
        wr[i] = w4[c]; gr[i] = g4[c];
        if (train_w) { mr[i] = m4c[c]; vr[i] = v4c[c]; }
      }
    }
  }
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int c = threadIdx.x + i * NT;
    if (cached && c < nvec) {
      bool in;
      float4 d = gr[i];
      ds = step_grad_acc(ds, wr[i].x, d.x, s_old, r_old, qmax, grid, in); d.x = (in || ds_in) ? d.x : 0.f;
      ds = step_grad_acc(ds, wr[i].y, d.y, s_old, r_old, qmax, grid, in); d.y = (in || ds_in) ? d.y : 0.f;
      ds = step_grad_acc(ds, wr[i].z, d.z, s_old, r_old, qmax, grid, in); d.z = (in || ds_in) ? d.z : 0.f;
      ds = step_grad_acc(ds, wr[i].w, d.w, s_old, r_old, qmax, grid, in); d.w = (in || ds_in) ? d.w : 0.f;
      gr[i] = d;
    }
  }
  if (!cached) {
    for (int c = threadIdx.x; c < nvec; c += NT) {
      const float4 wv = w4[c], d = g4[c];
      bool in;
      ds = step_grad_acc(ds, wv.x, d.x, s_old, r_old, qmax, grid, in);
      ds = step_grad_acc(ds, wv.y, d.y, s_old, r_old, qmax, grid, in);
      ds = step_grad_acc(ds, wv.z, d.z, s_old, r_old, qmax, grid, in);
      ds = step_grad_acc(ds, wv.w, d.w, s_old, r_old, qmax, grid, in);
    }
  }
  ds = block_sum(ds, sh);
  if (ds_in) ds = ds_in[row];          // gradients were masked and reduced before (same arithmetic)
  // 2. the row's step (its moments were fetched before the reduction)
  if (threadIdx.x == 0) {
    float s_new = s_old;
    if (train_s) {
      float ms = ms_pre, vs = vs_pre;
      s_new = adam_one(s_old, ds, ms, vs, o, 0.f, 1e-8f);
      m_s[row] = ms;
      v_s[row] = vs;
      steps[row] = s_new;
    }
    s_new_sh = s_new;
  }
  __syncthreads();
  const float s_new = s_new_sh, r_new = __frcp_rn(s_new);
  const float sc_new = grid == 0 ? s_new : 0.5f * s_new;
  // 3 + 4. weights, then their new codes
  float4* wo = reinterpret_cast<float4*>(w + base);
  float4* m4 = reinterpret_cast<float4*>(m + base);
  float4* v4 = reinterpret_cast<float4*>(v + base);
  int sum = 0;
  auto update = [&](int c, float4 wv, float4 d, float4 mm, float4 vv) {
    if (train_w) {
      wv.x = adam_one(wv.x, d.x, mm.x, vv.x, o, 1.f, -INFINITY);
      wv.y = adam_one(wv.y, d.y, mm.y, vv.y, o, 1.f, -INFINITY);
      wv.z = adam_one(wv.z, d.z, mm.z, vv.z, o, 1.f, -INFINITY);
      wv.w = adam_one(wv.w, d.w, mm.w, vv.w, o, 1.f, -INFINITY);
      wo[c] = wv;
      m4[c] = mm;
      v4[c] = vv;
    }
    float f0, f1, f2, f3;
    const int q0 = weight_code(wv.x, s_new, r_new, qmax, grid, f0), q1 = weight_code(wv.y, s_new, r_new, qmax, grid, f1);
    const int q2 = weight_code(wv.z, s_new, r_new, qmax, grid, f2), q3 = weight_code(wv.w, s_new, r_new, qmax, grid, f3);
    *reinterpret_cast<uint32_t*>(codes + base + 4 * c) =
        (uint32_t)(q0 & 0xff) | ((uint32_t)(q1 & 0xff) << 8) | ((uint32_t)(q2 & 0xff) << 16) | ((uint32_t)(q3 & 0xff) << 24);
    if (what) store_what4<T>(what + base + 4 * c, sc_new * f0, sc_new * f1, sc_new * f2, sc_new * f3);
    sum += q0 + q1 + q2 + q3;
  };
  if (cached) {
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const int c = threadIdx.x + i * NT;
      if (c < nvec) update(c, wr[i], gr[i], mr[i], vr[i]);
    }
  } else {
    for (int c = threadIdx.x; c < nvec; c += NT) {
      const float4 wv = w4[c];
      float4 d = g4[c];
      if (!ds_in) {
        bool in;
        float lvl;
        weight_ste(quotient(wv.x, s_old, r_old), qmax, grid, in, lvl); d.x = in ? d.x : 0.f;
        weight_ste(quotient(wv.y, s_old, r_old), qmax, grid, in, lvl); d.y = in ? d.y : 0.f;
        weight_ste(quotient(wv.z, s_old, r_old), qmax, grid, in, lvl); d.z = in ? d.z : 0.f;
        weight_ste(quotient(wv.w, s_old, r_old), qmax, grid, in, lvl); d.w = in ? d.w : 0.f;
      }
      update(c, wv, d, train_w ? m4[c] : make_float4(0, 0, 0, 0), train_w ? v4[c] : make_float4(0, 0, 0, 0));
    }
  }
  sum = warp_sum_i(sum);
  if ((threadIdx.x & 31) == 0) shi[threadIdx.x >> 5] = sum;
  __syncthreads();
  if (threadIdx.x < 32) {
    int t = threadIdx.x < (blockDim.x >> 5) ? shi[threadIdx.x] : 0;
    t = warp_sum_i(t);
    if (threadIdx.x == 0) {
      rowsum[row] = t;
      scale[row] = sc_new;
    }
  }
}

}  // namespace

void launch_fused_weight_update(float* w, const float* g, float* m, float* v, float* steps, const float* ds_in,
                                float* m_s, float* v_s, const OptimScalars* sc, int rows, int cols, int bits, int grid,
                                int train_w, int train_s, int8_t* codes, int32_t* rowsum, float* scale, void* what,
                                int dt, cudaStream_t st) {
  Scope scope("fused_weight_update", (double)rows * cols * (29.0 + (what ? (dt == 1 ? 2.0 : 4.0) : 0.0)), 0, st);
#define MREM_FWU_G(T, NV, NT, G) launch_k(fused_weight_update_kernel<T, NV, NT, G>, rows, NT, 0, st, w, g, m, v, steps, ds_in, m_s, v_s, sc, cols, bits, train_w, train_s, codes, rowsum, scale, (T*)what)
#define MREM_FWU(T, NV, NT) do { if (grid == 0) MREM_FWU_G(T, NV, NT, 0); else MREM_FWU_G(T, NV, NT, 1); } while (0)
  if (dt == 1) { if (cols <= 1024) MREM_FWU(bf16, 1, 256); else MREM_FWU(bf16, 2, 512); }
  else { if (cols <= 1024) MREM_FWU(float, 1, 256); else MREM_FWU(float, 2, 512); }
#undef MREM_FWU
#undef MREM_FWU_G
}

}  // namespace mrem
