// Output-logit term of the last module (Sec. 4.1: besides the grouped Transformer layers the MSE of the
// output logits is minimised): the classification head, which is not quantized (Sec. 3.1) and therefore
// the same on both sides, applied to the first token of the teacher's and of the student's last layer
// output; loss c * || z_hat - z ||^2 and its gradient with respect to the student's first-token rows,
// added to the loss gradient of the last layer.  The head works on `batch` rows only (about 0.2 GFLOP at
// hidden 1024), so it runs on the CUDA cores in float32 with fixed summation orders: one pass over the
// pooler matrix for the 2 x batch first-token vectors, one block per sequence for the classifier, and one
// pass over the pooler matrix for the gradient.
#include "kernels.h"

namespace mrem {

namespace {

constexpr int HV = 8;                  // vectors (sequences) per block in the two matrix passes

// pooled[v, j] = tanh(bp[j] + sum_i Wp[j, i] * cls[v, i]) for the 2B first-token vectors (student rows 0..B-1, teacher
// rows B..2B-1).  Block: HV vectors (in shared memory) x 32 outputs, one warp per output at a time, the row of Wp
// read once (coalesced) for the HV dot products.
template <typename T>
__global__ void __launch_bounds__(256) head_pool_kernel(const T* __restrict__ f_s, const T* __restrict__ f_t, long long seq_stride,
                                                        int B, int H, const float* __restrict__ wp, const float* __restrict__ bp,
                                                        float* __restrict__ pooled) {
  pdl_trigger();
  pdl_wait();
  extern __shared__ float cls[];                                    // [HV][H]
  const int v0 = blockIdx.y * HV, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int idx = threadIdx.x; idx < HV * H; idx += blockDim.x) {
    const int v = v0 + idx / H, i = idx % H;
    float val = 0.f;
    if (v < 2 * B) val = v < B ? to_f<T>(f_s[(long long)v * seq_stride + i]) : to_f<T>(f_t[(long long)(v - B) * seq_stride + i]);
    cls[idx] = val;
  }
  __syncthreads();
  for (int jj = warp; jj < 32; jj += 8) {
    const int j = blockIdx.x * 32 + jj;
    if (j >= H) break;
    const float* w = wp + (long long)j * H;
    float acc[HV];
#pragma unroll
    for (int v = 0; v < HV; ++v) acc[v] = 0.f;
    for (int i = lane; i < H; i += 32) {
      const float wv = w[i];
#pragma unroll
      for (int v = 0; v < HV; ++v) acc[v] = fmaf(wv, cls[v * H + i], acc[v]);
    }
#pragma unroll
    for (int v = 0; v < HV; ++v) {
      const float t = warp_sum(acc[v]);
      if (lane == 0 && v0 + v < 2 * B) pooled[(long long)(v0 + v) * H + j] = tanhf(t + bp[j]);
    }
  }
}

// One block per sequence: logits of both sides, the squared error, and d loss / d (pooler pre-activation) of the student.
__global__ void __launch_bounds__(256) head_logits_kernel(const float* __restrict__ pooled, int B, int H, int C,
                                                          const float* __restrict__ wc, const float* __restrict__ bc, float cc,
                                                          float* __restrict__ part, float* __restrict__ logits,
                                                          float* __restrict__ dpre) {
  pdl_trigger();
  pdl_wait();
  __shared__ float z_s[64], z_t[64], dz[64];
  const int b = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  const float* ps = pooled + (long long)b * H;
  const float* pt = pooled + (long long)(B + b) * H;
  for (int c = warp; c < C; c += nw) {
    const float* w = wc + (long long)c * H;
    float as = 0.f, at = 0.f;
    for (int i = lane; i < H; i += 32) { const float v = w[i]; as = fmaf(v, ps[i], as); at = fmaf(v, pt[i], at); }
    as = warp_sum(as); at = warp_sum(at);
    if (lane == 0) { z_s[c] = as + bc[c]; z_t[c] = at + bc[c]; }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    float acc = 0.f;
    for (int c = 0; c < C; ++c) {
      const float d = z_s[c] - z_t[c];
      acc += d * d;
      dz[c] = 2.f * cc * d;
      if (logits) { logits[(long long)b * C + c] = z_s[c]; logits[(long long)(B + b) * C + c] = z_t[c]; }
    }
    part[b] = acc;
  }
  __syncthreads();
  for (int i = threadIdx.x; i < H; i += blockDim.x) {
    float a = 0.f;
    for (int c = 0; c < C; ++c) a = fmaf(dz[c], wc[(long long)c * H + i], a);
    dpre[(long long)b * H + i] = a * (1.f - ps[i] * ps[i]);
  }
}

// dF[b, 0, i] += sum_j dpre[b, j] * Wp[j, i].  Block: HV sequences x 64 columns; thread (q, ci) adds the quarter q of
// the j range for column ci (rows of Wp read coalesced), the four quarters are added in index order.
template <typename T>
__global__ void __launch_bounds__(256) head_back_kernel(const float* __restrict__ dpre, int B, int H, const float* __restrict__ wp,
                                                        long long seq_stride, T* __restrict__ dF) {
  pdl_trigger();
  pdl_wait();
  extern __shared__ float sm[];                                     // dp[HV][H], then red[4][HV][64]
  float* dp = sm;
  float* red = sm + HV * H;
  const int b0 = blockIdx.y * HV, ci = threadIdx.x & 63, q = threadIdx.x >> 6, i = blockIdx.x * 64 + ci;
  for (int idx = threadIdx.x; idx < HV * H; idx += blockDim.x) {
    const int b = b0 + idx / H;
    dp[idx] = b < B ? dpre[(long long)b * H + idx % H] : 0.f;
  }
  __syncthreads();
  float acc[HV];
#pragma unroll
  for (int v = 0; v < HV; ++v) acc[v] = 0.f;
  const int per = (H + 3) / 4, j0 = q * per, j1 = min(H, j0 + per);
  if (i < H)
    for (int j = j0; j < j1; ++j) {
      const float w = wp[(long long)j * H + i];
#pragma unroll
      for (int v = 0; v < HV; ++v) acc[v] = fmaf(dp[v * H + j], w, acc[v]);
    }
#pragma unroll
  for (int v = 0; v < HV; ++v) red[(q * HV + v) * 64 + ci] = acc[v];
  __syncthreads();
  for (int idx = threadIdx.x; idx < HV * 64; idx += blockDim.x) {
    const int v = idx / 64, c2 = idx % 64, col = blockIdx.x * 64 + c2, b = b0 + v;
    if (b >= B || col >= H) continue;
    const float a = ((red[(0 * HV + v) * 64 + c2] + red[(1 * HV + v) * 64 + c2]) + red[(2 * HV + v) * 64 + c2]) + red[(3 * HV + v) * 64 + c2];
    T* g = dF + (long long)b * seq_stride + col;
    *g = from_f<T>(to_f<T>(*g) + a);
  }
}

__global__ void head_loss_final_kernel(const float* __restrict__ part, int B, float cc, float* __restrict__ loss_total,
                                       float* __restrict__ logit_loss) {
  pdl_trigger();
  pdl_wait();
  if (threadIdx.x == 0 && blockIdx.x == 0) {
    float acc = 0.f;
    for (int b = 0; b < B; ++b) acc += part[b];
    acc *= cc;
    if (logit_loss) *logit_loss = acc;
    *loss_total += acc;
  }
}

}  // namespace

size_t head_scratch_floats(int B, int H) { return (size_t)3 * B * H + B; }   // pooled [2B, H], dpre [B, H], part [B]

int launch_head_logit_loss(const void* f_s_last, const void* f_t_last, int B, int S, int H, int C, const float* wp,
                           const float* bp, const float* wc, const float* bc, float cc, void* dF_last, float* scratch,
                           float* logits, float* loss_total, float* logit_loss, int dt, cudaStream_t st) {
  if (C > 64 || (size_t)HV * H * sizeof(float) + 4 * HV * 64 * sizeof(float) > 96 * 1024) return -1;
  Scope sc("head_logit_loss", 2.0 * B * ((double)H * H + (double)C * H) * 4.0, 0, st);
  float* pooled = scratch;
  float* dpre = scratch + (size_t)2 * B * H;
  float* part = dpre + (size_t)B * H;
  const long long stride = (long long)S * H;
  const size_t smem_pool = sizeof(float) * HV * H, smem_back = smem_pool + sizeof(float) * 4 * HV * 64;
  const dim3 g_pool((H + 31) / 32, (2 * B + HV - 1) / HV), g_back((H + 63) / 64, (B + HV - 1) / HV);
#define MREM_HEAD(T) do { \
    if (smem_back > 48 * 1024) { \
      cudaFuncSetAttribute(head_pool_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024); \
      cudaFuncSetAttribute(head_back_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024); } \
    launch_k(head_pool_kernel<T>, g_pool, 256, smem_pool, st, (const T*)f_s_last, (const T*)f_t_last, stride, B, H, wp, bp, pooled); \
    launch_k(head_logits_kernel, B, 256, 0, st, (const float*)pooled, B, H, C, wc, bc, cc, part, logits, dpre); \
    launch_k(head_back_kernel<T>, g_back, 256, smem_back, st, (const float*)dpre, B, H, wp, stride, (T*)dF_last); } while (0)
  if (dt == 1) MREM_HEAD(bf16); else MREM_HEAD(float);
#undef MREM_HEAD
  launch_k(head_loss_final_kernel, 1, 32, 0, st, (const float*)part, B, cc, loss_total, logit_loss);
  return cudaGetLastError() == cudaSuccess ? 0 : -2;
}

}  // namespace mrem
