// Output-logit term of the last module (Sec. 4.1: besides the grouped Transformer layers the MSE of the
// output logits is minimised): the classification head, which is not quantized (Sec. 3.1) and therefore
// the same on both sides, applied to the first token of the teacher's and of the student's last layer
// output; loss c * || z_hat - z ||^2 and its gradient with respect to the student's first-token rows,
// added to the loss gradient of the last layer.  The head works on `batch` rows only (33 MFLOP at
// hidden 1024), so it is one block per sequence on the CUDA cores, float32, fixed summation orders.
#include "kernels.h"

namespace mrem {

namespace {

// dynamic shared memory: cls_s[H] cls_t[H] pooled_s[H] pooled_t[H] dpre[H] z_s[C] z_t[C] dz[C]
template <typename T>
__global__ void __launch_bounds__(256) head_logit_kernel(const T* __restrict__ f_s, const T* __restrict__ f_t,
                                                         long long seq_stride, int H, int C,
                                                         const float* __restrict__ wp, const float* __restrict__ bp,
                                                         const float* __restrict__ wc, const float* __restrict__ bc,
                                                         float cc, T* __restrict__ dF, float* __restrict__ part,
                                                         float* __restrict__ logits, int B) {
  pdl_trigger();
  pdl_wait();
  extern __shared__ float sm[];
  float *cls_s = sm, *cls_t = sm + H, *pl_s = sm + 2 * H, *pl_t = sm + 3 * H, *dpre = sm + 4 * H;
  float *z_s = sm + 5 * H, *z_t = z_s + C, *dz = z_t + C;
  const int b = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  const T* rs = f_s + (long long)b * seq_stride;          // first token of sequence b
  const T* rt = f_t + (long long)b * seq_stride;
  for (int i = threadIdx.x; i < H; i += blockDim.x) { cls_s[i] = to_f<T>(rs[i]); cls_t[i] = to_f<T>(rt[i]); }
  __syncthreads();
  // pooler: tanh(Wp cls + bp), one warp per output, both sides from one pass over the row of Wp
  for (int j = warp; j < H; j += nw) {
    const float* w = wp + (long long)j * H;
    float as = 0.f, at = 0.f;
    for (int i = lane; i < H; i += 32) { const float v = w[i]; as = fmaf(v, cls_s[i], as); at = fmaf(v, cls_t[i], at); }
    as = warp_sum(as); at = warp_sum(at);
    if (lane == 0) { pl_s[j] = tanhf(as + bp[j]); pl_t[j] = tanhf(at + bp[j]); }
  }
  __syncthreads();
  // classifier
  for (int c = warp; c < C; c += nw) {
    const float* w = wc + (long long)c * H;
    float as = 0.f, at = 0.f;
    for (int i = lane; i < H; i += 32) { const float v = w[i]; as = fmaf(v, pl_s[i], as); at = fmaf(v, pl_t[i], at); }
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
  // back through the classifier and the tanh
  for (int i = threadIdx.x; i < H; i += blockDim.x) {
    float a = 0.f;
    for (int c = 0; c < C; ++c) a = fmaf(dz[c], wc[(long long)c * H + i], a);
    dpre[i] = a * (1.f - pl_s[i] * pl_s[i]);
  }
  __syncthreads();
  // back through the pooler's matrix (column i of Wp: consecutive threads read consecutive addresses), added to the
  // loss gradient of the last layer at the first token
  T* g = dF + (long long)b * seq_stride;
  for (int i = threadIdx.x; i < H; i += blockDim.x) {
    float a = 0.f;
    for (int j = 0; j < H; ++j) a = fmaf(dpre[j], wp[(long long)j * H + i], a);
    g[i] = from_f<T>(to_f<T>(g[i]) + a);
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

int launch_head_logit_loss(const void* f_s_last, const void* f_t_last, int B, int S, int H, int C, const float* wp,
                           const float* bp, const float* wc, const float* bc, float cc, void* dF_last, float* part,
                           float* logits, float* loss_total, float* logit_loss, int dt, cudaStream_t st) {
  const size_t smem = sizeof(float) * (5 * (size_t)H + 3 * (size_t)C);
  if (smem > 48 * 1024) return -1;
  Scope sc("head_logit_loss", 2.0 * B * ((double)H * H + (double)C * H) * 4.0, 0, st);
  const long long stride = (long long)S * H;
  if (dt == 1)
    launch_k(head_logit_kernel<bf16>, B, 256, smem, st, (const bf16*)f_s_last, (const bf16*)f_t_last, stride, H, C, wp, bp, wc, bc, cc,
             (bf16*)dF_last, part, logits, B);
  else
    launch_k(head_logit_kernel<float>, B, 256, smem, st, (const float*)f_s_last, (const float*)f_t_last, stride, H, C, wp, bp, wc, bc,
             cc, (float*)dF_last, part, logits, B);
  launch_k(head_loss_final_kernel, 1, 32, 0, st, (const float*)part, B, cc, loss_total, logit_loss);
  return cudaGetLastError() == cudaSuccess ? 0 : -2;
}

}  // namespace mrem
