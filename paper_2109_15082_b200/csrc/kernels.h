// Launchers of the HBM-bound kernels of the reconstruction step.  `dt` is the storage type
// of activations: 0 = float32, 1 = bfloat16.  All launches are asynchronous on `st`.
#pragma once
#include "mrem_common.cuh"
#include "trace.h"

namespace mrem {

constexpr int RED_BLOCKS = 1184;    // grid of every kernel that emits per-block partial sums (8 x 148 SMs)

// ---- quantizers (Eq. 1)
// Weight quantizer: latent w[rows, cols] fp32 and steps (one per row, or one in all) ->
// int8 codes, int32 row sums of the codes, per-row dequantization scale (s, or s/2 on the
// half-integer 2-bit grid) and the dequantized matrix in the storage type.
void launch_quantize_weight(const float* w, int rows, int cols, const float* steps, int per_row, int bits, int grid,
                            int8_t* codes, int32_t* rowsum, float* scale, void* what, int dt, cudaStream_t st);

// Weight codes with a scale recomputed from the weights, one step-free rule per output row (Sec. 5.1 names one for
// 2-bit and one for 4-bit weights).  rule 2: ternary, delta = 0.7 mean|w|, codes sign(w) 1[|w| > delta], scale =
// mean of the kept |w|.  rule 3: codes in Omega(bits) and scale by alternating least squares (q = Pi(w / alpha),
// alpha = <q, w> / <q, q>) from min(3 mean|w|, max|w|) / qmax.  The fused update is AdamW with the gradient of
// w_hat passed through unchanged, then the rule on the new weights.
void launch_closed_form_quantize(const float* w, int rows, int cols, int rule, int bits, int8_t* codes, int32_t* rowsum,
                                 float* scale, void* what, int dt, cudaStream_t st);
struct OptimScalars;
void launch_closed_form_update(float* w, const float* g, float* m, float* v, const OptimScalars* sc, int rows, int cols,
                               int train_w, int rule, int bits, int8_t* codes, int32_t* rowsum, float* scale, void* what,
                               int dt, cudaStream_t st);

// Activation quantizer over a 2-D view x[rows, cols] with row stride ld_x:
// z = (x - offset) / step, q = rne(clip(z, lo, hi)).  Writes int8/uint8 codes (row stride
// ld_q8) and/or the codes as storage-type numbers (row stride ld_qt); either may be null.
void launch_quantize_act(const void* x, int dt, long long rows, int cols, long long ld_x, const float* step,
                         const float* offset, int lo, int hi, int8_t* q8, long long ld_q8, void* qt,
                         long long ld_qt, cudaStream_t st);

// Three adjacent column segments of width seg_cols (Q | K | V of the fused projection), each with its own
// symmetric step, in one pass; codes as storage-type numbers.
void launch_quantize_act3(const void* x, int dt, long long rows, int seg_cols, long long ld_x, const float* step0,
                          const float* step1, const float* step2, int lo, int hi, void* qt, long long ld_qt,
                          cudaStream_t st);

// dst[i] = (float)src[i] for a bfloat16 source
void launch_widen_bf16(const void* src, float* dst, long long n, cudaStream_t st);

// dst[i] = src[i] converted to the storage type
void launch_narrow(const float* src, void* dst, long long n, int dt, cudaStream_t st);

// Eq. 4: out = lam * f + (1 - lam) * f_hat
void launch_mix(const void* f, const void* f_hat, float lam, void* out, long long n, int dt, cudaStream_t st);

// ---- forward layer kernels
// out = LayerNorm(y) * gamma + beta (row-wise over `cols`), mean / rstd saved when non-null; with a
// step pointer the symmetric codes of the stored output are emitted as well.
void launch_layernorm_fwd(const void* y, const float* gamma, const float* beta, float eps, long long rows, int cols,
                          void* out, float* mean, float* rstd, const float* step, int qmax, int8_t* q8, void* qt,
                          int dt, cudaStream_t st);

// g = stored(gelu(u)); codes of g (asymmetric when offset != null) as int8/uint8 and storage-type numbers.
void launch_gelu_quant(const void* u, long long n, const float* step, const float* offset, int lo, int hi,
                       int8_t* q8, void* qt, int dt, cudaStream_t st);

// P = softmax(scores) over the last axis with keys >= valid_len[b] masked out; scores fp32
// [B, h, S, S]; optional codes of P as storage-type numbers.
void launch_softmax_fwd(const float* scores, const int* valid_len, int B, int h, int S, void* P, const float* step,
                        const float* offset, int lo, int hi, void* qt, int dt, cudaStream_t st);

// Fused attention forward on the tensor cores (bf16 storage, head size 64, seq <= 384, seq % 8 == 0):
// scores, masked softmax, quantizer of the probabilities, context product and (student) the context's
// codes in one kernel.  Returns a GemmRc.  Null p_step / c_step: no quantizer; null P: the probabilities are
// not written (a full-precision pass whose probabilities nobody reads); null P_qt: their codes are not written.
bool attention_fwd_supported(int S, int head_dim, int dt);
int launch_attention_fwd(const void* qkv, int B, int S, int h, int H, const int* valid_len, float alpha_const,
                         const float* a_p0, const float* a_p1, const float* c_p0, const float* c_p1,
                         const float* p_step, int p_lo, int p_hi, void* P, void* P_qt, void* ctx, const float* c_step,
                         int c_qmax, int8_t* ctx_q8, void* ctx_qt, int* status, cudaStream_t st);

// Fused attention backward of the student on the tensor cores (bf16 storage, head size 64, seq <= 128,
// seq % 8 == 0, batch * heads <= RED_BLOCKS): from the context gradient to the masked gradients of
// the pre-quantization Q, K, V ([B*S, 3H]) with the step-size partials of the Q, K, V, P sites
// (RED_BLOCKS slots each; unused slots are zeroed).  Returns a GemmRc.
bool attention_bwd_supported(int S, int head_dim, int dt, int batch_heads);
int launch_attention_bwd(const void* qkv_codes, const void* qkv, const void* P, const void* dctx, int B, int S, int h,
                         int H, const float* s_q, const float* s_k, const float* s_v, const float* s_p, int q_lo,
                         int q_hi, int p_lo, int p_hi, void* dqkv, float* part_q, float* part_k, float* part_v,
                         float* part_p, int* status, cudaStream_t st);

// ---- loss (Eq. 3)
// partial[l][block] = sum (f_hat - f)^2 over the block's share; dF = 2 c (f_hat - f).
void launch_loss(const void* f_hat, const void* f, int n_layers, long long n_per_layer, float c, void* dF,
                 float* partial, int* status, int dt, cudaStream_t st);
void launch_loss_finalize(const float* partial, int n_layers, float c, float* loss_total, float* loss_per_layer,
                          cudaStream_t st);

// Output-logit term of the last module: pooler (dense + tanh) and classifier on the first token of both last
// layer outputs [B, S, H]; adds cc * sum (z_hat - z)^2 to *loss_total (and writes it to *logit_loss when non-null),
// adds its gradient to dF_last at the first tokens; `scratch` >= head_scratch_floats(B, H) floats; `logits` null or
// [2, B, C] (student, teacher).  Returns 0, -1 when hidden / classes do not fit the kernel's shared memory, -2 on a launch error.
size_t head_scratch_floats(int B, int H);
int launch_head_logit_loss(const void* f_s_last, const void* f_t_last, int B, int S, int H, int C, const float* wp,
                           const float* bp, const float* wc, const float* bc, float cc, void* dF_last, float* scratch,
                           float* logits, float* loss_total, float* logit_loss, int dt, cudaStream_t st);

// ---- backward kernels
// Straight-through backward of an activation quantizer on a 2-D view:
// dx = dxhat * 1[lo <= z <= hi] (+ add), per-block partials of d l/d step (and d l/d offset).
void launch_ste_act(const void* x, long long ld_x, const void* dxhat, long long ld_d, const void* add,
                    long long ld_add, void* dx, long long ld_dx, long long rows, int cols, const float* step,
                    const float* offset, int lo, int hi, float* part_s, float* part_o, int dt, cudaStream_t st);

// GELU-site backward: recompute g = stored(gelu(u)), STE of its quantizer, dU = dGhat * inside * gelu'(u).
// GELU backward of a [rows, cols] tensor with the column sums of its result (the bias gradient of the linear layer
// before the GELU) in the same pass.  scratch: scratch_floats floats, counters: n_counters zero-initialised ints, both
// private to this call site.  Returns false (nothing launched) when the shape does not take the vector path.
bool launch_gelu_bwd_colsum(const void* u, const void* dghat, void* du, long long rows, int cols, const float* step,
                            const float* offset, int lo, int hi, int quantized, float* part_s, float* part_o,
                            float* bias_grad, float* scratch, long long scratch_floats, int* counters, int n_counters,
                            int dt, cudaStream_t st);
void launch_gelu_bwd(const void* u, const void* dghat, void* du, long long n, const float* step, const float* offset,
                     int lo, int hi, int quantized, float* part_s, float* part_o, int dt, cudaStream_t st);

// Softmax-site backward: STE of the P quantizer, then dS = P * (dP - sum_j dP * P) per row.
void launch_softmax_bwd(const void* P, const void* dphat, void* dS, long long rows, int S, const float* step,
                        int lo, int hi, int quantized, float* part_s, int dt, cudaStream_t st);

// LayerNorm backward: dy (storage type) from dout (+ dout2 when non-null).
void launch_layernorm_bwd(const void* dout, const void* dout2, const void* y, const float* mean, const float* rstd,
                          const float* gamma, long long rows, int cols, void* dy, void* dsum, int dt,
                          cudaStream_t st);

// The same with the incoming gradient assembled on the fly from a straight-through mask and a skip connection:
//   dv = dout (or 0 when null) + 1[lo <= x / *step <= hi] * dxhat + add;  dsum = dv;  dy = LayerNorm backward of dv.
// part_s gets RED_BLOCKS partial sums of the quantizer's step-size gradient.  Returns false (nothing launched)
// when the row does not fit the register-cached vector path; the caller then runs the separate kernels.
bool layernorm_bwd_ste_supported(int cols, int dt);      // the row width fits (16-byte aligned tensors assumed)
bool launch_layernorm_bwd_ste(const void* dout, const void* x, const void* dxhat, const void* add, const float* step,
                              int lo, int hi, const void* y, const float* mean, const float* rstd, const float* gamma,
                              long long rows, int cols, void* dy, void* dsum, float* part_s, int dt, cudaStream_t st);

// Column sums over rows: out0[c] = sum_r a[r,c]; with y/mean/rstd also out1[c] = sum_r a[r,c]*(y[r,c]-mean[r])*rstd[r];
// with a2 also out2[c] = sum_r a2[r,c].  One kernel: per-chunk partials in `scratch` (three planes of
// `plane_floats` floats each, plane_floats >= cols; the launcher takes as many row chunks as a plane holds),
// summed in a fixed order by the last block of each column group.  `counters` (>= cols/32 + 1 ints) must be
// zero before the first launch; the kernel leaves them zero.
constexpr int COL_CHUNKS = 32;      // row chunks a scratch plane holds at the widest tensor
void launch_col_reduce(const void* a, long long ld_a, const void* y, const float* mean, const float* rstd,
                       const void* a2, long long ld_a2, long long rows, int cols, float* out0, float* out1,
                       float* out2, float* scratch, long long plane_floats, int* counters, int dt, cudaStream_t st);

// Weight STE: dW = dWhat * inside (in place), ds[row] = sum_k dWhat * d what/d s.
void launch_ste_weight(const float* w, const float* steps, int per_row, int bits, int grid, float* dw, int rows,
                       int cols, float* ds_rows, cudaStream_t st);

// dst[i] = sum_j src_i[j], j in fixed order, for a table of reductions (one block each).
struct ReduceEntry { const float* src; int count; float* dst; };
// n traced launches of a kernel that does nothing: the tracer's own overhead per bracketed launch ("(empty kernel)").
void launch_trace_calibration(int n, cudaStream_t st);
void launch_reduce_table(const ReduceEntry* d_table, int n_entries, cudaStream_t st);

// out[i] = scale[0] * in[i]  (small vectors)
void launch_scale_vec(const float* in, const float* scale, float* out, int n, cudaStream_t st);
// beff[n] = b[n] + beta[0] * wscale[n] * rowsum[n]
void launch_effective_bias(const float* b, const float* beta, const float* wscale, const int32_t* rowsum, float* beff,
                           int n, cudaStream_t st);

// ---- optimizer (AdamW)
// bc = 1 - beta^t; lr_bc1 = lr / bc1, rsqrt_bc2 = 1 / sqrt(bc2)
struct OptimScalars { float lr, beta1, beta2, eps, bc1, bc2, weight_decay, lr_bc1, rsqrt_bc2; };
struct AdamEntry { float* p; const float* g; float* m; float* v; long long n; float wd; float min_value; };   // wd: 1 = decayed
// Computes the scalars of this step on the device: t = ++(*d_t) (or host_t when >= 1),
// lr = lr0 * (1 - (t-1)/total) when total > 0 else lr0.
void launch_optim_prepare(OptimScalars* d_out, int* d_t, int host_t, float lr0, int total_steps, float beta1,
                          float beta2, float eps, float weight_decay, cudaStream_t st);
void launch_adamw_table(const AdamEntry* d_table, int n_entries, long long total_elems, const OptimScalars* d_sc,
                        cudaStream_t st);

// Fused per-row update of a weight matrix and its per-row steps: step gradient (or ds_in when the
// gradients were already masked), AdamW on step and weights, re-quantization (codes, row sums,
// scale, dequantized row).
void launch_fused_weight_update(float* w, const float* g, float* m, float* v, float* steps, const float* ds_in,
                                float* m_s, float* v_s, const OptimScalars* sc, int rows, int cols, int bits, int grid,
                                int train_w, int train_s, int8_t* codes, int32_t* rowsum, float* scale, void* what,
                                int dt, cudaStream_t st);

// ---- step-size initialisation
// Per-row max|w| or mean|w| -> steps (per row, or one value when !per_row: two passes).
void launch_init_weight_steps(const float* w, int rows, int cols, int per_row, int rule, float qmax, float* steps,
                              float* scratch, cudaStream_t st);
// min and max of a 2-D view -> out[0] = min, out[1] = max (two kernels; scratch >= 2*RED_BLOCKS floats).
void launch_minmax(const void* x, long long ld, long long rows, int cols, float* out, float* scratch, int dt,
                   cudaStream_t st);
// step/offset from (min, max): mode 0 symmetric s = max|x|/qmax; 1 unsigned s = max/qmax, offset 0;
// 2 unsigned s = (max-min)/qmax, offset = min.
void launch_step_from_minmax(const float* minmax, int mode, float qmax, float* step, float* offset, cudaStream_t st);

// Gather rows of a calibration set: out[i] = src[idx[i]] for i < n_rows, row_bytes each (16-byte multiple).
void launch_gather_rows(const void* src, const int* d_idx, int n_rows, long long row_bytes, void* out,
                        cudaStream_t st);

}  // namespace mrem
