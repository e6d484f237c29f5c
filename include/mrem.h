/*
 * libmrem — the reconstruction step of module-wise reconstruction error minimization
 * (MREM) for post-training quantization of BERT-style encoders, on one B200 (sm_100a).
 *
 * One step (Algorithm 2 of the paper): a full-precision teacher module (a block of
 * encoder layers) and its fake-quantized student run on the same calibration batch; the
 * squared error between their layer outputs (Eq. 3) is back-propagated through the
 * quantizers (Eq. 1) with the straight-through estimator; AdamW updates the latent
 * weights and the quantization step sizes.
 *
 * Conventions
 *  - Every function returns an int32 status: 0 = MREM_OK, negative = error.  No exceptions,
 *    no exit, nothing printed.  mrem_last_error() returns text for the last failing call.
 *  - The library allocates NO device memory.  Tensors, parameters and the workspace are
 *    caller-owned DEVICE pointers (unless a parameter is named h_*: HOST pointer) that must
 *    stay valid while the context uses them and be 256-byte aligned.
 *  - All work is enqueued on the CUDA stream given at creation (a cudaStream_t passed as
 *    void*); calls do not block unless stated.  Scalars such as the loss are written to
 *    device addresses given by the caller.
 *  - Conditions detected on the device (a bounded wait that ran out, a non-finite loss) are
 *    recorded in a sticky device status word; mrem_poll_status() reads it.
 *  - A context is not thread-safe; independent contexts are independent.
 *  - Layouts are row-major.  Activations are [batch, seq, hidden]; a linear layer's weight
 *    is [out_features, in_features] (so y = x W^T + b).
 */
#ifndef MREM_H_
#define MREM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  MREM_OK = 0,
  MREM_ERR_ARG = -1,          /* null pointer, value out of range */
  MREM_ERR_ALIGN = -2,        /* pointer or stride not aligned as required */
  MREM_ERR_SHAPE = -3,        /* batch/seq/hidden combination not supported */
  MREM_ERR_WORKSPACE = -4,    /* workspace too small */
  MREM_ERR_ORDER = -5,        /* call made before the calls it depends on */
  MREM_ERR_CUDA = -6,         /* a CUDA runtime/driver call failed */
  MREM_ERR_TIMEOUT = -7,      /* device status: a bounded wait ran out */
  MREM_ERR_NONFINITE = -8,    /* device status: non-finite loss */
  MREM_ERR_UNSUPPORTED = -9
};

typedef struct mrem_ctx mrem_ctx;

typedef enum { MREM_TEACHER = 0, MREM_STUDENT = 1 } mrem_role;
typedef enum { MREM_F32 = 0, MREM_BF16 = 1 } mrem_dtype;

/* Parameter tensors of one encoder layer (post-LayerNorm BERT layout). */
enum {
  MREM_WQKV = 0, MREM_BQKV = 1,   /* [3H, H], [3H]: rows 0..H-1 query, H..2H-1 key, 2H..3H-1 value */
  MREM_WO = 2, MREM_BO = 3,       /* [H, H], [H]   attention output projection */
  MREM_LN1_G = 4, MREM_LN1_B = 5, /* [H]           LayerNorm after attention + skip */
  MREM_W1 = 6, MREM_B1 = 7,       /* [F, H], [F]   first FFN layer (GELU follows) */
  MREM_W2 = 8, MREM_B2 = 9,       /* [H, F], [H]   second FFN layer */
  MREM_LN2_G = 10, MREM_LN2_B = 11,
  MREM_N_PARAMS = 12
};

/* Quantizers of one layer.  0..3: weight steps of Wqkv, Wo, W1, W2 ([rows] or [1]).
 * 4..11: activation sites in forward order, one step each (a quantizer sits on both
 * operands of every matrix product, Sec. 3.1): layer input, Q, K, V, softmax output,
 * attention context, FFN input, GELU output. */
enum {
  MREM_Q_WQKV = 0, MREM_Q_WO = 1, MREM_Q_W1 = 2, MREM_Q_W2 = 3,
  MREM_Q_X = 4, MREM_Q_Q = 5, MREM_Q_K = 6, MREM_Q_V = 7, MREM_Q_P = 8, MREM_Q_C = 9, MREM_Q_A = 10, MREM_Q_G = 11,
  MREM_N_QUANTIZERS = 12
};
/* ids for mrem_get_grad: parameter ids 0..11; MREM_GRAD_STEP + quantizer id;
 * MREM_GRAD_OFFSET + quantizer id (only the GELU site has a learnable offset). */
enum { MREM_GRAD_STEP = 100, MREM_GRAD_OFFSET = 200 };

enum { MREM_TRAIN_WEIGHTS = 1, MREM_TRAIN_BIASES = 2, MREM_TRAIN_LAYERNORM = 4, MREM_TRAIN_W_STEPS = 8,
       MREM_TRAIN_A_STEPS = 16, MREM_TRAIN_ALL = 31 };

typedef struct {
  uint32_t struct_size;        /* sizeof(mrem_module_desc) */
  int32_t n_layers, hidden, n_heads, ffn;
  int32_t max_seq, max_batch;  /* the workspace is sized for max_batch * max_seq tokens */
  int32_t w_bits;              /* 2, 4 or 8 */
  int32_t a_bits;              /* 8 or 4 */
  int32_t w_grid;              /* 0: integer codes Omega(b) of Eq. 1; 1: 2-bit levels {-1.5,-.5,.5,1.5}*step;
                                  2: 2-bit ternary codes by the closed-form rule named in Sec. 5.1 (per output row:
                                  threshold 0.7 mean|w|, scale = mean of the kept |w|);
                                  3: codes in Omega(w_bits) with the scale refitted from the weights by the loss-aware
                                  rule Sec. 5.1 names for 4-bit weights, read with unit curvature weights (per output
                                  row, 16 rounds of q = Pi(w / alpha), alpha = <q, w> / <q, q> from
                                  alpha_0 = min(3 mean|w|, max|w|) / qmax).
                                  With 2 and 3 no weight steps are bound, learnt or reported and the weight gradient
                                  passes straight through; both need w_step_per_row = 1 */
  int32_t w_step_per_row;      /* 1: one step per output row; 0: one per matrix */
  int32_t act_asym_sites;      /* bit 0: softmax output unsigned (offset 0); bit 1: GELU output unsigned with
                                  learnable offset (Sec. 3.1: asymmetric for these two) */
  int32_t act_dtype;           /* mrem_dtype: storage type of activations (bf16: tensor cores; f32: exact path
                                  for small checks) */
  int32_t loss_mean;           /* 1: each layer's squared error divided by batch*seq*hidden; 0: plain sum (Eq. 3) */
  int32_t trainable_mask;      /* MREM_TRAIN_* */
  float ln_eps;
} mrem_module_desc;

typedef struct {
  float lr;                    /* learning rate of this step, or the initial one when decay_total_steps > 0 */
  float beta1, beta2, eps, weight_decay;   /* decay applies to the four weight matrices only */
  int32_t step;                /* 1-based step index t for the bias correction; 0: use and advance the
                                  context's device-side counter */
  int32_t decay_total_steps;   /* > 0: lr_t = lr * (1 - (t-1)/decay_total_steps), computed on the device (Sec. 5.1:
                                  linear decay) */
} mrem_optim;

/* ---- context ------------------------------------------------------------------------- */

/* Bytes of device workspace a context of this shape needs. */
int32_t mrem_workspace_bytes(const mrem_module_desc* desc, size_t* out_bytes);

/* Creates a context on the current device.  `workspace` (device, 256-byte aligned, at least
 * mrem_workspace_bytes) holds codes, stashed activations, gradients and optimizer moments;
 * it is zero-filled here (asynchronously).  Errors: ARG, ALIGN, SHAPE (hidden % n_heads != 0,
 * head size != 64 for bf16, hidden/ffn not multiples of 16), WORKSPACE, UNSUPPORTED. */
int32_t mrem_create(const mrem_module_desc* desc, void* workspace, size_t workspace_bytes, void* cuda_stream,
                    mrem_ctx** out);
int32_t mrem_destroy(mrem_ctx* ctx);
/* Text of the last error on this context (or of the last failed mrem_create when ctx is NULL).  Host string
 * owned by the library. */
const char* mrem_last_error(const mrem_ctx* ctx);

/* Binds caller-owned parameter storage.  Teacher: matrices in act_dtype, vectors float32, read-only.
 * Student: all float32 ("latent" full-precision values), updated in place by mrem_step. */
int32_t mrem_bind_param(mrem_ctx* ctx, int32_t role, int32_t layer, int32_t tensor_id, void* d_ptr, int32_t dtype);
/* Binds the step size(s) of one quantizer (float32, read-write) and, for MREM_Q_G, its offset
 * (float32 [1]; may be NULL for other sites). */
int32_t mrem_bind_steps(mrem_ctx* ctx, int32_t layer, int32_t quantizer_id, float* d_steps, float* d_offset);

/* Copies the teacher's parameters into the student's latent ones; zeroes the optimizer state. */
int32_t mrem_init_student_from_teacher(mrem_ctx* ctx);
/* rule 0: step = max|w| / qmax over the group (nothing clipped at the start); rule 1: mean|w| over the group. */
int32_t mrem_init_weight_steps(mrem_ctx* ctx, int32_t rule);
/* One unquantized pass of the student over the batch; each site's step = max|x|/qmax (symmetric) or
 * (max - min)/(2^b - 1) with offset min (GELU site) / max/(2^b-1) with offset 0 (softmax site). */
int32_t mrem_init_act_steps(mrem_ctx* ctx, const void* d_x, const int32_t* d_valid_len, int32_t batch, int32_t seq);

/* ---- one reconstruction step (Algorithm 2), in this order ------------------------------ */

/* Eq. 1 on every weight matrix of the student: latent weights + steps -> int8 codes, int32 row
 * sums of the codes, and the dequantized matrices used by the backward products. */
int32_t mrem_quantize_weights(mrem_ctx* ctx);
/* Tells the context that the caller wrote the student's weights or weight steps itself (through its own
 * pointers): the next mrem_quantize_weights then recomputes the codes instead of trusting the ones the
 * last mrem_step produced. */
int32_t mrem_invalidate_weight_codes(mrem_ctx* ctx);
/* Borrowed pointers to the codes [rows, cols] and row sums [rows] of one matrix (valid until destroy). */
int32_t mrem_get_weight_codes(mrem_ctx* ctx, int32_t layer, int32_t tensor_id, const int8_t** d_codes,
                              const int32_t** d_rowsum);

/* Runs one module forward.  d_x: [batch, seq, hidden] in act_dtype, this role's own input.
 * STUDENT with lambda != 0: the input becomes lambda * d_x_other + (1 - lambda) * d_x (Eq. 4, d_x_other =
 * the teacher-side input); otherwise d_x_other may be NULL.  d_valid_len: [batch] int32 key lengths
 * (positions >= length are masked out of the attention; a length below 1 counts as 1, above seq as seq) or NULL.  d_layer_outputs:
 * [n_layers, batch, seq, hidden] act_dtype, written; the last slice is the module output.
 * The student pass needs mrem_quantize_weights first (ERR_ORDER) and keeps d_x and d_layer_outputs
 * borrowed until mrem_module_backward has run. */
int32_t mrem_module_forward(mrem_ctx* ctx, int32_t role, const void* d_x, const void* d_x_other, float lambda,
                            const int32_t* d_valid_len, int32_t batch, int32_t seq, void* d_layer_outputs);
/* Eq. 3 over the layer outputs of the last teacher and student passes.  Writes the total to
 * d_loss_total (float32 [1]) and, when non-NULL, each layer's term to d_loss_per_layer
 * ([n_layers]); stores d loss / d f_hat_l for the backward. */
int32_t mrem_recon_loss(mrem_ctx* ctx, float* d_loss_total, float* d_loss_per_layer);
/* Sec. 3.1.1: back-propagation of the loss of Eq. 3 through the student module with the straight-through
 * estimator at every quantizer (the gradient passes where x / s lies inside the code range; step sizes and the
 * GELU-site offset get their own gradients, Sec. 4.1).  The loss gradient enters at every layer output of the
 * module (Eq. 3 sums over them) and stops at the module input (Sec. 4.2).  Needs the student pass and
 * mrem_recon_loss of this step (MREM_ERR_ORDER otherwise); fills the gradient buffers mrem_get_grad returns. */
int32_t mrem_module_backward(mrem_ctx* ctx);
/* Borrowed pointer to a gradient (float32, same shape as the parameter / step tensor).  Asking for a weight
 * matrix or a weight step applies the weight quantizers' straight-through masks on the spot. */
int32_t mrem_get_grad(mrem_ctx* ctx, int32_t layer, int32_t id, const float** d_grad);
/* Borrowed pointer to d loss / d (student module input), [batch, seq, hidden] in the storage type, after the
 * straight-through pass of the first layer's input quantizer and its skip connection.  The gradient stays
 * local to a module (Sec. 4.2) except in the model's first module, whose embedding layers receive it
 * (mrem_embed_step).  Valid from a backward pass (mrem_module_backward or mrem_backward_and_step) until the next
 * forward pass on this context (MREM_ERR_ORDER otherwise). */
int32_t mrem_get_input_grad(mrem_ctx* ctx, const void** d_grad);
/* Borrowed pointer to a tensor that a forward pass stored on its way through one layer (storage type, row-major;
 * for verification: each stored tensor is the rounding of one stage of the layer of Sec. 3.1 / Sec. 4.1 applied
 * to the stored tensors before it).  `which`:
 *   MREM_ACT_QKV  [tokens, 3*hidden]  input projection + bias
 *   MREM_ACT_P    [batch, heads, seq, seq]  softmax output (student pass only)
 *   MREM_ACT_CTX  [tokens, hidden]    attention context
 *   MREM_ACT_Y1   [tokens, hidden]    output projection + bias + layer input (before the first LayerNorm)
 *   MREM_ACT_A    [tokens, hidden]    first LayerNorm's output
 *   MREM_ACT_G    [tokens, ffn]       teacher: GELU output (it never stores the tensor before GELU);
 *                                     student: the tensor BEFORE GELU (its GELU output is recomputed, not kept)
 *   MREM_ACT_Y2   [tokens, hidden]    FFN2 + bias + first LayerNorm's output (before the second LayerNorm)
 * The teacher pass reuses one set of buffers for all layers, so only its last layer can be read
 * (MREM_ERR_ARG otherwise); the student pass keeps every layer.  Valid until the next forward pass of that role;
 * MREM_ERR_ORDER when there has been none. */
enum { MREM_ACT_QKV = 0, MREM_ACT_P = 1, MREM_ACT_CTX = 2, MREM_ACT_Y1 = 3, MREM_ACT_A = 4, MREM_ACT_G = 5, MREM_ACT_Y2 = 6,
       MREM_ACT_COUNT = 7 };
int32_t mrem_get_activation(mrem_ctx* ctx, int32_t role, int32_t layer, int32_t which, const void** d_ptr);
/* Algorithm 2's Update(w) and Update(s): AdamW (Sec. 4.2; learning rate decayed linearly, Sec. 5.1) on
 * everything in trainable_mask from the gradients of the last backward pass (MREM_ERR_ORDER without one);
 * weight decay on the four matrices only, steps clamped to >= 1e-8.  With per-row weight steps the update of
 * each matrix also re-quantizes it (Eq. 1 with the new weights and steps), so the next
 * mrem_quantize_weights has nothing left to do. */
int32_t mrem_step(mrem_ctx* ctx, const mrem_optim* optim);
/* mrem_module_backward and mrem_step as one call (the last two lines of Algorithm 2's inner loop).  With per-row
 * weight steps the matrices of a layer are updated, on a second stream the context owns, as soon as that
 * layer's gradients are complete, while the backward pass continues below it; the context's stream waits
 * for those updates before the call's work is considered done, so callers keep ordering everything on
 * their one stream.  Same kernels on the same data as the two separate calls: bitwise the same result.
 * The gradients are consumed: mrem_get_grad is not available afterwards.  mrem_recon_step_host and the
 * captured step use this form. */
int32_t mrem_backward_and_step(mrem_ctx* ctx, const mrem_optim* optim);

/* The whole step from HOST buffers: copies h_x_teacher / h_x_student ([batch, seq, hidden] act_dtype;
 * h_x_student may equal h_x_teacher) and h_valid_len (may be NULL) to the device, runs quantize_weights,
 * both forwards, loss, backward and step, copies the loss back to *h_loss and blocks until it is there.
 * With optim->step == 0 (device-side step counter) the step is captured into a CUDA graph on first use and
 * replayed while batch, seq, lambda, *optim and the presence of h_valid_len stay the same. */
int32_t mrem_recon_step_host(mrem_ctx* ctx, const void* h_x_teacher, const void* h_x_student,
                             const int32_t* h_valid_len, int32_t batch, int32_t seq, float lambda,
                             const mrem_optim* optim, float* h_loss);
/* The same step in two halves, so that the copy of the next batch overlaps the step in flight: submit
 * enqueues the host-to-device copies (on a copy stream the context owns, into one of two staging slots) and
 * the step, and returns at once; wait blocks until the OLDEST submitted step is done and returns its loss.
 * At most two steps may be in flight (MREM_ERR_ORDER beyond that).  The host buffers (pinned memory for the
 * copies to be asynchronous) must stay valid and unchanged until the matching wait has returned. */
int32_t mrem_recon_step_host_submit(mrem_ctx* ctx, const void* h_x_teacher, const void* h_x_student,
                                    const int32_t* h_valid_len, int32_t batch, int32_t seq, float lambda,
                                    const mrem_optim* optim);
int32_t mrem_recon_step_host_wait(mrem_ctx* ctx, float* h_loss);

/* Process-wide switch (default on): kernels are launched with programmatic stream serialization, i.e. a
 * kernel may be scheduled and run its set-up while its predecessor in the stream is still finishing; each
 * kernel waits for its predecessor's results before touching global memory, so results do not change.
 * Turn it off (0) to get plain stream-ordered launches, e.g. when comparing timings. */
int32_t mrem_set_programmatic_launch(int32_t on);

/* ---- data-parallel use (Sec. 4.2 trains on several devices; Algorithm 2's step is linear in the batch) ---------
 *
 * The loss of Eq. 3 is a sum over the batch, so its gradient is the sum of the gradients of the batch's parts: R
 * ranks that hold the same parameters and steps, each with batch/R of the sequences, obtain the whole batch's
 * gradient by adding theirs.  Two hooks make that exact without any arithmetic outside the library:
 * mrem_set_loss_share: from now on mrem_recon_loss multiplies its scale by `share` in (0, 1] (= this rank's sequences /
 *   all sequences of the step; default 1), so that the losses and every gradient of the ranks ADD UP to the whole
 *   batch's under loss_mean as under the plain sum.
 * mrem_grad_bucket: the contiguous float32 range [*d_ptr, *d_ptr + *n_floats) inside the workspace that holds ALL
 *   gradients of one layer after mrem_module_backward (the twelve parameters, then the weight-step, activation-step
 *   and offset gradients; alignment gaps between them hold no data).  Sum that range over the ranks (one all-reduce per
 *   layer, top layer first: the order in which the backward pass completes them), then call mrem_step.  The weight
 *   matrices' slots hold the gradient with respect to the QUANTIZED weights; the straight-through mask and the
 *   weight-step gradients are applied by mrem_step from the summed values (both are linear in it). */
int32_t mrem_set_loss_share(mrem_ctx* ctx, float share);
int32_t mrem_grad_bucket(mrem_ctx* ctx, int32_t layer, float** d_ptr, size_t* n_floats);

/* Failure detection.  Every device-side wait of the tensor-core kernels (on a TMA-filled stage, on a tensor-core
 * commit, on an accumulator hand-over) is bounded in time; a wait that runs out makes its kernel record a code in the
 * context's status word, stop issuing work, release what it holds and return, so the context stays usable and the host
 * learns of it through mrem_poll_status (MREM_ERR_TIMEOUT).
 * mrem_set_wait_limit_ns: process-wide limit of one such wait for all launches made afterwards (default 2 s;
 * 1 us .. 60 s, MREM_ERR_ARG otherwise).
 * mrem_selftest_wait_limit: enqueues, on the context's stream, one block whose single wait can never be satisfied (an
 * mbarrier nothing arrives at), using the library's own bounded wait and the current limit: after the limit the block
 * reports exactly as a starved product would and returns.  Nothing faults and nothing waits longer than the limit;
 * meant for checking the reporting path (set a limit of a millisecond or so first). */
int32_t mrem_set_wait_limit_ns(uint64_t ns);
int32_t mrem_selftest_wait_limit(mrem_ctx* ctx);

/* Per context (default on): inside a step the teacher pass runs on a second stream beside the student pass, and the
 * weight-gradient products, column reductions and weight updates of a layer beside the backward pass of the layers
 * below.  0 keeps everything on the context's stream (same kernels, same results; for timing comparisons: the replay
 * time of a step captured this way is the sum of its kernels' run times).  Takes effect at the next call or capture. */
int32_t mrem_set_two_streams(mrem_ctx* ctx, int32_t on);

/* Per context (default on): where the shapes allow it (bf16 storage, head size 64, seq <= 128, seq % 8 == 0)
 * the backward of the attention block (Sec. 3.1: the gradients of Q, K, V through the quantized scores,
 * softmax and context products, with the straight-through masks of the Q, K, V, P quantizers) runs as one
 * kernel; off (0) selects the kernel-per-operation path that covers every shape.  Both compute the same
 * quantities; they differ in where intermediates are rounded to the storage type.  Do not change it
 * between a student forward pass and its backward pass (the forward pass writes the codes of the attention
 * probabilities only for the kernel-per-operation path), nor between the capture and the replay of a graph. */
int32_t mrem_set_fused_attention_backward(mrem_ctx* ctx, int32_t on);

/* Reads the device status word (blocks on the stream): MREM_OK, MREM_ERR_TIMEOUT or MREM_ERR_NONFINITE in
 * *h_status; the word is cleared. */
int32_t mrem_poll_status(mrem_ctx* ctx, int32_t* h_status);

/* Optimizer state (moments of every trainable tensor and the step counter) as one blob. */
int32_t mrem_state_bytes(mrem_ctx* ctx, size_t* out_bytes);
int32_t mrem_export_state(mrem_ctx* ctx, void* d_blob, size_t bytes);
int32_t mrem_import_state(mrem_ctx* ctx, const void* d_blob, size_t bytes);

/* Captures quantize_weights .. step on fixed buffers into a CUDA graph owned by the context and
 * replays it.  Between replays the caller only rewrites the contents of the input buffers. */
int32_t mrem_graph_capture_step(mrem_ctx* ctx, const void* d_x_teacher, const void* d_x_student, float lambda,
                                const int32_t* d_valid_len, int32_t batch, int32_t seq, void* d_teacher_outputs,
                                void* d_student_outputs, float* d_loss_total, const mrem_optim* optim);
int32_t mrem_graph_launch(mrem_ctx* ctx);
/* Number of kernel nodes in the captured step. */
int32_t mrem_graph_num_kernels(mrem_ctx* ctx, int32_t* n_kernels);

/* Per-kernel timing of the eager calls (not of graph replays) with CUDA events on the context's stream.
 * `work` is the algorithmic work of all launches of that kernel: FLOPs (is_flops = 1: 2*M*N*K per product)
 * or bytes read plus written once at storage width (is_flops = 0).  mrem_trace_enable resets the totals
 * and blocks on the stream; mrem_trace_read blocks on the stream and fills up to max_entries entries.
 * A bracketed duration holds, beside the kernel's run time, what the event pair costs (event processing, launch and
 * drain of a grid: several microseconds); turning tracing on therefore launches 32 kernels that do nothing, bracketed
 * the same way, and reports them as the entry "(empty kernel)": its ms / launches is that overhead. */
typedef struct { char name[40]; double ms; double work; int64_t launches; int32_t is_flops; int32_t reserved; } mrem_trace_entry;
int32_t mrem_trace_enable(mrem_ctx* ctx, int32_t on);
int32_t mrem_trace_read(mrem_ctx* ctx, mrem_trace_entry* out, int32_t max_entries, int32_t* n_entries);

/* out[i] = src[idx[i]] for i < n_rows (rows of row_bytes bytes, a multiple of 16): draws a batch from a
 * calibration set resident on the device (Sec. 5.1). */
int32_t mrem_gather_rows(const void* d_src, const int32_t* d_idx, int32_t n_rows, size_t row_bytes, void* d_out,
                         void* cuda_stream);

/* ---- single operations (the building blocks above, exposed for verification) ----------- */

/* Eq. 1 on an activation tensor of n elements: z = (x - offset) / step (offset NULL = symmetric),
 * code = nearest integer (ties to even) of clip(z, lo, hi).  Writes 8-bit codes (d_codes8, may be
 * NULL) and/or the codes as numbers of type dtype (d_codes_t, may be NULL). */
int32_t mrem_quantize_act(const void* d_x, int32_t dtype, int64_t n, const float* d_step, const float* d_offset,
                          int32_t lo, int32_t hi, int8_t* d_codes8, void* d_codes_t, void* cuda_stream);
/* Eq. 1 on a weight matrix [rows, cols]; outputs as in mrem_quantize_weights (d_what may be NULL). */
int32_t mrem_quantize_weight(const float* d_w, int32_t rows, int32_t cols, const float* d_steps, int32_t per_row,
                             int32_t bits, int32_t grid, int8_t* d_codes, int32_t* d_rowsum, float* d_scale,
                             void* d_what, int32_t dtype, void* cuda_stream);
/* acc[m, n] = sum_k a[m, k] * b[n, k] in exact int32 on the int8 tensor cores.  a: [M, K] int8 (or uint8
 * when a_unsigned), b: [N, K] int8, K % 16 == 0, acc: [M, N] int32.  block_n 0 = automatic tile width; 64/128/256 force it.
 * d_status: device int32 receiving a DeviceStatus code on a bounded-wait timeout (0 otherwise). */
int32_t mrem_gemm_i8(const int8_t* d_a, int32_t a_unsigned, const int8_t* d_b, int32_t M, int32_t N, int32_t K,
                     int32_t* d_acc, int32_t block_n, int32_t* d_status, void* cuda_stream);
/* out[b, m, n] = alpha * sum_k A[b, m, k] * B[b, n, k] (float32 out).  dtype BF16: tcgen05 bf16 tensor
 * cores with fp32 accumulation; F32: CUDA cores.  a_mn / b_mn = 1 when the operand is stored with its
 * m / n index contiguous (lda/ldb then stride k), 0 when k is contiguous.  Batch strides in elements. */
int32_t mrem_gemm(int32_t dtype, const void* d_a, int32_t a_mn, int64_t lda, int64_t a_batch_stride, const void* d_b,
                  int32_t b_mn, int64_t ldb, int64_t b_batch_stride, int32_t M, int32_t N, int32_t K, int32_t batches,
                  float alpha, float* d_out, int64_t ldc, int64_t c_batch_stride, int32_t block_n, int32_t* d_status,
                  void* cuda_stream);

/* ---- the first module's embedding layers (Sec. 4.1) ---------------------------------------- */

/* Sec. 4.1: the embedding layers belong to the first module and the MSE of the Transformer embedding is
 * minimised beside the layer losses; Sec. 3.1: embeddings are quantized symmetrically like weights (the
 * "E" of the paper's W-E-A bit settings is the word-embedding width).  One call = one step of
 *     min  c * || e_hat - e ||^2,
 *     e     = LayerNorm(word[ids] + pos[0..seq) + type[type_ids])            (teacher tables)
 *     e_hat = LayerNorm(Q(word)[ids] + pos + type)                           (student tables),
 * Q = Eq. 1 with e_bits on the student's latent word table, one learnable step per row; position and
 * token-type tables and the LayerNorm are not quantized.  c = 1 / (batch * seq * hidden) with loss_mean.
 * Straight-through backward (a row gathered by several tokens gets the sum of their gradients, added in
 * token order); AdamW on word (with its row steps, kept >= 1e-8; the table is re-quantized in the same
 * pass), pos, type (decayed like weight matrices) and the LayerNorm parameters (not decayed).
 * Stateless: every tensor is the caller's; nothing is allocated. */
typedef struct {
  uint32_t struct_size;        /* sizeof(mrem_embed_desc) */
  int32_t vocab, hidden, max_pos, n_types;   /* hidden a multiple of 16 */
  int32_t e_bits;              /* 2, 4 or 8 */
  int32_t act_dtype;           /* mrem_dtype of e, e_hat */
  int32_t loss_mean;
  float ln_eps;
} mrem_embed_desc;

typedef struct {               /* device pointers, float32, 16-byte aligned */
  const float *t_word, *t_pos, *t_type, *t_ln_g, *t_ln_b;   /* teacher: [vocab,H] [max_pos,H] [n_types,H] [H] [H] */
  float *word, *pos, *type, *ln_g, *ln_b;                   /* student (latent), same shapes, updated */
  float* word_step;                                         /* [vocab], updated */
  float *g_word, *g_pos, *g_type, *g_ln_g, *g_ln_b, *g_word_step;   /* gradients, written by every call */
  float *m_word, *v_word, *m_pos, *v_pos, *m_type, *v_type, *m_ln_g, *v_ln_g, *m_ln_b, *v_ln_b,
        *m_word_step, *v_word_step;                         /* AdamW moments (zero before the first step); may be NULL when optim is NULL */
  int32_t* d_step_counter;                                  /* int32 [1], zero before the first step: AdamW's t when optim->step == 0 */
} mrem_embed_tensors;

int32_t mrem_embed_workspace_bytes(const mrem_embed_desc* desc, int32_t max_tokens, size_t* out_bytes);
/*   d_ids, d_type_ids  int32 [batch, seq] (d_type_ids NULL: all 0); an index outside its table is clamped and
 *                      reported in the status word
 *   requantize         non-zero on the first call and whenever the caller changed word or word_step: the
 *                      codes of the table (held in the workspace) are rebuilt first; updates keep them current
 *   d_e_teacher, d_e_student  [batch, seq, hidden] act_dtype, written (16-byte aligned)
 *   d_extra_grad       NULL or [batch, seq, hidden] act_dtype: a gradient with respect to the student's embedding
 *                      output that arrives from the layers it feeds (mrem_get_input_grad of the first module's
 *                      context after its backward pass); added to the gradient of the MSE
 *   optim              NULL: no update; g_word then holds the MASKED gradient of the latent table and g_word_step
 *                      the row-step gradients (with an update g_word is the unmasked sum, the mask being applied
 *                      inside the fused update, and g_word_step is not written)
 *   d_loss             float32 [1]: the loss before the update
 *   d_status           int32 [1], zero it once: 0 ok, 4 non-finite loss, 5 index out of range (sticky)
 * seq <= max_pos; workspace 256-byte aligned and at least mrem_embed_workspace_bytes(desc,
 * batch * seq).  Asynchronous on cuda_stream. */
int32_t mrem_embed_step(const mrem_embed_desc* desc, const mrem_embed_tensors* tensors, void* workspace,
                        size_t workspace_bytes, const int32_t* d_ids, const int32_t* d_type_ids, int32_t batch,
                        int32_t seq, int32_t requantize, void* d_e_teacher, void* d_e_student,
                        const void* d_extra_grad, const mrem_optim* optim, float* d_loss, int32_t* d_status,
                        void* cuda_stream);

/* ---- the last module's output logits (Sec. 4.1) -------------------------------------------- */

/* Sec. 4.1: "besides the grouped Transformer layers" the MSE of the output logits is minimised; the
 * classification head belongs to the last module and is not quantized (Sec. 3.1), so one set of head
 * parameters serves both sides and is not trained here.  After this call mrem_recon_loss adds
 *     c_z * || z_hat - z ||^2,   z = Wc tanh(Wp f_L[:, 0, :] + bp) + bc   (pooler and classifier on the first token
 * of the last layer's output; c_z = 1 / (batch * n_classes) with loss_mean, else 1) to the total loss and the
 * term's gradient to d loss / d f_hat_L, from where mrem_module_backward carries it through the module.
 *   d_wp [hidden, hidden], d_bp [hidden], d_wc [n_classes, hidden], d_bc [n_classes]: float32, device,
 *       caller-owned, borrowed until unbound (d_wp = NULL unbinds) or the context is destroyed
 *   d_logit_loss  NULL or float32 [1]: the term alone, written by every mrem_recon_loss
 *   d_logits      NULL or float32 [2, max_batch, n_classes]: student logits, then teacher logits ([2, batch, n_classes]
 *                 packed for the batch of the call)
 * hidden <= 2048, n_classes <= 64 (MREM_ERR_SHAPE).  Bind before a step graph is captured. */
int32_t mrem_bind_head(mrem_ctx* ctx, const float* d_wp, const float* d_bp, const float* d_wc, const float* d_bc,
                       int32_t n_classes, float* d_logit_loss, float* d_logits);

/* ---- the per-product objective (Eq. 2) ---------------------------------------------------- */

/* One optimisation step on the reconstruction error of ONE matrix product (Eq. 2, Sec. 2.2: the objective
 * that the module-wise loss of Eq. 3 generalises, and the building block of the layer-by-layer baseline
 * the paper compares with):
 *     min over w, s of  c * || Q(w)^T Q(a) - w^T a ||^2   over the rows of a,
 * w = the teacher's matrix `tensor_id` (MREM_WQKV, MREM_WO, MREM_W1 or MREM_W2) of `layer`, Q(w) = the
 * student's quantized matrix (Eq. 1, its own latent weights and steps), Q(a) = the activation quantizer
 * that sits at that product's input in the module (layer input, attention context, FFN1 input, GELU
 * output: the last one asymmetric with its offset when the context says so); c = 1 / (rows * out) with
 * loss_mean, else 1.  No bias on either side, as in Eq. 2.  The straight-through gradients (Sec. 3.1.1)
 * reach the latent matrix, its step(s), the activation step and offset; AdamW (mrem_optim, trainable_mask)
 * updates exactly those and the matrix is re-quantized.  Biases, LayerNorm parameters and every other
 * matrix are untouched.
 *   d_a     [rows, in] activations in the context's storage type, device, 16-byte aligned, 1 <= rows <=
 *           max_batch * max_seq
 *   optim   NULL: no update; the gradients of this product (matrix, its steps, the activation step and
 *           offset) can then be read with mrem_get_grad until the next step of any kind
 *   d_loss  float32 [1], device: the loss before the update
 * Needs per-row weight steps or the closed-form ternary weights (MREM_ERR_UNSUPPORTED otherwise), bound
 * teacher and student parameters and steps (MREM_ERR_ORDER).  Uses the context's workspace and stream;
 * asynchronous; invalidates the forward / loss / gradient state of a module step in progress. */
int32_t mrem_rem_step(mrem_ctx* ctx, int32_t layer, int32_t tensor_id, const void* d_a, int32_t rows,
                      const mrem_optim* optim, float* d_loss);

/* ---- for callers that cannot allocate device memory -------------------------------------- */

/* (The paper has no counterpart to this call; it exists for deployment reasons only.)
 *
 * The loss of Eq. 3 and its gradient WITHOUT a context and without any allocation: meant for callers
 * that have the two sets of layer outputs in hand but cannot call cudaMalloc or set up a workspace,
 * for example a plug-in inside a process whose device memory is handed out entirely by the host
 * application, a hook that runs while the application's allocator lock is held, or a latency-critical
 * loop where the device-wide synchronisation of cudaMalloc is not acceptable.  The scratch of the
 * two-stage reduction (one partial sum per layer and block) is a fixed array inside the library:
 * MREM_NOALLOC_MAX_LAYERS * 1184 floats (about 150 KB) that every GPU holds from the moment the library
 * is loaded on it until the process exits.
 *
 *   d_f_student, d_f_teacher  [n_layers, n_per_layer] of dtype (MREM_F32 / MREM_BF16), device, 16-byte aligned
 *   loss_mean                 1: each layer's squared error divided by n_per_layer; 0: plain sum
 *   d_grad                    [n_layers, n_per_layer] dtype, written: d loss / d f_student
 *   d_loss_total              float32 [1], written;  d_loss_per_layer: float32 [n_layers] or NULL
 *
 * Returns MREM_ERR_SHAPE when n_layers > MREM_NOALLOC_MAX_LAYERS (the built-in scratch is that large and
 * no larger), MREM_ERR_ARG for null pointers, a bad dtype or non-positive sizes, MREM_ERR_CUDA when the
 * device cannot be queried.  The first call on each device looks up the device address of the built-in
 * array (a one-off host-side query, made with that device current); make that first call before entering
 * any stream capture.  The address is remembered per device ordinal: `cuda_stream` must belong to the device
 * (and primary context) that is current at the call, and after cudaDeviceReset the library must not be
 * called again on that device.  All calls on a device share the one array: calls that may overlap on the GPU (two
 * streams, two threads) race on it and must be serialised by the caller.  Nothing in the array has to
 * be cleared between calls: each call rewrites every slot it later reads.  The call never allocates or
 * frees memory, on the host side of CUDA or otherwise. */
#define MREM_NOALLOC_MAX_LAYERS 32
int32_t mrem_recon_loss_noalloc(const void* d_f_student, const void* d_f_teacher, int32_t dtype, int32_t n_layers,
                                int64_t n_per_layer, int32_t loss_mean, void* d_grad, float* d_loss_total,
                                float* d_loss_per_layer, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* MREM_H_ */
