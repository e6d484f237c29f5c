// Host-side state of one reconstruction context: shapes, bound pointers and the layout of
// the caller-provided workspace.
#pragma once
#include <string>
#include <vector>

#include "../../include/mrem.h"
#include "gemm.h"
#include "kernels.h"

namespace mrem {

constexpr int N_SITES = 8;              // activation quantizer sites per layer
constexpr int N_WMAT = 4;               // weight matrices per layer

struct WeightBuf {                      // quantized form of one weight matrix
  int rows = 0, cols = 0;
  int8_t* codes = nullptr;              // [rows, cols]
  int32_t* rowsum = nullptr;            // [rows]
  float* scale = nullptr;               // [rows] dequantization scale (step, or step/2 on the half-integer grid)
  void* what = nullptr;                 // [rows, cols] dequantized, storage type
  float* beff = nullptr;                // [rows] bias + offset term (W2 only)
  float* ds_rows = nullptr;             // [rows] per-row step gradients before a per-matrix sum
};

struct LayerStash {                     // what the student forward keeps for the backward
  int8_t* x_q8; void* x_qt;
  void* qkv; void* qkv_qt;
  void* P; void* P_qt;
  void* ctx; int8_t* ctx_q8; void* ctx_qt;
  void* y1; float* mean1; float* rstd1;
  void* a; int8_t* a_q8; void* a_qt;
  void* u; int8_t* g_q8; void* g_qt;
  void* y2; float* mean2; float* rstd2;
  float* part;                          // [(N_SITES + 1) * RED_BLOCKS] per-block partial sums
};

struct LayerBind {
  void* teacher[MREM_N_PARAMS] = {};
  float* student[MREM_N_PARAMS] = {};
  float* w_steps[N_WMAT] = {};
  float* a_steps[N_SITES] = {};
  float* a_off[N_SITES] = {};
};

struct LayerGrad {
  float* p[MREM_N_PARAMS];              // parameter gradients
  float* ws[N_WMAT];                    // weight-step gradients
  float* a;                             // [N_SITES]
  float* off;                           // [N_SITES]
  float* m_p[MREM_N_PARAMS]; float* v_p[MREM_N_PARAMS];
  float* m_ws[N_WMAT]; float* v_ws[N_WMAT];
  float* m_a; float* v_a; float* m_off; float* v_off;
};

struct Arena {                          // bump allocator over the workspace (base may be null: sizing pass)
  char* base = nullptr;
  size_t off = 0;
  void* take(size_t bytes) {
    off = (off + 255) & ~size_t(255);
    void* p = base ? base + off : nullptr;
    off += bytes;
    return p;
  }
};

}  // namespace mrem

// w_grid 2 and 3: the weight scales are recomputed from the weights by a fixed rule, no weight steps exist
inline bool closed_form_weights(const mrem_module_desc& d) { return d.w_grid == 2 || d.w_grid == 3; }

struct mrem_ctx {
  mrem_module_desc d;
  cudaStream_t stream = nullptr;
  int sm_count = 148;
  int dt = 1;                           // storage type id (0 f32, 1 bf16)
  size_t esz = 2;
  long long max_tokens = 0;
  std::string err;
  char* ws_base = nullptr;

  std::vector<mrem::LayerBind> bind;
  std::vector<mrem::LayerStash> stash;
  std::vector<mrem::LayerGrad> grad;
  std::vector<std::vector<mrem::WeightBuf>> wq;     // [layer][4]

  // shared scratch
  void *t_qkv, *t_P, *t_ctx, *t_y1, *t_a, *t_g, *t_y2;   // teacher activations
  float* scores;
  void* x_mix;                                          // Eq. 4 input of the student
  void* dF;                                             // [L, M, H] loss gradients
  void *d_y2, *d_ghat, *d_u, *d_ahat, *d_a, *d_y1, *d_ctxhat, *d_ctx, *d_phat, *d_s, *d_qkvhat, *d_qkv, *d_xhat,
      *d_sum, *carry[2];
  float* col_scratch;
  long long col_plane = 0;               // floats per plane of col_scratch
  int* col_counters;
  float* gb_scratch = nullptr;           // chunk partials and tickets of the column sums the GELU backward takes along
  long long gb_floats = 0;               // (its own: column reductions of the side stream run at the same time)
  int* gb_counters = nullptr;
  int gb_n_counters = 0;
  float* rowbias;
  // second copy of the backward buffers the side stream reads (layers alternate between the two copies, so the
  // main stream may start the layer below while the side stream still works on this one)
  void *alt_d_y2 = nullptr, *alt_d_sum = nullptr, *alt_d_u = nullptr, *alt_d_a = nullptr, *alt_d_y1 = nullptr, *alt_d_qkv = nullptr;
  float* alt_rowbias = nullptr;
  float* loss_partial;
  float* head_scratch = nullptr;         // pooled vectors, gradient and per-sequence errors of the output-logit term
  float* minmax;
  int* status;
  int* t_counter;
  mrem::OptimScalars* optim_sc;
  mrem::ReduceEntry* reduce_table;   int reduce_per_layer = 0;
  mrem::AdamEntry* adam_table;       int adam_entries = 0;  long long adam_elems = 0;   // every trainable tensor
  mrem::AdamEntry* adam_rest;        int rest_entries = 0;  long long rest_elems = 0;   // all but matrices and their steps
  mrem::AdamEntry* rem_table = nullptr;                                                // the two scalar entries of mrem_rem_step
  bool w_ste_done = false;           // the weight gradients have been masked and the step gradients reduced
  // second stream (lowest priority) and its fork/join events: the memory-bound weight updates of a layer
  // run there while the main stream goes on with the tensor-core work of the layer below
  cudaStream_t side_stream = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  cudaEvent_t ev_layer[2] = {nullptr, nullptr};   // side stream done with the gradient buffers of a layer parity
  cudaStream_t teacher_stream = nullptr;   // set for the duration of a step that runs the teacher pass beside the student's
  // classification head of the model's last module (null: none): the output-logit term of the loss
  struct { const float *wp = nullptr, *bp = nullptr, *wc = nullptr, *bc = nullptr; int n_classes = 0; float* logit_loss = nullptr; float* logits = nullptr; } head;
  float loss_share = 1.f;            // this context's share of the whole batch (data parallel: local / global sequences)
  bool use_side_stream = true;       // run the teacher pass and the weight-gradient / update work on the second stream
  bool fused_attention_bwd = true;   // use the single-kernel attention backward where it applies
  bool codes_fresh = false;          // the weight codes match the current latent weights and steps
  mrem::Tracer tracer;               bool trace_on = false;
  void *h2d_xt, *h2d_xs; int32_t* h2d_len; float* d_loss_e2e;   // inputs and loss of the host-buffer step (fixed: graph inputs)
  void* stage_x[2][2]; int32_t* stage_len[2];                   // [slot][teacher|student]: where the copies from the host land
  cudaStream_t copy_stream = nullptr;                           // host -> device copies of the host-buffer step
  cudaEvent_t ev_h2d[2] = {nullptr, nullptr}, ev_host_done[2] = {nullptr, nullptr};
  bool slot_used[2] = {false, false};
  unsigned host_head = 0, host_tail = 0;                        // submitted / waited-for steps
  cudaGraph_t host_graph = nullptr; cudaGraphExec_t host_graph_exec = nullptr;
  struct HostKey { int batch = -1, seq = -1, same = 0, has_len = 0; float lambda = 0.f; mrem_optim optim{}; } host_key;
  void *e2e_t_out, *e2e_s_out;                                  // its layer outputs [L, M, H]
  size_t state_off = 0, state_bytes = 0;                          // optimizer moments: one contiguous range
  bool tables_dirty = true;

  // per-step state
  bool have_input_grad = false;      // carry[0] holds d loss / d module input of the last backward pass
  bool weights_quantized = false, have_teacher = false, have_student = false, have_loss = false, have_grads = false;
  const void* s_in = nullptr;  void* s_out = nullptr;  const void* t_out = nullptr;
  const int32_t* cur_len = nullptr;
  int cur_batch = 0, cur_seq = 0;

  cudaGraph_t graph = nullptr;
  cudaGraphExec_t graph_exec = nullptr;
  float* h_pinned_loss = nullptr;
};
