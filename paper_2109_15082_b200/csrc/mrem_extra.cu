// C-ABI entry points built on the step: activation-step initialisation, the host-buffer
// step, CUDA-graph capture of a step, and the single operations exposed for verification.
#include <cstring>
#include <string>

#include "mrem_ctx.h"

using namespace mrem;

namespace mrem {
int fail(mrem_ctx* c, int code, const char* msg);
int build_tables(mrem_ctx* c);
int float_forward(mrem_ctx* c, const void* x, const int32_t* len, int B, int S, void* outs, bool student_params,
                  bool init_steps);
}  // namespace mrem

namespace {

int enqueue_step(mrem_ctx* c, const void* xt, const void* xs, float lambda, const int32_t* len, int batch, int seq,
                 void* t_out, void* s_out, float* d_loss, const mrem_optim* o) {
  int rc = mrem_quantize_weights(c);
  // Without teacher forcing the two passes are independent until the loss: the teacher's runs on the side
  // stream beside the student's (its tensor-core products under the student's quantizer kernels).  Only
  // with the fused attention kernel, whose path shares no scratch between the passes.
  const bool beside = lambda == 0.f && c->use_side_stream && c->side_stream && !c->trace_on && c->d.n_heads > 0 &&
                      attention_fwd_supported(seq, c->d.hidden / c->d.n_heads, c->dt);
  if (rc == MREM_OK && beside) {
    if (cudaEventRecord(c->ev_fork, c->stream) != cudaSuccess || cudaStreamWaitEvent(c->side_stream, c->ev_fork, 0) != cudaSuccess)
      return fail(c, MREM_ERR_CUDA, "step: stream fork failed");
    c->teacher_stream = c->side_stream;
  }
  if (rc == MREM_OK) rc = mrem_module_forward(c, MREM_TEACHER, xt, nullptr, 0.f, len, batch, seq, t_out);
  c->teacher_stream = nullptr;
  if (rc == MREM_OK) rc = mrem_module_forward(c, MREM_STUDENT, xs, xt, lambda, len, batch, seq, s_out);
  if (beside && (cudaEventRecord(c->ev_join, c->side_stream) != cudaSuccess || cudaStreamWaitEvent(c->stream, c->ev_join, 0) != cudaSuccess))
    return fail(c, MREM_ERR_CUDA, "step: stream join failed");
  if (rc == MREM_OK) rc = mrem_recon_loss(c, d_loss, nullptr);
  if (rc == MREM_OK) rc = mrem_backward_and_step(c, o);
  return rc;
}

int map_gemm_rc(int rc) {
  return rc == GEMM_OK ? MREM_OK : (rc == GEMM_ERR_ALIGN ? MREM_ERR_ALIGN : (rc == GEMM_ERR_ARG ? MREM_ERR_ARG : MREM_ERR_CUDA));
}

}  // namespace

extern "C" {

int32_t mrem_init_act_steps(mrem_ctx* c, const void* x, const int32_t* len, int32_t batch, int32_t seq) {
  if (!c || !x) return MREM_ERR_ARG;
  if (batch < 1 || seq < 1 || batch > c->d.max_batch || seq > c->d.max_seq) return fail(c, MREM_ERR_SHAPE, "init_act_steps: batch/seq outside the context's maximum");
  for (int l = 0; l < c->d.n_layers; ++l) {
    for (int k = 0; k < N_SITES; ++k) if (!c->bind[l].a_steps[k]) return fail(c, MREM_ERR_ORDER, "init_act_steps: activation steps not bound");
    if ((c->d.act_asym_sites & 2) && !c->bind[l].a_off[7]) return fail(c, MREM_ERR_ORDER, "init_act_steps: GELU-site offset not bound");
  }
  const int rc = float_forward(c, x, len, batch, seq, c->e2e_s_out, true, true);
  c->weights_quantized = false;      // the w_hat buffers were used as scratch
  c->codes_fresh = false;
  return rc;
}

// Captures enqueue_step on the context's stream into (*graph, *exec); any earlier pair is destroyed.
static int capture_step_graph(mrem_ctx* c, const void* xt, const void* xs, float lambda, const int32_t* len, int batch,
                              int seq, void* t_out, void* s_out, float* d_loss, const mrem_optim* o, cudaGraph_t* graph,
                              cudaGraphExec_t* exec, const char* who) {
  if (c->tables_dirty) { const int rc = build_tables(c); if (rc != MREM_OK) return rc; }
  if (*exec) { cudaGraphExecDestroy(*exec); *exec = nullptr; }
  if (*graph) { cudaGraphDestroy(*graph); *graph = nullptr; }
  // quantize once outside the graph: inside it the fused update keeps the codes current
  { const int qrc = mrem_quantize_weights(c); if (qrc != MREM_OK) return qrc; }
  if (!c->d.w_step_per_row) c->codes_fresh = false;      // per-matrix steps: every step re-quantizes, inside the graph
  const bool was_tracing = c->trace_on;
  c->trace_on = false;              // event pairs are not recorded inside a captured graph
  struct Restore { mrem_ctx* c; bool v; ~Restore() { c->trace_on = v; } } restore{c, was_tracing};
  if (cudaStreamBeginCapture(c->stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
    cudaGetLastError();   // clear the sticky-until-read error: the legacy default stream cannot be captured
    c->err = std::string(who) + ": begin capture failed (the context's stream must not be the legacy default stream)";
    return MREM_ERR_CUDA;
  }
  const int rc = enqueue_step(c, xt, xs, lambda, len, batch, seq, t_out, s_out, d_loss, o);
  cudaGraph_t g = nullptr;
  const cudaError_t e = cudaStreamEndCapture(c->stream, &g);
  if (rc != MREM_OK) { if (g) cudaGraphDestroy(g); return rc; }
  if (e != cudaSuccess || !g) return fail(c, MREM_ERR_CUDA, "graph capture failed at end capture");
  *graph = g;
  if (cudaGraphInstantiate(exec, g, 0) != cudaSuccess) return fail(c, MREM_ERR_CUDA, "graph instantiate failed");
  return MREM_OK;
}

int32_t mrem_recon_step_host_submit(mrem_ctx* c, const void* h_xt, const void* h_xs, const int32_t* h_len, int32_t batch,
                                    int32_t seq, float lambda, const mrem_optim* o) {
  if (!c || !h_xt || !h_xs || !o) return MREM_ERR_ARG;
  if (batch < 1 || seq < 1 || batch > c->d.max_batch || seq > c->d.max_seq) return fail(c, MREM_ERR_SHAPE, "recon_step_host: batch/seq outside the context's maximum");
  if (c->host_head - c->host_tail >= 2) return fail(c, MREM_ERR_ORDER, "recon_step_host_submit: two steps already in flight; call mrem_recon_step_host_wait");
  const int k = (int)(c->host_head & 1u);
  const size_t bytes = (size_t)batch * seq * c->d.hidden * c->esz;
  const bool same = h_xs == h_xt;
  // copies from the host go to slot k on the copy stream, beside whatever the context's stream is computing
  if (c->slot_used[k] && cudaStreamWaitEvent(c->copy_stream, c->ev_host_done[k], 0) != cudaSuccess) return fail(c, MREM_ERR_CUDA, "recon_step_host: stream wait failed");
  bool okc = cudaMemcpyAsync(c->stage_x[k][0], h_xt, bytes, cudaMemcpyHostToDevice, c->copy_stream) == cudaSuccess;
  if (!same) okc = okc && cudaMemcpyAsync(c->stage_x[k][1], h_xs, bytes, cudaMemcpyHostToDevice, c->copy_stream) == cudaSuccess;
  if (h_len) okc = okc && cudaMemcpyAsync(c->stage_len[k], h_len, sizeof(int32_t) * batch, cudaMemcpyHostToDevice, c->copy_stream) == cudaSuccess;
  okc = okc && cudaEventRecord(c->ev_h2d[k], c->copy_stream) == cudaSuccess && cudaStreamWaitEvent(c->stream, c->ev_h2d[k], 0) == cudaSuccess;
  // from the slot into the step's fixed input buffers (device to device: microseconds)
  okc = okc && cudaMemcpyAsync(c->h2d_xt, c->stage_x[k][0], bytes, cudaMemcpyDeviceToDevice, c->stream) == cudaSuccess;
  if (!same) okc = okc && cudaMemcpyAsync(c->h2d_xs, c->stage_x[k][1], bytes, cudaMemcpyDeviceToDevice, c->stream) == cudaSuccess;
  if (h_len) okc = okc && cudaMemcpyAsync(c->h2d_len, c->stage_len[k], sizeof(int32_t) * batch, cudaMemcpyDeviceToDevice, c->stream) == cudaSuccess;
  if (!okc) return fail(c, MREM_ERR_CUDA, "recon_step_host: copy failed");
  const void* xs = same ? c->h2d_xt : c->h2d_xs;
  const int32_t* len = h_len ? c->h2d_len : nullptr;
  int rc;
  const bool capturable = c->stream != nullptr && c->stream != cudaStreamLegacy;
  if (o->step > 0 || c->trace_on || !capturable) {
    // an explicit step number is baked into the launch arguments, traced kernels are timed one by one, and the
    // legacy default stream cannot be captured: no graph
    rc = enqueue_step(c, c->h2d_xt, xs, lambda, len, batch, seq, c->e2e_t_out, c->e2e_s_out, c->d_loss_e2e, o);
  } else {
    mrem_ctx::HostKey key;
    key.batch = batch; key.seq = seq; key.same = same; key.has_len = h_len != nullptr; key.lambda = lambda; key.optim = *o;
    const mrem_ctx::HostKey& old = c->host_key;
    const bool hit = c->host_graph_exec && old.batch == key.batch && old.seq == key.seq && old.same == key.same &&
                     old.has_len == key.has_len && old.lambda == key.lambda && memcmp(&old.optim, &key.optim, sizeof(mrem_optim)) == 0;
    rc = MREM_OK;
    if (!hit) {
      rc = capture_step_graph(c, c->h2d_xt, xs, lambda, len, batch, seq, c->e2e_t_out, c->e2e_s_out, c->d_loss_e2e, o,
                              &c->host_graph, &c->host_graph_exec, "recon_step_host");
      if (rc == MREM_OK) c->host_key = key;
    } else if (!c->codes_fresh && c->d.w_step_per_row) {
      rc = mrem_quantize_weights(c);          // weights or steps were written from outside since the last step
    }
    if (rc == MREM_OK && cudaGraphLaunch(c->host_graph_exec, c->stream) != cudaSuccess) rc = fail(c, MREM_ERR_CUDA, "recon_step_host: graph launch failed");
    if (rc == MREM_OK) {                      // the host-side state the eager call sequence would have left
      c->t_out = c->e2e_t_out; c->s_out = c->e2e_s_out; c->s_in = xs;
      c->cur_batch = batch; c->cur_seq = seq; c->cur_len = len;
      c->have_grads = false; c->have_loss = false; c->have_student = false; c->have_teacher = false;
      c->codes_fresh = c->d.w_step_per_row != 0;
      c->weights_quantized = c->codes_fresh;
    }
  }
  if (rc != MREM_OK) return rc;
  if (cudaMemcpyAsync(c->h_pinned_loss + k, c->d_loss_e2e, sizeof(float), cudaMemcpyDeviceToHost, c->stream) != cudaSuccess ||
      cudaEventRecord(c->ev_host_done[k], c->stream) != cudaSuccess)
    return fail(c, MREM_ERR_CUDA, "recon_step_host: device error");
  c->slot_used[k] = true;
  ++c->host_head;
  return MREM_OK;
}

int32_t mrem_recon_step_host_wait(mrem_ctx* c, float* h_loss) {
  if (!c || !h_loss) return MREM_ERR_ARG;
  if (c->host_tail == c->host_head) return fail(c, MREM_ERR_ORDER, "recon_step_host_wait: no step in flight");
  const int k = (int)(c->host_tail & 1u);
  if (cudaEventSynchronize(c->ev_host_done[k]) != cudaSuccess) return fail(c, MREM_ERR_CUDA, "recon_step_host_wait: device error");
  *h_loss = c->h_pinned_loss[k];
  ++c->host_tail;
  return MREM_OK;
}

int32_t mrem_recon_step_host(mrem_ctx* c, const void* h_xt, const void* h_xs, const int32_t* h_len, int32_t batch,
                             int32_t seq, float lambda, const mrem_optim* o, float* h_loss) {
  if (!c || !h_loss) return MREM_ERR_ARG;
  if (c->host_tail != c->host_head) return fail(c, MREM_ERR_ORDER, "recon_step_host: submitted steps are still in flight; wait for them first");
  const int rc = mrem_recon_step_host_submit(c, h_xt, h_xs, h_len, batch, seq, lambda, o);
  return rc != MREM_OK ? rc : mrem_recon_step_host_wait(c, h_loss);
}

int32_t mrem_graph_capture_step(mrem_ctx* c, const void* xt, const void* xs, float lambda, const int32_t* len,
                                int32_t batch, int32_t seq, void* t_out, void* s_out, float* d_loss,
                                const mrem_optim* o) {
  if (!c || !xt || !xs || !t_out || !s_out || !d_loss || !o) return MREM_ERR_ARG;
  if (o->step > 0) return fail(c, MREM_ERR_ARG, "graph_capture_step: optim.step must be 0 (device-side counter)");
  return capture_step_graph(c, xt, xs, lambda, len, batch, seq, t_out, s_out, d_loss, o, &c->graph, &c->graph_exec,
                            "graph_capture_step");
}

int32_t mrem_graph_num_kernels(mrem_ctx* c, int32_t* n_kernels) {
  if (!c || !n_kernels) return MREM_ERR_ARG;
  if (!c->graph) return fail(c, MREM_ERR_ORDER, "graph_num_kernels: no captured step");
  size_t n = 0;
  if (cudaGraphGetNodes(c->graph, nullptr, &n) != cudaSuccess) return fail(c, MREM_ERR_CUDA, "graph_num_kernels failed");
  std::vector<cudaGraphNode_t> nodes(n);
  if (n && cudaGraphGetNodes(c->graph, nodes.data(), &n) != cudaSuccess) return fail(c, MREM_ERR_CUDA, "graph_num_kernels failed");
  int k = 0;
  for (size_t i = 0; i < n; ++i) {
    cudaGraphNodeType t;
    if (cudaGraphNodeGetType(nodes[i], &t) == cudaSuccess && t == cudaGraphNodeTypeKernel) ++k;
  }
  *n_kernels = k;
  return MREM_OK;
}

int32_t mrem_graph_launch(mrem_ctx* c) {
  if (!c) return MREM_ERR_ARG;
  if (!c->graph_exec) return fail(c, MREM_ERR_ORDER, "graph_launch: no captured step");
  return cudaGraphLaunch(c->graph_exec, c->stream) == cudaSuccess ? MREM_OK : fail(c, MREM_ERR_CUDA, "graph_launch failed");
}

// ------------------------------------------------------------------ single operations

int32_t mrem_quantize_act(const void* x, int32_t dtype, int64_t n, const float* step, const float* offset, int32_t lo,
                          int32_t hi, int8_t* q8, void* qt, void* st) {
  if (!x || !step || n < 0 || (dtype != MREM_F32 && dtype != MREM_BF16) || lo > hi || lo < -128 || hi > 255) return MREM_ERR_ARG;
  if (n == 0) return MREM_OK;
  // a flat tensor is a view of `rows` rows of 2^k columns (largest power of two <= 4096 dividing n)
  int cols = 1;
  while (cols < 4096 && n % (cols * 2) == 0) cols *= 2;
  const long long rows = n / cols;
  launch_quantize_act(x, dtype, rows, cols, cols, step, offset, lo, hi, q8, cols, qt, cols, (cudaStream_t)st);
  return cudaGetLastError() == cudaSuccess ? MREM_OK : MREM_ERR_CUDA;
}

int32_t mrem_quantize_weight(const float* w, int32_t rows, int32_t cols, const float* steps, int32_t per_row,
                             int32_t bits, int32_t grid, int8_t* codes, int32_t* rowsum, float* scale, void* what,
                             int32_t dtype, void* st) {
  if (!w || !steps || !codes || !rowsum || !scale || rows < 0 || cols < 1) return MREM_ERR_ARG;
  if ((bits != 2 && bits != 4 && bits != 8) || (grid != 0 && !(grid == 1 && bits == 2))) return MREM_ERR_UNSUPPORTED;
  if (dtype != MREM_F32 && dtype != MREM_BF16) return MREM_ERR_ARG;
  if (rows == 0) return MREM_OK;
  launch_quantize_weight(w, rows, cols, steps, per_row, bits, grid, codes, rowsum, scale, what, dtype, (cudaStream_t)st);
  return cudaGetLastError() == cudaSuccess ? MREM_OK : MREM_ERR_CUDA;
}

int32_t mrem_gemm_i8(const int8_t* a, int32_t a_unsigned, const int8_t* b, int32_t M, int32_t N, int32_t K,
                     int32_t* acc, int32_t block_n, int32_t* d_status, void* st) {
  if (!a || !b || !acc || !d_status || M < 0 || N < 0 || K < 1) return MREM_ERR_ARG;
  if (K % 16) return MREM_ERR_ALIGN;
  if (M == 0 || N == 0) return MREM_OK;
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return MREM_ERR_CUDA;
  OperandDesc A{a, K, 0, 0, 0}, B{b, K, 0, 0, 0};
  GemmShape g{M, N, K, 1, 1};
  Epilogue e{};
  e.out = acc; e.out_kind = OUT_I32; e.ldc = N; e.alpha_const = 1.f;
  return map_gemm_rc(tc_gemm(1, a_unsigned, A, B, g, e, block_n, d_status, sms, (cudaStream_t)st));
}

int32_t mrem_gemm(int32_t dtype, const void* a, int32_t a_mn, int64_t lda, int64_t a_bs, const void* b, int32_t b_mn,
                  int64_t ldb, int64_t b_bs, int32_t M, int32_t N, int32_t K, int32_t batches, float alpha, float* out,
                  int64_t ldc, int64_t c_bs, int32_t block_n, int32_t* d_status, void* st) {
  if (!a || !b || !out || !d_status || M < 0 || N < 0 || K < 1 || batches < 1) return MREM_ERR_ARG;
  if (dtype != MREM_F32 && dtype != MREM_BF16) return MREM_ERR_ARG;
  if (M == 0 || N == 0) return MREM_OK;
  OperandDesc A{a, lda, a_bs, 0, a_mn}, B{b, ldb, b_bs, 0, b_mn};
  GemmShape g{M, N, K, batches, 1};
  Epilogue e{};
  e.out = out; e.out_kind = OUT_F32; e.ldc = ldc; e.c_b0 = c_bs; e.alpha_const = alpha;
  if (dtype == MREM_F32) return map_gemm_rc(simt_gemm_f32(A, B, g, e, (cudaStream_t)st));
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return MREM_ERR_CUDA;
  return map_gemm_rc(tc_gemm(0, 0, A, B, g, e, block_n, d_status, sms, (cudaStream_t)st));
}

}  // extern "C"
