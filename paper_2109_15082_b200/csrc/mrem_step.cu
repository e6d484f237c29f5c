// The reconstruction step (Algorithm 2): weight quantization, teacher and student forward,
// loss (Eq. 3), straight-through backward and the AdamW update, as sequences of kernel
// launches on the context's stream.  No host synchronisation, no allocation.
#include <cmath>

#include "mrem_ctx.h"

using namespace mrem;

namespace mrem {
int fail(mrem_ctx* c, int code, const char* msg);
void param_shape(const mrem_module_desc& d, int id, int* rows, int* cols);
int build_tables(mrem_ctx* c);
}  // namespace mrem

namespace {

const int kMatParam[N_WMAT] = {MREM_WQKV, MREM_WO, MREM_W1, MREM_W2};
enum { W_QKV = 0, W_O = 1, W_1 = 2, W_2 = 3 };
enum { S_X = 0, S_Q = 1, S_K = 2, S_V = 3, S_P = 4, S_C = 5, S_A = 6, S_G = 7 };

struct View {                      // an operand: pointer, stride of the non-contiguous index, batch strides
  const void* p; long long ld, sb0, sb1; int mn; int is_static;
};
inline View view(const void* p, long long ld, int mn = 0, long long sb0 = 0, long long sb1 = 0) {
  return View{p, ld, sb0, sb1, mn, 0};
}
// a weight matrix (or its dequantized form): written by no kernel that directly precedes a product reading it, so the
// product may fetch its first tiles before its predecessor in the stream has finished
inline View weights(const void* p, long long ld, int mn = 0) { return View{p, ld, 0, 0, mn, 1}; }

struct Epi {                       // shorthand builder of an Epilogue
  Epilogue e{};
  Epi(void* out, int kind, long long ldc, long long cb0 = 0, long long cb1 = 0) {
    e.out = out; e.out_kind = kind; e.ldc = ldc; e.c_b0 = cb0; e.c_b1 = cb1; e.alpha_const = 1.f;
  }
  Epi& alpha(float a, const float* p0 = nullptr, const float* p1 = nullptr) { e.alpha_const = a; e.alpha_p0 = p0; e.alpha_p1 = p1; return *this; }
  Epi& colscale(const float* p) { e.col_scale = p; return *this; }
  Epi& colbias(const float* p) { e.col_bias = p; return *this; }
  Epi& rowbias(const float* p) { e.row_bias = p; return *this; }
  Epi& residual(const void* p) { e.residual = p; return *this; }
  Epi& gelu() { e.act = 1; return *this; }
};

struct Runner {
  mrem_ctx* c;
  int rc = MREM_OK;
  cudaStream_t st;
  explicit Runner(mrem_ctx* ctx) : c(ctx), st(ctx->stream) {}
  Runner(mrem_ctx* ctx, cudaStream_t stream) : c(ctx), st(stream) {}
  int okind() const { return c->dt == 1 ? OUT_BF16 : OUT_F32; }
  void* at(const void* p, long long elems) const { return (char*)p + elems * (long long)c->esz; }

  void note(int grc, const char* what) {
    if (grc != GEMM_OK && rc == MREM_OK) {
      rc = grc == GEMM_ERR_ALIGN ? MREM_ERR_ALIGN : (grc == GEMM_ERR_ARG ? MREM_ERR_ARG : MREM_ERR_CUDA);
      c->err = what;
    }
  }
  // storage-type product on the tensor cores (bf16) or CUDA cores (f32)
  void gemm(const View& A, const View& B, int M, int N, int K, int nb0, int nb1, const Epilogue& e) {
    OperandDesc a{A.p, A.ld, A.sb0, A.sb1, A.mn, 0}, b{B.p, B.ld, B.sb0, B.sb1, B.mn, B.is_static};
    GemmShape g{M, N, K, nb0, nb1};
    if (c->dt == 1) note(tc_gemm(0, 0, a, b, g, e, 0, c->status, c->sm_count, st), "bf16 GEMM launch failed");
    else note(simt_gemm_f32(a, b, g, e, st), "f32 GEMM launch failed");
  }
  // weight-gradient products (bf16 in, fp32 out) of one layer: collected, then launched as one grouped kernel
  // over the joint tile list where the tensor-core path takes them, else one by one
  std::vector<GemmGroupItem> deferred;
  void defer(const View& A, const View& B, int M, int N, int K, const Epilogue& e) {
    if (c->dt != 1) { gemm(A, B, M, N, K, 1, 1, e); return; }
    GemmGroupItem it{OperandDesc{A.p, A.ld, A.sb0, A.sb1, A.mn}, OperandDesc{B.p, B.ld, B.sb0, B.sb1, B.mn}, GemmShape{M, N, K, 1, 1}, e};
    deferred.push_back(it);
  }
  void flush_deferred() {
    if (deferred.empty()) return;
    if ((int)deferred.size() <= MAX_GEMM_GROUP && tc_gemm_group_eligible(deferred.data(), (int)deferred.size())) {
      note(tc_gemm_group(deferred.data(), (int)deferred.size(), c->status, c->sm_count, st), "grouped weight-gradient GEMM launch failed");
    } else {
      for (const GemmGroupItem& it : deferred)
        note(tc_gemm(0, 0, it.A, it.B, it.g, it.epi, 0, c->status, c->sm_count, st), "bf16 GEMM launch failed");
    }
    deferred.clear();
  }
  // integer-code product with exact int32 accumulation
  void gemm_i8(const int8_t* A, int a_unsigned, const int8_t* B, int M, int N, int K, const Epilogue& e) {
    OperandDesc a{A, K, 0, 0, 0, 0}, b{B, K, 0, 0, 0, 1};      // B: weight codes, written by the last update
    GemmShape g{M, N, K, 1, 1};
    note(tc_gemm(1, a_unsigned, a, b, g, e, 0, c->status, c->sm_count, st), "int8 GEMM launch failed");
  }
};

struct ActRange { int lo, hi; bool asym; };
ActRange site_range(const mrem_module_desc& d, int site) {
  const bool asym = (site == S_P && (d.act_asym_sites & 1)) || (site == S_G && (d.act_asym_sites & 2));
  if (asym) return {0, (1 << d.a_bits) - 1, true};
  const int q = (1 << (d.a_bits - 1)) - 1;
  return {-q, q, false};
}

int check_io(mrem_ctx* c, const void* x, int batch, int seq, void* outs) {
  if (!x || !outs) return fail(c, MREM_ERR_ARG, "forward: NULL tensor");
  if (batch < 1 || seq < 1 || batch > c->d.max_batch || seq > c->d.max_seq) return fail(c, MREM_ERR_SHAPE, "forward: batch/seq outside the context's maximum");
  if (c->dt == 1 && seq % 8) return fail(c, MREM_ERR_SHAPE, "forward: bf16 path needs seq % 8 == 0");
  if ((reinterpret_cast<uintptr_t>(x) & 15) || (reinterpret_cast<uintptr_t>(outs) & 15)) return fail(c, MREM_ERR_ALIGN, "forward: tensors must be 16-byte aligned");
  return MREM_OK;
}

// Sets one activation step (and offset) from the range of a 2-D view.
void init_site(mrem_ctx* c, const LayerBind& b, int site, const void* x, long long ld, long long rows, int cols) {
  const ActRange r = site_range(c->d, site);
  launch_minmax(x, ld, rows, cols, c->minmax, c->col_scratch, c->dt, c->stream);
  const int mode = !r.asym ? 0 : (site == S_P ? 1 : 2);
  launch_step_from_minmax(c->minmax, mode, (float)r.hi, b.a_steps[site], mode == 2 ? b.a_off[site] : nullptr, c->stream);
}

}  // namespace

namespace mrem {
// ------------------------------------------------------------------ full-precision forward
// The teacher pass.  With `student_params` the same graph runs on the student's latent
// parameters (matrices narrowed to the storage type in the w_hat buffers) and, with
// `init_steps`, sets every activation step of the student from the ranges it sees.
int float_forward(mrem_ctx* c, const void* x, const int32_t* len, int B, int S, void* outs, bool student_params,
                  bool init_steps) {
  const mrem_module_desc& d = c->d;
  const int H = d.hidden, F = d.ffn, h = d.n_heads, hd = H / h;
  const long long M = (long long)B * S;
  cudaStream_t st = (!student_params && !init_steps && c->teacher_stream) ? c->teacher_stream : c->stream;
  Runner r(c, st);
  const int ok = r.okind();
  const void* cur = x;
  for (int l = 0; l < d.n_layers; ++l) {
    LayerBind b = c->bind[l];
    if (student_params) {
      for (int k = 0; k < MREM_N_PARAMS; ++k) {
        if (!b.student[k]) return fail(c, MREM_ERR_ORDER, "forward: student parameters not bound");
        b.teacher[k] = b.student[k];
      }
      for (int k = 0; k < N_WMAT; ++k) {
        WeightBuf& w = c->wq[l][k];
        launch_narrow(b.student[kMatParam[k]], w.what, (long long)w.rows * w.cols, c->dt, st);
        b.teacher[kMatParam[k]] = w.what;
      }
    }
    for (int k = 0; k < MREM_N_PARAMS; ++k) if (!b.teacher[k]) return fail(c, MREM_ERR_ORDER, "forward: teacher parameters not bound");
    void* out = r.at(outs, (long long)l * M * H);
    if (init_steps) init_site(c, b, S_X, cur, H, M, H);
    r.gemm(view(cur, H), (student_params ? view(b.teacher[MREM_WQKV], H) : weights(b.teacher[MREM_WQKV], H)), (int)M, 3 * H, H, 1, 1,
           Epi(c->t_qkv, ok, 3 * H).colbias((float*)b.teacher[MREM_BQKV]).e);
    if (init_steps)
      for (int seg = 0; seg < 3; ++seg) init_site(c, b, S_Q + seg, r.at(c->t_qkv, seg * H), 3 * H, M, H);
    if (attention_fwd_supported(S, hd, c->dt)) {
      // (the probabilities of the full-precision pass are read only when the activation steps are initialised)
      r.note(launch_attention_fwd(c->t_qkv, B, S, h, H, len, 1.f / sqrtf((float)hd), nullptr, nullptr, nullptr, nullptr,
                                  nullptr, 0, 0, init_steps ? c->t_P : nullptr, nullptr, c->t_ctx, nullptr, 0, nullptr, nullptr, c->status, st),
             "attention launch failed");
    } else {
      r.gemm(view(c->t_qkv, 3 * H, 0, hd, (long long)S * 3 * H), view(r.at(c->t_qkv, H), 3 * H, 0, hd, (long long)S * 3 * H),
             S, S, hd, h, B, Epi(c->scores, OUT_F32, S, (long long)S * S, (long long)h * S * S).alpha(1.f / sqrtf((float)hd)).e);
      launch_softmax_fwd(c->scores, len, B, h, S, c->t_P, nullptr, nullptr, 0, 0, nullptr, c->dt, st);
      r.gemm(view(c->t_P, S, 0, (long long)S * S, (long long)h * S * S), view(r.at(c->t_qkv, 2 * H), 3 * H, 1, hd, (long long)S * 3 * H),
             S, hd, S, h, B, Epi(c->t_ctx, ok, H, hd, (long long)S * H).e);
    }
    if (init_steps) init_site(c, b, S_P, c->t_P, S, (long long)B * h * S, S);
    if (init_steps) init_site(c, b, S_C, c->t_ctx, H, M, H);
    r.gemm(view(c->t_ctx, H), (student_params ? view(b.teacher[MREM_WO], H) : weights(b.teacher[MREM_WO], H)), (int)M, H, H, 1, 1,
           Epi(c->t_y1, ok, H).colbias((float*)b.teacher[MREM_BO]).residual(cur).e);
    launch_layernorm_fwd(c->t_y1, (float*)b.teacher[MREM_LN1_G], (float*)b.teacher[MREM_LN1_B], d.ln_eps, M, H, c->t_a,
                         nullptr, nullptr, nullptr, 0, nullptr, nullptr, c->dt, st);
    if (init_steps) init_site(c, b, S_A, c->t_a, H, M, H);
    r.gemm(view(c->t_a, H), (student_params ? view(b.teacher[MREM_W1], H) : weights(b.teacher[MREM_W1], H)), (int)M, F, H, 1, 1,
           Epi(c->t_g, ok, F).colbias((float*)b.teacher[MREM_B1]).gelu().e);
    if (init_steps) init_site(c, b, S_G, c->t_g, F, M, F);
    r.gemm(view(c->t_g, F), (student_params ? view(b.teacher[MREM_W2], F) : weights(b.teacher[MREM_W2], F)), (int)M, H, F, 1, 1,
           Epi(c->t_y2, ok, H).colbias((float*)b.teacher[MREM_B2]).residual(c->t_a).e);
    launch_layernorm_fwd(c->t_y2, (float*)b.teacher[MREM_LN2_G], (float*)b.teacher[MREM_LN2_B], d.ln_eps, M, H, out,
                         nullptr, nullptr, nullptr, 0, nullptr, nullptr, c->dt, st);
    cur = out;
  }
  if (r.rc != MREM_OK) return r.rc;
  return cudaGetLastError() == cudaSuccess ? MREM_OK : fail(c, MREM_ERR_CUDA, "forward: launch failed");
}
}  // namespace mrem

namespace {

// ------------------------------------------------------------------ student
// The fake-quantized pass: a quantizer on both operands of every matrix product.
// Linear layers run on int8 codes with exact int32 accumulation; attention products on codes held as storage-type numbers.
int student_forward(mrem_ctx* c, const void* x, const int32_t* len, int B, int S, void* outs) {
  const mrem_module_desc& d = c->d;
  const int H = d.hidden, F = d.ffn, h = d.n_heads, hd = H / h;
  const long long M = (long long)B * S;
  Runner r(c);
  const int ok = r.okind();
  const void* cur = x;
  for (int l = 0; l < d.n_layers; ++l) {
    const LayerBind& b = c->bind[l];
    LayerStash& s = c->stash[l];
    std::vector<WeightBuf>& w = c->wq[l];
    for (int k = 0; k < MREM_N_PARAMS; ++k) if (!b.student[k]) return fail(c, MREM_ERR_ORDER, "forward: student parameters not bound");
    for (int k = 0; k < N_SITES; ++k) if (!b.a_steps[k]) return fail(c, MREM_ERR_ORDER, "forward: activation steps not bound");
    if ((d.act_asym_sites & 2) && !b.a_off[S_G]) return fail(c, MREM_ERR_ORDER, "forward: GELU-site offset not bound");
    void* out = r.at(outs, (long long)l * M * H);
    const ActRange rx = site_range(d, S_X), rp = site_range(d, S_P), rg = site_range(d, S_G);

    // (layers above the first get the codes of their input from the LayerNorm that produced it)
    if (l == 0) launch_quantize_act(cur, c->dt, M, H, H, b.a_steps[S_X], nullptr, rx.lo, rx.hi, s.x_q8, H, s.x_qt, H, c->stream);
    r.gemm_i8(s.x_q8, 0, w[W_QKV].codes, (int)M, 3 * H, H,
              Epi(s.qkv, ok, 3 * H).alpha(1.f, b.a_steps[S_X]).colscale(w[W_QKV].scale).colbias(b.student[MREM_BQKV]).e);
    launch_quantize_act3(s.qkv, c->dt, M, H, 3 * H, b.a_steps[S_Q], b.a_steps[S_K], b.a_steps[S_V], rx.lo, rx.hi, s.qkv_qt,
                         3 * H, c->stream);
    if (attention_fwd_supported(S, hd, c->dt)) {
      // (the single-kernel attention backward takes the codes of the probabilities from the probabilities themselves:
      //  they are written out only for the kernel-per-operation backward)
      const bool codes_needed = !(c->fused_attention_bwd && attention_bwd_supported(S, hd, c->dt, B * h));
      r.note(launch_attention_fwd(s.qkv_qt, B, S, h, H, len, 1.f / sqrtf((float)hd), b.a_steps[S_Q], b.a_steps[S_K],
                                  b.a_steps[S_P], b.a_steps[S_V], b.a_steps[S_P], rp.lo, rp.hi, s.P, codes_needed ? s.P_qt : nullptr, s.ctx,
                                  b.a_steps[S_C], rx.hi, s.ctx_q8, s.ctx_qt, c->status, c->stream),
             "attention launch failed");
    } else {
      r.gemm(view(s.qkv_qt, 3 * H, 0, hd, (long long)S * 3 * H), view(r.at(s.qkv_qt, H), 3 * H, 0, hd, (long long)S * 3 * H),
             S, S, hd, h, B,
             Epi(c->scores, OUT_F32, S, (long long)S * S, (long long)h * S * S).alpha(1.f / sqrtf((float)hd), b.a_steps[S_Q], b.a_steps[S_K]).e);
      launch_softmax_fwd(c->scores, len, B, h, S, s.P, b.a_steps[S_P], nullptr, rp.lo, rp.hi, s.P_qt, c->dt, c->stream);
      r.gemm(view(s.P_qt, S, 0, (long long)S * S, (long long)h * S * S), view(r.at(s.qkv_qt, 2 * H), 3 * H, 1, hd, (long long)S * 3 * H),
             S, hd, S, h, B, Epi(s.ctx, ok, H, hd, (long long)S * H).alpha(1.f, b.a_steps[S_P], b.a_steps[S_V]).e);
      launch_quantize_act(s.ctx, c->dt, M, H, H, b.a_steps[S_C], nullptr, rx.lo, rx.hi, s.ctx_q8, H, s.ctx_qt, H, c->stream);
    }
    r.gemm_i8(s.ctx_q8, 0, w[W_O].codes, (int)M, H, H,
              Epi(s.y1, ok, H).alpha(1.f, b.a_steps[S_C]).colscale(w[W_O].scale).colbias(b.student[MREM_BO]).residual(cur).e);
    launch_layernorm_fwd(s.y1, b.student[MREM_LN1_G], b.student[MREM_LN1_B], d.ln_eps, M, H, s.a, s.mean1, s.rstd1,
                         b.a_steps[S_A], rx.hi, s.a_q8, s.a_qt, c->dt, c->stream);
    r.gemm_i8(s.a_q8, 0, w[W_1].codes, (int)M, F, H,
              Epi(s.u, ok, F).alpha(1.f, b.a_steps[S_A]).colscale(w[W_1].scale).colbias(b.student[MREM_B1]).e);
    launch_gelu_quant(s.u, M * F, b.a_steps[S_G], rg.asym ? b.a_off[S_G] : nullptr, rg.lo, rg.hi, s.g_q8, s.g_qt, c->dt, c->stream);
    const float* bias2 = b.student[MREM_B2];
    if (rg.asym) {
      launch_effective_bias(b.student[MREM_B2], b.a_off[S_G], w[W_2].scale, w[W_2].rowsum, w[W_2].beff, H, c->stream);
      bias2 = w[W_2].beff;
    }
    r.gemm_i8(s.g_q8, rg.asym ? 1 : 0, w[W_2].codes, (int)M, H, F,
              Epi(s.y2, ok, H).alpha(1.f, b.a_steps[S_G]).colscale(w[W_2].scale).colbias(bias2).residual(s.a).e);
    if (l + 1 < d.n_layers)
      launch_layernorm_fwd(s.y2, b.student[MREM_LN2_G], b.student[MREM_LN2_B], d.ln_eps, M, H, out, s.mean2, s.rstd2,
                           c->bind[l + 1].a_steps[S_X], rx.hi, c->stash[l + 1].x_q8, c->stash[l + 1].x_qt, c->dt, c->stream);
    else
      launch_layernorm_fwd(s.y2, b.student[MREM_LN2_G], b.student[MREM_LN2_B], d.ln_eps, M, H, out, s.mean2, s.rstd2,
                           nullptr, 0, nullptr, nullptr, c->dt, c->stream);
    cur = out;
  }
  if (r.rc != MREM_OK) return r.rc;
  return cudaGetLastError() == cudaSuccess ? MREM_OK : fail(c, MREM_ERR_CUDA, "student forward: launch failed");
}

// The fused update of one layer's four matrices and their row steps (Algorithm 2: Update(w), Update(s)).
void enqueue_matrix_update(mrem_ctx* c, int l, int k, cudaStream_t st) {
  const mrem_module_desc& d = c->d;
  const int train_w = (d.trainable_mask & MREM_TRAIN_WEIGHTS) != 0, train_s = (d.trainable_mask & MREM_TRAIN_W_STEPS) != 0;
  const int pid = kMatParam[k];
  WeightBuf& w = c->wq[l][k];
  LayerGrad& g = c->grad[l];
  if (closed_form_weights(d)) {
    launch_closed_form_update(c->bind[l].student[pid], g.p[pid], g.m_p[pid], g.v_p[pid], c->optim_sc, w.rows, w.cols, train_w,
                              d.w_grid, d.w_bits, w.codes, w.rowsum, w.scale, w.what, c->dt, st);
    return;
  }
  launch_fused_weight_update(c->bind[l].student[pid], g.p[pid], g.m_p[pid], g.v_p[pid], c->bind[l].w_steps[k],
                             c->w_ste_done ? g.ws[k] : nullptr, g.m_ws[k], g.v_ws[k], c->optim_sc, w.rows, w.cols,
                             d.w_bits, d.w_grid, train_w, train_s, w.codes, w.rowsum, w.scale, w.what, c->dt, st);
}
void enqueue_matrix_updates(mrem_ctx* c, int l, cudaStream_t st) {
  for (int k = 0; k < N_WMAT; ++k) enqueue_matrix_update(c, l, k, st);
}

// ------------------------------------------------------------------ backward
// Two streams: the weight-gradient products (tensor-core bound, results needed only by the update) are
// issued on the side stream and run under the main stream's element-wise and row kernels (memory bound);
// the main stream waits for them before the next layer reuses the gradient buffers they read.  With
// `update_as_you_go` (per-row steps; the optimizer scalars of this step are already on the device) each
// layer's matrices are also updated on the side stream as soon as their gradients are complete.  The main
// stream joins the side stream before returning.  While kernels are being timed one by one (tracing) all
// of it stays on the main stream.
int student_backward(mrem_ctx* c, bool update_as_you_go) {
  const mrem_module_desc& d = c->d;
  const int H = d.hidden, F = d.ffn, h = d.n_heads, hd = H / h, B = c->cur_batch, S = c->cur_seq;
  const long long M = (long long)B * S;
  const long long sSS = (long long)S * S, sHSS = (long long)h * S * S, sQKV = (long long)S * 3 * H;
  Runner r(c);
  const bool two_streams = c->use_side_stream && c->side_stream && !c->trace_on;
  cudaStream_t side = two_streams ? c->side_stream : c->stream;
  Runner rw(c, side);                            // weight-gradient products
  bool sync_failed = false;
  auto fork = [&]() {                            // side stream: wait for what the main stream has enqueued so far
    if (two_streams && (cudaEventRecord(c->ev_fork, c->stream) != cudaSuccess || cudaStreamWaitEvent(side, c->ev_fork, 0) != cudaSuccess))
      sync_failed = true;
  };
  auto join = [&]() {                            // main stream: wait for what the side stream has enqueued so far
    if (two_streams && (cudaEventRecord(c->ev_join, side) != cudaSuccess || cudaStreamWaitEvent(c->stream, c->ev_join, 0) != cudaSuccess))
      sync_failed = true;
  };
  const int ok = r.okind();
  const float inv_sqrt_d = 1.f / sqrtf((float)hd);
  // Buffers the side stream reads, two copies used by alternate layers: the main stream starts the layer below while
  // the side stream still reduces and multiplies this layer's gradients, and waits (ev_layer) only before it
  // overwrites the copy of the layer two above.
  struct SideBufs { void *d_y2, *d_sum, *d_u, *d_a, *d_y1, *d_qkv; float* rowbias; };
  const SideBufs copies[2] = {{c->d_y2, c->d_sum, c->d_u, c->d_a, c->d_y1, c->d_qkv, c->rowbias},
                              {c->alt_d_y2, c->alt_d_sum, c->alt_d_u, c->alt_d_a, c->alt_d_y1, c->alt_d_qkv, c->alt_rowbias}};
  const void* carry = nullptr;
  // the straight-through passes that feed a LayerNorm's backward run inside it where the row fits its registers
  const bool fuse_ln = layernorm_bwd_ste_supported(H, c->dt);
  struct { const void* x; const void* add; const float* step; float* part; } pending = {nullptr, nullptr, nullptr, nullptr};
  for (int l = d.n_layers - 1; l >= 0; --l) {
    const LayerBind& b = c->bind[l];
    LayerStash& s = c->stash[l];
    LayerGrad& g = c->grad[l];
    std::vector<WeightBuf>& w = c->wq[l];
    const void* x_in = l == 0 ? c->s_in : r.at(c->s_out, (long long)(l - 1) * M * H);
    const void* dF = r.at(c->dF, (long long)l * M * H);
    const ActRange rx = site_range(d, S_X), rp = site_range(d, S_P), rg = site_range(d, S_G);
    float* part = s.part;
    cudaStream_t st = c->stream;
    const SideBufs& q = copies[l & 1];
    if (two_streams && l + 2 < d.n_layers && cudaStreamWaitEvent(c->stream, c->ev_layer[l & 1], 0) != cudaSuccess) sync_failed = true;

    // second LayerNorm: total gradient at the layer output = loss term + what the next layer sent back
    // (with `pending` the layer above left its input gradient unmasked: the straight-through pass of its input
    //  quantizer and its skip connection are applied while this LayerNorm's backward reads them)
    bool sent_back = carry != nullptr;
    if (pending.x) {
      const bool fused = launch_layernorm_bwd_ste(dF, pending.x, c->d_xhat, pending.add, pending.step, rx.lo, rx.hi, s.y2, s.mean2, s.rstd2,
                                                  b.student[MREM_LN2_G], M, H, q.d_y2, q.d_sum, pending.part, c->dt, st);
      if (!fused) {
        launch_ste_act(pending.x, H, c->d_xhat, H, pending.add, H, c->carry[0], H, M, H, pending.step, nullptr, rx.lo, rx.hi,
                       pending.part, nullptr, c->dt, st);
        launch_layernorm_bwd(dF, c->carry[0], s.y2, s.mean2, s.rstd2, b.student[MREM_LN2_G], M, H, q.d_y2, q.d_sum, c->dt, st);
      }
      sent_back = true;
      pending.x = nullptr;
    } else {
      launch_layernorm_bwd(dF, carry, s.y2, s.mean2, s.rstd2, b.student[MREM_LN2_G], M, H, q.d_y2, carry ? q.d_sum : nullptr, c->dt, st);
    }
    // LayerNorm parameter gradients and the bias gradient of FFN2 (y2 = G_hat W2_hat^T + b2 + a) in one pass
    // (column sums feed only the update and the weight-gradient epilogue: side stream)
    fork();
    launch_col_reduce(sent_back ? q.d_sum : dF, H, s.y2, s.mean2, s.rstd2, q.d_y2, H, M, H, g.p[MREM_LN2_B], g.p[MREM_LN2_G],
                      g.p[MREM_B2], c->col_scratch, c->col_plane, c->col_counters, c->dt, side);
    r.gemm(view(q.d_y2, H), weights(w[W_2].what, F, 1), (int)M, F, H, 1, 1, Epi(c->d_ghat, ok, F).e);
    {
      Epi e(g.p[MREM_W2], OUT_F32, F);
      e.alpha(1.f, b.a_steps[S_G]);
      if (rg.asym) { launch_scale_vec(g.p[MREM_B2], b.a_off[S_G], q.rowbias, H, side); e.rowbias(q.rowbias); }
      rw.defer(view(q.d_y2, H, 1), view(s.g_qt, F, 1), H, F, (int)M, e.e);
    }
    // (the bias gradient of FFN1, the column sums of d_u, rides along where the vector path applies)
    const bool b1_done = launch_gelu_bwd_colsum(s.u, c->d_ghat, q.d_u, M, F, b.a_steps[S_G], rg.asym ? b.a_off[S_G] : nullptr, rg.lo, rg.hi, 1,
                                                part + S_G * RED_BLOCKS, part + N_SITES * RED_BLOCKS, g.p[MREM_B1], c->gb_scratch,
                                                c->gb_floats, c->gb_counters, c->gb_n_counters, c->dt, st);
    if (!b1_done)
      launch_gelu_bwd(s.u, c->d_ghat, q.d_u, M * F, b.a_steps[S_G], rg.asym ? b.a_off[S_G] : nullptr, rg.lo, rg.hi, 1,
                      part + S_G * RED_BLOCKS, part + N_SITES * RED_BLOCKS, c->dt, st);
    // FFN1:  u = A_hat W1_hat^T + b1
    fork();
    if (!b1_done)
      launch_col_reduce(q.d_u, F, nullptr, nullptr, nullptr, nullptr, 0, M, F, g.p[MREM_B1], nullptr, nullptr, c->col_scratch, c->col_plane, c->col_counters, c->dt, side);
    r.gemm(view(q.d_u, F), weights(w[W_1].what, H, 1), (int)M, H, F, 1, 1, Epi(c->d_ahat, ok, H).e);
    rw.defer(view(q.d_u, F, 1), view(s.a_qt, H, 1), F, H, (int)M, Epi(g.p[MREM_W1], OUT_F32, H).alpha(1.f, b.a_steps[S_A]).e);
    // straight-through pass of the FFN1 input quantizer + skip connection -> d_a, and the first LayerNorm's backward
    if (!(fuse_ln && launch_layernorm_bwd_ste(nullptr, s.a, c->d_ahat, q.d_y2, b.a_steps[S_A], rx.lo, rx.hi, s.y1, s.mean1, s.rstd1,
                                              b.student[MREM_LN1_G], M, H, q.d_y1, q.d_a, part + S_A * RED_BLOCKS, c->dt, st))) {
      launch_ste_act(s.a, H, c->d_ahat, H, q.d_y2, H, q.d_a, H, M, H, b.a_steps[S_A], nullptr, rx.lo, rx.hi,
                     part + S_A * RED_BLOCKS, nullptr, c->dt, st);
      launch_layernorm_bwd(q.d_a, nullptr, s.y1, s.mean1, s.rstd1, b.student[MREM_LN1_G], M, H, q.d_y1, nullptr, c->dt, st);
    }
    // attention output projection:  y1 = ctx_hat Wo_hat^T + bo + x  (its bias gradient rides along)
    fork();
    launch_col_reduce(q.d_a, H, s.y1, s.mean1, s.rstd1, q.d_y1, H, M, H, g.p[MREM_LN1_B], g.p[MREM_LN1_G], g.p[MREM_BO],
                      c->col_scratch, c->col_plane, c->col_counters, c->dt, side);
    r.gemm(view(q.d_y1, H), weights(w[W_O].what, H, 1), (int)M, H, H, 1, 1, Epi(c->d_ctxhat, ok, H).e);
    rw.defer(view(q.d_y1, H, 1), view(s.ctx_qt, H, 1), H, H, (int)M, Epi(g.p[MREM_WO], OUT_F32, H).alpha(1.f, b.a_steps[S_C]).e);
    launch_ste_act(s.ctx, H, c->d_ctxhat, H, nullptr, 0, c->d_ctx, H, M, H, b.a_steps[S_C], nullptr, rx.lo, rx.hi,
                   part + S_C * RED_BLOCKS, nullptr, c->dt, st);
    // attention:  ctx = P_hat V_hat,  P = softmax(Q_hat K_hat^T / sqrt(d))
    if (c->fused_attention_bwd && attention_bwd_supported(S, hd, c->dt, B * h)) {
      r.note(launch_attention_bwd(s.qkv_qt, s.qkv, s.P, c->d_ctx, B, S, h, H, b.a_steps[S_Q], b.a_steps[S_K], b.a_steps[S_V],
                                  b.a_steps[S_P], rx.lo, rx.hi, rp.lo, rp.hi, q.d_qkv, part + S_Q * RED_BLOCKS,
                                  part + S_K * RED_BLOCKS, part + S_V * RED_BLOCKS, part + S_P * RED_BLOCKS, c->status, st),
             "attention backward launch failed");
    } else {
      r.gemm(view(c->d_ctx, H, 0, hd, (long long)S * H), view(r.at(s.qkv_qt, 2 * H), 3 * H, 0, hd, sQKV), S, S, hd, h, B,
             Epi(c->d_phat, ok, S, sSS, sHSS).alpha(1.f, b.a_steps[S_V]).e);
      r.gemm(view(s.P_qt, S, 1, sSS, sHSS), view(c->d_ctx, H, 1, hd, (long long)S * H), S, hd, S, h, B,
             Epi(r.at(c->d_qkvhat, 2 * H), ok, 3 * H, hd, sQKV).alpha(1.f, b.a_steps[S_P]).e);
      launch_softmax_bwd(s.P, c->d_phat, c->d_s, (long long)B * h * S, S, b.a_steps[S_P], rp.lo, rp.hi, 1, part + S_P * RED_BLOCKS, c->dt, st);
      r.gemm(view(c->d_s, S, 0, sSS, sHSS), view(r.at(s.qkv_qt, H), 3 * H, 1, hd, sQKV), S, hd, S, h, B,
             Epi(c->d_qkvhat, ok, 3 * H, hd, sQKV).alpha(inv_sqrt_d, b.a_steps[S_K]).e);
      r.gemm(view(c->d_s, S, 1, sSS, sHSS), view(s.qkv_qt, 3 * H, 1, hd, sQKV), S, hd, S, h, B,
             Epi(r.at(c->d_qkvhat, H), ok, 3 * H, hd, sQKV).alpha(inv_sqrt_d, b.a_steps[S_Q]).e);
      for (int seg = 0; seg < 3; ++seg)
        launch_ste_act(r.at(s.qkv, seg * H), 3 * H, r.at(c->d_qkvhat, seg * H), 3 * H, nullptr, 0, r.at(q.d_qkv, seg * H), 3 * H, M, H,
                       b.a_steps[S_Q + seg], nullptr, rx.lo, rx.hi, part + (S_Q + seg) * RED_BLOCKS, nullptr, c->dt, st);
    }
    // QKV projection:  qkv = X_hat Wqkv_hat^T + bqkv
    fork();
    launch_col_reduce(q.d_qkv, 3 * H, nullptr, nullptr, nullptr, nullptr, 0, M, 3 * H, g.p[MREM_BQKV], nullptr, nullptr, c->col_scratch, c->col_plane, c->col_counters, c->dt, side);
    r.gemm(view(q.d_qkv, 3 * H), weights(w[W_QKV].what, H, 1), (int)M, H, 3 * H, 1, 1, Epi(c->d_xhat, ok, H).e);
    rw.defer(view(q.d_qkv, 3 * H, 1), view(s.x_qt, H, 1), 3 * H, H, (int)M, Epi(g.p[MREM_WQKV], OUT_F32, H).alpha(1.f, b.a_steps[S_X]).e);
    rw.flush_deferred();                              // the layer's four weight-gradient products, one launch
    if (fuse_ln && l > 0) {
      // left to the LayerNorm backward of the layer below, which reads d_xhat and d_y1 before anything overwrites them
      pending.x = x_in; pending.add = q.d_y1; pending.step = b.a_steps[S_X]; pending.part = part + S_X * RED_BLOCKS;
      carry = nullptr;
    } else {
      void* next_carry = c->carry[l & 1];
      launch_ste_act(x_in, H, c->d_xhat, H, q.d_y1, H, next_carry, H, M, H, b.a_steps[S_X], nullptr, rx.lo, rx.hi,
                     part + S_X * RED_BLOCKS, nullptr, c->dt, st);
      carry = next_carry;
    }
    // (the weight quantizers' masks and step gradients are applied inside the fused update of mrem_step,
    //  or on demand by mrem_get_grad)
    // the side stream is done with this layer's copy of the gradient buffers once the grouped products have run
    if (two_streams && cudaEventRecord(c->ev_layer[l & 1], side) != cudaSuccess) sync_failed = true;
    // nothing below reads what the update writes: the latent weights, moments, row steps and this layer's codes
    if (update_as_you_go) enqueue_matrix_updates(c, l, side);
  }
  // step-size and offset gradients of every layer's activation quantizers: the per-block partial sums the
  // kernels above left, added in index order (one launch for the whole module; only the update reads them)
  launch_reduce_table(c->reduce_table, c->reduce_per_layer * d.n_layers, c->stream);
  join();
  c->have_input_grad = true;           // layer 0's straight-through pass wrote it to carry[0]
  if (sync_failed) return fail(c, MREM_ERR_CUDA, "backward: stream fork/join failed");
  if (rw.rc != MREM_OK) { c->err = "weight-gradient GEMM launch failed"; return rw.rc; }
  if (r.rc != MREM_OK) return r.rc;
  return cudaGetLastError() == cudaSuccess ? MREM_OK : fail(c, MREM_ERR_CUDA, "backward: launch failed");
}

}  // namespace

extern "C" {

int32_t mrem_quantize_weights(mrem_ctx* c) {
  if (!c) return MREM_ERR_ARG;
  TracerGuard tg(c->trace_on ? &c->tracer : nullptr);
  if (c->codes_fresh) { c->weights_quantized = true; return MREM_OK; }   // the last update already re-quantized
  for (int l = 0; l < c->d.n_layers; ++l)
    for (int k = 0; k < N_WMAT; ++k) {
      const LayerBind& b = c->bind[l];
      if (!b.student[kMatParam[k]] || (!b.w_steps[k] && !closed_form_weights(c->d))) return fail(c, MREM_ERR_ORDER, "quantize_weights: weights or steps not bound");
      WeightBuf& w = c->wq[l][k];
      if (closed_form_weights(c->d)) {
        launch_closed_form_quantize(b.student[kMatParam[k]], w.rows, w.cols, c->d.w_grid, c->d.w_bits, w.codes, w.rowsum,
                                    w.scale, w.what, c->dt, c->stream);
        continue;
      }
      launch_quantize_weight(b.student[kMatParam[k]], w.rows, w.cols, b.w_steps[k], c->d.w_step_per_row, c->d.w_bits,
                             c->d.w_grid, w.codes, w.rowsum, w.scale, w.what, c->dt, c->stream);
    }
  if (cudaGetLastError() != cudaSuccess) return fail(c, MREM_ERR_CUDA, "quantize_weights: launch failed");
  c->weights_quantized = true;
  c->codes_fresh = true;
  return MREM_OK;
}

int32_t mrem_module_forward(mrem_ctx* c, int32_t role, const void* x, const void* x_other, float lambda,
                            const int32_t* len, int32_t batch, int32_t seq, void* outs) {
  if (!c) return MREM_ERR_ARG;
  TracerGuard tg(c->trace_on ? &c->tracer : nullptr);
  int rc = check_io(c, x, batch, seq, outs);
  if (rc != MREM_OK) return rc;
  if (c->have_teacher || c->have_student) {
    if (batch != c->cur_batch || seq != c->cur_seq) { c->have_teacher = c->have_student = false; }
  }
  mrem::g_plain_next_launch = 1;          // the pass's first kernel is a full barrier towards everything before it
  if (role == MREM_TEACHER) {
    rc = float_forward(c, x, len, batch, seq, outs, false, false);
    if (rc != MREM_OK) return rc;
    c->t_out = outs; c->have_teacher = true;
  } else if (role == MREM_STUDENT) {
    if (!c->weights_quantized) return fail(c, MREM_ERR_ORDER, "forward(student): call mrem_quantize_weights first");
    const void* in = x;
    if (lambda != 0.f) {
      if (!x_other) return fail(c, MREM_ERR_ARG, "forward(student): lambda != 0 needs d_x_other");
      if (!(lambda >= 0.f && lambda <= 1.f)) return fail(c, MREM_ERR_ARG, "forward(student): lambda outside [0, 1]");
      launch_mix(x_other, x, lambda, c->x_mix, (long long)batch * seq * c->d.hidden, c->dt, c->stream);
      in = c->x_mix;
    }
    rc = student_forward(c, in, len, batch, seq, outs);
    if (rc != MREM_OK) return rc;
    c->s_in = in; c->s_out = outs; c->have_student = true;
  } else {
    return fail(c, MREM_ERR_ARG, "forward: role");
  }
  c->cur_batch = batch; c->cur_seq = seq; c->cur_len = len;
  c->have_loss = false; c->have_grads = false; c->have_input_grad = false;
  return MREM_OK;
}

int32_t mrem_recon_loss(mrem_ctx* c, float* loss_total, float* loss_per_layer) {
  if (!c || !loss_total) return MREM_ERR_ARG;
  TracerGuard tg(c->trace_on ? &c->tracer : nullptr);
  if (!c->have_teacher || !c->have_student) return fail(c, MREM_ERR_ORDER, "recon_loss: needs a teacher and a student forward of the same batch");
  const long long n = (long long)c->cur_batch * c->cur_seq * c->d.hidden;
  const float cc = (c->d.loss_mean ? 1.f / (float)n : 1.f) * c->loss_share;
  launch_loss(c->s_out, c->t_out, c->d.n_layers, n, cc, c->dF, c->loss_partial, c->status, c->dt, c->stream);
  launch_loss_finalize(c->loss_partial, c->d.n_layers, cc, loss_total, loss_per_layer, c->stream);
  if (c->head.wp) {
    // last module of the model: the output-logit term, its gradient added to the last layer's loss gradient
    const int L = c->d.n_layers, C = c->head.n_classes;
    const float cz = (c->d.loss_mean ? 1.f / (float)((long long)c->cur_batch * C) : 1.f) * c->loss_share;
    const long long last = (long long)(L - 1) * n;
    const int hrc = launch_head_logit_loss((const char*)c->s_out + last * c->esz, (const char*)c->t_out + last * c->esz, c->cur_batch,
                                           c->cur_seq, c->d.hidden, C, c->head.wp, c->head.bp, c->head.wc, c->head.bc, cz,
                                           (char*)c->dF + last * c->esz, c->head_scratch, c->head.logits, loss_total,
                                           c->head.logit_loss, c->dt, c->stream);
    if (hrc == -1) return fail(c, MREM_ERR_SHAPE, "recon_loss: hidden size / class count too large for the logit term");
    if (hrc != 0) return fail(c, MREM_ERR_CUDA, "recon_loss: launch failed");
  }
  if (cudaGetLastError() != cudaSuccess) return fail(c, MREM_ERR_CUDA, "recon_loss: launch failed");
  c->have_loss = true;
  return MREM_OK;
}

int32_t mrem_module_backward(mrem_ctx* c) {
  if (!c) return MREM_ERR_ARG;
  TracerGuard tg(c->trace_on ? &c->tracer : nullptr);
  if (!c->have_student || !c->have_loss) return fail(c, MREM_ERR_ORDER, "backward: needs forward(student) and recon_loss of this step");
  for (int l = 0; l < c->d.n_layers; ++l)
    for (int k = 0; k < N_WMAT; ++k) if (!c->bind[l].w_steps[k] && !closed_form_weights(c->d)) return fail(c, MREM_ERR_ORDER, "backward: weight steps not bound");
  if (c->tables_dirty) { const int rc = build_tables(c); if (rc != MREM_OK) return rc; }
  const int rc = student_backward(c, false);
  if (rc != MREM_OK) return rc;
  c->have_grads = true;
  c->w_ste_done = false;
  return MREM_OK;
}

// mrem_module_backward followed by mrem_step, with the matrix updates overlapped with the backward pass
// (same kernels on the same data: the results are bitwise those of the two separate calls).
int32_t mrem_backward_and_step(mrem_ctx* c, const mrem_optim* o) {
  if (!c || !o) return MREM_ERR_ARG;
  if (!c->d.w_step_per_row) {
    const int rc = mrem_module_backward(c);
    return rc != MREM_OK ? rc : mrem_step(c, o);
  }
  TracerGuard tg(c->trace_on ? &c->tracer : nullptr);
  if (!c->have_student || !c->have_loss) return fail(c, MREM_ERR_ORDER, "backward: needs forward(student) and recon_loss of this step");
  for (int l = 0; l < c->d.n_layers; ++l)
    for (int k = 0; k < N_WMAT; ++k) if (!c->bind[l].w_steps[k] && !closed_form_weights(c->d)) return fail(c, MREM_ERR_ORDER, "backward: weight steps not bound");
  if (c->tables_dirty) { const int rc = build_tables(c); if (rc != MREM_OK) return rc; }
  launch_optim_prepare(c->optim_sc, c->t_counter, o->step, o->lr, o->decay_total_steps, o->beta1, o->beta2, o->eps,
                       o->weight_decay, c->stream);
  c->w_ste_done = false;
  const int rc = student_backward(c, true);
  if (rc != MREM_OK) return rc;
  launch_adamw_table(c->adam_rest, c->rest_entries, c->rest_elems, c->optim_sc, c->stream);
  if (cudaGetLastError() != cudaSuccess) return fail(c, MREM_ERR_CUDA, "step: launch failed");
  c->have_grads = false; c->have_loss = false; c->have_student = false; c->have_teacher = false;
  c->codes_fresh = true;
  c->weights_quantized = true;
  return MREM_OK;
}

int32_t mrem_step(mrem_ctx* c, const mrem_optim* o) {
  if (!c || !o) return MREM_ERR_ARG;
  TracerGuard tg(c->trace_on ? &c->tracer : nullptr);
  if (!c->have_grads) return fail(c, MREM_ERR_ORDER, "step: needs mrem_module_backward of this step");
  if (c->tables_dirty) { const int rc = build_tables(c); if (rc != MREM_OK) return rc; }
  launch_optim_prepare(c->optim_sc, c->t_counter, o->step, o->lr, o->decay_total_steps, o->beta1, o->beta2, o->eps,
                       o->weight_decay, c->stream);
  const mrem_module_desc& d = c->d;
  if (d.w_step_per_row) {
    // every tensor but the matrices and their steps, then one fused pass per matrix
    launch_adamw_table(c->adam_rest, c->rest_entries, c->rest_elems, c->optim_sc, c->stream);
    for (int l = 0; l < d.n_layers; ++l) enqueue_matrix_updates(c, l, c->stream);
  } else {
    if (!c->w_ste_done) {
      for (int l = 0; l < d.n_layers; ++l)
        for (int k = 0; k < N_WMAT; ++k) {
          WeightBuf& w = c->wq[l][k];
          launch_ste_weight(c->bind[l].student[kMatParam[k]], c->bind[l].w_steps[k], 0, d.w_bits, d.w_grid,
                            c->grad[l].p[kMatParam[k]], w.rows, w.cols, w.ds_rows, c->stream);
          launch_reduce_table(c->reduce_table + (size_t)l * c->reduce_per_layer + N_SITES + 1 + k, 1, c->stream);
        }
    }
    launch_adamw_table(c->adam_table, c->adam_entries, c->adam_elems, c->optim_sc, c->stream);
  }
  if (cudaGetLastError() != cudaSuccess) return fail(c, MREM_ERR_CUDA, "step: launch failed");
  c->have_grads = false; c->have_loss = false; c->have_student = false; c->have_teacher = false;
  c->codes_fresh = d.w_step_per_row != 0;
  c->weights_quantized = c->codes_fresh;
  return MREM_OK;
}


// Eq. 2: one optimisation step on the reconstruction error of ONE matrix product of one layer,
//   min_{w, s} || Q(w)^T Q(a) - w^T a ||^2  over the rows of a,
// with the same kernels as the module step: the full-precision product on the bf16 (or fp32) path, the
// quantized one on integer codes, the loss kernel of Eq. 3 on the pair, the straight-through backward of
// the two quantizers, the fused update of the matrix and AdamW on the input quantizer's step (and offset).
int32_t mrem_rem_step(mrem_ctx* c, int32_t layer, int32_t tensor_id, const void* a, int32_t rows, const mrem_optim* o,
                      float* d_loss) {
  if (!c || !a || !d_loss) return MREM_ERR_ARG;
  TracerGuard tg(c->trace_on ? &c->tracer : nullptr);
  const mrem_module_desc& d = c->d;
  if (layer < 0 || layer >= d.n_layers) return fail(c, MREM_ERR_ARG, "rem_step: layer");
  int k = -1;
  for (int i = 0; i < N_WMAT; ++i) if (kMatParam[i] == tensor_id) k = i;
  if (k < 0) return fail(c, MREM_ERR_ARG, "rem_step: tensor_id must name one of the four weight matrices");
  if (rows < 1 || rows > c->max_tokens) return fail(c, MREM_ERR_SHAPE, "rem_step: rows outside the context's maximum (max_batch * max_seq)");
  if (reinterpret_cast<uintptr_t>(a) & 15) return fail(c, MREM_ERR_ALIGN, "rem_step: d_a must be 16-byte aligned");
  if (!d.w_step_per_row && !closed_form_weights(d)) return fail(c, MREM_ERR_UNSUPPORTED, "rem_step: needs per-row weight steps or closed-form weight scales");
  const int site = k == W_QKV ? S_X : (k == W_O ? S_C : (k == W_1 ? S_A : S_G));
  const LayerBind& b = c->bind[layer];
  if (!b.teacher[tensor_id] || !b.student[tensor_id] || (!b.w_steps[k] && !closed_form_weights(d)) || !b.a_steps[site])
    return fail(c, MREM_ERR_ORDER, "rem_step: parameters or steps not bound");
  const ActRange ar = site_range(d, site);
  if (ar.asym && !b.a_off[site]) return fail(c, MREM_ERR_ORDER, "rem_step: offset of the GELU-site quantizer not bound");
  if (c->tables_dirty) { const int rc = build_tables(c); if (rc != MREM_OK) return rc; }
  int rc = mrem_quantize_weights(c);
  if (rc != MREM_OK) return rc;

  LayerStash& s = c->stash[layer];
  LayerGrad& g = c->grad[layer];
  WeightBuf& w = c->wq[layer][k];
  const int N = w.rows, K = w.cols, F = d.ffn;
  const long long M = rows;
  cudaStream_t st = c->stream;
  Runner r(c);
  const int ok = r.okind();
  // scratch of the module step, by width: codes of the input, the two products, the loss gradient, d a_hat
  int8_t* q8 = K == F ? s.g_q8 : s.x_q8;
  void* qt = K == F ? s.g_qt : s.x_qt;
  void* target = N == F ? c->t_g : c->t_qkv;
  void* y = N == F ? s.u : s.qkv;
  void* dy = N == F ? c->d_u : c->d_qkv;
  void* dxhat = K == F ? c->d_ghat : c->d_ahat;
  const float* step = b.a_steps[site];
  const float* off = ar.asym ? b.a_off[site] : nullptr;
  const int bias_id = tensor_id + 1;                     // the bias follows its matrix in the parameter list

  // w^T a  (launched as a full barrier: the codes the quantizer above may just have written are complete for all that follows)
  mrem::g_plain_next_launch = 1;
  r.gemm(view(a, K), view(b.teacher[tensor_id], K), (int)M, N, K, 1, 1, Epi(target, ok, N).e);
  // Q(w)^T Q(a): integer codes, exact accumulation, dequantized in the epilogue (offset term as a column bias)
  launch_quantize_act(a, c->dt, M, K, K, step, off, ar.lo, ar.hi, q8, K, qt, K, st);
  Epi fe(y, ok, N);
  fe.alpha(1.f, step).colscale(w.scale);
  if (ar.asym) {
    if (cudaMemsetAsync(c->alt_rowbias, 0, sizeof(float) * N, st) != cudaSuccess) return fail(c, MREM_ERR_CUDA, "rem_step: memset failed");
    launch_effective_bias(c->alt_rowbias, off, w.scale, w.rowsum, w.beff, N, st);
    fe.colbias(w.beff);
  }
  r.gemm_i8(q8, ar.asym ? 1 : 0, w.codes, (int)M, N, K, fe.e);
  // loss and its gradient
  const long long n = M * N;
  const float cc = d.loss_mean ? 1.f / (float)n : 1.f;
  launch_loss(y, target, 1, n, cc, dy, c->loss_partial, c->status, c->dt, st);
  launch_loss_finalize(c->loss_partial, 1, cc, d_loss, nullptr, st);
  // d l / d w_hat = dy^T a_hat, a_hat = step * codes (+ offset: a row bias of offset * column sums of dy)
  Epi we(g.p[tensor_id], OUT_F32, K);
  we.alpha(1.f, step);
  if (ar.asym) {
    launch_col_reduce(dy, N, nullptr, nullptr, nullptr, nullptr, 0, M, N, g.p[bias_id], nullptr, nullptr, c->col_scratch, c->col_plane,
                      c->col_counters, c->dt, st);
    launch_scale_vec(g.p[bias_id], off, c->rowbias, N, st);
    we.rowbias(c->rowbias);
  }
  r.gemm(view(dy, N, 1), view(qt, K, 1), N, K, (int)M, 1, 1, we.e);
  // d l / d a_hat = dy w_hat, then the straight-through factors of the input quantizer
  r.gemm(view(dy, N), view(w.what, K, 1), (int)M, K, N, 1, 1, Epi(dxhat, ok, K).e);
  launch_ste_act(a, K, dxhat, K, nullptr, 0, dxhat, K, M, K, step, off, ar.lo, ar.hi, s.part + site * RED_BLOCKS,
                 ar.asym ? s.part + N_SITES * RED_BLOCKS : nullptr, c->dt, st);
  const ReduceEntry* red = c->reduce_table + (size_t)layer * c->reduce_per_layer;
  launch_reduce_table(red + site, 1, st);
  if (ar.asym) launch_reduce_table(red + N_SITES, 1, st);
  c->w_ste_done = false;
  if (o) {
    // update: the matrix and its steps (which also re-quantizes it), the input quantizer's step and offset
    launch_optim_prepare(c->optim_sc, c->t_counter, o->step, o->lr, o->decay_total_steps, o->beta1, o->beta2, o->eps,
                         o->weight_decay, st);
    enqueue_matrix_update(c, layer, k, st);
    if (d.trainable_mask & MREM_TRAIN_A_STEPS) {
      AdamEntry host[2];
      int ne = 0;
      host[ne++] = AdamEntry{b.a_steps[site], g.a + site, g.m_a + site, g.v_a + site, 1, 0.f, 1e-8f};
      if (ar.asym) host[ne++] = AdamEntry{b.a_off[site], g.off + site, g.m_off + site, g.v_off + site, 1, 0.f, -INFINITY};
      if (cudaMemcpyAsync(c->rem_table, host, sizeof(AdamEntry) * ne, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return fail(c, MREM_ERR_CUDA, "rem_step: table upload failed");
      launch_adamw_table(c->rem_table, ne, ne, c->optim_sc, st);
    }
  }
  if (r.rc != MREM_OK) return r.rc;
  if (cudaGetLastError() != cudaSuccess) return fail(c, MREM_ERR_CUDA, "rem_step: launch failed");
  c->have_grads = o == nullptr;        // without an update the gradients stay readable (mrem_get_grad)
  c->have_loss = false; c->have_student = false; c->have_teacher = false;
  c->codes_fresh = true;
  c->weights_quantized = true;
  return MREM_OK;
}

}  // extern "C"
