// C-ABI of libmrem: context, workspace layout, parameter binding, initialisation, state.
// The step itself (forward, loss, backward, update) lives in mrem_step.cu.
#include <cstring>

#include "mrem_ctx.h"

using namespace mrem;

namespace mrem {
thread_local Tracer* g_tracer = nullptr;
int g_programmatic_launch = 1;
thread_local int g_plain_next_launch = 0;
unsigned long long g_wait_limit_ns = 2000000000ull;   // 2 s
}

namespace {
thread_local std::string g_create_err;   // mrem_last_error(NULL): the calling thread's last create / workspace-size error

const int kParamIsMatrix[MREM_N_PARAMS] = {1, 0, 1, 0, 0, 0, 1, 0, 1, 0, 0, 0};
const int kMatParam[N_WMAT] = {MREM_WQKV, MREM_WO, MREM_W1, MREM_W2};
const int kBiasOfMat[N_WMAT] = {MREM_BQKV, MREM_BO, MREM_B1, MREM_B2};
}  // namespace

namespace mrem {

void param_shape(const mrem_module_desc& d, int id, int* rows, int* cols) {
  const int H = d.hidden, F = d.ffn;
  switch (id) {
    case MREM_WQKV: *rows = 3 * H; *cols = H; break;
    case MREM_BQKV: *rows = 1; *cols = 3 * H; break;
    case MREM_WO: *rows = H; *cols = H; break;
    case MREM_W1: *rows = F; *cols = H; break;
    case MREM_B1: *rows = 1; *cols = F; break;
    case MREM_W2: *rows = H; *cols = F; break;
    default: *rows = 1; *cols = H; break;       // bo, b2, LayerNorm vectors
  }
}

int fail(mrem_ctx* c, int code, const char* msg) {
  if (c) c->err = msg; else g_create_err = msg;
  return code;
}

static int validate(const mrem_module_desc* d, std::string* why) {
  if (!d || d->struct_size != sizeof(mrem_module_desc)) { *why = "desc is NULL or struct_size mismatch"; return MREM_ERR_ARG; }
  if (d->n_layers < 1 || d->hidden < 16 || d->n_heads < 1 || d->ffn < 16 || d->max_seq < 1 || d->max_batch < 1) {
    *why = "non-positive dimension"; return MREM_ERR_ARG; }
  if (d->hidden % d->n_heads) { *why = "hidden not divisible by n_heads"; return MREM_ERR_SHAPE; }
  if (d->hidden % 16 || d->ffn % 16) { *why = "hidden and ffn must be multiples of 16"; return MREM_ERR_SHAPE; }
  if (d->act_dtype != MREM_F32 && d->act_dtype != MREM_BF16) { *why = "act_dtype"; return MREM_ERR_ARG; }
  const int hd = d->hidden / d->n_heads;
  if (d->act_dtype == MREM_BF16 && (hd % 64 || d->max_seq % 8)) {
    *why = "bf16 path needs head size multiple of 64 and seq multiple of 8"; return MREM_ERR_SHAPE; }
  if (d->w_bits != 2 && d->w_bits != 4 && d->w_bits != 8) { *why = "w_bits must be 2, 4 or 8"; return MREM_ERR_UNSUPPORTED; }
  if (d->a_bits != 8 && d->a_bits != 4) { *why = "a_bits must be 8 or 4"; return MREM_ERR_UNSUPPORTED; }
  if (d->w_grid < 0 || d->w_grid > 3) { *why = "w_grid must be 0, 1, 2 or 3"; return MREM_ERR_UNSUPPORTED; }
  if ((d->w_grid == 1 || d->w_grid == 2) && d->w_bits != 2) { *why = "w_grid 1 and 2 need w_bits 2"; return MREM_ERR_UNSUPPORTED; }
  if (closed_form_weights(*d) && !d->w_step_per_row) { *why = "w_grid 2 and 3 (closed-form weight scales) work per output row"; return MREM_ERR_UNSUPPORTED; }
  if ((long long)d->max_batch * d->n_heads > 65535) { *why = "batch * heads too large"; return MREM_ERR_SHAPE; }
  return MREM_OK;
}

// Lays the workspace out; with a null base only the size is computed.
static void layout(mrem_ctx* c, char* base, size_t* total) {
  const mrem_module_desc& d = c->d;
  Arena A; A.base = base;
  const size_t es = c->esz;
  const long long M = c->max_tokens, H = d.hidden, F = d.ffn;
  const long long PS = (long long)d.max_batch * d.n_heads * d.max_seq * d.max_seq;
  const int L = d.n_layers;

  c->status = (int*)A.take(256);
  c->t_counter = (int*)A.take(256);
  c->optim_sc = (OptimScalars*)A.take(256);
  c->minmax = (float*)A.take(256);
  c->d_loss_e2e = (float*)A.take(256);
  c->loss_partial = (float*)A.take(sizeof(float) * RED_BLOCKS * L);
  c->head_scratch = (float*)A.take(sizeof(float) * head_scratch_floats(d.max_batch, H));
  c->col_plane = (long long)COL_CHUNKS * (3 * H > F ? 3 * H : F);
  c->col_scratch = (float*)A.take(sizeof(float) * 3 * c->col_plane);
  c->col_counters = (int*)A.take(sizeof(int) * ((3 * H > F ? 3 * H : F) / 32 + 2));
  c->gb_floats = (long long)(RED_BLOCKS / ((F + 127) / 128) + 1) * F;     // one row of partials per chunk of the GELU backward's grid
  c->gb_scratch = (float*)A.take(sizeof(float) * c->gb_floats);
  c->gb_n_counters = F / 32 + 2;
  c->gb_counters = (int*)A.take(sizeof(int) * c->gb_n_counters);
  c->rowbias = (float*)A.take(sizeof(float) * (3 * H > F ? 3 * H : F));
  c->alt_rowbias = (float*)A.take(sizeof(float) * (3 * H > F ? 3 * H : F));
  c->reduce_per_layer = N_SITES + 1 + N_WMAT;
  c->reduce_table = (ReduceEntry*)A.take(sizeof(ReduceEntry) * c->reduce_per_layer * L);
  c->adam_table = (AdamEntry*)A.take(sizeof(AdamEntry) * (MREM_N_PARAMS + N_WMAT + N_SITES + 1) * L);
  c->adam_rest = (AdamEntry*)A.take(sizeof(AdamEntry) * (MREM_N_PARAMS + N_WMAT + N_SITES + 1) * L);
  c->rem_table = (AdamEntry*)A.take(sizeof(AdamEntry) * 2);
  c->h2d_xt = A.take(M * H * es);
  c->h2d_xs = A.take(M * H * es);
  c->h2d_len = (int32_t*)A.take(sizeof(int32_t) * d.max_batch);
  for (int k = 0; k < 2; ++k) {
    c->stage_x[k][0] = A.take(M * H * es);
    c->stage_x[k][1] = A.take(M * H * es);
    c->stage_len[k] = (int32_t*)A.take(sizeof(int32_t) * d.max_batch);
  }
  c->e2e_t_out = A.take((size_t)L * M * H * es);
  c->e2e_s_out = A.take((size_t)L * M * H * es);

  c->t_qkv = A.take(M * 3 * H * es); c->t_P = A.take(PS * es); c->t_ctx = A.take(M * H * es);
  c->t_y1 = A.take(M * H * es); c->t_a = A.take(M * H * es); c->t_g = A.take(M * F * es);
  c->t_y2 = A.take(M * H * es);
  c->scores = (float*)A.take(PS * sizeof(float));
  c->x_mix = A.take(M * H * es);
  c->dF = A.take((size_t)L * M * H * es);
  c->d_y2 = A.take(M * H * es); c->d_ghat = A.take(M * F * es); c->d_u = A.take(M * F * es);
  c->d_ahat = A.take(M * H * es); c->d_a = A.take(M * H * es); c->d_y1 = A.take(M * H * es);
  c->d_ctxhat = A.take(M * H * es); c->d_ctx = A.take(M * H * es);
  c->d_phat = A.take(PS * es); c->d_s = A.take(PS * es);
  c->d_qkvhat = A.take(M * 3 * H * es); c->d_qkv = A.take(M * 3 * H * es);
  c->d_xhat = A.take(M * H * es); c->d_sum = A.take(M * H * es);
  c->carry[0] = A.take(M * H * es); c->carry[1] = A.take(M * H * es);
  c->alt_d_y2 = A.take(M * H * es); c->alt_d_sum = A.take(M * H * es); c->alt_d_u = A.take(M * F * es);
  c->alt_d_a = A.take(M * H * es); c->alt_d_y1 = A.take(M * H * es); c->alt_d_qkv = A.take(M * 3 * H * es);

  c->stash.resize(L); c->wq.assign(L, std::vector<WeightBuf>(N_WMAT)); c->grad.resize(L);
  for (int l = 0; l < L; ++l) {
    LayerStash& s = c->stash[l];
    s.x_q8 = (int8_t*)A.take(M * H); s.x_qt = A.take(M * H * es);
    s.qkv = A.take(M * 3 * H * es); s.qkv_qt = A.take(M * 3 * H * es);
    s.P = A.take(PS * es); s.P_qt = A.take(PS * es);
    s.ctx = A.take(M * H * es); s.ctx_q8 = (int8_t*)A.take(M * H); s.ctx_qt = A.take(M * H * es);
    s.y1 = A.take(M * H * es); s.mean1 = (float*)A.take(M * 4); s.rstd1 = (float*)A.take(M * 4);
    s.a = A.take(M * H * es); s.a_q8 = (int8_t*)A.take(M * H); s.a_qt = A.take(M * H * es);
    s.u = A.take(M * F * es); s.g_q8 = (int8_t*)A.take(M * F); s.g_qt = A.take(M * F * es);
    s.y2 = A.take(M * H * es); s.mean2 = (float*)A.take(M * 4); s.rstd2 = (float*)A.take(M * 4);
    s.part = (float*)A.take(sizeof(float) * (N_SITES + 1) * RED_BLOCKS);
    for (int k = 0; k < N_WMAT; ++k) {
      WeightBuf& w = c->wq[l][k];
      param_shape(d, kMatParam[k], &w.rows, &w.cols);
      const size_t n = (size_t)w.rows * w.cols;
      w.codes = (int8_t*)A.take(n); w.rowsum = (int32_t*)A.take(4 * w.rows); w.scale = (float*)A.take(4 * w.rows);
      w.what = A.take(n * es); w.beff = (float*)A.take(4 * w.rows); w.ds_rows = (float*)A.take(4 * w.rows);
    }
    LayerGrad& g = c->grad[l];
    for (int k = 0; k < MREM_N_PARAMS; ++k) {
      int r, q; param_shape(d, k, &r, &q);
      g.p[k] = (float*)A.take(sizeof(float) * r * q);
    }
    for (int k = 0; k < N_WMAT; ++k) g.ws[k] = (float*)A.take(sizeof(float) * (d.w_step_per_row ? c->wq[l][k].rows : 1));
    g.a = (float*)A.take(sizeof(float) * N_SITES);
    g.off = (float*)A.take(sizeof(float) * N_SITES);
  }
  // optimizer moments: one contiguous range so that export/import is a single copy
  A.take(0);
  c->state_off = (A.off + 255) & ~size_t(255);
  for (int l = 0; l < L; ++l) {
    LayerGrad& g = c->grad[l];
    for (int k = 0; k < MREM_N_PARAMS; ++k) {
      int r, q; param_shape(d, k, &r, &q);
      g.m_p[k] = (float*)A.take(sizeof(float) * r * q); g.v_p[k] = (float*)A.take(sizeof(float) * r * q);
    }
    for (int k = 0; k < N_WMAT; ++k) {
      const size_t n = d.w_step_per_row ? c->wq[l][k].rows : 1;
      g.m_ws[k] = (float*)A.take(4 * n); g.v_ws[k] = (float*)A.take(4 * n);
    }
    g.m_a = (float*)A.take(4 * N_SITES); g.v_a = (float*)A.take(4 * N_SITES);
    g.m_off = (float*)A.take(4 * N_SITES); g.v_off = (float*)A.take(4 * N_SITES);
  }
  c->state_bytes = ((A.off + 255) & ~size_t(255)) - c->state_off;
  *total = (A.off + 255) & ~size_t(255);
}

// Device tables of the per-layer scalar reductions and of the AdamW entries; rebuilt after binds.
int build_tables(mrem_ctx* c) {
  const mrem_module_desc& d = c->d;
  const int L = d.n_layers;
  std::vector<ReduceEntry> red;
  std::vector<AdamEntry> adam, rest;
  for (int l = 0; l < L; ++l) {
    LayerStash& s = c->stash[l];
    LayerGrad& g = c->grad[l];
    LayerBind& b = c->bind[l];
    for (int site = 0; site < N_SITES; ++site) red.push_back({s.part + site * RED_BLOCKS, RED_BLOCKS, g.a + site});
    red.push_back({s.part + N_SITES * RED_BLOCKS, RED_BLOCKS, g.off + 7});
    for (int k = 0; k < N_WMAT; ++k) {
      // per-matrix steps: sum the per-row contributions; per-row steps: a 1-element copy keeps the table uniform
      if (d.w_step_per_row) red.push_back({g.ws[k], 1, g.ws[k]});
      else red.push_back({c->wq[l][k].ds_rows, c->wq[l][k].rows, g.ws[k]});
    }
    for (int k = 0; k < MREM_N_PARAMS; ++k) {
      const bool mat = kParamIsMatrix[k];
      const bool ln = (k == MREM_LN1_G || k == MREM_LN1_B || k == MREM_LN2_G || k == MREM_LN2_B);
      const int bit = mat ? MREM_TRAIN_WEIGHTS : (ln ? MREM_TRAIN_LAYERNORM : MREM_TRAIN_BIASES);
      if (!(d.trainable_mask & bit)) continue;
      if (!b.student[k]) return fail(c, MREM_ERR_ORDER, "student parameter not bound");
      int r, q; param_shape(d, k, &r, &q);
      adam.push_back({b.student[k], g.p[k], g.m_p[k], g.v_p[k], (long long)r * q, mat ? 1.f : 0.f, -INFINITY});
      if (!mat) rest.push_back(adam.back());
    }
    if ((d.trainable_mask & MREM_TRAIN_W_STEPS) && !closed_form_weights(d))
      for (int k = 0; k < N_WMAT; ++k) {
        if (!b.w_steps[k]) return fail(c, MREM_ERR_ORDER, "weight steps not bound");
        adam.push_back({b.w_steps[k], g.ws[k], g.m_ws[k], g.v_ws[k], d.w_step_per_row ? c->wq[l][k].rows : 1, 0.f, 1e-8f});
      }
    if (d.trainable_mask & MREM_TRAIN_A_STEPS) {
      for (int site = 0; site < N_SITES; ++site) {
        if (!b.a_steps[site]) return fail(c, MREM_ERR_ORDER, "activation steps not bound");
        adam.push_back({b.a_steps[site], g.a + site, g.m_a + site, g.v_a + site, 1, 0.f, 1e-8f});
        rest.push_back(adam.back());
      }
      if ((d.act_asym_sites & 2) && b.a_off[7])
        { adam.push_back({b.a_off[7], g.off + 7, g.m_off + 7, g.v_off + 7, 1, 0.f, -INFINITY}); rest.push_back(adam.back()); }
    }
  }
  if (cudaMemcpyAsync(c->reduce_table, red.data(), sizeof(ReduceEntry) * red.size(), cudaMemcpyHostToDevice, c->stream) != cudaSuccess)
    return fail(c, MREM_ERR_CUDA, "table upload failed");
  c->adam_entries = (int)adam.size();
  c->adam_elems = 0;
  for (const AdamEntry& e : adam) c->adam_elems += e.n;
  c->rest_entries = (int)rest.size();
  c->rest_elems = 0;
  for (const AdamEntry& e : rest) c->rest_elems += e.n;
  if (!rest.empty() && cudaMemcpyAsync(c->adam_rest, rest.data(), sizeof(AdamEntry) * rest.size(), cudaMemcpyHostToDevice, c->stream) != cudaSuccess)
    return fail(c, MREM_ERR_CUDA, "table upload failed");
  if (cudaMemcpyAsync(c->adam_table, adam.data(), sizeof(AdamEntry) * adam.size(), cudaMemcpyHostToDevice, c->stream) != cudaSuccess)
    return fail(c, MREM_ERR_CUDA, "table upload failed");
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) return fail(c, MREM_ERR_CUDA, "sync failed");
  c->tables_dirty = false;
  return MREM_OK;
}

}  // namespace mrem

extern "C" {

int32_t mrem_workspace_bytes(const mrem_module_desc* desc, size_t* out_bytes) {
  std::string why;
  const int rc = validate(desc, &why);
  if (rc != MREM_OK) return fail(nullptr, rc, why.c_str());
  if (!out_bytes) return fail(nullptr, MREM_ERR_ARG, "out_bytes is NULL");
  mrem_ctx tmp;
  tmp.d = *desc;
  tmp.dt = desc->act_dtype; tmp.esz = desc->act_dtype == MREM_BF16 ? 2 : 4;
  tmp.max_tokens = (long long)desc->max_batch * desc->max_seq;
  layout(&tmp, nullptr, out_bytes);
  return MREM_OK;
}

int32_t mrem_create(const mrem_module_desc* desc, void* workspace, size_t workspace_bytes, void* cuda_stream,
                    mrem_ctx** out) {
  std::string why;
  const int rc = validate(desc, &why);
  if (rc != MREM_OK) return fail(nullptr, rc, why.c_str());
  if (!workspace || !out) return fail(nullptr, MREM_ERR_ARG, "workspace or out is NULL");
  if (reinterpret_cast<uintptr_t>(workspace) & 255) return fail(nullptr, MREM_ERR_ALIGN, "workspace not 256-byte aligned");
  mrem_ctx* c = new mrem_ctx();
  c->d = *desc;
  c->dt = desc->act_dtype; c->esz = desc->act_dtype == MREM_BF16 ? 2 : 4;
  c->max_tokens = (long long)desc->max_batch * desc->max_seq;
  c->stream = (cudaStream_t)cuda_stream;
  size_t need = 0;
  layout(c, nullptr, &need);
  if (workspace_bytes < need) { delete c; return fail(nullptr, MREM_ERR_WORKSPACE, "workspace too small"); }
  layout(c, (char*)workspace, &need);
  c->ws_base = (char*)workspace;
  c->bind.resize(desc->n_layers);
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    delete c; return fail(nullptr, MREM_ERR_CUDA, "no CUDA device");
  }
  if (cudaMemsetAsync(workspace, 0, need, c->stream) != cudaSuccess) { delete c; return fail(nullptr, MREM_ERR_CUDA, "memset failed"); }
  if (cudaMallocHost((void**)&c->h_pinned_loss, 256) != cudaSuccess) { delete c; return fail(nullptr, MREM_ERR_CUDA, "pinned alloc failed"); }
  int pri_lo = 0, pri_hi = 0;
  if (cudaDeviceGetStreamPriorityRange(&pri_lo, &pri_hi) != cudaSuccess ||
      cudaStreamCreateWithPriority(&c->side_stream, cudaStreamNonBlocking, pri_lo) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->ev_layer[0], cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->ev_layer[1], cudaEventDisableTiming) != cudaSuccess ||
      cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->ev_h2d[0], cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->ev_h2d[1], cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->ev_host_done[0], cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->ev_host_done[1], cudaEventDisableTiming) != cudaSuccess) {
    mrem_destroy(c);
    return fail(nullptr, MREM_ERR_CUDA, "stream or event creation failed");
  }
  *out = c;
  return MREM_OK;
}

int32_t mrem_destroy(mrem_ctx* c) {
  if (!c) return MREM_ERR_ARG;
  if (c->graph_exec) cudaGraphExecDestroy(c->graph_exec);
  if (c->graph) cudaGraphDestroy(c->graph);
  if (c->h_pinned_loss) cudaFreeHost(c->h_pinned_loss);
  if (c->host_graph_exec) cudaGraphExecDestroy(c->host_graph_exec);
  if (c->host_graph) cudaGraphDestroy(c->host_graph);
  for (int k = 0; k < 2; ++k) {
    if (c->ev_h2d[k]) cudaEventDestroy(c->ev_h2d[k]);
    if (c->ev_host_done[k]) cudaEventDestroy(c->ev_host_done[k]);
  }
  if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
  if (c->ev_fork) cudaEventDestroy(c->ev_fork);
  if (c->ev_join) cudaEventDestroy(c->ev_join);
  for (cudaEvent_t e : c->ev_layer) if (e) cudaEventDestroy(e);
  if (c->side_stream) cudaStreamDestroy(c->side_stream);
  delete c;
  return MREM_OK;
}

const char* mrem_last_error(const mrem_ctx* c) { return c ? c->err.c_str() : g_create_err.c_str(); }

int32_t mrem_bind_param(mrem_ctx* c, int32_t role, int32_t layer, int32_t id, void* p, int32_t dtype) {
  if (!c) return MREM_ERR_ARG;
  if (layer < 0 || layer >= c->d.n_layers || id < 0 || id >= MREM_N_PARAMS || !p) return fail(c, MREM_ERR_ARG, "bind_param: bad layer, id or pointer");
  if (reinterpret_cast<uintptr_t>(p) & 255) return fail(c, MREM_ERR_ALIGN, "bind_param: pointer not 256-byte aligned");
  if (role == MREM_TEACHER) {
    const int want = kParamIsMatrix[id] ? c->d.act_dtype : MREM_F32;
    if (dtype != want) return fail(c, MREM_ERR_ARG, "bind_param: teacher matrices are act_dtype, vectors float32");
    c->bind[layer].teacher[id] = p;
  } else if (role == MREM_STUDENT) {
    if (dtype != MREM_F32) return fail(c, MREM_ERR_ARG, "bind_param: student parameters are float32");
    c->bind[layer].student[id] = (float*)p;
  } else {
    return fail(c, MREM_ERR_ARG, "bind_param: role");
  }
  c->tables_dirty = true;
  c->codes_fresh = false;
  return MREM_OK;
}

int32_t mrem_bind_steps(mrem_ctx* c, int32_t layer, int32_t q, float* steps, float* offset) {
  if (!c) return MREM_ERR_ARG;
  if (layer < 0 || layer >= c->d.n_layers || q < 0 || q >= MREM_N_QUANTIZERS || !steps) return fail(c, MREM_ERR_ARG, "bind_steps: bad layer, id or pointer");
  if (reinterpret_cast<uintptr_t>(steps) & 3) return fail(c, MREM_ERR_ALIGN, "bind_steps: pointer not aligned");
  if (q < N_WMAT) c->bind[layer].w_steps[q] = steps;
  else { c->bind[layer].a_steps[q - N_WMAT] = steps; c->bind[layer].a_off[q - N_WMAT] = offset; }
  c->tables_dirty = true;
  c->codes_fresh = false;
  return MREM_OK;
}

int32_t mrem_get_weight_codes(mrem_ctx* c, int32_t layer, int32_t id, const int8_t** codes, const int32_t** rowsum) {
  if (!c) return MREM_ERR_ARG;
  int k = -1;
  for (int i = 0; i < N_WMAT; ++i) if (kMatParam[i] == id) k = i;
  if (layer < 0 || layer >= c->d.n_layers || k < 0) return fail(c, MREM_ERR_ARG, "get_weight_codes: bad layer or id");
  if (codes) *codes = c->wq[layer][k].codes;
  if (rowsum) *rowsum = c->wq[layer][k].rowsum;
  return MREM_OK;
}

int32_t mrem_get_grad(mrem_ctx* c, int32_t layer, int32_t id, const float** g) {
  if (!c || !g) return MREM_ERR_ARG;
  if (layer < 0 || layer >= c->d.n_layers) return fail(c, MREM_ERR_ARG, "get_grad: bad layer");
  if (!c->have_grads) return fail(c, MREM_ERR_ORDER, "get_grad: no backward has run");
  const bool weight_id = (id >= 0 && id < MREM_N_PARAMS && kParamIsMatrix[id]) || (id >= MREM_GRAD_STEP && id < MREM_GRAD_STEP + N_WMAT);
  if (closed_form_weights(c->d) && id >= MREM_GRAD_STEP && id < MREM_GRAD_STEP + N_WMAT)
    return fail(c, MREM_ERR_UNSUPPORTED, "get_grad: closed-form weight scales have no step gradient");
  if (weight_id && !c->w_ste_done && !closed_form_weights(c->d)) {
    // The backward leaves the matrices' gradients unmasked for the fused update; a caller who wants
    // to read them gets the straight-through masks and the step gradients applied now.
    TracerGuard tg(nullptr);
    for (int l = 0; l < c->d.n_layers; ++l)
      for (int k = 0; k < N_WMAT; ++k) {
        const WeightBuf& w = c->wq[l][k];
        launch_ste_weight(c->bind[l].student[kMatParam[k]], c->bind[l].w_steps[k], c->d.w_step_per_row, c->d.w_bits,
                          c->d.w_grid, c->grad[l].p[kMatParam[k]], w.rows, w.cols,
                          c->d.w_step_per_row ? c->grad[l].ws[k] : w.ds_rows, c->stream);
        if (!c->d.w_step_per_row)
          launch_reduce_table(c->reduce_table + (size_t)l * c->reduce_per_layer + N_SITES + 1 + k, 1, c->stream);
      }
    if (cudaGetLastError() != cudaSuccess) return fail(c, MREM_ERR_CUDA, "get_grad: launch failed");
    c->w_ste_done = true;
  }
  LayerGrad& G = c->grad[layer];
  if (id >= 0 && id < MREM_N_PARAMS) *g = G.p[id];
  else if (id >= MREM_GRAD_STEP && id < MREM_GRAD_STEP + N_WMAT) *g = G.ws[id - MREM_GRAD_STEP];
  else if (id >= MREM_GRAD_STEP + N_WMAT && id < MREM_GRAD_STEP + MREM_N_QUANTIZERS) *g = G.a + (id - MREM_GRAD_STEP - N_WMAT);
  else if (id >= MREM_GRAD_OFFSET + N_WMAT && id < MREM_GRAD_OFFSET + MREM_N_QUANTIZERS) *g = G.off + (id - MREM_GRAD_OFFSET - N_WMAT);
  else return fail(c, MREM_ERR_ARG, "get_grad: bad id");
  return MREM_OK;
}

int32_t mrem_get_input_grad(mrem_ctx* c, const void** g) {
  if (!c || !g) return MREM_ERR_ARG;
  if (!c->have_input_grad) return fail(c, MREM_ERR_ORDER, "get_input_grad: no backward pass since the last forward pass");
  *g = c->carry[0];
  return MREM_OK;
}

int32_t mrem_get_activation(mrem_ctx* c, int32_t role, int32_t layer, int32_t which, const void** ptr) {
  if (!c || !ptr) return MREM_ERR_ARG;
  if (layer < 0 || layer >= c->d.n_layers) return fail(c, MREM_ERR_ARG, "get_activation: layer");
  const void* p = nullptr;
  if (role == MREM_TEACHER) {
    if (!c->have_teacher) return fail(c, MREM_ERR_ORDER, "get_activation: no teacher pass to read");
    if (layer != c->d.n_layers - 1) return fail(c, MREM_ERR_ARG, "get_activation: the teacher pass keeps its last layer's tensors only");
    const void* t[MREM_ACT_COUNT] = {c->t_qkv, nullptr, c->t_ctx, c->t_y1, c->t_a, c->t_g, c->t_y2};
    if (which >= 0 && which < MREM_ACT_COUNT) p = t[which];
  } else if (role == MREM_STUDENT) {
    if (!c->have_student) return fail(c, MREM_ERR_ORDER, "get_activation: no student pass to read");
    const LayerStash& s = c->stash[layer];
    const void* t[MREM_ACT_COUNT] = {s.qkv, s.P, s.ctx, s.y1, s.a, s.u, s.y2};
    if (which >= 0 && which < MREM_ACT_COUNT) p = t[which];
  } else {
    return fail(c, MREM_ERR_ARG, "get_activation: role");
  }
  if (!p) return fail(c, MREM_ERR_ARG, "get_activation: this tensor is not kept by that pass");
  *ptr = p;
  return MREM_OK;
}

int32_t mrem_init_student_from_teacher(mrem_ctx* c) {
  if (!c) return MREM_ERR_ARG;
  for (int l = 0; l < c->d.n_layers; ++l)
    for (int k = 0; k < MREM_N_PARAMS; ++k) {
      const LayerBind& b = c->bind[l];
      if (!b.teacher[k] || !b.student[k]) return fail(c, MREM_ERR_ORDER, "init_student: parameters not bound");
      int r, q; param_shape(c->d, k, &r, &q);
      const long long n = (long long)r * q;
      if (kParamIsMatrix[k] && c->dt == 1) {
        launch_widen_bf16(b.teacher[k], b.student[k], n, c->stream);
      } else if (cudaMemcpyAsync(b.student[k], b.teacher[k], n * 4, cudaMemcpyDeviceToDevice, c->stream) != cudaSuccess) {
        return fail(c, MREM_ERR_CUDA, "copy failed");
      }
    }
  char* base = c->ws_base;
  if (cudaMemsetAsync(base + c->state_off, 0, c->state_bytes, c->stream) != cudaSuccess) return fail(c, MREM_ERR_CUDA, "memset failed");
  if (cudaMemsetAsync(c->t_counter, 0, 4, c->stream) != cudaSuccess) return fail(c, MREM_ERR_CUDA, "memset failed");
  c->weights_quantized = false;
  c->codes_fresh = false;
  return MREM_OK;
}

int32_t mrem_init_weight_steps(mrem_ctx* c, int32_t rule) {
  if (!c) return MREM_ERR_ARG;
  TracerGuard tg(nullptr);
  if (rule != 0 && rule != 1) return fail(c, MREM_ERR_ARG, "init_weight_steps: rule");
  if (closed_form_weights(c->d)) return MREM_OK;          // closed-form scales: nothing to initialise
  const float qmax = c->d.w_grid == 0 ? (float)((1 << (c->d.w_bits - 1)) - 1) : 1.5f;
  for (int l = 0; l < c->d.n_layers; ++l)
    for (int k = 0; k < N_WMAT; ++k) {
      const LayerBind& b = c->bind[l];
      if (!b.student[kMatParam[k]] || !b.w_steps[k]) return fail(c, MREM_ERR_ORDER, "init_weight_steps: weights or steps not bound");
      const WeightBuf& w = c->wq[l][k];
      launch_init_weight_steps(b.student[kMatParam[k]], w.rows, w.cols, c->d.w_step_per_row, rule, qmax, b.w_steps[k], w.ds_rows, c->stream);
    }
  c->weights_quantized = false;
  c->codes_fresh = false;
  return cudaGetLastError() == cudaSuccess ? MREM_OK : fail(c, MREM_ERR_CUDA, "launch failed");
}

int32_t mrem_invalidate_weight_codes(mrem_ctx* c) {
  if (!c) return MREM_ERR_ARG;
  c->codes_fresh = false;
  c->weights_quantized = false;
  return MREM_OK;
}

int32_t mrem_set_programmatic_launch(int32_t on) {
  mrem::g_programmatic_launch = on ? 1 : 0;
  return MREM_OK;
}

int32_t mrem_set_loss_share(mrem_ctx* c, float share) {
  if (!c) return MREM_ERR_ARG;
  if (!(share > 0.f && share <= 1.f)) return fail(c, MREM_ERR_ARG, "set_loss_share: share outside (0, 1]");
  c->loss_share = share;
  return MREM_OK;
}

int32_t mrem_grad_bucket(mrem_ctx* c, int32_t layer, float** d_ptr, size_t* n_floats) {
  if (!c || !d_ptr || !n_floats) return MREM_ERR_ARG;
  if (layer < 0 || layer >= c->d.n_layers) return fail(c, MREM_ERR_ARG, "grad_bucket: layer");
  const LayerGrad& g = c->grad[layer];
  // the layer's gradients were carved back to back: parameters, weight steps, activation steps, offsets
  *d_ptr = g.p[0];
  *n_floats = (size_t)((g.off + N_SITES) - g.p[0]);
  return MREM_OK;
}

int32_t mrem_set_wait_limit_ns(uint64_t ns) {
  if (ns < 1000ull || ns > 60000000000ull) return MREM_ERR_ARG;       // 1 us .. 60 s
  mrem::g_wait_limit_ns = ns;
  return MREM_OK;
}

int32_t mrem_selftest_wait_limit(mrem_ctx* c) {
  if (!c) return MREM_ERR_ARG;
  if (launch_wait_probe(c->status, mrem::g_wait_limit_ns, c->stream) != cudaSuccess || cudaGetLastError() != cudaSuccess)
    return fail(c, MREM_ERR_CUDA, "selftest_wait_limit: launch failed");
  return MREM_OK;
}

int32_t mrem_set_fused_attention_backward(mrem_ctx* c, int32_t on) {
  if (!c) return MREM_ERR_ARG;
  c->fused_attention_bwd = on != 0;
  return MREM_OK;
}

int32_t mrem_bind_head(mrem_ctx* c, const float* wp, const float* bp, const float* wc, const float* bc, int32_t n_classes,
                       float* d_logit_loss, float* d_logits) {
  if (!c) return MREM_ERR_ARG;
  if (!wp) { c->head = {}; return MREM_OK; }                 // unbind
  if (!bp || !wc || !bc) return fail(c, MREM_ERR_ARG, "bind_head: NULL tensor");
  if (n_classes < 1 || n_classes > 64) return fail(c, MREM_ERR_SHAPE, "bind_head: 1 <= n_classes <= 64");
  if (c->d.hidden > 2048) return fail(c, MREM_ERR_SHAPE, "bind_head: hidden size up to 2048");
  c->head.wp = wp; c->head.bp = bp; c->head.wc = wc; c->head.bc = bc;
  c->head.n_classes = n_classes; c->head.logit_loss = d_logit_loss; c->head.logits = d_logits;
  return MREM_OK;
}

int32_t mrem_poll_status(mrem_ctx* c, int32_t* h_status) {
  if (!c || !h_status) return MREM_ERR_ARG;
  int v = 0;
  if (cudaMemcpyAsync(&v, c->status, 4, cudaMemcpyDeviceToHost, c->stream) != cudaSuccess ||
      cudaMemsetAsync(c->status, 0, 4, c->stream) != cudaSuccess || cudaStreamSynchronize(c->stream) != cudaSuccess)
    return fail(c, MREM_ERR_CUDA, "poll_status: CUDA error");
  *h_status = v == DEV_OK ? MREM_OK : (v == DEV_NONFINITE ? MREM_ERR_NONFINITE : MREM_ERR_TIMEOUT);
  return MREM_OK;
}

int32_t mrem_state_bytes(mrem_ctx* c, size_t* out) {
  if (!c || !out) return MREM_ERR_ARG;
  *out = c->state_bytes + 256;
  return MREM_OK;
}
int32_t mrem_export_state(mrem_ctx* c, void* blob, size_t bytes) {
  if (!c || !blob) return MREM_ERR_ARG;
  if (bytes < c->state_bytes + 256) return fail(c, MREM_ERR_ARG, "export_state: blob too small");
  char* base = c->ws_base;
  if (cudaMemcpyAsync(blob, c->t_counter, 256, cudaMemcpyDeviceToDevice, c->stream) != cudaSuccess ||
      cudaMemcpyAsync((char*)blob + 256, base + c->state_off, c->state_bytes, cudaMemcpyDeviceToDevice, c->stream) != cudaSuccess)
    return fail(c, MREM_ERR_CUDA, "export_state: copy failed");
  return MREM_OK;
}
int32_t mrem_import_state(mrem_ctx* c, const void* blob, size_t bytes) {
  if (!c || !blob) return MREM_ERR_ARG;
  if (bytes < c->state_bytes + 256) return fail(c, MREM_ERR_ARG, "import_state: blob too small");
  char* base = c->ws_base;
  if (cudaMemcpyAsync(c->t_counter, blob, 256, cudaMemcpyDeviceToDevice, c->stream) != cudaSuccess ||
      cudaMemcpyAsync(base + c->state_off, (const char*)blob + 256, c->state_bytes, cudaMemcpyDeviceToDevice, c->stream) != cudaSuccess)
    return fail(c, MREM_ERR_CUDA, "import_state: copy failed");
  return MREM_OK;
}

int32_t mrem_trace_enable(mrem_ctx* c, int32_t on) {
  if (!c) return MREM_ERR_ARG;
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) return fail(c, MREM_ERR_CUDA, "trace_enable: sync failed");
  c->tracer.reset();
  c->trace_on = on != 0;
  if (c->trace_on) {
    // what a bracketed launch measures beyond the kernel itself: reported as the entry "(empty kernel)"
    TracerGuard tg(&c->tracer);
    launch_trace_calibration(32, c->stream);
  }
  return MREM_OK;
}

int32_t mrem_set_two_streams(mrem_ctx* c, int32_t on) {
  if (!c) return MREM_ERR_ARG;
  c->use_side_stream = on != 0;
  return MREM_OK;
}

int32_t mrem_trace_read(mrem_ctx* c, mrem_trace_entry* out, int32_t max_entries, int32_t* n_entries) {
  if (!c || !out || !n_entries || max_entries < 0) return MREM_ERR_ARG;
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) return fail(c, MREM_ERR_CUDA, "trace_read: sync failed");
  c->tracer.collect();
  int n = 0;
  for (const auto& kv : c->tracer.totals()) {
    if (n >= max_entries) break;
    mrem_trace_entry& e = out[n++];
    std::memset(&e, 0, sizeof(e));
    std::strncpy(e.name, kv.first.c_str(), sizeof(e.name) - 1);
    e.ms = kv.second.ms; e.work = kv.second.work; e.launches = kv.second.launches; e.is_flops = kv.second.is_flops;
  }
  *n_entries = n;
  return MREM_OK;
}

int32_t mrem_gather_rows(const void* src, const int32_t* idx, int32_t n_rows, size_t row_bytes, void* out, void* st) {
  if (!src || !idx || !out || n_rows < 1 || n_rows > 65535) return MREM_ERR_ARG;
  if (row_bytes % 16 || (reinterpret_cast<uintptr_t>(src) & 15) || (reinterpret_cast<uintptr_t>(out) & 15)) return MREM_ERR_ALIGN;
  launch_gather_rows(src, idx, n_rows, (long long)row_bytes, out, (cudaStream_t)st);
  return cudaGetLastError() == cudaSuccess ? MREM_OK : MREM_ERR_CUDA;
}

}  // extern "C"
