// Embedding layers of the first module (Sec. 4.1: besides the grouped Transformer layers the MSE of the
// Transformer embedding is minimised; Sec. 3.1: embeddings are quantized symmetrically like weights).
//   teacher  e     = LayerNorm(word[ids] + pos[0..S) + type[type_ids])
//   student  e_hat = LayerNorm(Q(word)[ids] + pos + type),  Q = Eq. 1 on the word table, one step per row
//   loss     c * || e_hat - e ||^2,  straight-through backward, AdamW on the student's tables, the word
//            table's row steps and the LayerNorm parameters; the update re-quantizes the word table.
// The word table is treated as a weight matrix with `vocab` output rows: its quantizer, straight-through
// mask and fused AdamW + re-quantization are the kernels of the encoder matrices; LayerNorm, loss and
// column reductions likewise.  New here: the gather (codes x row scale, exact), the scatter of the token
// gradients into table rows (every token that gathered a row, added in token order: no atomics) and the
// reductions over the batch for the position and token-type tables.  Nothing is allocated: the caller
// brings every tensor and one workspace.
#include <cmath>

#include "../../include/mrem.h"
#include "kernels.h"
#include "vec.cuh"

namespace mrem {

namespace {

// y[t, :] = row(ids[t]) + pos[t % S, :] + type[type_ids[t], :], rounded as stored; one block of 128 threads per token.
// With codes the row is scale[id] * codes[id, :] (the quantized table), else word[id, :].
template <typename T>
__global__ void __launch_bounds__(128) embed_sum_kernel(const float* __restrict__ word, const int8_t* __restrict__ codes,
                                                        const float* __restrict__ scale, const float* __restrict__ pos,
                                                        const float* __restrict__ type, const int* __restrict__ ids,
                                                        const int* __restrict__ type_ids, int S, int H, int vocab, int n_types,
                                                        T* __restrict__ y, int* __restrict__ status) {
  pdl_trigger();
  pdl_wait();
  const long long t = blockIdx.x;
  int id = ids[t], tt = type_ids ? type_ids[t] : 0;
  if (id < 0 || id >= vocab || tt < 0 || tt >= n_types) {          // recorded, then clamped: no out-of-range access
    if (threadIdx.x == 0) atomicCAS(status, 0, (int)DEV_BAD_INDEX);
    id = min(max(id, 0), vocab - 1);
    tt = min(max(tt, 0), n_types - 1);
  }
  const int s = (int)(t % S);
  const float sc = codes ? scale[id] : 0.f;
  for (int c = threadIdx.x; c < H; c += blockDim.x) {
    const float w = codes ? sc * (float)codes[(long long)id * H + c] : word[(long long)id * H + c];
    y[t * H + c] = from_f<T>(w + pos[(long long)s * H + c] + type[(long long)tt * H + c]);
  }
}

// Occurrence lists of the batch's ids, without sorting and without atomics.  Per token t (one thread each):
//   lead[t] = index of the first token with the id of token t,  rank[t] = number of earlier tokens with that id.
__global__ void __launch_bounds__(256) embed_lead_kernel(const int* __restrict__ ids, int M, int vocab, int* __restrict__ lead,
                                                         int* __restrict__ rank) {
  pdl_trigger();
  pdl_wait();
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= M) return;
  const int id = min(max(ids[t], 0), vocab - 1);
  int first = t, r = 0;
  for (int i = t - 1; i >= 0; --i)
    if (min(max(ids[i], 0), vocab - 1) == id) { first = i; ++r; }
  lead[t] = first;
  rank[t] = r;
}
// list = the tokens grouped by id (groups ordered by their first token, token order inside a group):
//   position of token t = number of tokens whose group starts before t's group + rank[t];
// for the first token of a group also start[t] = that position and count[t] = size of the group (count 0 elsewhere).
__global__ void __launch_bounds__(256) embed_list_kernel(const int* __restrict__ lead, const int* __restrict__ rank, int M,
                                                         int* __restrict__ list, int* __restrict__ start, int* __restrict__ count) {
  pdl_trigger();
  pdl_wait();
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= M) return;
  const int mine = lead[t];
  int before = 0, same = 0;
  for (int i = 0; i < M; ++i) {
    const int l = lead[i];
    before += l < mine;
    same += l == mine;
  }
  list[before + rank[t]] = t;
  start[t] = before;
  count[t] = mine == t ? same : 0;
}

// g_word[id, :] = sum over the tokens t with ids[t] == id of dy[t, :], in token order: the block of the first
// token with an id adds that id's group of the list for its 128 columns (independent loads); rows no token gathered
// keep the zeros the caller put there.
template <typename T>
__global__ void __launch_bounds__(128) embed_scatter_kernel(const T* __restrict__ dy, const int* __restrict__ ids,
                                                            const int* __restrict__ list, const int* __restrict__ start,
                                                            const int* __restrict__ count, int H, int vocab,
                                                            float* __restrict__ g_word) {
  pdl_trigger();
  pdl_wait();
  const int t0 = blockIdx.x, n = count[t0];
  if (n == 0) return;                                               // block-uniform: not the first token of its id
  const int c = blockIdx.y * blockDim.x + threadIdx.x;
  if (c >= H) return;
  const int id = min(max(ids[t0], 0), vocab - 1);
  const int* grp = list + start[t0];
  float acc = 0.f;
  for (int j = 0; j < n; ++j) acc += to_f<T>(dy[(long long)grp[j] * H + c]);
  g_word[(long long)id * H + c] = acc;
}

// g_pos[s, c] = sum_b dy[b, s, c] (rows of the table beyond seq get zero).
template <typename T>
__global__ void __launch_bounds__(256) embed_pos_kernel(const T* __restrict__ dy, int B, int S, int H, float* __restrict__ g_pos) {
  pdl_trigger();
  pdl_wait();
  const int c = blockIdx.x * blockDim.x + threadIdx.x, row = blockIdx.y;
  if (c >= H) return;
  float acc = 0.f;
  if (row < S)
    for (int b = 0; b < B; ++b) acc += to_f<T>(dy[((long long)b * S + row) * H + c]);
  g_pos[(long long)row * H + c] = acc;
}

// Token-type table, two stages with fixed orders: partial[chunk, k, c] = sum over the chunk's tokens of type k (token
// order), then g_type[k, c] = sum over the chunks in index order.
constexpr int TYPE_CHUNKS = 64;
template <typename T>
__global__ void __launch_bounds__(256) embed_type_partial_kernel(const T* __restrict__ dy, const int* __restrict__ type_ids,
                                                                 long long M, int H, int n_types, float* __restrict__ partial) {
  pdl_trigger();
  pdl_wait();
  const int c = blockIdx.x * blockDim.x + threadIdx.x, chunk = blockIdx.y, k = blockIdx.z;
  if (c >= H) return;
  const long long per = (M + TYPE_CHUNKS - 1) / TYPE_CHUNKS, t0 = chunk * per, t1 = t0 + per < M ? t0 + per : M;
  float acc = 0.f;
  for (long long t = t0; t < t1; ++t) {
    const int tt = type_ids ? min(max(type_ids[t], 0), n_types - 1) : 0;
    if (tt == k) acc += to_f<T>(dy[t * H + c]);
  }
  partial[((long long)chunk * n_types + k) * H + c] = acc;
}
__global__ void __launch_bounds__(256) embed_type_final_kernel(const float* __restrict__ partial, int H, int n_types,
                                                               float* __restrict__ g_type) {
  pdl_trigger();
  pdl_wait();
  const int c = blockIdx.x * blockDim.x + threadIdx.x, k = blockIdx.y;
  if (c >= H) return;
  float acc = 0.f;
  for (int chunk = 0; chunk < TYPE_CHUNKS; ++chunk) acc += partial[((long long)chunk * n_types + k) * H + c];
  g_type[(long long)k * H + c] = acc;
}

struct Carve {                         // the workspace, cut the same way by the sizing call and by the step
  char* base; size_t off = 0;
  explicit Carve(void* b) : base((char*)b) {}
  void* take(size_t bytes) { off = (off + 255) & ~size_t(255); void* p = base ? base + off : nullptr; off += bytes; return p; }
};
struct EmbedScratch {
  void *y_t, *y_s, *dE, *dy, *dsum;
  float *mean, *rstd, *col_scratch, *loss_partial;
  long long col_plane;
  int* col_counters;
  int8_t* codes; int32_t* rowsum; float* scale;
  OptimScalars* optim_sc; AdamEntry* table;
  int *lead, *rank, *list, *start, *count; float* type_partial;
  size_t bytes;
};
EmbedScratch carve(const mrem_embed_desc& d, long long max_tokens, void* base) {
  Carve A(base);
  EmbedScratch s;
  const size_t es = d.act_dtype == MREM_BF16 ? 2 : 4;
  const size_t MH = (size_t)max_tokens * d.hidden;
  s.y_t = A.take(MH * es); s.y_s = A.take(MH * es); s.dE = A.take(MH * es); s.dy = A.take(MH * es); s.dsum = A.take(MH * es);
  s.mean = (float*)A.take(4 * max_tokens); s.rstd = (float*)A.take(4 * max_tokens);
  s.col_plane = (long long)COL_CHUNKS * d.hidden;
  s.col_scratch = (float*)A.take(sizeof(float) * 3 * s.col_plane);
  s.col_counters = (int*)A.take(sizeof(int) * (d.hidden / 32 + 2));
  s.loss_partial = (float*)A.take(sizeof(float) * RED_BLOCKS);
  s.codes = (int8_t*)A.take((size_t)d.vocab * d.hidden);
  s.rowsum = (int32_t*)A.take(sizeof(int32_t) * d.vocab);
  s.scale = (float*)A.take(sizeof(float) * d.vocab);
  s.optim_sc = (OptimScalars*)A.take(sizeof(OptimScalars));
  s.table = (AdamEntry*)A.take(sizeof(AdamEntry) * 4);
  s.lead = (int*)A.take(sizeof(int) * max_tokens); s.rank = (int*)A.take(sizeof(int) * max_tokens);
  s.list = (int*)A.take(sizeof(int) * max_tokens); s.start = (int*)A.take(sizeof(int) * max_tokens);
  s.count = (int*)A.take(sizeof(int) * max_tokens);
  s.type_partial = (float*)A.take(sizeof(float) * (size_t)TYPE_CHUNKS * d.n_types * d.hidden);
  s.bytes = (A.off + 255) & ~size_t(255);
  return s;
}

int check_desc(const mrem_embed_desc* d) {
  if (!d || d->struct_size != sizeof(mrem_embed_desc)) return MREM_ERR_ARG;
  if (d->vocab < 1 || d->hidden < 16 || d->hidden % 16 || d->max_pos < 1 || d->n_types < 1) return MREM_ERR_SHAPE;
  if (d->e_bits != 2 && d->e_bits != 4 && d->e_bits != 8) return MREM_ERR_UNSUPPORTED;
  if (d->act_dtype != MREM_F32 && d->act_dtype != MREM_BF16) return MREM_ERR_ARG;
  return MREM_OK;
}

}  // namespace
}  // namespace mrem

using namespace mrem;

extern "C" {

int32_t mrem_embed_workspace_bytes(const mrem_embed_desc* d, int32_t max_tokens, size_t* out_bytes) {
  const int rc = check_desc(d);
  if (rc != MREM_OK) return rc;
  if (!out_bytes || max_tokens < 1) return MREM_ERR_ARG;
  *out_bytes = carve(*d, max_tokens, nullptr).bytes;
  return MREM_OK;
}

int32_t mrem_embed_step(const mrem_embed_desc* d, const mrem_embed_tensors* x, void* workspace, size_t workspace_bytes,
                        const int32_t* d_ids, const int32_t* d_type_ids, int32_t batch, int32_t seq, int32_t requantize,
                        void* d_e_teacher, void* d_e_student, const void* d_extra_grad, const mrem_optim* o, float* d_loss,
                        int32_t* d_status, void* cuda_stream) {
  int rc = check_desc(d);
  if (rc != MREM_OK) return rc;
  if (!x || !workspace || !d_ids || !d_e_teacher || !d_e_student || !d_loss || !d_status) return MREM_ERR_ARG;
  if (batch < 1 || seq < 1 || seq > d->max_pos) return MREM_ERR_SHAPE;
  const float* need[] = {x->t_word, x->t_pos, x->t_type, x->t_ln_g, x->t_ln_b, x->word, x->pos, x->type, x->ln_g, x->ln_b,
                         x->word_step, x->g_word, x->g_word_step, x->g_pos, x->g_type, x->g_ln_g, x->g_ln_b};
  for (const float* p : need) if (!p) return MREM_ERR_ARG;
  if (o && (!x->m_word || !x->v_word || !x->m_word_step || !x->v_word_step || !x->m_pos || !x->v_pos || !x->m_type || !x->v_type ||
            !x->m_ln_g || !x->v_ln_g || !x->m_ln_b || !x->v_ln_b || !x->d_step_counter))
    return MREM_ERR_ARG;
  const long long M = (long long)batch * seq;
  const int H = d->hidden, V = d->vocab, dt = d->act_dtype == MREM_BF16 ? 1 : 0;
  const EmbedScratch s = carve(*d, M, workspace);
  if (s.bytes > workspace_bytes) return MREM_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255) || (reinterpret_cast<uintptr_t>(d_e_teacher) & 15) ||
      (reinterpret_cast<uintptr_t>(d_e_student) & 15) || (reinterpret_cast<uintptr_t>(x->word) & 15) ||
      (reinterpret_cast<uintptr_t>(x->g_word) & 15))
    return MREM_ERR_ALIGN;
  cudaStream_t st = (cudaStream_t)cuda_stream;

  // Eq. 1 on the word table (only when the caller changed it or its steps since the last update)
  if (requantize) launch_quantize_weight(x->word, V, H, x->word_step, 1, d->e_bits, 0, s.codes, s.rowsum, s.scale, nullptr, dt, st);
  // both embedding outputs
#define MREM_EMB(T) do { \
    launch_k(embed_sum_kernel<T>, (unsigned)M, 128, 0, st, x->t_word, (const int8_t*)nullptr, (const float*)nullptr, x->t_pos, x->t_type, d_ids, d_type_ids, (int)seq, H, V, (int)d->n_types, (T*)s.y_t, d_status); \
    launch_k(embed_sum_kernel<T>, (unsigned)M, 128, 0, st, (const float*)x->word, (const int8_t*)s.codes, (const float*)s.scale, (const float*)x->pos, (const float*)x->type, d_ids, d_type_ids, (int)seq, H, V, (int)d->n_types, (T*)s.y_s, d_status); } while (0)
  if (dt == 1) MREM_EMB(bf16); else MREM_EMB(float);
#undef MREM_EMB
  launch_layernorm_fwd(s.y_t, x->t_ln_g, x->t_ln_b, d->ln_eps, M, H, d_e_teacher, nullptr, nullptr, nullptr, 0, nullptr, nullptr, dt, st);
  launch_layernorm_fwd(s.y_s, x->ln_g, x->ln_b, d->ln_eps, M, H, d_e_student, s.mean, s.rstd, nullptr, 0, nullptr, nullptr, dt, st);
  // loss and its gradient
  const long long n = M * H;
  const float cc = d->loss_mean ? 1.f / (float)n : 1.f;
  launch_loss(d_e_student, d_e_teacher, 1, n, cc, s.dE, s.loss_partial, d_status, dt, st);
  launch_loss_finalize(s.loss_partial, 1, cc, d_loss, nullptr, st);
  // LayerNorm backward and its parameter gradients
  // (with a gradient arriving from the layers the embedding feeds, the LayerNorm sees the sum of the two)
  if (d_extra_grad && (reinterpret_cast<uintptr_t>(d_extra_grad) & 15)) return MREM_ERR_ALIGN;
  launch_layernorm_bwd(s.dE, d_extra_grad, s.y_s, s.mean, s.rstd, x->ln_g, M, H, s.dy, d_extra_grad ? s.dsum : nullptr, dt, st);
  if (cudaMemsetAsync(s.col_counters, 0, sizeof(int) * (H / 32 + 2), st) != cudaSuccess) return MREM_ERR_CUDA;
  launch_col_reduce(d_extra_grad ? s.dsum : s.dE, H, s.y_s, s.mean, s.rstd, nullptr, 0, M, H, x->g_ln_b, x->g_ln_g, nullptr, s.col_scratch, s.col_plane,
                    s.col_counters, dt, st);
  // position / token-type tables: sums over the batch; word table: every token's gradient into the row it gathered
  if (cudaMemsetAsync(x->g_word, 0, sizeof(float) * (size_t)V * H, st) != cudaSuccess) return MREM_ERR_CUDA;
  launch_k(embed_lead_kernel, (unsigned)((M + 255) / 256), 256, 0, st, d_ids, (int)M, V, s.lead, s.rank);
  launch_k(embed_list_kernel, (unsigned)((M + 255) / 256), 256, 0, st, (const int*)s.lead, (const int*)s.rank, (int)M, s.list, s.start, s.count);
  const dim3 gcol((H + 255) / 256), gscat((unsigned)M, (H + 127) / 128);
#define MREM_EMB_BWD(T) do { \
    launch_k(embed_pos_kernel<T>, dim3(gcol.x, d->max_pos), 256, 0, st, (const T*)s.dy, (int)batch, (int)seq, H, x->g_pos); \
    launch_k(embed_type_partial_kernel<T>, dim3(gcol.x, TYPE_CHUNKS, d->n_types), 256, 0, st, (const T*)s.dy, d_type_ids, M, H, (int)d->n_types, s.type_partial); \
    launch_k(embed_scatter_kernel<T>, gscat, 128, 0, st, (const T*)s.dy, d_ids, (const int*)s.list, (const int*)s.start, (const int*)s.count, H, V, x->g_word); } while (0)
  if (dt == 1) MREM_EMB_BWD(bf16); else MREM_EMB_BWD(float);
#undef MREM_EMB_BWD
  launch_k(embed_type_final_kernel, dim3(gcol.x, d->n_types), 256, 0, st, (const float*)s.type_partial, H, (int)d->n_types, x->g_type);
  if (!o) {
    // gradients only: the word table's straight-through mask and its row-step gradients, left in g_word / g_word_step
    launch_ste_weight(x->word, x->word_step, 1, d->e_bits, 0, x->g_word, V, H, x->g_word_step, st);
    return cudaGetLastError() == cudaSuccess ? MREM_OK : MREM_ERR_CUDA;
  }
  // update: mask + step gradient + AdamW on the steps and the table + Eq. 1 with the new values in one pass;
  // the small tensors through the table kernel (embedding tables decayed like weight matrices, LayerNorm not)
  launch_optim_prepare(s.optim_sc, x->d_step_counter, o->step, o->lr, o->decay_total_steps, o->beta1, o->beta2, o->eps, o->weight_decay, st);
  launch_fused_weight_update(x->word, x->g_word, x->m_word, x->v_word, x->word_step, nullptr, x->m_word_step, x->v_word_step, s.optim_sc,
                             V, H, d->e_bits, 0, 1, 1, s.codes, s.rowsum, s.scale, nullptr, dt, st);
  const AdamEntry host[4] = {
      {x->pos, x->g_pos, x->m_pos, x->v_pos, (long long)d->max_pos * H, 1.f, -INFINITY},
      {x->type, x->g_type, x->m_type, x->v_type, (long long)d->n_types * H, 1.f, -INFINITY},
      {x->ln_g, x->g_ln_g, x->m_ln_g, x->v_ln_g, H, 0.f, -INFINITY},
      {x->ln_b, x->g_ln_b, x->m_ln_b, x->v_ln_b, H, 0.f, -INFINITY}};
  if (cudaMemcpyAsync(s.table, host, sizeof(host), cudaMemcpyHostToDevice, st) != cudaSuccess) return MREM_ERR_CUDA;
  launch_adamw_table(s.table, 4, (long long)(d->max_pos + d->n_types + 2) * H, s.optim_sc, st);
  return cudaGetLastError() == cudaSuccess ? MREM_OK : MREM_ERR_CUDA;
}

}  // extern "C"
