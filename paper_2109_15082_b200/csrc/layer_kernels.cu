// LayerNorm, softmax, loss and straight-through backward kernels of the reconstruction step.
// All are HBM/L2-bound passes: 16-byte vector access where the view allows it, one warp per
// row for row-wise ops, warp-shuffle reductions, and fixed-order two-stage sums (per-block
// partials, then one block adds them in index order) so results are reproducible run to run.
#include "kernels.h"
#include "optim.cuh"
#include "vec.cuh"

namespace mrem {

namespace {

// (x - offset) / step for the straight-through factors (see quotient)
__device__ __forceinline__ float qz(float x, float s, float r_s, float off, bool has_off) {
  return quotient(has_off ? __fsub_rn(x, off) : x, s, r_s);
}
__device__ __forceinline__ int qcode(float z, float lo, float hi) { return __float2int_rn(fminf(fmaxf(z, lo), hi)); }

// ------------------------------------------------------------------ loss (Eq. 3) and its gradient
template <typename T, int V>
__global__ void __launch_bounds__(256) loss_kernel(const T* __restrict__ fh, const T* __restrict__ f,
                                                   long long n, float c, T* __restrict__ dF,
                                                   float* __restrict__ partial, int* __restrict__ status) {
  pdl_trigger();
  pdl_wait();
  __shared__ float sh[32];
  const long long base = (long long)blockIdx.y * n;
  float acc = 0.f;
  for (long long i = (blockIdx.x * (long long)blockDim.x + threadIdx.x) * V; i < n; i += (long long)gridDim.x * blockDim.x * V) {
    float a[V], b[V];
    load_vec<T, V>(fh + base + i, a);
    load_vec<T, V>(f + base + i, b);
#pragma unroll
    for (int j = 0; j < V; ++j) {
      const float d = a[j] - b[j];
      acc += d * d;
      a[j] = 2.f * c * d;
    }
    store_vec<T, V>(dF + base + i, a);
  }
  acc = block_sum(acc, sh);
  if (threadIdx.x == 0) {
    partial[blockIdx.y * gridDim.x + blockIdx.x] = acc;
    if (!isfinite(acc) && status) atomicCAS(status, 0, (int)DEV_NONFINITE);
  }
}
__global__ void loss_final_kernel(const float* __restrict__ partial, int n_layers, int nb, float c,
                                  float* __restrict__ total, float* __restrict__ per_layer) {
  pdl_trigger();
  pdl_wait();
  __shared__ float sh[32];
  float tot = 0.f;
  for (int l = 0; l < n_layers; ++l) {
    float a = 0.f;
    for (int i = threadIdx.x; i < nb; i += blockDim.x) a += partial[l * nb + i];
    a = block_sum(a, sh) * c;
    if (threadIdx.x == 0 && per_layer) per_layer[l] = a;
    tot += a;
  }
  if (threadIdx.x == 0 && total) *total = tot;
}

// ------------------------------------------------------------------ STE of an activation quantizer on a 2-D view
template <typename T, int V>
__global__ void __launch_bounds__(256) ste_act_kernel(const T* __restrict__ x, long long ld_x,
                                                      const T* __restrict__ dxhat, long long ld_d,
                                                      const T* __restrict__ add, long long ld_add,
                                                      T* __restrict__ dx, long long ld_dx, long long rows, int cols,
                                                      const float* __restrict__ step,
                                                      const float* __restrict__ offset, float lo, float hi,
                                                      float* __restrict__ part_s, float* __restrict__ part_o) {
  pdl_trigger();
  pdl_wait();
  __shared__ float sh[32];
  const float s = *step, r_s = __frcp_rn(s);
  const bool has_off = offset != nullptr;
  const float off = has_off ? *offset : 0.f;
  const int vcols = cols / V;
  const long long total = rows * vcols;
  float ds = 0.f, dofs = 0.f;
  // (row, vector) of this thread's element, advanced by the grid stride without a division per element
  const long long stride = (long long)gridDim.x * blockDim.x, i0 = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  const long long r_step = stride / vcols;
  const int v_step = (int)(stride - r_step * vcols);
  long long r = i0 / vcols;
  int cv = (int)(i0 - r * vcols);
  for (long long i = i0; i < total; i += stride) {
    const int c = cv * V;
    float xv[V], d[V];
    load_vec<T, V>(x + r * ld_x + c, xv);
    load_vec<T, V>(dxhat + r * ld_d + c, d);
#pragma unroll
    for (int j = 0; j < V; ++j) {
      const float z = qz(xv[j], s, r_s, off, has_off);
      const bool in = z >= lo && z <= hi;
      ds += d[j] * (rne_magic(fminf(fmaxf(z, lo), hi)) - (in ? z : 0.f));
      dofs += in ? 0.f : d[j];
      d[j] = in ? d[j] : 0.f;
    }
    if (add) {
      float e[V];
      load_vec<T, V>(add + r * ld_add + c, e);
#pragma unroll
      for (int j = 0; j < V; ++j) d[j] += e[j];
    }
    store_vec<T, V>(dx + r * ld_dx + c, d);
    r += r_step;
    cv += v_step;
    if (cv >= vcols) { cv -= vcols; ++r; }
  }
  ds = block_sum(ds, sh);
  dofs = block_sum(dofs, sh);
  if (threadIdx.x == 0) {
    part_s[blockIdx.x] = ds;
    if (part_o) part_o[blockIdx.x] = dofs;
  }
}

// ------------------------------------------------------------------ GELU backward with the STE of its output quantizer
template <typename T, int V>
__global__ void __launch_bounds__(256) gelu_bwd_kernel(const T* __restrict__ u, const T* __restrict__ dghat,
                                                       T* __restrict__ du, long long n,
                                                       const float* __restrict__ step,
                                                       const float* __restrict__ offset, float lo, float hi,
                                                       int quantized, float* __restrict__ part_s,
                                                       float* __restrict__ part_o) {
  pdl_trigger();
  pdl_wait();
  __shared__ float sh[32];
  const float s = quantized ? *step : 1.f, r_s = __frcp_rn(s);
  const bool has_off = offset != nullptr;
  const float off = has_off ? *offset : 0.f;
  float ds = 0.f, dofs = 0.f;
  for (long long i = (blockIdx.x * (long long)blockDim.x + threadIdx.x) * V; i < n; i += (long long)gridDim.x * blockDim.x * V) {
    float uv[V], d[V];
    load_vec<T, V>(u + i, uv);
    load_vec<T, V>(dghat + i, d);
#pragma unroll
    for (int j = 0; j < V; ++j) {
      float tail, ex;
      gelu_parts(uv[j], tail, ex);
      if (quantized) {
        const float z = qz(stored<T>(gelu_from_tail(uv[j], tail)), s, r_s, off, has_off);
        const bool in = z >= lo && z <= hi;
        ds += d[j] * (rne_magic(fminf(fmaxf(z, lo), hi)) - (in ? z : 0.f));
        dofs += in ? 0.f : d[j];
        d[j] = in ? d[j] : 0.f;
      }
      d[j] *= gelu_grad_from_parts(uv[j], tail, ex);
    }
    store_vec<T, V>(du + i, d);
  }
  ds = block_sum(ds, sh);
  dofs = block_sum(dofs, sh);
  if (threadIdx.x == 0) {
    if (part_s) part_s[blockIdx.x] = ds;
    if (part_o) part_o[blockIdx.x] = dofs;
  }
}

// ------------------------------------------------------------------ STE of the weight quantizer (one block per row)
// The same pass with the bias gradient of the linear layer before the GELU riding along: b1_grad[c] = sum over rows of
// du[r, c].  A block of 16 x 16 threads owns 16 vectors of columns of one chunk of rows (gridDim.y chunks): a thread adds
// its rows in row order, the block adds its 16 row lanes in index order, and the last block to finish a column group
// (ticket counter) adds the chunks' partials in index order, so the sums do not depend on scheduling.  Block b = y *
// gridDim.x + x leaves its partial step / offset gradient in slot b; slots from the grid size up to n_slots are zeroed.
constexpr int GB_TX = 16, GB_TY = 16;
template <typename T, int V>
__global__ void __launch_bounds__(256) gelu_bwd_colsum_kernel(const T* __restrict__ u, const T* __restrict__ dghat,
                                                              T* __restrict__ du, long long rows, int cols,
                                                              const float* __restrict__ step,
                                                              const float* __restrict__ offset, float lo, float hi,
                                                              int quantized, float* __restrict__ part_s,
                                                              float* __restrict__ part_o, int n_slots,
                                                              float* __restrict__ bias_grad, float* __restrict__ scratch,
                                                              int* __restrict__ counters) {
  pdl_trigger();
  pdl_wait();
  constexpr int BC = GB_TX * V;                              // columns per block
  __shared__ float sh[32];
  __shared__ float cs[GB_TY][BC + 1];
  __shared__ int is_last;
  const float s = quantized ? *step : 1.f, r_s = __frcp_rn(s);
  const bool has_off = offset != nullptr;
  const float off = has_off ? *offset : 0.f;
  const int tx = threadIdx.x % GB_TX, ty = threadIdx.x / GB_TX;
  const int c = blockIdx.x * BC + tx * V;
  const int chunks = gridDim.y;
  const long long per = (rows + chunks - 1) / chunks;
  const long long r0 = blockIdx.y * per, r1 = r0 + per < rows ? r0 + per : rows;
  float acc[V];
#pragma unroll
  for (int j = 0; j < V; ++j) acc[j] = 0.f;
  float ds = 0.f, dofs = 0.f;
  if (c < cols) {
    for (long long r = r0 + ty; r < r1; r += GB_TY) {
      const long long i = r * cols + c;
      float uv[V], d[V];
      load_vec<T, V>(u + i, uv);
      load_vec<T, V>(dghat + i, d);
#pragma unroll
      for (int j = 0; j < V; ++j) {
        float tail, ex;
        gelu_parts(uv[j], tail, ex);
        if (quantized) {
          const float z = qz(stored<T>(gelu_from_tail(uv[j], tail)), s, r_s, off, has_off);
          const bool in = z >= lo && z <= hi;
          ds += d[j] * (rne_magic(fminf(fmaxf(z, lo), hi)) - (in ? z : 0.f));
          dofs += in ? 0.f : d[j];
          d[j] = in ? d[j] : 0.f;
        }
        d[j] *= gelu_grad_from_parts(uv[j], tail, ex);
        acc[j] += d[j];
      }
      store_vec<T, V>(du + i, d);
    }
  }
  ds = block_sum(ds, sh);
  dofs = block_sum(dofs, sh);
  const int bid = blockIdx.y * gridDim.x + blockIdx.x, n_blocks = gridDim.x * gridDim.y;
  if (threadIdx.x == 0) {
    if (part_s) part_s[bid] = ds;
    if (part_o) part_o[bid] = dofs;
  }
  if (bid == 0)
    for (int i = n_blocks + threadIdx.x; i < n_slots; i += blockDim.x) {
      if (part_s) part_s[i] = 0.f;
      if (part_o) part_o[i] = 0.f;
    }
#pragma unroll
  for (int j = 0; j < V; ++j) cs[ty][tx * V + j] = acc[j];
  __syncthreads();
  const int col = threadIdx.x, cc = blockIdx.x * BC + col;
  if (col < BC && cc < cols) {
    float t = 0.f;
#pragma unroll
    for (int k = 0; k < GB_TY; ++k) t += cs[k][col];
    scratch[(long long)blockIdx.y * cols + cc] = t;
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) is_last = atomicAdd(&counters[blockIdx.x], 1) == chunks - 1;
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  if (col < BC && cc < cols) {
    const float* src = scratch + cc;
    float t = 0.f;
    for (int k0 = 0; k0 < chunks; k0 += 8) {                 // eight loads in flight, added in index order
      float q[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) q[k] = k0 + k < chunks ? src[(long long)(k0 + k) * cols] : 0.f;
#pragma unroll
      for (int k = 0; k < 8; ++k) t += q[k];
    }
    bias_grad[cc] = t;
  }
  if (threadIdx.x == 0) counters[blockIdx.x] = 0;           // ready for the next launch
}

__global__ void __launch_bounds__(256) ste_weight_kernel(const float* __restrict__ w, const float* __restrict__ steps,
                                                         int per_row, int bits, int grid, float* __restrict__ dw,
                                                         int cols, float* __restrict__ ds_rows) {
  pdl_trigger();
  pdl_wait();
  __shared__ float sh[32];
  const int row = blockIdx.x;
  const float s = steps[per_row ? row : 0];
  const float r_s = __frcp_rn(s);
  const float qmax = (float)((1 << (bits - 1)) - 1);
  const float4* wr = reinterpret_cast<const float4*>(w + (long long)row * cols);
  float4* dr = reinterpret_cast<float4*>(dw + (long long)row * cols);
  float ds = 0.f;
  for (int c = threadIdx.x; c < cols / 4; c += blockDim.x) {     // cols is a multiple of 16
    const float4 wv = wr[c];
    float4 d = dr[c];
    bool in;
    ds = step_grad_acc(ds, wv.x, d.x, s, r_s, qmax, grid, in); d.x = in ? d.x : 0.f;
    ds = step_grad_acc(ds, wv.y, d.y, s, r_s, qmax, grid, in); d.y = in ? d.y : 0.f;
    ds = step_grad_acc(ds, wv.z, d.z, s, r_s, qmax, grid, in); d.z = in ? d.z : 0.f;
    ds = step_grad_acc(ds, wv.w, d.w, s, r_s, qmax, grid, in); d.w = in ? d.w : 0.f;
    dr[c] = d;
  }
  ds = block_sum(ds, sh);
  if (threadIdx.x == 0) ds_rows[row] = ds;
}

__global__ void __launch_bounds__(256) reduce_table_kernel(const ReduceEntry* __restrict__ table) {
  pdl_trigger();
  pdl_wait();
  __shared__ float sh[32];
  const ReduceEntry e = table[blockIdx.x];
  float a = 0.f;
  for (int i = threadIdx.x; i < e.count; i += blockDim.x) a += e.src[i];
  a = block_sum(a, sh);
  if (threadIdx.x == 0) *e.dst = a;
}

__global__ void scale_vec_kernel(const float* __restrict__ in, const float* __restrict__ scale, float* __restrict__ out, int n) {
  pdl_trigger();
  pdl_wait();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = scale[0] * in[i];
}
__global__ void effective_bias_kernel(const float* __restrict__ b, const float* __restrict__ beta,
                                      const float* __restrict__ wscale, const int32_t* __restrict__ rowsum,
                                      float* __restrict__ beff, int n) {
  pdl_trigger();
  pdl_wait();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) beff[i] = b[i] + beta[0] * wscale[i] * (float)rowsum[i];
}

// ------------------------------------------------------------------ AdamW
__global__ void optim_prepare_kernel(OptimScalars* out, int* d_t, int host_t, float lr0, int total, float b1, float b2,
                                     float eps, float wd) {
  pdl_trigger();
  pdl_wait();
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  int t = host_t >= 1 ? host_t : (*d_t + 1);
  *d_t = t;
  OptimScalars o;
  o.lr = total > 0 ? lr0 * fmaxf(1.f - (float)(t - 1) / (float)total, 0.f) : lr0;
  o.beta1 = b1;
  o.beta2 = b2;
  o.eps = eps;
  o.weight_decay = wd;
  o.bc1 = (float)(1.0 - pow((double)b1, (double)t));
  o.bc2 = (float)(1.0 - pow((double)b2, (double)t));
  o.lr_bc1 = (float)((double)o.lr / (1.0 - pow((double)b1, (double)t)));
  o.rsqrt_bc2 = (float)(1.0 / sqrt(1.0 - pow((double)b2, (double)t)));
  *out = o;
}

__global__ void __launch_bounds__(256) adamw_table_kernel(const AdamEntry* __restrict__ table,
                                                          const OptimScalars* __restrict__ sc) {
  pdl_trigger();
  pdl_wait();
  const AdamEntry e = table[blockIdx.y];
  const OptimScalars o = *sc;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < e.n; i += (long long)gridDim.x * blockDim.x) {
    float m = e.m[i], v = e.v[i];
    e.p[i] = adam_one(e.p[i], e.g[i], m, v, o, e.wd, e.min_value);
    e.m[i] = m;
    e.v[i] = v;
  }
}

inline int grid_for(long long work_items, int threads = 256, int cap = 148 * 8) {
  long long b = (work_items + threads - 1) / threads;
  if (b < 1) b = 1;
  return (int)(b < cap ? b : cap);
}
inline bool al16(const void* p) { return p == nullptr || (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

}  // namespace

#define MREM_DT(dt, T, ...)            \
  do {                                 \
    if ((dt) == 1) { using T = bf16; __VA_ARGS__; } else { using T = float; __VA_ARGS__; } \
  } while (0)

void launch_loss(const void* f_hat, const void* f, int n_layers, long long n_per_layer, float c, void* dF,
                 float* partial, int* status, int dt, cudaStream_t st) {
  Scope sc("recon_loss", (double)n_layers * n_per_layer * 3 * (dt == 1 ? 2.0 : 4.0), 0, st);
  dim3 grid(RED_BLOCKS, n_layers);
  MREM_DT(dt, T, {
    constexpr int V = 16 / (int)sizeof(T);
    if (n_per_layer % V == 0 && al16(f_hat) && al16(f) && al16(dF))
      launch_k(loss_kernel<T, V>, grid, 256, 0, st, (const T*)f_hat, (const T*)f, n_per_layer, c, (T*)dF, partial, status);
    else
      launch_k(loss_kernel<T, 1>, grid, 256, 0, st, (const T*)f_hat, (const T*)f, n_per_layer, c, (T*)dF, partial, status);
  });
}
void launch_loss_finalize(const float* partial, int n_layers, float c, float* loss_total, float* loss_per_layer,
                          cudaStream_t st) {
  launch_k(loss_final_kernel, 1, 256, 0, st, partial, n_layers, RED_BLOCKS, c, loss_total, loss_per_layer);
}

void launch_ste_act(const void* x, long long ld_x, const void* dxhat, long long ld_d, const void* add,
                    long long ld_add, void* dx, long long ld_dx, long long rows, int cols, const float* step,
                    const float* offset, int lo, int hi, float* part_s, float* part_o, int dt, cudaStream_t st) {
  Scope sc("ste_act", (double)rows * cols * (dt == 1 ? 2.0 : 4.0) * (add ? 4 : 3), 0, st);
  MREM_DT(dt, T, {
    constexpr int V = 16 / (int)sizeof(T);
    const bool v = cols % V == 0 && ld_x % V == 0 && ld_d % V == 0 && ld_dx % V == 0 && (!add || ld_add % V == 0) &&
                   al16(x) && al16(dxhat) && al16(add) && al16(dx);
    if (v) launch_k(ste_act_kernel<T, V>, RED_BLOCKS, 256, 0, st, (const T*)x, ld_x, (const T*)dxhat, ld_d, (const T*)add, ld_add, (T*)dx, ld_dx, rows, cols, step, offset, (float)lo, (float)hi, part_s, part_o);
    else launch_k(ste_act_kernel<T, 1>, RED_BLOCKS, 256, 0, st, (const T*)x, ld_x, (const T*)dxhat, ld_d, (const T*)add, ld_add, (T*)dx, ld_dx, rows, cols, step, offset, (float)lo, (float)hi, part_s, part_o);
  });
}

bool launch_gelu_bwd_colsum(const void* u, const void* dghat, void* du, long long rows, int cols, const float* step,
                             const float* offset, int lo, int hi, int quantized, float* part_s, float* part_o,
                             float* bias_grad, float* scratch, long long scratch_floats, int* counters, int n_counters,
                             int dt, cudaStream_t st) {
  if (rows <= 0 || cols <= 0) return false;
  bool done = false;
  MREM_DT(dt, T, {
    constexpr int V = 16 / (int)sizeof(T);
    constexpr int BC = GB_TX * V;
    const int col_blocks = (cols + BC - 1) / BC;
    long long chunks = RED_BLOCKS / col_blocks;                       // the grid fills the RED_BLOCKS partial-sum slots
    if (chunks > (rows + GB_TY - 1) / GB_TY) chunks = (rows + GB_TY - 1) / GB_TY;
    if (chunks > scratch_floats / cols) chunks = scratch_floats / cols;
    if (cols % V == 0 && al16(u) && al16(dghat) && al16(du) && chunks >= 1 && col_blocks <= n_counters && col_blocks <= RED_BLOCKS) {
      Scope sc("gelu_bwd", (double)rows * cols * 3 * (dt == 1 ? 2.0 : 4.0), 0, st);
      dim3 grid(col_blocks, (unsigned)chunks);
      launch_k(gelu_bwd_colsum_kernel<T, V>, grid, 256, 0, st, (const T*)u, (const T*)dghat, (T*)du, rows, cols, step, offset,
               (float)lo, (float)hi, quantized, part_s, part_o, RED_BLOCKS, bias_grad, scratch, counters);
      done = true;
    }
  });
  return done;
}

void launch_gelu_bwd(const void* u, const void* dghat, void* du, long long n, const float* step, const float* offset,
                     int lo, int hi, int quantized, float* part_s, float* part_o, int dt, cudaStream_t st) {
  Scope sc("gelu_bwd", (double)n * 3 * (dt == 1 ? 2.0 : 4.0), 0, st);
  MREM_DT(dt, T, {
    constexpr int V = 16 / (int)sizeof(T);
    if (n % V == 0 && al16(u) && al16(dghat) && al16(du))
      launch_k(gelu_bwd_kernel<T, V>, RED_BLOCKS, 256, 0, st, (const T*)u, (const T*)dghat, (T*)du, n, step, offset, (float)lo, (float)hi, quantized, part_s, part_o);
    else
      launch_k(gelu_bwd_kernel<T, 1>, RED_BLOCKS, 256, 0, st, (const T*)u, (const T*)dghat, (T*)du, n, step, offset, (float)lo, (float)hi, quantized, part_s, part_o);
  });
}

void launch_ste_weight(const float* w, const float* steps, int per_row, int bits, int grid, float* dw, int rows,
                       int cols, float* ds_rows, cudaStream_t st) {
  Scope sc("ste_weight", (double)rows * cols * 12.0, 0, st);
  launch_k(ste_weight_kernel, rows, 256, 0, st, w, steps, per_row, bits, grid, dw, cols, ds_rows);
}

// A kernel that does nothing, bracketed by the tracer like every other launch: what the event pair itself measures
// (event processing, launch and drain of a grid) and therefore what every traced duration contains on top of the
// kernel's own run time.
__global__ void empty_kernel() {
  pdl_trigger();
  pdl_wait();
}
void launch_trace_calibration(int n, cudaStream_t st) {
  for (int i = 0; i < n; ++i) {
    Scope sc("(empty kernel)", 0.0, 0, st);
    launch_k(empty_kernel, 148, 256, 0, st);
  }
}

void launch_reduce_table(const ReduceEntry* d_table, int n_entries, cudaStream_t st) {
  if (n_entries > 0) launch_k(reduce_table_kernel, n_entries, 256, 0, st, d_table);
}

void launch_scale_vec(const float* in, const float* scale, float* out, int n, cudaStream_t st) {
  launch_k(scale_vec_kernel, (n + 255) / 256, 256, 0, st, in, scale, out, n);
}
void launch_effective_bias(const float* b, const float* beta, const float* wscale, const int32_t* rowsum, float* beff,
                           int n, cudaStream_t st) {
  launch_k(effective_bias_kernel, (n + 255) / 256, 256, 0, st, b, beta, wscale, rowsum, beff, n);
}

void launch_optim_prepare(OptimScalars* d_out, int* d_t, int host_t, float lr0, int total_steps, float beta1,
                          float beta2, float eps, float weight_decay, cudaStream_t st) {
  launch_k(optim_prepare_kernel, 1, 32, 0, st, d_out, d_t, host_t, lr0, total_steps, beta1, beta2, eps, weight_decay);
}
void launch_adamw_table(const AdamEntry* d_table, int n_entries, long long total_elems, const OptimScalars* d_sc,
                        cudaStream_t st) {
  if (n_entries <= 0) return;
  Scope sc("adamw", (double)total_elems * 28.0, 0, st);
  dim3 grid(64, n_entries);
  launch_k(adamw_table_kernel, grid, 256, 0, st, d_table, d_sc);
}

}  // namespace mrem
