// Shared pieces of the tensor-core GEMM kernels: launch parameters, tile decoding and the epilogue
// (TMEM accumulators -> scale / bias / residual / activation -> bf16 rows through a small shared-memory box and a
// tiled store, or global stores straight from registers, every lane writing whole 32-byte sectors of its own row).
#pragma once
#include "gemm.h"
#include "tc_ptx.cuh"

namespace mrem {
namespace tc {

constexpr int BLOCK_M = 128;
constexpr int A_STAGE_BYTES = BLOCK_M * 128;          // 128 rows x 128 B
constexpr int SINGLE_CTA_SMEM_BUDGET = 204800;        // bytes of operand stages per CTA (the rest: barriers, column terms,
                                                      // output boxes)
constexpr int COLVEC = 128;                           // columns one epilogue warp drains per tile, at most
constexpr int OUT_BOX_BYTES = 2048;                   // per epilogue warp: 32 rows x 32 bf16 columns
constexpr int MAX_STAGES = 8;
constexpr int GEMM_THREADS = 320;                    // TMA warp, MMA warp, 8 epilogue warps
constexpr int EPI_WARPS = 8;
constexpr int TMEM_COLS = 512;

struct TcParams {
  int M, N, K, nb0, nb1;
  int m_tiles, n_tiles, k_blocks, num_tiles;
  int block_n, block_k, num_stages, stage_bytes;
  int a_mn, b_mn;
  int b_static;                        // the B operand does not depend on the preceding kernel: prefetch its first tiles
  int c_tma;                           // bf16 output written with tiled stores (a tensor map of C was built)
  uint32_t idesc;
  Epilogue epi;
  int* status;
  unsigned long long wait_ns;          // limit of each wait on an mbarrier
};

__device__ __forceinline__ void fail(const TcParams& p, int code, volatile int* abort_flag) {
  atomicCAS(p.status, 0, code);
  *abort_flag = 1;
}

struct TileCoord { int m0, n0, b0, b1; };
__device__ __forceinline__ TileCoord decode_tile(const TcParams& p, int tile) {
  TileCoord t;
  const int per_batch = p.m_tiles * p.n_tiles;
  const int z = tile / per_batch, r = tile - z * per_batch;
  t.n0 = (r / p.m_tiles) * p.block_n;      // consecutive tiles walk down one column block
  t.m0 = (r % p.m_tiles) * BLOCK_M;
  t.b0 = z % p.nb0;
  t.b1 = z / p.nb0;
  return t;
}

// ------------------------------------------------------------------ epilogue of 32 columns of one row: ragged
// or unaligned edges (element-wise bounds checks, run-time terms)
template <int KIND>
__device__ __forceinline__ void epilogue_chunk(const TcParams& p, const uint32_t* r, float alpha, long long row_off,
                                               int row, int col0, bool row_ok, bool vec_ok) {
  const Epilogue& e = p.epi;
  if (!row_ok) return;
  const int ncol = min(32, p.N - col0);
  if (ncol <= 0) return;
  if (e.out_kind == OUT_I32) {
    int* out = reinterpret_cast<int*>(e.out) + row_off + col0;
    if (vec_ok && ncol == 32) {
#pragma unroll
      for (int j = 0; j < 32; j += 4)
        *reinterpret_cast<uint4*>(out + j) = make_uint4(r[j], r[j + 1], r[j + 2], r[j + 3]);
    } else {
      _Pragma("unroll") for (int j = 0; j < 32; ++j) if (j < ncol) out[j] = (int)r[j];
    }
    return;
  }
  float v[32];
  const float rb = e.row_bias ? e.row_bias[row] : 0.f;
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    const int n = min(col0 + j, p.N - 1);
    const float acc = (KIND == 1) ? (float)(int)r[j] : __uint_as_float(r[j]);
    const float sc = e.col_scale ? alpha * e.col_scale[n] : alpha;
    v[j] = acc * sc + (e.col_bias ? e.col_bias[n] : 0.f) + rb;
  }
  const bool full = vec_ok && ncol == 32;
  if (e.residual) {
    if (e.out_kind == OUT_BF16) {
      const bf16* res = reinterpret_cast<const bf16*>(e.residual) + row_off + col0;
      if (full) {
#pragma unroll
        for (int j = 0; j < 32; j += 8) {
          const uint4 u = *reinterpret_cast<const uint4*>(res + j);
          const bf16* h = reinterpret_cast<const bf16*>(&u);
#pragma unroll
          for (int t = 0; t < 8; ++t) v[j + t] += __bfloat162float(h[t]);
        }
      } else {
        _Pragma("unroll") for (int j = 0; j < 32; ++j) if (j < ncol) v[j] += __bfloat162float(res[j]);
      }
    } else {
      const float* res = reinterpret_cast<const float*>(e.residual) + row_off + col0;
      _Pragma("unroll") for (int j = 0; j < 32; ++j) if (j < ncol) v[j] += res[j];
    }
  }
  if (e.act == 1) {
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = gelu_erf(v[j]);
  }
  if (e.out_kind == OUT_BF16) {
    bf16* out = reinterpret_cast<bf16*>(e.out) + row_off + col0;
    if (full) {
#pragma unroll
      for (int j = 0; j < 32; j += 8) {
        uint4 u;
        __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&u);
#pragma unroll
        for (int t = 0; t < 4; ++t) h[t] = __floats2bfloat162_rn(v[j + 2 * t], v[j + 2 * t + 1]);
        *reinterpret_cast<uint4*>(out + j) = u;
      }
    } else {
      _Pragma("unroll") for (int j = 0; j < 32; ++j) if (j < ncol) out[j] = __float2bfloat16_rn(v[j]);
    }
  } else {
    float* out = reinterpret_cast<float*>(e.out) + row_off + col0;
    if (full) {
#pragma unroll
      for (int j = 0; j < 32; j += 4) *reinterpret_cast<float4*>(out + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
    } else {
      _Pragma("unroll") for (int j = 0; j < 32; ++j) if (j < ncol) out[j] = v[j];
    }
  }
}

// ------------------------------------------------------------------ epilogue of whole 32-column chunks
// One warp drains its 32 accumulator rows (TMEM lane = row = lane of the warp) over a range of columns in
// chunks of 32: tcgen05.ld gives every lane 32 consecutive columns of its row and the lane applies the
// epilogue.  fp32 / int32 rows (128 contiguous bytes per lane) and bf16 rows without a tensor map of C are written
// with 32-byte vector stores that fill whole sectors; bf16 rows otherwise go through the warp's shared-memory box
// and a tiled store (StoreCtx).  The load of chunk c + 1 and the fetch of its residual are in flight while chunk c
// is processed.
__device__ __forceinline__ void ldg256(const void* p, uint32_t* r) {
  asm volatile("ld.global.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "l"(p));
}
__device__ __forceinline__ void stg256(void* p, const uint32_t* r) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "r"(r[0]), "r"(r[1]), "r"(r[2]),
               "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
               : "memory");
}

// Where one epilogue warp's bf16 chunks go.  map == nullptr: st.global from registers.  Otherwise every lane writes
// its 64 bytes into the warp's shared-memory box (32 rows x 64 bytes, 64-byte swizzle: 16-byte piece j of row r sits at
// piece j ^ ((r >> 1) & 3), so a quarter-warp's 16-byte stores cover all banks) and lane 0 issues one tiled store of the
// box; rows and columns outside C are clipped by the store.  The global stores of a lane-per-row layout touch 32
// lines per instruction and hold up the memory pipe that the MMA and TMA warps issue through; the tiled store does not.
struct StoreCtx {
  const CUtensorMap* map;
  uint32_t box;               // shared address of the warp's box (1024-byte aligned)
  int row0, b0, b1;           // C row of lane 0, batch coordinates
  int lane;
};

// MODE >= 0: bit 0 column scale, bit 1 column bias, bit 2 residual, bit 3 GELU, known at compile time;
// MODE < 0: the same four read from the Epilogue at run time.
template <int MODE> struct EpiFlags {
  bool scale, bias, res, act;
  __device__ __forceinline__ explicit EpiFlags(const Epilogue& e)
      : scale(MODE >= 0 ? (MODE & 1) != 0 : e.col_scale != nullptr), bias(MODE >= 0 ? (MODE & 2) != 0 : e.col_bias != nullptr),
        res(MODE >= 0 ? (MODE & 4) != 0 : e.residual != nullptr), act(MODE >= 0 ? (MODE & 8) != 0 : e.act == 1) {}
};

// Residual of one chunk of a bf16 output row: 32 values = 64 bytes.
__device__ __forceinline__ void fetch_res_bf16(const Epilogue& e, long long off, bool row_ok, uint32_t* res) {
  if (row_ok) {
    const bf16* src = reinterpret_cast<const bf16*>(e.residual) + off;
    ldg256(src, res);
    ldg256(src + 16, res + 8);
  }
}

// acc[32] of one row -> out[off .. off + 32).  `cv` = the chunk's column terms in shared memory: cv[j] = alpha *
// col_scale of column j of the chunk, cv[COLVEC + j] = its col_bias (staged by the warp before it waited for the
// accumulator; every lane reads the same address, one broadcast per load).
template <int KIND, int OUT, int MODE>
__device__ __forceinline__ void finish_chunk(const Epilogue& e, const uint32_t* r, const uint32_t* res, float alpha, float rb,
                                             const float* cv, long long off, bool row_ok, const StoreCtx& sx, int n) {
  if (OUT == OUT_I32) {
    if (row_ok) {
      int* out = reinterpret_cast<int*>(e.out) + off;
#pragma unroll
      for (int j = 0; j < 32; j += 8) stg256(out + j, r + j);
    }
    return;
  }
  const EpiFlags<MODE> f(e);
  float v[32];
#pragma unroll
  for (int j = 0; j < 32; j += 4) {
    float4 sc = make_float4(alpha, alpha, alpha, alpha), bi = make_float4(rb, rb, rb, rb);
    if (f.scale) sc = *reinterpret_cast<const float4*>(cv + j);
    if (f.bias) {
      const float4 t = *reinterpret_cast<const float4*>(cv + COLVEC + j);
      bi.x += t.x; bi.y += t.y; bi.z += t.z; bi.w += t.w;
    }
    const float a0 = (KIND == 1) ? (float)(int)r[j] : __uint_as_float(r[j]);
    const float a1 = (KIND == 1) ? (float)(int)r[j + 1] : __uint_as_float(r[j + 1]);
    const float a2 = (KIND == 1) ? (float)(int)r[j + 2] : __uint_as_float(r[j + 2]);
    const float a3 = (KIND == 1) ? (float)(int)r[j + 3] : __uint_as_float(r[j + 3]);
    v[j] = a0 * sc.x + bi.x; v[j + 1] = a1 * sc.y + bi.y; v[j + 2] = a2 * sc.z + bi.z; v[j + 3] = a3 * sc.w + bi.w;
  }
  if (OUT == OUT_BF16) {
    if (f.res) {
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const float2 t = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&res[j]));
        v[2 * j] += t.x;
        v[2 * j + 1] += t.y;
      }
    }
    if (f.act) {
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] = gelu_erf(v[j]);
    }
    uint32_t o[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * j], v[2 * j + 1]);
      o[j] = *reinterpret_cast<const uint32_t*>(&h);
    }
    if (sx.map) {
      if (sx.lane == 0) tma_store_wait_read<0>();          // the box's previous store has read it
      __syncwarp();
      const uint32_t row_addr = sx.box + (uint32_t)sx.lane * 64u, sw = ((uint32_t)sx.lane >> 1) & 3u;
#pragma unroll
      for (uint32_t j = 0; j < 4; ++j) sts128(row_addr + ((j ^ sw) << 4), o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
      fence_async_shared();
      __syncwarp();
      if (sx.lane == 0) {
        tma_store_4d(sx.map, sx.box, n, sx.row0, sx.b0, sx.b1);
        tma_store_commit();
      }
    } else if (row_ok) {
      bf16* out = reinterpret_cast<bf16*>(e.out) + off;
      stg256(out, o);
      stg256(out + 16, o + 8);
    }
  } else {
    if (f.res && row_ok) {
      const float* src = reinterpret_cast<const float*>(e.residual) + off;
#pragma unroll
      for (int j = 0; j < 32; j += 8) {
        uint32_t t[8];
        ldg256(src + j, t);
#pragma unroll
        for (int k = 0; k < 8; ++k) v[j + k] += __uint_as_float(t[k]);
      }
    }
    if (f.act) {
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] = gelu_erf(v[j]);
    }
    if (row_ok) {
      float* out = reinterpret_cast<float*>(e.out) + off;
#pragma unroll
      for (int j = 0; j < 32; j += 8) {
        uint32_t t[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) t[k] = __float_as_uint(v[j + k]);
        stg256(out + j, t);
      }
    }
  }
}

// `nchunks` whole chunks starting at accumulator column c0 (tile-relative) = global column n; `cv` = column terms of
// the first.
// `res0` holds the residual of the first chunk (bf16 output with residual only), fetched by the caller
// before it waited for the accumulator.
template <int KIND, int OUT, int MODE>
__device__ __forceinline__ void drain_chunks(const Epilogue& e, uint32_t taddr, int nchunks, float alpha, float rb,
                                             const float* cv, long long off, bool row_ok, uint32_t* res0, const StoreCtx& sx,
                                             int n) {
  const bool pipelined_res = OUT == OUT_BF16 && EpiFlags<MODE>(e).res;
  uint32_t ra[32], rb2[32], res1[16];
  tmem_ld32_issue(taddr, ra);
  for (int c = 0; c < nchunks; c += 2) {
    tmem_ld_wait();
    tmem_ld_pin(ra);
    const bool more1 = c + 1 < nchunks;
    if (more1) {
      tmem_ld32_issue(taddr + 32u * (uint32_t)(c + 1), rb2);
      if (pipelined_res) fetch_res_bf16(e, off + 32 * (c + 1), row_ok, res1);
    }
    finish_chunk<KIND, OUT, MODE>(e, ra, res0, alpha, rb, cv + 32 * c, off + 32 * c, row_ok, sx, n + 32 * c);
    if (more1) {
      tmem_ld_wait();
      tmem_ld_pin(rb2);
      if (c + 2 < nchunks) {
        tmem_ld32_issue(taddr + 32u * (uint32_t)(c + 2), ra);
        if (pipelined_res) fetch_res_bf16(e, off + 32 * (c + 2), row_ok, res0);
      }
      finish_chunk<KIND, OUT, MODE>(e, rb2, res1, alpha, rb, cv + 32 * (c + 1), off + 32 * (c + 1), row_ok, sx, n + 32 * (c + 1));
    }
  }
}

// One warp stages the column terms of its `ncols` (<= COLVEC) columns from global column n on: 4 per lane, alpha
// folded into the scale.  Columns at or beyond N are left alone (no whole chunk reaches them).
template <int MODE>
__device__ __forceinline__ void stage_col_terms(const Epilogue& e, float* cv, float alpha, int n, int ncols, int N, int lane) {
  const EpiFlags<MODE> f(e);
  if (!f.scale && !f.bias) return;
  __syncwarp();                                   // the previous tile's reads of cv are done
  const int c = 4 * lane;
  if (c < ncols && n + c + 3 < N) {
    if (f.scale) {
      float4 t = __ldg(reinterpret_cast<const float4*>(e.col_scale + n + c));
      t.x *= alpha; t.y *= alpha; t.z *= alpha; t.w *= alpha;
      *reinterpret_cast<float4*>(cv + c) = t;
    }
    if (f.bias) *reinterpret_cast<float4*>(cv + COLVEC + c) = __ldg(reinterpret_cast<const float4*>(e.col_bias + n + c));
  }
  __syncwarp();
}

// MODE >= 0: bf16 output (fp32 with bit 4) with the epilogue terms of MODE; MODE < 0: output kind and terms read
// at run time.
template <int KIND, int MODE>
__device__ __forceinline__ void drain_dispatch(const Epilogue& e, uint32_t taddr, int nchunks, float alpha, float rb,
                                               const float* cv, long long off, bool row_ok, uint32_t* res0,
                                               const StoreCtx& sx, int n) {
  if (MODE >= 16) {
    drain_chunks<KIND, OUT_F32, MODE>(e, taddr, nchunks, alpha, rb, cv, off, row_ok, res0, sx, n);
  } else if (MODE >= 0 || e.out_kind == OUT_BF16) {
    drain_chunks<KIND, OUT_BF16, MODE>(e, taddr, nchunks, alpha, rb, cv, off, row_ok, res0, sx, n);
  } else if (e.out_kind == OUT_F32) {
    drain_chunks<KIND, OUT_F32, -1>(e, taddr, nchunks, alpha, rb, cv, off, row_ok, res0, sx, n);
  } else {
    drain_chunks<KIND, OUT_I32, 0>(e, taddr, nchunks, alpha, rb, cv, off, row_ok, res0, sx, n);
  }
}

// The epilogue variant a launch takes: bf16 outputs with one of the term sets the encoder uses, and plain fp32
// outputs (the weight gradients), get a kernel compiled for exactly those terms (bit 0 column scale, bit 1
// column bias, bit 2 residual, bit 3 GELU, bit 4 fp32 output; alpha and the row bias are always applied);
// everything else runs the variant that reads them at run time (-1).
inline int epilogue_mode(int kind, const Epilogue& e) {
  const int mode = (e.col_scale ? 1 : 0) | (e.col_bias ? 2 : 0) | (e.residual ? 4 : 0) | (e.act == 1 ? 8 : 0);
  if (e.out_kind == OUT_F32) return (kind == 0 && mode == 0) ? 16 : -1;
  if (e.out_kind != OUT_BF16) return -1;
  if (kind == 0) return (mode == 0 || mode == 2 || mode == 6 || mode == 10) ? mode : -1;
  return (mode == 3 || mode == 7) ? mode : -1;
}

// True when rows of out (and residual) start on 32-byte boundaries for every row, batch and 32-column chunk,
// and the column vectors can be fetched as float4.
__device__ __forceinline__ bool direct_epilogue_ok(const Epilogue& e) {
  const int per32 = e.out_kind == OUT_BF16 ? 16 : 8;
  bool ok = (e.ldc % per32 == 0) && (e.c_b0 % per32 == 0) && (e.c_b1 % per32 == 0) && ((reinterpret_cast<uintptr_t>(e.out) & 31) == 0);
  if (e.residual) ok = ok && ((reinterpret_cast<uintptr_t>(e.residual) & 31) == 0);
  return ok && ((reinterpret_cast<uintptr_t>(e.col_scale) & 15) == 0) && ((reinterpret_cast<uintptr_t>(e.col_bias) & 15) == 0);
}

}  // namespace tc
}  // namespace mrem
