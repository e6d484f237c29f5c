// Tensor-core GEMM for sm_100a: C[b][m][n] = epilogue( sum_k A[b][m][k] * B[b][n][k] ).
//
// One persistent CTA per SM.  Warp 0 streams operand tiles into a ring of shared-memory
// stages with TMA (128-byte swizzle), warp 1 issues tcgen05.mma (bf16 -> fp32, or
// int8 -> int32 with exact accumulation) into one of two TMEM accumulator buffers, and
// warps 2..9 drain the other buffer with tcgen05.ld, apply the epilogue (column scale and
// bias staged in shared memory before the accumulator is ready) and write their rows: bf16
// through a 2 KB shared-memory box per warp and tiled stores, anything else straight from
// registers with 32-byte vector stores.  The epilogue of tile i overlaps the main loop of
// tile i+1.
// Either operand may be stored k-contiguous ("K-major") or m/n-contiguous ("MN-major");
// the second form serves the backward products (dX = dY * W_hat, dW = dY^T * X_hat) and
// the attention products without any transposed copy.
//
// Every wait on an mbarrier is bounded in time; when one runs out the kernel records a
// code in the status word, stops issuing work, frees its TMEM and returns.
#include <cuda.h>

#include <cstdio>

#include "gemm_epi.cuh"

namespace mrem {

using namespace tc;

namespace {

// ------------------------------------------------------------------ the kernel
template <int KIND, int MODE>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_c, const __grid_constant__ TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t empty_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t tfull_bar[2];
  __shared__ __align__(8) uint64_t tempty_bar[2];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  __shared__ __align__(16) float col_terms[EPI_WARPS][2 * COLVEC];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  pdl_trigger();

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.num_stages; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(smem_u32(&tfull_bar[a]), 1);
      mbar_init(smem_u32(&tempty_bar[a]), EPI_WARPS);
    }
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // A B operand that the preceding kernel does not write (weights): the producer fetches the B tiles of its first
  // stages now, while that kernel is still finishing; the matching A tiles follow after the wait.
  int prefetched = 0;
  if (threadIdx.x == 0 && p.b_static && (int)blockIdx.x < p.num_tiles) {
    const TileCoord t = decode_tile(p, blockIdx.x);
    prefetched = p.k_blocks < p.num_stages ? p.k_blocks : p.num_stages;
    for (int kb = 0; kb < prefetched; ++kb) {
      const uint32_t bar = smem_u32(&full_bar[kb]);
      const uint32_t sb = tiles_base + kb * p.stage_bytes + A_STAGE_BYTES;
      mbar_expect_tx(bar, (uint32_t)p.stage_bytes);
      const int k0 = kb * p.block_k;
      if (!p.b_mn) {
        tma_load_4d(sb, &map_b, bar, k0, t.n0, t.b0, t.b1);
      } else if (p.b_mn == 2) {
        tma_load_5d(sb, &map_b, bar, 0, k0, t.n0 >> 6, t.b0, t.b1);
      } else {
        for (int j = 0; j < p.block_n / 64; ++j) tma_load_4d(sb + j * 8192, &map_b, bar, t.n0 + 64 * j, k0, t.b0, t.b1);
      }
    }
  }
  pdl_wait();                            // set-up done; from here on the predecessor's results are needed
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&tmem_slot);
  volatile int* vabort = &abort_flag;

  if (warp == 0) {
    // ---------------- TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x) {
        const TileCoord t = decode_tile(p, tile);
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!mbar_wait_or_abort(smem_u32(&empty_bar[stage]), phase ^ 1u, vabort, p.wait_ns)) {
            if (!*vabort) fail(p, DEV_TIMEOUT_MMA, vabort);
            ok = false;
            break;
          }
          const uint32_t bar = smem_u32(&full_bar[stage]);
          const uint32_t sa = tiles_base + stage * p.stage_bytes, sb = sa + A_STAGE_BYTES;
          const bool b_done = tile == (int)blockIdx.x && kb < prefetched;     // fetched (and announced) before the wait
          if (!b_done) mbar_expect_tx(bar, (uint32_t)p.stage_bytes);
          const int k0 = kb * p.block_k;
          if (!p.a_mn) {
            tma_load_4d(sa, &map_a, bar, k0, t.m0, t.b0, t.b1);
          } else if (p.a_mn == 2) {
            tma_load_5d(sa, &map_a, bar, 0, k0, t.m0 >> 6, t.b0, t.b1);
          } else {
            for (int j = 0; j < BLOCK_M / 64; ++j) tma_load_4d(sa + j * 8192, &map_a, bar, t.m0 + 64 * j, k0, t.b0, t.b1);
          }
          if (b_done) {
          } else if (!p.b_mn) {
            tma_load_4d(sb, &map_b, bar, k0, t.n0, t.b0, t.b1);
          } else if (p.b_mn == 2) {
            tma_load_5d(sb, &map_b, bar, 0, k0, t.n0 >> 6, t.b0, t.b1);
          } else {
            for (int j = 0; j < p.block_n / 64; ++j) tma_load_4d(sb + j * 8192, &map_b, bar, t.n0 + 64 * j, k0, t.b0, t.b1);
          }
          if (++stage == p.num_stages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // let the copies already in flight land before the CTA may exit
        for (int s = 0; s < p.num_stages; ++s) {
          const unsigned long long t0 = global_ns();
          while (global_ns() - t0 < 1000000ull) { }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer
    if (lane == 0) {
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      // descriptor words: high word fixed (stride between 8-row groups, version, 128-byte swizzle); low word =
      // address >> 4 plus the leading-dimension offset field, advanced per 16-deep step and per stage
      const uint32_t adv_a = (p.a_mn ? 2048u : 32u) >> 4, adv_b = (p.b_mn ? 2048u : 32u) >> 4;
      const uint64_t proto_a = smem_desc(tiles_base, p.a_mn ? 8192u : 16u, 1024u);
      const uint64_t proto_b = smem_desc(tiles_base + A_STAGE_BYTES, p.b_mn ? 8192u : 16u, 1024u);
      const uint32_t a_hi = (uint32_t)(proto_a >> 32), b_hi = (uint32_t)(proto_b >> 32);
      const uint32_t a_lo0 = (uint32_t)proto_a, b_lo0 = (uint32_t)proto_b, stage_adv = (uint32_t)p.stage_bytes >> 4;
      uint32_t a_lo = a_lo0, b_lo = b_lo0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x) {
        if (!mbar_wait_or_abort(smem_u32(&tempty_bar[acc]), acc_phase ^ 1u, vabort, p.wait_ns)) {
          if (!*vabort) fail(p, DEV_TIMEOUT_EPI, vabort);
          break;
        }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + (uint32_t)(acc * p.block_n);
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!mbar_wait_or_abort(smem_u32(&full_bar[stage]), phase, vabort, p.wait_ns)) {
            if (!*vabort) fail(p, DEV_TIMEOUT_TMA, vabort);
            ok = false;
            break;
          }
          tc_fence_after();
          tc_mma_lohi<KIND>(tmem_d, a_lo, a_hi, b_lo, b_hi, p.idesc, (uint32_t)(kb != 0));
          tc_mma_lohi<KIND>(tmem_d, a_lo + adv_a, a_hi, b_lo + adv_b, b_hi, p.idesc, 1u);
          tc_mma_lohi<KIND>(tmem_d, a_lo + 2 * adv_a, a_hi, b_lo + 2 * adv_b, b_hi, p.idesc, 1u);
          tc_mma_lohi<KIND>(tmem_d, a_lo + 3 * adv_a, a_hi, b_lo + 3 * adv_b, b_hi, p.idesc, 1u);
          tc_commit(smem_u32(&empty_bar[stage]));
          a_lo += stage_adv; b_lo += stage_adv;
          if (++stage == p.num_stages) { stage = 0; phase ^= 1u; a_lo = a_lo0; b_lo = b_lo0; }
        }
        if (!ok) break;
        tc_commit(smem_u32(&tfull_bar[acc]));
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
    }
  } else {
    // ---------------- epilogue warps: TMEM lane quadrant = warp % 4, two warps per quadrant, each draining
    // its 32 rows over one half of the tile's columns
    const int quad = warp & 3, half = (warp - 2) >> 2;
    const Epilogue& e = p.epi;
    float alpha = e.alpha_const;
    if (e.alpha_p0) alpha *= *e.alpha_p0;
    if (e.alpha_p1) alpha *= *e.alpha_p1;
    const bool direct = direct_epilogue_ok(e);
    const bool res_bf16 = e.residual != nullptr && e.out_kind == OUT_BF16;
    const int cols_per_warp = p.block_n >> 1, c_begin = half * cols_per_warp;
    // bf16 rows leave through this warp's shared-memory box (behind the operand stages) and tiled stores
    const bool boxed = direct && p.c_tma;
    StoreCtx sx{boxed ? &map_c : nullptr, tiles_base + (uint32_t)(p.num_stages * p.stage_bytes) + (uint32_t)((warp - 2) * OUT_BOX_BYTES),
                0, 0, 0, lane};
    int acc = 0;
    uint32_t acc_phase = 0;
    for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x) {
      const TileCoord t = decode_tile(p, tile);
      const int row = t.m0 + quad * 32 + lane, col_begin = t.n0 + c_begin;
      const bool row_ok = row < p.M;
      const long long row_off = (long long)t.b0 * e.c_b0 + (long long)t.b1 * e.c_b1 + (long long)row * e.ldc;
      // whole 32-column chunks of this warp's range that lie inside N take the vector path
      int nfull = 0;
      if (direct && col_begin < p.N) nfull = min((p.N - col_begin) >> 5, cols_per_warp >> 5);
      uint32_t res0[16];
      if (nfull > 0 && res_bf16) fetch_res_bf16(e, row_off + col_begin, row_ok, res0);   // in flight during the wait
      const float rb = (e.row_bias && row_ok) ? e.row_bias[row] : 0.f;
      float* cv = col_terms[warp - 2];
      if (nfull > 0) stage_col_terms<MODE>(e, cv, alpha, col_begin, cols_per_warp, p.N, lane);   // before the wait as well
      // every lane polls; the decision is made warp-uniform before any .sync.aligned instruction
      const bool got = mbar_wait_or_abort(smem_u32(&tfull_bar[acc]), acc_phase, vabort, p.wait_ns);
      if (!__all_sync(0xffffffffu, got)) {
        if (lane == 0 && !*vabort) fail(p, DEV_TIMEOUT_MMA, vabort);
        break;
      }
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * p.block_n);
      sx.row0 = t.m0 + quad * 32; sx.b0 = t.b0; sx.b1 = t.b1;
      if (nfull > 0) drain_dispatch<KIND, MODE>(e, taddr + (uint32_t)c_begin, nfull, alpha, rb, cv, row_off + col_begin, row_ok, res0, sx, col_begin);
      for (int c = c_begin + 32 * nfull; c < c_begin + cols_per_warp && t.n0 + c < p.N; c += 32) {   // ragged or unaligned rest
        uint32_t r[32];
        tmem_ld32(taddr + (uint32_t)c, r);
        epilogue_chunk<KIND>(p, r, alpha, row_off, row, t.n0 + c, row_ok, false);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&tempty_bar[acc]));
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
    if (boxed && lane == 0) tma_store_wait_all();          // the boxes are read and written out before the CTA ends
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

// One thread waits, with the library's bounded wait, on an mbarrier that nothing ever arrives at; when the limit runs
// out it reports through the same status word and code as a product whose operand tile never landed, and returns.
__global__ void wait_probe_kernel(int* status, unsigned long long limit_ns) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0 && !mbar_wait_or_abort(smem_u32(&bar), 0u, &abort_flag, limit_ns)) atomicCAS(status, 0, (int)DEV_TIMEOUT_TMA);
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

}  // namespace

// Tensor map of one operand: 4-D (contiguous index, strided index, batch0, batch1).
int make_operand_map(CUtensorMap* map, const OperandDesc& op, int elem_bytes, int mn_extent, int K, int nb0, int nb1,
             int tile_mn, int block_k, int* chunked) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return GEMM_ERR_CUDA;
  if (chunked) *chunked = 0;
  if (chunked && op.mn_contig && elem_bytes == 2 && mn_extent % 64 == 0 && tile_mn % 64 == 0) {
    // (64 contiguous, k rows, chunk of 64, batch0, batch1): one box = every 64-wide piece of the tile, piece after piece
    const cuuint64_t s1 = (cuuint64_t)op.ld * 2, rows = (cuuint64_t)K;
    const cuuint64_t s3 = nb0 > 1 ? (cuuint64_t)op.s_b0 * 2 : s1 * rows;
    const cuuint64_t s4 = nb1 > 1 ? (cuuint64_t)op.s_b1 * 2 : s3 * (cuuint64_t)nb0;
    if ((reinterpret_cast<uintptr_t>(op.ptr) & 15) || (s1 & 15) || (s3 & 15) || (s4 & 15)) return GEMM_ERR_ALIGN;
    if (s1 < (cuuint64_t)mn_extent * 2) return GEMM_ERR_ARG;
    cuuint64_t dims[5] = {64, rows, (cuuint64_t)(mn_extent / 64), (cuuint64_t)nb0, (cuuint64_t)nb1};
    cuuint64_t strides[4] = {s1, 128, s3, s4};
    cuuint32_t box[5] = {64, (cuuint32_t)block_k, (cuuint32_t)(tile_mn / 64), 1, 1};
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(op.ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return GEMM_ERR_CUDA;
    *chunked = 1;
    return GEMM_OK;
  }
  const cuuint64_t inner = op.mn_contig ? (cuuint64_t)mn_extent : (cuuint64_t)K;
  const cuuint64_t rows = op.mn_contig ? (cuuint64_t)K : (cuuint64_t)mn_extent;
  cuuint64_t dims[4] = {inner, rows, (cuuint64_t)nb0, (cuuint64_t)nb1};
  cuuint64_t s1 = (cuuint64_t)op.ld * elem_bytes;
  cuuint64_t s2 = nb0 > 1 ? (cuuint64_t)op.s_b0 * elem_bytes : s1 * rows;
  cuuint64_t s3 = nb1 > 1 ? (cuuint64_t)op.s_b1 * elem_bytes : s2 * (cuuint64_t)nb0;
  if ((reinterpret_cast<uintptr_t>(op.ptr) & 15) || (s1 & 15) || (s2 & 15) || (s3 & 15)) return GEMM_ERR_ALIGN;
  if (s1 < inner * elem_bytes) return GEMM_ERR_ARG;
  cuuint64_t strides[3] = {s1, s2, s3};
  cuuint32_t box[4];
  if (op.mn_contig) {
    box[0] = 128 / elem_bytes;
    box[1] = (cuuint32_t)block_k;
  } else {
    box[0] = (cuuint32_t)block_k;
    box[1] = (cuuint32_t)tile_mn;
  }
  box[2] = box[3] = 1;
  cuuint32_t estr[4] = {1, 1, 1, 1};
  const CUtensorMapDataType dt = elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8;
  CUresult r = fn(map, dt, 4, const_cast<void*>(op.ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? GEMM_OK : GEMM_ERR_CUDA;
}

namespace {

// Tile width by a cost model fitted to event timings on the encoder shapes: a persistent CTA works through
// `waves` tiles one after the other, a tile costs k_blocks main-loop steps plus an epilogue share that is
// not hidden.  A step of a narrow tile is cheaper, but far from proportionally (the A tile is re-fetched
// for every column block and the shared-memory traffic per flop grows), so wide tiles win unless they
// leave most SMs idle.
int pick_block_n(int M, int N, int k_blocks, int batches, int sm_count) {
  const int m_tiles = (M + BLOCK_M - 1) / BLOCK_M;
  int best = 64;
  double best_cost = 1e30;
  for (int bn = 64; bn <= 256; bn *= 2) {
    if (bn > 64 && bn / 2 >= N) break;
    const long long tiles = (long long)m_tiles * ((N + bn - 1) / bn) * batches;
    const long long waves = (tiles + sm_count - 1) / sm_count;
    const double step_us = bn == 64 ? 0.32 : (bn == 128 ? 0.43 : 0.50);
    const double epi_us = bn == 64 ? 0.5 : (bn == 128 ? 1.0 : 2.0);
    const double cost = (double)waves * (k_blocks * step_us + epi_us);
    if (cost < best_cost - 1e-9) { best_cost = cost; best = bn; }
  }
  return best;
}

}  // namespace

int tc_gemm(int kind, int a_unsigned, const OperandDesc& A, const OperandDesc& B, const GemmShape& g,
            const Epilogue& epi, int block_n, int* d_status, int sm_count, cudaStream_t stream) {
  if (g.M <= 0 || g.N <= 0 || g.K <= 0 || g.nb0 <= 0 || g.nb1 <= 0) return GEMM_ERR_ARG;
  const int es = kind == 0 ? 2 : 1;
  if (kind == 1 && (A.mn_contig || B.mn_contig)) return GEMM_ERR_ARG;
  TcParams p;
  p.M = g.M; p.N = g.N; p.K = g.K; p.nb0 = g.nb0; p.nb1 = g.nb1;
  p.block_n = block_n > 0 ? block_n : pick_block_n(g.M, g.N, (g.K + 128 / es - 1) / (128 / es), g.nb0 * g.nb1, sm_count);
  if (p.block_n != 64 && p.block_n != 128 && p.block_n != 256) return GEMM_ERR_ARG;
  p.block_k = 128 / es;
  p.m_tiles = (g.M + BLOCK_M - 1) / BLOCK_M;
  p.n_tiles = (g.N + p.block_n - 1) / p.block_n;
  p.k_blocks = (g.K + p.block_k - 1) / p.block_k;
  p.num_tiles = p.m_tiles * p.n_tiles * g.nb0 * g.nb1;
  p.stage_bytes = A_STAGE_BYTES + p.block_n * 128;
  p.num_stages = SINGLE_CTA_SMEM_BUDGET / p.stage_bytes;
  if (p.num_stages > MAX_STAGES) p.num_stages = MAX_STAGES;
  p.a_mn = A.mn_contig; p.b_mn = B.mn_contig;
  p.b_static = B.is_static;
  p.epi = epi;
  p.status = d_status;
  p.wait_ns = g_wait_limit_ns;
  // instruction descriptor: D format, A/B formats, majors, N >> 3, M >> 4
  uint32_t idesc = 0;
  if (kind == 0) {
    idesc |= 1u << 4;                          // fp32 accumulate
    idesc |= 1u << 7;                          // A = bf16
    idesc |= 1u << 10;                         // B = bf16
  } else {
    idesc |= 2u << 4;                          // int32 accumulate
    idesc |= (a_unsigned ? 0u : 1u) << 7;      // A = u8 / s8
    idesc |= 1u << 10;                         // B = s8
  }
  idesc |= (uint32_t)(A.mn_contig ? 1 : 0) << 15;
  idesc |= (uint32_t)(B.mn_contig ? 1 : 0) << 16;
  idesc |= (uint32_t)(p.block_n >> 3) << 17;
  idesc |= (uint32_t)(BLOCK_M >> 4) << 24;
  p.idesc = idesc;

  CUtensorMap ma, mb;
  int a_chunked = 0, b_chunked = 0;           // MN-major operands: one 5-D load per stage where the extent allows it
  int rc = make_operand_map(&ma, A, es, g.M, g.K, g.nb0, g.nb1, BLOCK_M, p.block_k, &a_chunked);
  if (rc != GEMM_OK) return rc;
  rc = make_operand_map(&mb, B, es, g.N, g.K, g.nb0, g.nb1, p.block_n, p.block_k, &b_chunked);
  if (rc != GEMM_OK) return rc;
  if (a_chunked) p.a_mn = 2;
  if (b_chunked) p.b_mn = 2;
  // bf16 output whose rows and batches start on 16-byte boundaries: tiled stores of 32 x 32 boxes
  CUtensorMap mc = ma;
  p.c_tma = 0;
  if (epi.out_kind == OUT_BF16 && (reinterpret_cast<uintptr_t>(epi.out) & 15) == 0 && epi.ldc % 8 == 0 && epi.ldc >= g.N &&
      (g.nb0 == 1 || epi.c_b0 % 8 == 0) && (g.nb1 == 1 || epi.c_b1 % 8 == 0)) {
    const cuuint64_t s1 = (cuuint64_t)epi.ldc * 2;
    const cuuint64_t s2 = g.nb0 > 1 ? (cuuint64_t)epi.c_b0 * 2 : s1 * (cuuint64_t)g.M;
    const cuuint64_t s3 = g.nb1 > 1 ? (cuuint64_t)epi.c_b1 * 2 : s2 * (cuuint64_t)g.nb0;
    cuuint64_t dims[4] = {(cuuint64_t)g.N, (cuuint64_t)g.M, (cuuint64_t)g.nb0, (cuuint64_t)g.nb1};
    cuuint64_t strides[3] = {s1, s2, s3};
    cuuint32_t box[4] = {32, 32, 1, 1}, estr[4] = {1, 1, 1, 1};
    EncodeTiledFn fn = encode_fn();
    if (fn && fn(&mc, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, epi.out, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                 CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS)
      p.c_tma = 1;
  }

  const int smem = p.num_stages * p.stage_bytes + 1024 + EPI_WARPS * OUT_BOX_BYTES;
  typedef void (*Kern)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const TcParams);
  static const struct { int kind, mode; Kern fn; } variants[] = {
      {0, -1, tc_gemm_kernel<0, -1>}, {0, 0, tc_gemm_kernel<0, 0>}, {0, 2, tc_gemm_kernel<0, 2>}, {0, 6, tc_gemm_kernel<0, 6>},
      {0, 10, tc_gemm_kernel<0, 10>}, {0, 16, tc_gemm_kernel<0, 16>}, {1, -1, tc_gemm_kernel<1, -1>}, {1, 3, tc_gemm_kernel<1, 3>}, {1, 7, tc_gemm_kernel<1, 7>}};
  constexpr int n_variants = sizeof(variants) / sizeof(variants[0]);
  static bool attr_set[n_variants] = {};
  const int mode = epilogue_mode(kind, epi);
  int vi = 0;
  while (vi < n_variants && !(variants[vi].kind == kind && variants[vi].mode == mode)) ++vi;
  if (vi == n_variants) return GEMM_ERR_ARG;
  Kern kern = variants[vi].fn;
  if (!attr_set[vi]) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SINGLE_CTA_SMEM_BUDGET + 1024 + EPI_WARPS * OUT_BOX_BYTES) != cudaSuccess)
      return GEMM_ERR_CUDA;
    attr_set[vi] = true;
  }
  const int grid = p.num_tiles < sm_count ? p.num_tiles : sm_count;
  Scope sc([&] {
    char buf[40];
    snprintf(buf, sizeof(buf), "%s %dx%dx%d%s%s b%d", kind == 0 ? "gemm_bf16" : "gemm_i8", g.M, g.N, g.K,
             A.mn_contig ? "T" : "N", B.mn_contig ? "N" : "T", g.nb0 * g.nb1);
    return std::string(buf);
  }, 2.0 * g.M * g.N * (double)g.K * g.nb0 * g.nb1, 1, stream, 0);
  if (launch_k(kern, grid, GEMM_THREADS, smem, stream, ma, mb, mc, p) != cudaSuccess) return GEMM_ERR_CUDA;
  return cudaGetLastError() == cudaSuccess ? GEMM_OK : GEMM_ERR_CUDA;
}

cudaError_t launch_wait_probe(int* d_status, unsigned long long limit_ns, cudaStream_t stream) {
  return launch_k(wait_probe_kernel, 1, 32, 0, stream, d_status, limit_ns);
}

}  // namespace mrem
