// Several bf16 products with fp32 outputs in ONE persistent launch (sm_100a): the four weight-gradient
// products of an encoder layer, dW = alpha * dY^T X_hat (+ row bias), each of which alone fills the
// 148 SMs badly (128, 128, 32 and 96 tiles of 128 x 256) and pays the launch, pipeline fill and drain
// of a kernel of its own.  The tiles of all problems form one list that the CTAs walk round-robin with
// the pipeline of tc_gemm_kernel: warp 0 streams operand tiles by TMA into a ring of shared-memory
// stages, warp 1 issues tcgen05.mma into one of two TMEM accumulators, warps 2..9 drain the other one.
// Every problem brings its own tensor maps, shape, operand layouts and epilogue; the tile width (256)
// and therefore the stage layout are common.  All waits on mbarriers are bounded in time.
#include <cuda.h>

#include <cstdio>

#include "gemm_epi.cuh"

namespace mrem {

using namespace tc;

namespace {

struct GroupParams {
  int n;                              // problems
  int tile_end[MAX_GEMM_GROUP];       // running tile count: problem i owns tiles [tile_end[i-1], tile_end[i])
  int num_stages, stage_bytes;
  TcParams p[MAX_GEMM_GROUP];
};
struct GroupMaps { CUtensorMap a[MAX_GEMM_GROUP], b[MAX_GEMM_GROUP]; };

__device__ __forceinline__ int find_problem(const GroupParams& g, int tile, int& local) {
  int pi = 0;
  while (pi + 1 < g.n && tile >= g.tile_end[pi]) ++pi;
  local = tile - (pi ? g.tile_end[pi - 1] : 0);
  return pi;
}

__global__ void __launch_bounds__(GEMM_THREADS, 1)
tc_gemm_group_kernel(const __grid_constant__ GroupMaps maps, const __grid_constant__ GroupParams g) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t full_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t empty_bar[MAX_STAGES];
  __shared__ __align__(8) uint64_t tfull_bar[2];
  __shared__ __align__(8) uint64_t tempty_bar[2];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int total_tiles = g.tile_end[g.n - 1];
  pdl_trigger();

  if (threadIdx.x == 0) {
    for (int s = 0; s < g.num_stages; ++s) {
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
  pdl_wait();                            // set-up done; from here on the predecessors' results are needed
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&tmem_slot);
  volatile int* vabort = &abort_flag;

  if (warp == 0) {
    // ---------------- TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        int local;
        const int pi = find_problem(g, tile, local);
        const TcParams& p = g.p[pi];
        const CUtensorMap* map_a = &maps.a[pi];
        const CUtensorMap* map_b = &maps.b[pi];
        const TileCoord t = decode_tile(p, local);
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!mbar_wait_or_abort(smem_u32(&empty_bar[stage]), phase ^ 1u, vabort, g.p[0].wait_ns)) {
            if (!*vabort) fail(p, DEV_TIMEOUT_MMA, vabort);
            ok = false;
            break;
          }
          const uint32_t bar = smem_u32(&full_bar[stage]);
          const uint32_t sa = tiles_base + stage * g.stage_bytes, sb = sa + A_STAGE_BYTES;
          mbar_expect_tx(bar, (uint32_t)g.stage_bytes);
          const int k0 = kb * p.block_k;
          if (!p.a_mn) {
            tma_load_4d(sa, map_a, bar, k0, t.m0, t.b0, t.b1);
          } else if (p.a_mn == 2) {
            tma_load_5d(sa, map_a, bar, 0, k0, t.m0 >> 6, t.b0, t.b1);
          } else {
            for (int j = 0; j < BLOCK_M / 64; ++j) tma_load_4d(sa + j * 8192, map_a, bar, t.m0 + 64 * j, k0, t.b0, t.b1);
          }
          if (!p.b_mn) {
            tma_load_4d(sb, map_b, bar, k0, t.n0, t.b0, t.b1);
          } else if (p.b_mn == 2) {
            tma_load_5d(sb, map_b, bar, 0, k0, t.n0 >> 6, t.b0, t.b1);
          } else {
            for (int j = 0; j < p.block_n / 64; ++j) tma_load_4d(sb + j * 8192, map_b, bar, t.n0 + 64 * j, k0, t.b0, t.b1);
          }
          if (++stage == g.num_stages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // let the copies already in flight land before the CTA may exit
        for (int s = 0; s < g.num_stages; ++s) {
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
      const uint32_t stage_adv = (uint32_t)g.stage_bytes >> 4;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        int local;
        const TcParams& p = g.p[find_problem(g, tile, local)];
        // descriptor words of this problem's operand layouts (see tc_gemm_kernel)
        const uint32_t adv_a = (p.a_mn ? 2048u : 32u) >> 4, adv_b = (p.b_mn ? 2048u : 32u) >> 4;
        const uint64_t proto_a = smem_desc(tiles_base, p.a_mn ? 8192u : 16u, 1024u);
        const uint64_t proto_b = smem_desc(tiles_base + A_STAGE_BYTES, p.b_mn ? 8192u : 16u, 1024u);
        const uint32_t a_hi = (uint32_t)(proto_a >> 32), b_hi = (uint32_t)(proto_b >> 32);
        const uint32_t a_lo0 = (uint32_t)proto_a, b_lo0 = (uint32_t)proto_b;
        uint32_t a_lo = a_lo0 + (uint32_t)stage * stage_adv, b_lo = b_lo0 + (uint32_t)stage * stage_adv;
        if (!mbar_wait_or_abort(smem_u32(&tempty_bar[acc]), acc_phase ^ 1u, vabort, g.p[0].wait_ns)) {
          if (!*vabort) fail(p, DEV_TIMEOUT_EPI, vabort);
          break;
        }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + (uint32_t)(acc * p.block_n);
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!mbar_wait_or_abort(smem_u32(&full_bar[stage]), phase, vabort, g.p[0].wait_ns)) {
            if (!*vabort) fail(p, DEV_TIMEOUT_TMA, vabort);
            ok = false;
            break;
          }
          tc_fence_after();
          tc_mma_lohi<0>(tmem_d, a_lo, a_hi, b_lo, b_hi, p.idesc, (uint32_t)(kb != 0));
          tc_mma_lohi<0>(tmem_d, a_lo + adv_a, a_hi, b_lo + adv_b, b_hi, p.idesc, 1u);
          tc_mma_lohi<0>(tmem_d, a_lo + 2 * adv_a, a_hi, b_lo + 2 * adv_b, b_hi, p.idesc, 1u);
          tc_mma_lohi<0>(tmem_d, a_lo + 3 * adv_a, a_hi, b_lo + 3 * adv_b, b_hi, p.idesc, 1u);
          tc_commit(smem_u32(&empty_bar[stage]));
          a_lo += stage_adv; b_lo += stage_adv;
          if (++stage == g.num_stages) { stage = 0; phase ^= 1u; a_lo = a_lo0; b_lo = b_lo0; }
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
    int acc = 0;
    uint32_t acc_phase = 0;
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
      int local;
      const TcParams& p = g.p[find_problem(g, tile, local)];
      const Epilogue& e = p.epi;
      float alpha = e.alpha_const;
      if (e.alpha_p0) alpha *= *e.alpha_p0;
      if (e.alpha_p1) alpha *= *e.alpha_p1;
      const int cols_per_warp = p.block_n >> 1, c_begin = half * cols_per_warp;
      const TileCoord t = decode_tile(p, local);
      const int row = t.m0 + quad * 32 + lane, col_begin = t.n0 + c_begin;
      const bool row_ok = row < p.M;
      const long long row_off = (long long)t.b0 * e.c_b0 + (long long)t.b1 * e.c_b1 + (long long)row * e.ldc;
      const int nfull = col_begin < p.N ? min((p.N - col_begin) >> 5, cols_per_warp >> 5) : 0;   // N % 32 == 0 (host)
      const float rb = (e.row_bias && row_ok) ? e.row_bias[row] : 0.f;
      const bool got = mbar_wait_or_abort(smem_u32(&tfull_bar[acc]), acc_phase, vabort, g.p[0].wait_ns);
      if (!__all_sync(0xffffffffu, got)) {
        if (lane == 0 && !*vabort) fail(p, DEV_TIMEOUT_MMA, vabort);
        break;
      }
      tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * p.block_n);
      uint32_t res0[16];
      if (nfull > 0) drain_dispatch<0, 16>(e, taddr + (uint32_t)c_begin, nfull, alpha, rb, nullptr, row_off + col_begin, row_ok, res0,
                                       StoreCtx{nullptr, 0u, 0, 0, 0, lane}, col_begin);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&tempty_bar[acc]));
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1u;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

}  // namespace

bool tc_gemm_group_eligible(const GemmGroupItem* items, int n) {
  if (n < 1 || n > MAX_GEMM_GROUP) return false;
  for (int i = 0; i < n; ++i) {
    const GemmGroupItem& it = items[i];
    const Epilogue& e = it.epi;
    if (it.g.M <= 0 || it.g.N <= 0 || it.g.K <= 0 || it.g.nb0 != 1 || it.g.nb1 != 1) return false;
    if (e.out_kind != OUT_F32 || e.col_scale || e.col_bias || e.residual || e.act || !e.out) return false;
    if (it.g.N % 32 || e.ldc % 8 || (reinterpret_cast<uintptr_t>(e.out) & 31)) return false;   // whole chunks, 32-byte stores
  }
  return true;
}

int tc_gemm_group(const GemmGroupItem* items, int n, int* d_status, int sm_count, cudaStream_t stream) {
  if (!tc_gemm_group_eligible(items, n)) return GEMM_ERR_ARG;
  GroupParams gp;
  GroupMaps maps;
  gp.n = n;
  const int block_n = 256, block_k = 64;
  gp.stage_bytes = A_STAGE_BYTES + block_n * 128;
  gp.num_stages = SINGLE_CTA_SMEM_BUDGET / gp.stage_bytes;
  int tiles = 0;
  double flops = 0;
  for (int i = 0; i < MAX_GEMM_GROUP; ++i) {
    const GemmGroupItem& it = items[i < n ? i : n - 1];        // unused slots repeat the last problem (never reached)
    TcParams& p = gp.p[i];
    p.M = it.g.M; p.N = it.g.N; p.K = it.g.K; p.nb0 = 1; p.nb1 = 1;
    p.block_n = block_n; p.block_k = block_k;
    p.m_tiles = (p.M + BLOCK_M - 1) / BLOCK_M;
    p.n_tiles = (p.N + block_n - 1) / block_n;
    p.k_blocks = (p.K + block_k - 1) / block_k;
    p.num_tiles = p.m_tiles * p.n_tiles;
    p.stage_bytes = gp.stage_bytes; p.num_stages = gp.num_stages;
    p.a_mn = it.A.mn_contig; p.b_mn = it.B.mn_contig;
    p.epi = it.epi;
    p.status = d_status;
    p.wait_ns = g_wait_limit_ns;
    p.idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(it.A.mn_contig ? 1 : 0) << 15) |
              ((uint32_t)(it.B.mn_contig ? 1 : 0) << 16) | ((uint32_t)(block_n >> 3) << 17) | ((uint32_t)(BLOCK_M >> 4) << 24);
    int a_chunked = 0, b_chunked = 0;         // MN-major operands: one 5-D load per stage where the extent allows it
    int rc = make_operand_map(&maps.a[i], it.A, 2, p.M, p.K, 1, 1, BLOCK_M, block_k, &a_chunked);
    if (rc != GEMM_OK) return rc;
    rc = make_operand_map(&maps.b[i], it.B, 2, p.N, p.K, 1, 1, block_n, block_k, &b_chunked);
    if (rc != GEMM_OK) return rc;
    if (a_chunked) p.a_mn = 2;
    if (b_chunked) p.b_mn = 2;
    if (i < n) {
      tiles += p.num_tiles;
      flops += 2.0 * p.M * p.N * (double)p.K;
    }
    gp.tile_end[i] = tiles;
  }
  const int smem = gp.num_stages * gp.stage_bytes + 1024;
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(tc_gemm_group_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SINGLE_CTA_SMEM_BUDGET + 1024) != cudaSuccess)
      return GEMM_ERR_CUDA;
    attr_set = true;
  }
  const int grid = tiles < sm_count ? tiles : sm_count;
  Scope sc([&] {
    char buf[48];
    snprintf(buf, sizeof(buf), "gemm_bf16 group of %d, %d tiles", n, tiles);
    return std::string(buf);
  }, flops, 1, stream, 0);
  if (launch_k(tc_gemm_group_kernel, grid, GEMM_THREADS, smem, stream, maps, gp) != cudaSuccess) return GEMM_ERR_CUDA;
  return cudaGetLastError() == cudaSuccess ? GEMM_OK : GEMM_ERR_CUDA;
}

}  // namespace mrem
