// Fused attention backward of the student for one (batch, head) per CTA on sm_100a, sequences up
// to 128 tokens, head size 64.  Inputs: the gradient of the context, the codes of Q, K, V, the stored
// probabilities P and the pre-quantization Q, K, V.  One kernel does what otherwise takes four
// batched products, the softmax backward and three straight-through kernels:
//   dP_hat = s_v * dctx V_q^T                      (tcgen05, accumulators in TMEM)
//   STE of the P quantizer, softmax backward dS = P * (dP - sum_j dP P), by 256 threads (two per
//     query row) reading TMEM; P_hat codes and dS are written to swizzled shared memory
//   dV_hat = s_p * P_q^T dctx,  dQ_hat = s_k/sqrt(d) * dS K_q,  dK_hat = s_q/sqrt(d) * dS^T Q_q
//     (three tcgen05 products; the same shared-memory tile serves as K-major A operand of one
//     product and as MN-major A operand of another, so nothing is transposed; the codes of P and
//     dS share one tile, dQ and dK take over the TMEM columns of dP, so two CTAs fit on an SM)
//   STE of the Q, K, V quantizers on the way out, with their step-size gradients.
// Step-size gradients leave as one partial sum per CTA and site (summed later in CTA order).
// All waits are time-bounded.
#include "gemm.h"
#include "kernels.h"
#include "tc_ptx.cuh"

#include <type_traits>

namespace mrem {

namespace {

constexpr int ATB_THREADS = 288;          // warp 0: TMA + MMA issue; warps 1..8: row work, two threads per row
constexpr int HD = 64;
// TMEM columns: dP in 0..127; once dS has been formed from it, dQ and dK take its place
constexpr int TMEM_DP = 0, TMEM_DV = 128, TMEM_DQ = 0, TMEM_DK = 64, TMEM_ALLOC = 256;

struct AttnBwdParams {
  int S, h, B, H;
  int n16;                   // S rounded up to 16
  int n_kb;                  // 64-wide blocks covering S
  float inv_sqrt_d;
  const float *s_q, *s_k, *s_v, *s_p;
  float q_lo, q_hi;          // code range of the symmetric Q/K/V sites
  float p_lo, p_hi;          // code range of the P site
  const bf16* P;             // [B, h, S, S]
  const bf16* qkv;           // [B*S, 3H] values before quantization
  bf16* dqkv;                // [B*S, 3H] out
  float *part_q, *part_k, *part_v, *part_p;   // [red_slots] each: one partial per CTA, the rest zeroed
  int red_slots;
  int* status;
  unsigned long long wait_ns;  // limit of each wait on an mbarrier
};

__device__ __forceinline__ void ld16(const void* p, uint32_t* w) {
  const uint4 u = *reinterpret_cast<const uint4*>(p);
  w[0] = u.x; w[1] = u.y; w[2] = u.z; w[3] = u.w;
}
__device__ __forceinline__ void st16(void* p, const uint32_t* w) {
  *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
}
__device__ __forceinline__ float2 unpack2(uint32_t w) {
  return __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w));
}
__device__ __forceinline__ uint32_t pack2(float a, float b) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// The epilogue of one gradient: scale the accumulator, apply the straight-through mask of the site's
// quantizer, store 32 head columns of one token, return this thread's share of the step-size gradient.
__device__ __forceinline__ float ste_store(const uint32_t* a, bool row_ok, const bf16* x, bf16* out, float scale,
                                           float step, float lo, float hi) {
  float acc = 0.f;
  const float r_step = __frcp_rn(step);
  if (row_ok) {
    uint32_t xw[16], ow[16];
#pragma unroll
    for (int t = 0; t < 4; ++t) ld16(x + t * 8, xw + 4 * t);
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const float2 xv = unpack2(xw[j]);
      const float g0 = scale * __uint_as_float(a[2 * j]), g1 = scale * __uint_as_float(a[2 * j + 1]);
      const float z0 = quotient(xv.x, step, r_step), z1 = quotient(xv.y, step, r_step);
      const float c0 = fminf(fmaxf(z0, lo), hi), c1 = fminf(fmaxf(z1, lo), hi);
      const bool in0 = c0 == z0, in1 = c1 == z1;              // inside the code range
      const float q0 = rne_magic(c0), q1 = rne_magic(c1);
      acc += g0 * (in0 ? q0 - z0 : q0) + g1 * (in1 ? q1 - z1 : q1);
      ow[j] = pack2(in0 ? g0 : 0.f, in1 ? g1 : 0.f);
    }
#pragma unroll
    for (int t = 0; t < 4; ++t) st16(out + t * 8, ow + 4 * t);
  }
  return acc;
}

__global__ void __launch_bounds__(ATB_THREADS, 2) attention_bwd_kernel(const __grid_constant__ CUtensorMap map_codes,
                                                                       const __grid_constant__ CUtensorMap map_dctx,
                                                                       const __grid_constant__ AttnBwdParams p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full, bar_a, bar_p, bar_b, bar_s, bar_o;
  __shared__ uint32_t tmem_slot;
  __shared__ float red_dot[2][128];
  __shared__ float red_part[8][4];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int head = blockIdx.x, b = blockIdx.y;
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  // sX holds the codes of P (A operand of the dV product) first and dS (A operand of dQ and dK) afterwards
  const uint32_t sQ = base, sK = sQ + 16384, sV = sK + 16384, sD = sV + 16384, sX = sD + 16384;
  uint8_t* gX = smem_raw + (sX - smem_u32(smem_raw));
  pdl_trigger();

  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar_full), 1);
    mbar_init(smem_u32(&bar_a), 1);
    mbar_init(smem_u32(&bar_p), 256);
    mbar_init(smem_u32(&bar_b), 1);
    mbar_init(smem_u32(&bar_s), 256);
    mbar_init(smem_u32(&bar_o), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(TMEM_ALLOC)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  pdl_wait();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&tmem_slot);
  const int ksteps = p.n16 / 16;

  if (warp == 0) {
    if (lane == 0) {
      const uint32_t bar = smem_u32(&bar_full);
      mbar_expect_tx(bar, 4u * 16384u);
      tma_load_4d(sD, &map_dctx, bar, 0, 0, head, b);
      tma_load_4d(sV, &map_codes, bar, 0, 0, 2 * p.h + head, b);
      tma_load_4d(sK, &map_codes, bar, 0, 0, p.h + head, b);
      tma_load_4d(sQ, &map_codes, bar, 0, 0, head, b);
      bool ok = mbar_wait(bar, 0, p.wait_ns);
      if (!ok) atomicCAS(p.status, 0, (int)DEV_TIMEOUT_TMA);
      tc_fence_after();
      if (ok) {      // dP_hat [queries x keys] = dctx [q x d] * V_q^T
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.n16 >> 3) << 17) | (8u << 24);
#pragma unroll
        for (int k = 0; k < 4; ++k)
          tc_mma<0>(tmem + TMEM_DP, smem_desc(sD + k * 32, 16u, 1024u), smem_desc(sV + k * 32, 16u, 1024u), idesc, (uint32_t)(k != 0));
      }
      tc_commit(smem_u32(&bar_a));
      const uint32_t f = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(HD >> 3) << 17) | (8u << 24);
      const uint32_t id_tt = f | (1u << 15) | (1u << 16);     // A and B MN-major
      const uint32_t id_nt = f | (1u << 16);                  // A K-major, B MN-major
      ok = ok && mbar_wait(smem_u32(&bar_p), 0, p.wait_ns);
      if (!ok) atomicCAS(p.status, 0, (int)DEV_TIMEOUT_EPI);
      tc_fence_after();
      if (ok)
        for (int ks = 0; ks < ksteps; ++ks)       // dV_hat [keys x d] = P_q^T [keys x q] * dctx [q x d]
          tc_mma<0>(tmem + TMEM_DV, smem_desc(sX + ks * 2048, 16384u, 1024u), smem_desc(sD + ks * 2048, 8192u, 1024u), id_tt, (uint32_t)(ks != 0));
      tc_commit(smem_u32(&bar_b));
      ok = ok && mbar_wait(smem_u32(&bar_s), 0, p.wait_ns);
      if (!ok) atomicCAS(p.status, 0, (int)DEV_TIMEOUT_EPI);
      tc_fence_after();
      if (ok) {
        for (int ks = 0; ks < ksteps; ++ks)       // dQ_hat [q x d] = dS [q x keys] * K_q [keys x d]
          tc_mma<0>(tmem + TMEM_DQ, smem_desc(sX + (ks >> 2) * 16384 + (ks & 3) * 32, 16u, 1024u), smem_desc(sK + ks * 2048, 8192u, 1024u), id_nt, (uint32_t)(ks != 0));
        for (int ks = 0; ks < ksteps; ++ks)       // dK_hat [keys x d] = dS^T [keys x q] * Q_q [q x d]
          tc_mma<0>(tmem + TMEM_DK, smem_desc(sX + ks * 2048, 16384u, 1024u), smem_desc(sQ + ks * 2048, 8192u, 1024u), id_tt, (uint32_t)(ks != 0));
      }
      tc_commit(smem_u32(&bar_o));
    }
  } else {
    const int quad = warp & 3, half = (warp - 1) >> 2;
    const int r = quad * 32 + lane;                       // row of the tile: a query for dP/dS/dQ, a key for dK/dV
    const bool row_ok = r < p.S;
    const uint32_t trow = tmem + ((uint32_t)(quad * 32) << 16);
    const float s_p = *p.s_p, s_v = *p.s_v, s_q = *p.s_q, s_k = *p.s_k;
    const float r_p = __frcp_rn(s_p);
    const int n_chunks = (p.S + 31) / 32;
    const long long prow = (((long long)b * p.h + head) * p.S + r) * p.S;
    float ds_p = 0.f;
    bool got = mbar_wait(smem_u32(&bar_a), 0, p.wait_ns);
    tc_fence_after();
    // ---- pass A: STE of the P quantizer, row dot product, the codes of P into the operand tile
    float dot = 0.f;
    for (int c = half; c < 2 * p.n_kb; c += 2) {
      uint32_t cw[16];
      if (c < n_chunks) {                   // warp-uniform: the TMEM accesses below are warp-collective
        uint32_t a[32], pw[16];
        tmem_ld32(trow + TMEM_DP + (uint32_t)(c * 32), a);
        const int ncol = row_ok ? p.S - c * 32 : 0;
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          if (t * 8 < ncol) ld16(p.P + prow + c * 32 + t * 8, pw + 4 * t);
          else { pw[4 * t] = pw[4 * t + 1] = pw[4 * t + 2] = pw[4 * t + 3] = 0u; }
        }
        // FULL: every lane's 32 keys lie inside the sequence (the common case), no per-element bounds
        auto chunk = [&](auto full_tag) {
          constexpr bool FULL = decltype(full_tag)::value;
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float2 pv = unpack2(pw[j]);
            float d0 = s_v * __uint_as_float(a[2 * j]), d1 = s_v * __uint_as_float(a[2 * j + 1]);
            const float z0 = quotient(pv.x, s_p, r_p), z1 = quotient(pv.y, s_p, r_p);
            const float c0 = fminf(fmaxf(z0, p.p_lo), p.p_hi), c1 = fminf(fmaxf(z1, p.p_lo), p.p_hi);
            const bool in0 = c0 == z0, in1 = c1 == z1;            // inside the code range
            const float q0 = rne_magic(c0), q1 = rne_magic(c1);
            const bool v0 = FULL || 2 * j < ncol, v1 = FULL || 2 * j + 1 < ncol;      // inside the sequence (row and key)
            if (v0) ds_p += d0 * (in0 ? q0 - z0 : q0);
            if (v1) ds_p += d1 * (in1 ? q1 - z1 : q1);
            d0 = (in0 && v0) ? d0 : 0.f;
            d1 = (in1 && v1) ? d1 : 0.f;
            dot += d0 * pv.x + d1 * pv.y;
            a[2 * j] = __float_as_uint(d0);
            a[2 * j + 1] = __float_as_uint(d1);
            cw[j] = pack2(v0 ? q0 : 0.f, v1 ? q1 : 0.f);
          }
        };
        if (__all_sync(0xffffffffu, ncol >= 32)) chunk(std::true_type{}); else chunk(std::false_type{});
        tmem_st32(trow + TMEM_DP + (uint32_t)(c * 32), a);        // masked dP kept in place for pass B
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) cw[j] = 0u;
      }
      uint8_t* rowp = gX + (c >> 1) * 16384 + r * 128;
#pragma unroll
      for (int t = 0; t < 4; ++t) st16(rowp + ((((c & 1) * 4 + t) ^ (r & 7)) * 16), cw + 4 * t);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tc_fence_before();
    mbar_arrive(smem_u32(&bar_p));
    red_dot[half][r] = dot;
    asm volatile("bar.sync 1, 256;" ::: "memory");
    dot = red_dot[0][r] + red_dot[1][r];
    // ---- pass B: dS = P * (dP - dot), held in registers until the dV product has consumed the codes of P
    uint32_t sw[2][16];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int c = half + 2 * i;
      if (c < n_chunks) {
        uint32_t a[32], pw[16];
        tmem_ld32(trow + TMEM_DP + (uint32_t)(c * 32), a);
        const int ncol = row_ok ? p.S - c * 32 : 0;
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          if (t * 8 < ncol) ld16(p.P + prow + c * 32 + t * 8, pw + 4 * t);
          else { pw[4 * t] = pw[4 * t + 1] = pw[4 * t + 2] = pw[4 * t + 3] = 0u; }
        }
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const float2 pv = unpack2(pw[j]);
          sw[i][j] = pack2(pv.x * (__uint_as_float(a[2 * j]) - dot), pv.y * (__uint_as_float(a[2 * j + 1]) - dot));
        }
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) sw[i][j] = 0u;
      }
    }
    got = mbar_wait(smem_u32(&bar_b), 0, p.wait_ns) && got;
    tc_fence_after();
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int c = half + 2 * i;
      if (c < 2 * p.n_kb) {
        uint8_t* rowp = gX + (c >> 1) * 16384 + r * 128;
#pragma unroll
        for (int t = 0; t < 4; ++t) st16(rowp + ((((c & 1) * 4 + t) ^ (r & 7)) * 16), sw[i] + 4 * t);
      }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tc_fence_before();
    mbar_arrive(smem_u32(&bar_s));
    // ---- the three gradients: STE of the Q, K, V quantizers, 32 of the 64 head columns per thread
    const long long grow = ((long long)b * p.S + r) * 3 * p.H + head * HD + half * 32;
    uint32_t a[32];
    tmem_ld32(trow + (uint32_t)(TMEM_DV + half * 32), a);           // complete since bar_b
    const float ds_v = ste_store(a, row_ok, p.qkv + grow + 2 * p.H, p.dqkv + grow + 2 * p.H, s_p, s_v, p.q_lo, p.q_hi);
    got = mbar_wait(smem_u32(&bar_o), 0, p.wait_ns) && got;
    if (!__all_sync(0xffffffffu, got) && lane == 0) atomicCAS(p.status, 0, (int)DEV_TIMEOUT_MMA);
    tc_fence_after();
    tmem_ld32(trow + (uint32_t)(TMEM_DQ + half * 32), a);
    const float ds_q = ste_store(a, row_ok, p.qkv + grow, p.dqkv + grow, p.inv_sqrt_d * s_k, s_q, p.q_lo, p.q_hi);
    tmem_ld32(trow + (uint32_t)(TMEM_DK + half * 32), a);
    const float ds_k = ste_store(a, row_ok, p.qkv + grow + p.H, p.dqkv + grow + p.H, p.inv_sqrt_d * s_q, s_k, p.q_lo, p.q_hi);
    tc_fence_before();
    // ---- one partial per CTA and site, added in a fixed order
    const float w_p = warp_sum(ds_p), w_q = warp_sum(ds_q), w_k = warp_sum(ds_k), w_v = warp_sum(ds_v);
    if (lane == 0) { red_part[warp - 1][0] = w_p; red_part[warp - 1][1] = w_q; red_part[warp - 1][2] = w_k; red_part[warp - 1][3] = w_v; }
    asm volatile("bar.sync 1, 256;" ::: "memory");
    if (warp == 1 && lane < 4) {
      float t = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) t += red_part[w][lane];
      float* dst = lane == 0 ? p.part_p : (lane == 1 ? p.part_q : (lane == 2 ? p.part_k : p.part_v));
      dst[b * p.h + head] = t;
    }
    if (head == 0 && b == 0)             // the slots no CTA owns
      for (int i = p.B * p.h + (int)threadIdx.x - 32; i < p.red_slots; i += 256) {
        p.part_p[i] = 0.f; p.part_q[i] = 0.f; p.part_k[i] = 0.f; p.part_v[i] = 0.f;
      }
  }
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_ALLOC) : "memory");
  }
}

}  // namespace

bool attention_bwd_supported(int S, int head_dim, int dt, int batch_heads) {
  return dt == 1 && head_dim == HD && S % 8 == 0 && S <= 128 && batch_heads <= RED_BLOCKS;
}

int launch_attention_bwd(const void* qkv_codes, const void* qkv, const void* P, const void* dctx, int B, int S, int h,
                         int H, const float* s_q, const float* s_k, const float* s_v, const float* s_p, int q_lo,
                         int q_hi, int p_lo, int p_hi, void* dqkv, float* part_q, float* part_k, float* part_v,
                         float* part_p, int* status, cudaStream_t st) {
  AttnBwdParams p;
  p.S = S; p.h = h; p.B = B; p.H = H;
  p.n16 = (S + 15) / 16 * 16;
  p.n_kb = (S + 63) / 64;
  p.inv_sqrt_d = 1.f / sqrtf((float)HD);
  p.s_q = s_q; p.s_k = s_k; p.s_v = s_v; p.s_p = s_p;
  p.q_lo = (float)q_lo; p.q_hi = (float)q_hi; p.p_lo = (float)p_lo; p.p_hi = (float)p_hi;
  p.P = (const bf16*)P; p.qkv = (const bf16*)qkv; p.dqkv = (bf16*)dqkv;
  p.part_q = part_q; p.part_k = part_k; p.part_v = part_v; p.part_p = part_p;
  p.red_slots = RED_BLOCKS;
  p.status = status;
  p.wait_ns = g_wait_limit_ns;
  CUtensorMap mc, md;
  OperandDesc oc{qkv_codes, 3LL * H, HD, (long long)S * 3 * H, 0};
  int rc = make_operand_map(&mc, oc, 2, S, HD, 3 * h, B, 128, HD);
  if (rc != GEMM_OK) return rc;
  OperandDesc od{dctx, (long long)H, HD, (long long)S * H, 0};
  rc = make_operand_map(&md, od, 2, S, HD, h, B, 128, HD);
  if (rc != GEMM_OK) return rc;
  const int smem = 1024 + 4 * 16384 + 32768;      // two CTAs per SM
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(attention_bwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return GEMM_ERR_CUDA;
    attr_set = true;
  }
  Scope sc("attention_bwd_tcgen05", 8.0 * B * h * (double)S * S * HD, 1, st);
  if (launch_k(attention_bwd_kernel, dim3(h, B), ATB_THREADS, smem, st, mc, md, p) != cudaSuccess) return GEMM_ERR_CUDA;
  return cudaGetLastError() == cudaSuccess ? GEMM_OK : GEMM_ERR_CUDA;
}

}  // namespace mrem
