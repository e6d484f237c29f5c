// Fused attention forward for one (batch, head, 128-query block) per CTA on sm_100a:
//   S = Q K^T (tcgen05, fp32 accumulators in TMEM)  ->  masked softmax by 256 threads, two per
//   query row (alternate 32-key chunks), straight out of TMEM  ->  (student) Eq. 1 on the probabilities  ->
//   ctx = P V with P taken from shared memory as the A operand of a second tcgen05 product.
// The scores never touch HBM.  Operands are the Q/K/V slices of the [tokens, 3*hidden] tensor
// (bf16 values for the teacher, integer codes held as bf16 for the student: every product of
// codes is exact in fp32), fetched by TMA with 128-byte swizzle.  Outputs: the probabilities
// (and their codes) for the backward pass, the context rows, and for the student the codes of
// the context (int8 for the next int8 product, bf16 for the backward).
// Head size 64, sequence length up to 384 (scores + context accumulators fit the 512 TMEM
// columns).  All waits are time-bounded.
#include "gemm.h"
#include "kernels.h"
#include "tc_ptx.cuh"

namespace mrem {

namespace {

constexpr int ATT_THREADS = 288;          // warp 0: TMA + MMA issue; warps 1..8: softmax / epilogue, two per row quadrant
constexpr int HD = 64;

struct AttnParams {
  int S, h, B, H;
  int n_kb;                  // key blocks of 64
  int n16;                   // keys rounded up to 16 (width of the score product)
  int tmem_cols;             // allocation (power of two >= n16 + 64)
  float alpha_const;         // score scale = alpha_const * (*a_p0) * (*a_p1)
  const float *a_p0, *a_p1;
  const float *c_p0, *c_p1;  // context scale = (*c_p0) * (*c_p1); null = 1
  const int* valid_len;
  const float* p_step;       // quantizer of the probabilities (student), null = none
  float p_lo, p_hi;
  const float* c_step;       // symmetric quantizer of the context (student), null = none
  float c_qmax;
  bf16 *P, *P_qt;            // [B, h, S, S]
  bf16* ctx;                 // [B*S, H]
  int8_t* ctx_q8;            // [B*S, H]
  bf16* ctx_qt;              // [B*S, H]
  int* status;
  unsigned long long wait_ns;  // limit of each wait on an mbarrier
};

__device__ __forceinline__ void store16(void* p, const uint32_t* w) {
  *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
}

__global__ void __launch_bounds__(ATT_THREADS) attention_fwd_kernel(const __grid_constant__ CUtensorMap map_qkv,
                                                                    const __grid_constant__ AttnParams p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full, bar_s, bar_p, bar_o;
  __shared__ uint32_t tmem_slot;
  __shared__ float red[2][2][128];                           // [max | sum][column half][row]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qb = blockIdx.x, head = blockIdx.y, b = blockIdx.z;
  const int q0 = qb * 128;
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int n_box = (p.S + 127) / 128;                       // 128-row TMA boxes of keys / values
  const uint32_t sQ = base, sK = sQ + 16384, sV = sK + n_box * 16384, sP = sV + n_box * 16384;
  uint8_t* gP = smem_raw + (sP - smem_u32(smem_raw));        // generic pointer to the P operand tile
  pdl_trigger();

  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar_full), 1);
    mbar_init(smem_u32(&bar_s), 1);
    mbar_init(smem_u32(&bar_p), 256);
    mbar_init(smem_u32(&bar_o), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                 "r"(p.tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  pdl_wait();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&tmem_slot);
  const uint32_t tmem_ctx = tmem + (uint32_t)p.n16;

  if (warp == 0) {
    if (lane == 0) {
      // ---- loads: Q block, all keys, all values (slots of the qkv tensor: head, h + head, 2h + head)
      const uint32_t bar = smem_u32(&bar_full);
      const int kv_boxes = n_box;
      mbar_expect_tx(bar, 16384u + (uint32_t)kv_boxes * 2u * 16384u);
      tma_load_4d(sQ, &map_qkv, bar, 0, q0, head, b);
      for (int i = 0; i < kv_boxes; ++i) {
        tma_load_4d(sK + i * 16384, &map_qkv, bar, 0, i * 128, p.h + head, b);
        tma_load_4d(sV + i * 16384, &map_qkv, bar, 0, i * 128, 2 * p.h + head, b);
      }
      bool ok = mbar_wait(bar, 0, p.wait_ns);
      if (!ok) atomicCAS(p.status, 0, (int)DEV_TIMEOUT_TMA);
      tc_fence_after();
      // ---- scores: [128 x n16] = Q [128 x 64] * K^T, in pieces of at most 256 keys
      if (ok) {
        for (int n0 = 0; n0 < p.n16; n0 += 256) {
          const int n = min(256, p.n16 - n0);
          const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | (8u << 24);
#pragma unroll
          for (int k = 0; k < 4; ++k)
            tc_mma<0>(tmem + (uint32_t)n0, smem_desc(sQ + k * 32, 16u, 1024u), smem_desc(sK + n0 * 128 + k * 32, 16u, 1024u),
                      idesc, (uint32_t)(k != 0));
        }
      }
      tc_commit(smem_u32(&bar_s));
      // ---- context: [128 x 64] = P [128 x keys] * V [keys x 64]  (V is the MN-major operand)
      ok = ok && mbar_wait(smem_u32(&bar_p), 0, p.wait_ns);
      if (!ok) atomicCAS(p.status, 0, (int)DEV_TIMEOUT_EPI);
      tc_fence_after();
      if (ok) {
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(HD >> 3) << 17) | (8u << 24);
        const int ksteps = p.n_kb * 4;
        for (int ks = 0; ks < ksteps; ++ks)
          tc_mma<0>(tmem_ctx, smem_desc(sP + (ks >> 2) * 16384 + (ks & 3) * 32, 16u, 1024u),
                    smem_desc(sV + ks * 2048, 8192u, 1024u), idesc, (uint32_t)(ks != 0));
      }
      tc_commit(smem_u32(&bar_o));
    }
  } else {
    // ---- two threads per query row; TMEM lane quadrant = warp % 4, 32-key chunks alternate between them
    const int quad = warp & 3, half = (warp - 1) >> 2;
    const int r = quad * 32 + lane;                      // row inside the block
    const int q = q0 + r;
    const bool row_ok = q < p.S;
    int len = p.valid_len ? p.valid_len[b] : p.S;
    len = len < 1 ? 1 : (len > p.S ? p.S : len);
    float alpha = p.alpha_const;
    if (p.a_p0) alpha *= *p.a_p0;
    if (p.a_p1) alpha *= *p.a_p1;
    const bool quant = p.p_step != nullptr;
    const float ps = quant ? *p.p_step : 1.f, r_ps = __frcp_rn(ps);
    const uint32_t trow = tmem + ((uint32_t)(quad * 32) << 16);
    const int n_chunks = (p.S + 31) / 32;
    const bool got = mbar_wait(smem_u32(&bar_s), 0, p.wait_ns);
    if (!__all_sync(0xffffffffu, got) && lane == 0) atomicCAS(p.status, 0, (int)DEV_TIMEOUT_MMA);
    tc_fence_after();
    // scores in units of log2(e): exp(alpha * a - max) = 2^(alpha2 * a - max2); alpha > 0, so the maximum
    // can be taken over the raw accumulators
    const float alpha2 = alpha * 1.4426950408889634f;
    float mx = -INFINITY;
    for (int c = half; c < n_chunks; c += 2) {
      uint32_t a[32];
      tmem_ld32(trow + (uint32_t)(c * 32), a);
      if (c * 32 + 32 <= len) {                          // all 32 keys valid (warp-uniform)
#pragma unroll
        for (int j = 0; j < 32; ++j) mx = fmaxf(mx, __uint_as_float(a[j]));
      } else {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (c * 32 + j < len) mx = fmaxf(mx, __uint_as_float(a[j]));
      }
    }
    red[0][half][r] = mx;
    asm volatile("bar.sync 1, 256;" ::: "memory");
    const float mx2 = alpha2 * fmaxf(red[0][0][r], red[0][1][r]);
    float sum = 0.f;
    for (int c = half; c < n_chunks; c += 2) {            // exp once: kept in TMEM in place of the score
      uint32_t a[32];
      tmem_ld32(trow + (uint32_t)(c * 32), a);
      if (c * 32 + 32 <= len) {
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const float e = exp2_approx(fmaf(alpha2, __uint_as_float(a[j]), -mx2));
          sum += e;
          a[j] = __float_as_uint(e);
        }
      } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const float e = c * 32 + j < len ? exp2_approx(fmaf(alpha2, __uint_as_float(a[j]), -mx2)) : 0.f;
          sum += e;
          a[j] = __float_as_uint(e);
        }
      }
      tmem_st32(trow + (uint32_t)(c * 32), a);
    }
    red[1][half][r] = sum;
    asm volatile("bar.sync 1, 256;" ::: "memory");
    sum = red[1][0][r] + red[1][1][r];
    const float inv_sum = __frcp_rn(sum);
    const long long prow = (((long long)b * p.h + head) * p.S + q) * p.S;
    for (int c = half; c < 2 * p.n_kb; c += 2) {          // 32-key chunks up to the padded key count
      uint32_t pw[16], cw[16];                            // 32 probabilities / codes packed as bf16 pairs
      if (c < n_chunks) {
        uint32_t a[32];
        tmem_ld32(trow + (uint32_t)(c * 32), a);
#pragma unroll
        for (int j = 0; j < 32; j += 2) {
          const float v0 = __uint_as_float(a[j]) * inv_sum, v1 = __uint_as_float(a[j + 1]) * inv_sum;
          const __nv_bfloat162 pb = __floats2bfloat162_rn(v0, v1);
          pw[j >> 1] = *reinterpret_cast<const uint32_t*>(&pb);
          if (quant) {
            const float2 f = __bfloat1622float2(pb);
            // f is bf16-valued: quotient() equals the IEEE division of Eq. 1 for every such value and every step
            const float c0 = rne_magic(fminf(fmaxf(quotient(f.x, ps, r_ps), p.p_lo), p.p_hi));
            const float c1 = rne_magic(fminf(fmaxf(quotient(f.y, ps, r_ps), p.p_lo), p.p_hi));
            const __nv_bfloat162 cb = __floats2bfloat162_rn(c0, c1);
            cw[j >> 1] = *reinterpret_cast<const uint32_t*>(&cb);
          } else {
            cw[j >> 1] = pw[j >> 1];
          }
        }
        if (row_ok && p.P) {                              // (no P: a pass whose probabilities nobody reads)
          const int ncol = p.S - c * 32;                  // columns of this chunk inside the tensor (S % 8 == 0)
#pragma unroll
          for (int t = 0; t < 4; ++t)
            if (t * 8 < ncol) {
              store16(p.P + prow + c * 32 + t * 8, pw + 4 * t);
              if (quant && p.P_qt) store16(p.P_qt + prow + c * 32 + t * 8, cw + 4 * t);
            }
        }
      } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) cw[j] = 0u;
      }
      // operand tile: block of 64 keys, row r, 16-byte chunk index XOR (r & 7)  (128-byte swizzle)
      uint8_t* rowp = gP + (c >> 1) * 16384 + r * 128;
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const int chunk = ((c & 1) * 4 + t) ^ (r & 7);
        store16(rowp + chunk * 16, cw + 4 * t);
      }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> visible to the MMA
    tc_fence_before();
    mbar_arrive(smem_u32(&bar_p));
    // ---- context row
    const bool got2 = mbar_wait(smem_u32(&bar_o), 0, p.wait_ns);
    if (!__all_sync(0xffffffffu, got2) && lane == 0) atomicCAS(p.status, 0, (int)DEV_TIMEOUT_MMA);
    tc_fence_after();
    float calpha = 1.f;
    if (p.c_p0) calpha *= *p.c_p0;
    if (p.c_p1) calpha *= *p.c_p1;
    const float cs = p.c_step ? *p.c_step : 1.f, r_cs = __frcp_rn(cs);
    const long long crow = ((long long)b * p.S + q) * p.H + head * HD;
    {
      const int hh = half;
      uint32_t a[32];
      tmem_ld32(trow + (uint32_t)(p.n16 + hh * 32), a);
      uint32_t w[16], cq[16], c8[8];
#pragma unroll
      for (int j = 0; j < 32; j += 2) {
        const __nv_bfloat162 vb = __floats2bfloat162_rn(calpha * __uint_as_float(a[j]), calpha * __uint_as_float(a[j + 1]));
        w[j >> 1] = *reinterpret_cast<const uint32_t*>(&vb);
        if (p.c_step) {
          const float2 f = __bfloat1622float2(vb);
          uint32_t b0, b1;                                 // rounding words: low byte = the 8-bit code
          const float i0 = rne_magic(fminf(fmaxf(quotient(f.x, cs, r_cs), -p.c_qmax), p.c_qmax), b0);
          const float i1 = rne_magic(fminf(fmaxf(quotient(f.y, cs, r_cs), -p.c_qmax), p.c_qmax), b1);
          const __nv_bfloat162 cb = __floats2bfloat162_rn(i0, i1);
          cq[j >> 1] = *reinterpret_cast<const uint32_t*>(&cb);
          const uint32_t two = __byte_perm(b0, b1, 0x0040) & 0xffffu;
          if ((j & 2) == 0) c8[j >> 2] = two; else c8[j >> 2] |= two << 16;
        }
      }
      if (row_ok) {
#pragma unroll
        for (int t = 0; t < 4; ++t) store16(p.ctx + crow + hh * 32 + t * 8, w + 4 * t);
        if (p.c_step) {
#pragma unroll
          for (int t = 0; t < 4; ++t) store16(p.ctx_qt + crow + hh * 32 + t * 8, cq + 4 * t);
          store16(p.ctx_q8 + crow + hh * 32, c8);
          store16(p.ctx_q8 + crow + hh * 32 + 16, c8 + 4);
        }
      }
    }
    tc_fence_before();
  }
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(p.tmem_cols) : "memory");
  }
}

}  // namespace

bool attention_fwd_supported(int S, int head_dim, int dt) { return dt == 1 && head_dim == HD && S % 8 == 0 && S <= 384; }

// qkv: [B*S, 3H] storage-type tensor (values or codes).  Null p_step / c_step: no quantizer (teacher).
int launch_attention_fwd(const void* qkv, int B, int S, int h, int H, const int* valid_len, float alpha_const,
                         const float* a_p0, const float* a_p1, const float* c_p0, const float* c_p1,
                         const float* p_step, int p_lo, int p_hi, void* P, void* P_qt, void* ctx, const float* c_step,
                         int c_qmax, int8_t* ctx_q8, void* ctx_qt, int* status, cudaStream_t st) {
  AttnParams p;
  p.S = S; p.h = h; p.B = B; p.H = H;
  p.n_kb = (S + 63) / 64;
  p.n16 = (S + 15) / 16 * 16;
  int cols = 32;
  while (cols < p.n16 + HD) cols *= 2;
  p.tmem_cols = cols;
  p.alpha_const = alpha_const; p.a_p0 = a_p0; p.a_p1 = a_p1; p.c_p0 = c_p0; p.c_p1 = c_p1;
  p.valid_len = valid_len;
  p.p_step = p_step; p.p_lo = (float)p_lo; p.p_hi = (float)p_hi;
  p.c_step = c_step; p.c_qmax = (float)c_qmax;
  p.P = (bf16*)P; p.P_qt = (bf16*)P_qt; p.ctx = (bf16*)ctx; p.ctx_q8 = ctx_q8; p.ctx_qt = (bf16*)ctx_qt;
  p.status = status;
  p.wait_ns = g_wait_limit_ns;
  // one map over the [tokens, 3H] tensor: (64 of a head, S rows, 3h head slots, B)
  OperandDesc op{qkv, 3LL * H, HD, (long long)S * 3 * H, 0};
  CUtensorMap map;
  const int rc = make_operand_map(&map, op, 2, S, HD, 3 * h, B, 128, HD);
  if (rc != GEMM_OK) return rc;
  const int n_box = (S + 127) / 128;
  const int smem = 1024 + 16384 + n_box * 16384 * 2 + p.n_kb * 16384;
  static int max_set = 0;
  if (smem > max_set) {
    if (cudaFuncSetAttribute(attention_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 1024 + 16384 + 3 * 16384 * 2 + 6 * 16384) != cudaSuccess)
      return GEMM_ERR_CUDA;
    max_set = 1 << 30;
  }
  const long long rows = (long long)B * h * S;
  Scope sc("attention_fwd_tcgen05", 4.0 * rows * S * HD, 1, st);
  dim3 grid((S + 127) / 128, h, B);
  if (launch_k(attention_fwd_kernel, grid, ATT_THREADS, smem, st, map, p) != cudaSuccess) return GEMM_ERR_CUDA;
  return cudaGetLastError() == cudaSuccess ? GEMM_OK : GEMM_ERR_CUDA;
}

}  // namespace mrem
