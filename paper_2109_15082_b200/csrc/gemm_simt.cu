// Plain fp32 GEMM on the CUDA cores: C[b][m][n] = epilogue( sum_k A[b][m][k] * B[b][n][k] ).
// Serves the float32 storage mode (small correctness configurations), where tensor-core
// input rounding would not meet float32 accuracy.  64x64 tiles, 4x4 outputs per thread,
// operands addressed through generic strides so that every transposition is one code path.
#include "gemm.h"

namespace mrem {

namespace {

constexpr int TS = 64, TK = 16;

struct SimtParams {
  OperandDesc A, B;
  GemmShape g;
  Epilogue epi;
};

__device__ __forceinline__ float load_op(const OperandDesc& o, long long base, int mn, int k, int mn_extent, int K) {
  if (mn >= mn_extent || k >= K) return 0.f;
  const long long off = o.mn_contig ? (long long)k * o.ld + mn : (long long)mn * o.ld + k;
  return reinterpret_cast<const float*>(o.ptr)[base + off];
}

__global__ void __launch_bounds__(256) simt_gemm_kernel(const SimtParams p) {
  pdl_trigger();
  pdl_wait();
  __shared__ float sa[TK][TS + 1];
  __shared__ float sb[TK][TS + 1];
  const int z = blockIdx.z, b0 = z % p.g.nb0, b1 = z / p.g.nb0;
  const int m0 = blockIdx.y * TS, n0 = blockIdx.x * TS;
  const long long abase = (long long)b0 * p.A.s_b0 + (long long)b1 * p.A.s_b1;
  const long long bbase = (long long)b0 * p.B.s_b0 + (long long)b1 * p.B.s_b1;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float acc[4][4] = {};
  for (int k0 = 0; k0 < p.g.K; k0 += TK) {
    for (int i = threadIdx.x; i < TS * TK; i += 256) {
      int mn, k;
      if (p.A.mn_contig) { mn = i % TS; k = i / TS; } else { k = i % TK; mn = i / TK; }
      sa[k][mn] = load_op(p.A, abase, m0 + mn, k0 + k, p.g.M, p.g.K);
      if (p.B.mn_contig) { mn = i % TS; k = i / TS; } else { k = i % TK; mn = i / TK; }
      sb[k][mn] = load_op(p.B, bbase, n0 + mn, k0 + k, p.g.N, p.g.K);
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < TK; ++k) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = sa[k][ty * 4 + i]; b[i] = sb[k][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
  const Epilogue& e = p.epi;
  float alpha = e.alpha_const;
  if (e.alpha_p0) alpha *= *e.alpha_p0;
  if (e.alpha_p1) alpha *= *e.alpha_p1;
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= p.g.M) continue;
    const long long row_off = (long long)b0 * e.c_b0 + (long long)b1 * e.c_b1 + (long long)m * e.ldc;
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= p.g.N) continue;
      float v = acc[i][j] * (e.col_scale ? alpha * e.col_scale[n] : alpha);
      v += (e.col_bias ? e.col_bias[n] : 0.f) + (e.row_bias ? e.row_bias[m] : 0.f);
      if (e.residual) v += reinterpret_cast<const float*>(e.residual)[row_off + n];
      if (e.act == 1) v = gelu_erf(v);
      reinterpret_cast<float*>(e.out)[row_off + n] = v;
    }
  }
}

}  // namespace

int simt_gemm_f32(const OperandDesc& A, const OperandDesc& B, const GemmShape& g, const Epilogue& epi,
                  cudaStream_t stream) {
  if (g.M <= 0 || g.N <= 0 || g.K <= 0 || g.nb0 <= 0 || g.nb1 <= 0) return GEMM_ERR_ARG;
  if (epi.out_kind != OUT_F32) return GEMM_ERR_ARG;
  SimtParams p{A, B, g, epi};
  dim3 grid((g.N + TS - 1) / TS, (g.M + TS - 1) / TS, g.nb0 * g.nb1);
  if (grid.y > 65535 || grid.z > 65535) return GEMM_ERR_ARG;
  Scope sc("gemm_f32_simt", 2.0 * g.M * g.N * (double)g.K * g.nb0 * g.nb1, 1, stream);
  launch_k(simt_gemm_kernel, grid, 256, 0, stream, p);
  return cudaGetLastError() == cudaSuccess ? GEMM_OK : GEMM_ERR_CUDA;
}

}  // namespace mrem
