// Internal interface of the two GEMM back ends.
#pragma once
#include <cuda.h>

#include "mrem_common.cuh"
#include "trace.h"

namespace mrem {

enum GemmRc : int { GEMM_OK = 0, GEMM_ERR_ARG = -1, GEMM_ERR_ALIGN = -2, GEMM_ERR_CUDA = -6 };

// Tensor-core path (tcgen05).  kind 0: bf16 x bf16 -> fp32; kind 1: (u8|s8) x s8 -> int32 (exact).
// block_n 0 picks the tile width.  Operands need 16-byte aligned bases and strides.
int tc_gemm(int kind, int a_unsigned, const OperandDesc& A, const OperandDesc& B, const GemmShape& g,
            const Epilogue& epi, int block_n, int* d_status, int sm_count, cudaStream_t stream);

// Verification aid: one block that lets a bounded wait run out (limit_ns) and reports DEV_TIMEOUT_TMA in *d_status.
cudaError_t launch_wait_probe(int* d_status, unsigned long long limit_ns, cudaStream_t stream);

// Several bf16 products with plain fp32 outputs (alpha and row bias only) as one persistent launch over the
// joint tile list: the weight-gradient products of a layer.  Operands as in tc_gemm, one batch each.
constexpr int MAX_GEMM_GROUP = 4;
struct GemmGroupItem { OperandDesc A, B; GemmShape g; Epilogue epi; };
bool tc_gemm_group_eligible(const GemmGroupItem* items, int n);
int tc_gemm_group(const GemmGroupItem* items, int n, int* d_status, int sm_count, cudaStream_t stream);

// 4-D TMA tensor map (128-byte swizzle) of an operand: (contiguous index, strided index, batch0, batch1).
// K-major operands get boxes of block_k x tile_mn elements, MN-major ones 64 x block_k.
// With `chunked` given, an MN-major 16-bit operand whose MN extent is a multiple of 64 gets a 5-D map instead
// (64 contiguous elements, k, 64-element chunk index, batch0, batch1) whose box holds ALL 64 x block_k pieces of a tile, so
// that one TMA instruction loads what otherwise takes tile_mn / 64 of them (same shared-memory layout); *chunked says which.
int make_operand_map(CUtensorMap* map, const OperandDesc& op, int elem_bytes, int mn_extent, int K, int nb0, int nb1,
                     int tile_mn, int block_k, int* chunked = nullptr);

// Plain fp32 SIMT path, used when activations are stored in float32 (small correctness
// configurations); same operand and epilogue conventions, no alignment requirements.
int simt_gemm_f32(const OperandDesc& A, const OperandDesc& B, const GemmShape& g, const Epilogue& epi,
                  cudaStream_t stream);

}  // namespace mrem
