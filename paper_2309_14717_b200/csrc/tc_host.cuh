// Host helpers shared by the tensor-core kernels' launch code (defined in gemm_tc.cu).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace qalora {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_fn();      // cuTensorMapEncodeTiled through the runtime, or null

// bf16 matrix [rows][cols] row-major, box = 64 columns x box_rows rows, 128-byte swizzle, zero fill
bool make_act_map(CUtensorMap* map, const void* base, long long rows, int cols, int box_rows);
// packed codes as 8-byte elements; box = the run of tile_cols pack units x kb_rows k-block rows
bool make_codes_map(CUtensorMap* map, const uint32_t* codes, int K, int N, int bits, int tile_cols, int kb_rows);
// (alpha, beta) float32 [G][2N]; box = 2 * tile_cols floats x rows
bool make_qp_map(CUtensorMap* map, const float2* qp, int G, int N, int tile_cols, int rows);
// out[i] = bf16(sum over parts of partial[part][i]) in part order; count a multiple of 8
int launch_sum_parts_bf16(const float* partial, __nv_bfloat16* out, size_t count, int parts, cudaStream_t st);

}  // namespace qalora
