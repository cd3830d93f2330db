// Host interface of the tcgen05 projection GEMM (fp16 operands, fp32 accumulation).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace cs {

enum GemmEpilogue {
  kEpiStoreF16 = 0,  // out fp16 [M,N] = a * w^T
  kEpiResidAdd = 1,   // out fp32 [M,N] += a * w^T   (added by the copy engine; long k ranges are split over the SMs)
  kEpiSwiGLU = 2,     // out fp16 [M,N] = silu(a * w^T) * (a * w2^T)
  kEpiStoreRope = 3,  // out fp16 [M,N] = a * w^T with the rotary turn applied to the leading heads (QKV projection)
  kEpiStoreNormRope = 4   // as kEpiStoreRope, each turned head RMS-normalised over its columns first (gains qk_gain)
};

// 2D tensor map over a row-major [rows, cols] matrix of 16-bit floats (fp16, or bf16 for the kv cache);
// box = [box_rows, box_cols].
bool make_tensor_map_16b(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows,
                         uint32_t box_cols, bool swizzle128, bool is_bf16);
// 3D fp16 tensor map over a row-major [tokens, heads, head_dim] view (token stride = row_elems elements):
// box = [box_tokens, box_heads, 64], 128-byte swizzle. Used to fetch a query tile whose rows are
// (token, head-in-group) pairs.
bool make_tensor_map_heads3d(CUtensorMap* tm, const void* base, uint64_t tokens, uint64_t heads, uint32_t head_dim,
                             uint64_t row_elems, uint32_t box_tokens, uint32_t box_heads);
// 4D fp16 tensor maps that deliver rows of `hd` columns (hd = 64 * halves) as
// [8-row group][64-column half][8 rows][128 bytes] with the 128-byte swizzle, the shared-memory layout of the
// attention kernel's K and V tiles. Dimensions, innermost first: 64 columns, 8 rows (stride = one row), halves
// (stride 128 bytes), groups.
//  - make_kv_group_map: over a matrix of `rows` rows (a multiple of 8) of exactly hd columns; the last coordinate
//    is the 8-row group index; one box = groups_per_box groups. Used for the cache pool (one 16-row page per box).
//  - make_kv_rows_map: over a row-major [rows_alloc, row_elems] matrix whose rows hold many 64-column blocks; the
//    second coordinate is the first row (any value < rows), the third the 64-column block index, the last is
//    always 0 and spans 16 groups, so one box = 128 consecutive rows starting at any row. The box may reach up to
//    127 rows past `rows`: the allocation must hold them (rows_alloc >= rows + 128) and they must be finite.
bool make_kv_group_map(CUtensorMap* tm, const void* base, uint64_t rows, uint32_t hd, uint32_t groups_per_box);
bool make_kv_rows_map(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t row_elems, uint32_t hd);
// Tensor map of a GEMM operand ([rows, k] fp16, K-major): 128-row x 64-column boxes, 128-byte swizzle.
bool make_gemm_operand_map(CUtensorMap* tm, const void* base, int rows, int k);

// Rotary position turn fused into the store epilogue of the QKV projection: columns [0, n_rot_cols) are heads of
// 2 * half columns in which the pair (j, j + half) of row t turns by the angle whose (cos, sin) is table[t * half + j];
// the remaining columns (the V heads) are stored as they are. half is 32 or 64; N and n_rot_cols multiples of 2 * half.
// With qk_gain != nullptr every turned head is first RMS-normalised over its 2 * half columns (in fp32, on the
// accumulator): x / sqrt(mean(x^2) + eps) * g, g = qk_gain[0 .. 2 half) for heads in columns [0, q_cols) (queries)
// and qk_gain[2 half .. 4 half) for the turned heads after them (keys).
struct RopeEpilogue {
  const float2* table;
  int half;
  int n_rot_cols;
  const float* qk_gain = nullptr;
  int q_cols = 0;
  float eps = 0.f;
};
cudaError_t gemm_f16_rope(const CUtensorMap& ta, const CUtensorMap& tb, void* out, int M, int N, int K,
                          const RopeEpilogue& rope, uint32_t* status, cudaStream_t stream);

// Ordered mode of the residual epilogue (kEpiResidAdd): `flags` is a zero-initialised device array of
// kTurnWords words that only these launches touch, `epoch` a host counter that every ordered launch advances. With it the pieces
// of a tile are added in a fixed order and the result is bit-identical from run to run; launches that share the array
// must be ordered on one stream.
constexpr int kTurnWords = 148 + 8;
struct TurnOrder {
  uint32_t* flags;
  uint32_t* epoch;
};
cudaError_t gemm_f16(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap* tb2, void* out, int M, int N,
                      int K, int epilogue, uint32_t* status, cudaStream_t stream, const TurnOrder* turn = nullptr);

}  // namespace cs
