// Helpers shared by the tcgen05 versions of the fused layer halves (fused_layer_tc.cu, fused_layer_tc128.cu).
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "ptx.cuh"
#include "tensor_map.cuh"
#include "tmem_ldst.cuh"

namespace gsit {
namespace {

using namespace ptx;

constexpr int TM = 128;           // rows per tile
constexpr int T_THREADS = 192;
constexpr int XBOX = TM * 128;     // TMA box of 128 rows x 128 bytes (32 floats or 64 bf16 per row), swizzled

__device__ __forceinline__ void t_bar_rows() { asm volatile("bar.sync 1, 128;" ::: "memory"); }  // the four row warps
// 16-byte chunk `ch` (0..7) of row r in a tile of 128-byte rows with the 128-byte swizzle.
__device__ __forceinline__ uint32_t sw128(uint32_t tile, int r, int ch) { return tile + r * 128 + ((ch ^ (r & 7)) << 4); }

__device__ __forceinline__ float4 ld_v4f(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}
// Copies n floats of a per-feature vector into shared memory (or `fill` when the pointer is null): vectors such as
// gamma, beta and the biases are read by every thread for every row, as 16-byte broadcasts.
__device__ __forceinline__ void stage_vector(float* dst, const float* src, int n, float fill, int tid, int nthreads) {
  for (int i = tid; i < n; i += nthreads) dst[i] = (src != nullptr) ? src[i] : fill;
}
// Row validity with 32-bit arithmetic (the library limits B * L to 2^29).
__device__ __forceinline__ bool row_real32(const Geometry& g, int row, int rows) {
  if (row >= rows) return false;
  if (g.row_start != nullptr) return true;  // packed layout: every row below the end is taken as real
  const int b = row / g.L, p = row - b * g.L;
  const int sgm = segment_of(g, p);
  return (p - g.seg_off[sgm]) < valid_rows(g, b, sgm);
}

// 2-D map over a [rows, cols] float view with row pitch `row_stride` elements; box = [32 columns, box_rows rows] (128
// bytes wide), 128-byte swizzle.
bool make_map_f32(CUtensorMap* tm, const void* basep, int64_t rows, int cols, int64_t row_stride, int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (fn == nullptr) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)row_stride * 4};
  const cuuint32_t box[2] = {32u, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(basep), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int t_sm_count() {
  int n = 0;
  return (sm_count_and_smem_once(nullptr, 0, &n) == cudaSuccess) ? n : 0;
}

}  // namespace
}  // namespace gsit
