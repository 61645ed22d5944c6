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

// Kernels whose rows are split between two threads -- the same TMEM lane in warps w and w + 4, each owning half of the
// columns -- have eight row warps.
constexpr int T_THREADS8 = 320;
__device__ __forceinline__ void t_bar_rows8() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// LayerNorm statistics of a row whose columns are split between two threads.  Each takes the mean and the centred sum
// of squares of its own NC values; the pair exchanges them through `s_stat` (2 x 128 float pairs) and merges them with
// the pairwise update of Chan, Golub and LeVeque, which is symmetric in the two halves, so both threads get the same
// bits.  Every row thread calls it (it contains a barrier of the eight row warps).
template <int NC>
__device__ __forceinline__ void split_row_stats(const float (&v)[NC], uint32_t s_stat, int r, int hf, float eps, bool real,
                                                float& mean, float& rstd) {
  // packed f32x2 arithmetic: two columns per instruction
  float2 s0 = make_float2(0.f, 0.f), s1 = s0;
#pragma unroll
  for (int e = 0; e < NC; e += 4) {
    s0 = __fadd2_rn(s0, make_float2(v[e], v[e + 1]));
    s1 = __fadd2_rn(s1, make_float2(v[e + 2], v[e + 3]));
  }
  const float mean_h = ((s0.x + s0.y) + (s1.x + s1.y)) * (1.f / NC);
  const float2 nm = make_float2(-mean_h, -mean_h);
  float2 q0 = make_float2(0.f, 0.f), q1 = q0;
#pragma unroll
  for (int e = 0; e < NC; e += 4) {
    const float2 a = __fadd2_rn(make_float2(v[e], v[e + 1]), nm), b = __fadd2_rn(make_float2(v[e + 2], v[e + 3]), nm);
    q0 = __ffma2_rn(a, a, q0);
    q1 = __ffma2_rn(b, b, q1);
  }
  const float m2_h = (q0.x + q0.y) + (q1.x + q1.y);
  asm volatile("st.shared.v2.f32 [%0], {%1, %2};" ::"r"(s_stat + (uint32_t)(hf * TM + r) * 8u), "f"(mean_h), "f"(m2_h) : "memory");
  t_bar_rows8();
  float mean_p, m2_p;
  asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(mean_p), "=f"(m2_p) : "r"(s_stat + (uint32_t)((hf ^ 1) * TM + r) * 8u) : "memory");
  const float delta = mean_p - mean_h;
  mean = 0.5f * (mean_h + mean_p);
  const float m2 = (m2_h + m2_p) + (delta * delta) * (0.5f * NC);
  rstd = real ? rsqrtf(m2 * (1.f / (2 * NC)) + eps) : 0.f;
}
// Normalises the thread's NC columns (the row's columns col0 .. col0 + NC - 1) and writes them as bf16 into row r of a
// tile of 128-byte rows in the 128-byte swizzle, 16-byte chunks chunk0 .. chunk0 + NC / 8 - 1 (zeros when !real).
// Per pair of columns: (v * rstd - mean * rstd) as one packed fused multiply-add, then * gamma + beta as another.
template <int NC>
__device__ __forceinline__ void normalise_to_tile(const float (&v)[NC], float mean, float rstd, bool real, uint32_t s_gamma,
                                                  uint32_t s_beta, int col0, uint32_t tile, int r, int chunk0) {
  const float2 rs = make_float2(rstd, rstd), nmr = make_float2(-mean * rstd, -mean * rstd);
#pragma unroll
  for (int ch = 0; ch < NC / 8; ++ch) {
    const uint32_t off = (uint32_t)(col0 + ch * 8) * 4u;
    const float4 g0 = ld_v4f(s_gamma + off), g1 = ld_v4f(s_gamma + off + 16);
    const float4 b0 = ld_v4f(s_beta + off), b1 = ld_v4f(s_beta + off + 16);
    const float2 gm[4] = {make_float2(g0.x, g0.y), make_float2(g0.z, g0.w), make_float2(g1.x, g1.y), make_float2(g1.z, g1.w)};
    const float2 bt[4] = {make_float2(b0.x, b0.y), make_float2(b0.z, b0.w), make_float2(b1.x, b1.y), make_float2(b1.z, b1.w)};
    uint32_t pk[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int e = ch * 8 + 2 * k;
      const float2 t = __ffma2_rn(make_float2(v[e], v[e + 1]), rs, nmr);
      const float2 y = __ffma2_rn(t, gm[k], bt[k]);
      pk[k] = real ? pack_bf16(y.x, y.y) : 0u;
    }
    st_shared_v4(sw128(tile, r, chunk0 + ch), pk[0], pk[1], pk[2], pk[3]);
  }
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
