// Helpers shared by the tcgen05 versions of the fused layer halves (fused_layer_tc.cu, fused_layer_tc128.cu).
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "tensor_map.cuh"
#include "tmem_ldst.cuh"

namespace gsit {
namespace {

constexpr int TM = 128;           // rows per tile
constexpr int T_THREADS = 192;
constexpr int T_SPIN = 1 << 16;
constexpr int XBOX = TM * 128;     // TMA box of 128 rows x 128 bytes (32 floats or 64 bf16 per row), swizzled

__device__ __forceinline__ void t_mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void t_mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void t_mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void t_mbar_wait(const Geometry& g, uint32_t bar, uint32_t parity) {
  for (int it = 0; it < T_SPIN; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    if (ok) return;
    if ((it & 63) == 63 && (*reinterpret_cast<volatile unsigned int*>(g.status) & GSIT_DEVFLAG_TIMEOUT)) return;
  }
  raise_flag(g, GSIT_DEVFLAG_TIMEOUT);
}
__device__ __forceinline__ void t_tma_2d(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void t_tma_store_2d(const CUtensorMap* tm, uint32_t src, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(src) : "memory");
}
__device__ __forceinline__ bool t_elect() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred != 0;
}
// K-major operand tile with 128-byte rows and 128-byte swizzle: 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t t_desc(uint32_t addr) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)(1024u >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
__host__ __device__ constexpr uint32_t t_idesc(int n) {  // D = f32, A = B = bf16 K-major, M = 128, N = n
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}
__device__ __forceinline__ void t_umma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void t_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void t_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void t_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void t_fence_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void t_bar_rows() { asm volatile("bar.sync 1, 128;" ::: "memory"); }  // the four row warps
__device__ __forceinline__ uint32_t t_bf2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
// 16-byte chunk `ch` (0..7) of row r in a tile of 128-byte rows with the 128-byte swizzle.
__device__ __forceinline__ uint32_t sw128(uint32_t tile, int r, int ch) { return tile + r * 128 + ((ch ^ (r & 7)) << 4); }
__device__ __forceinline__ void st_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

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
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) n = 0;
  }
  return n;
}

}  // namespace
}  // namespace gsit
