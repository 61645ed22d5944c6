// Packed row layout: the plan (where each segment of each sample starts among the real rows), and the copies between
// the padded [B, L, cols] layout and the packed [rows, cols] one.  Section "Inner Decomposition for Efficiency" drops
// padded positions from the computation; packed, they are not stored either, so the row-wise parts of the layer
// (LayerNorm, projections, MLP) do no work for them at all.
#include "common.cuh"
#include "ptx.cuh"

namespace gsit {
namespace {

// One CTA; thread i owns the pairs (b, s) = i, i + 1024, ...; an exclusive scan in (b, s) order.
__global__ void __launch_bounds__(1024) plan_rows_kernel(const Geometry g, const int split_sample, int32_t* __restrict__ row_start) {
  __shared__ int part[1024];
  __shared__ int split_sum;
  const int n = 3 * g.batch, tid = threadIdx.x;
  const int per = (n + 1023) / 1024;                 // consecutive entries per thread
  const int lo = min(n, tid * per), hi = min(n, lo + per);
  int sum = 0;
  for (int e = lo; e < hi; ++e) sum += valid_rows(g, e / 3, e % 3);
  part[tid] = sum;
  __syncthreads();
  for (int off = 1; off < 1024; off <<= 1) {         // inclusive scan of the per-thread sums
    const int v = (tid >= off) ? part[tid - off] : 0;
    __syncthreads();
    part[tid] += v;
    __syncthreads();
  }
  int run = part[tid] - sum;                          // exclusive prefix of this thread's first entry
  // rows before the split sample, to find the padding that aligns it
  if (tid == 0) split_sum = -1;
  __syncthreads();
  const int split_e = 3 * split_sample;
  {
    int r2 = run;
    for (int e = lo; e < hi; ++e) {
      if (e == split_e) split_sum = r2;
      r2 += valid_rows(g, e / 3, e % 3);
    }
  }
  __syncthreads();
  const int pad = (split_sample > 0 && split_sample < g.batch && split_sum >= 0) ? ((split_sum + 127) / 128 * 128 - split_sum) : 0;
  for (int e = lo; e < hi; ++e) {
    row_start[e] = run + ((pad > 0 && e >= split_e) ? pad : 0);
    run += valid_rows(g, e / 3, e % 3);
  }
  if (tid == 1023) row_start[n] = part[1023] + pad;
}

// Copies between the two layouts.  A thread moves MOVE_UNROLL 16-byte chunks that lie a quarter of the matrix apart
// (consecutive threads take consecutive chunks, so a warp covers whole rows and both sides of every copy are coalesced);
// all its loads are issued before its first store, so that enough bytes are in flight to cover the memory latency.
// All index arithmetic is 32-bit (the library limits B * L to 2^29 rows).
constexpr int MOVE_UNROLL = 4;
template <bool PACK>
__global__ void __launch_bounds__(256) move_rows_kernel(const Geometry g, const float* __restrict__ src, const int64_t src_stride,
                                                        float* __restrict__ dst, const int64_t dst_stride, const int cpr /* chunks per row */,
                                                        const unsigned total /* chunks in all */, const unsigned quarter) {
  ptx::grid_dep_wait();  // the source comes from the kernel before this one (and the row plan from an earlier one)
  ptx::grid_dep_launch();
  const unsigned idx0 = blockIdx.x * 256u + threadIdx.x;
  if (idx0 >= quarter) return;
  float4 v[MOVE_UNROLL];
  float4* out[MOVE_UNROLL];
#pragma unroll
  for (int u = 0; u < MOVE_UNROLL; ++u) {
    const unsigned idx = idx0 + (unsigned)u * quarter;
    out[u] = nullptr;
    v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (idx >= total) continue;
    const unsigned w = idx / (unsigned)cpr, c = idx - w * (unsigned)cpr;  // padded-layout row, chunk in the row
    const int b = (int)(w / (unsigned)g.L), p = (int)(w - (unsigned)b * (unsigned)g.L);
    const int s = segment_of(g, p), i = p - g.seg_off[s];
    const bool real = i < valid_rows(g, b, s);
    if (PACK) {
      if (!real) continue;
      const int64_t packed = (int64_t)g.row_start[3 * b + s] + i;
      out[u] = reinterpret_cast<float4*>(dst + packed * dst_stride) + c;
      v[u] = __ldg(reinterpret_cast<const float4*>(src + (int64_t)w * src_stride) + c);
    } else {
      out[u] = reinterpret_cast<float4*>(dst + (int64_t)w * dst_stride) + c;
      if (real) v[u] = __ldg(reinterpret_cast<const float4*>(src + ((int64_t)g.row_start[3 * b + s] + i) * src_stride) + c);
    }
  }
#pragma unroll
  for (int u = 0; u < MOVE_UNROLL; ++u)
    if (out[u] != nullptr) *out[u] = v[u];
}

}  // namespace

cudaError_t launch_plan_rows(const Geometry& g, int split_sample, int32_t* row_start, cudaStream_t st) {
  plan_rows_kernel<<<1, 1024, 0, st>>>(g, split_sample, row_start);
  return cudaGetLastError();
}

cudaError_t launch_move_rows(const Geometry& g, bool pack, const float* src, int64_t src_stride, float* dst, int64_t dst_stride,
                             int cols, cudaStream_t st) {
  const int cpr = cols / 4;
  const int64_t total = (int64_t)g.batch * g.L * cpr;
  if (total > 0xffffffffLL) return cudaErrorNotSupported;
  const unsigned quarter = (unsigned)((total + MOVE_UNROLL - 1) / MOVE_UNROLL);
  const unsigned blocks = (quarter + 255u) / 256u;
  if (blocks == 0) return cudaSuccess;
  if (pack)
    return launch_overlapped(move_rows_kernel<true>, dim3(blocks), dim3(256), 0, st, g, src, src_stride, dst, dst_stride, cpr,
                             (unsigned)total, quarter);
  return launch_overlapped(move_rows_kernel<false>, dim3(blocks), dim3(256), 0, st, g, src, src_stride, dst, dst_stride, cpr,
                           (unsigned)total, quarter);
}

}  // namespace gsit
