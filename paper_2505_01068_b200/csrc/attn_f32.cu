// fp32 IM attention on CUDA cores: one warp per (sample, head, query row).
// The warp walks only the real keys of the open key segments of its row's block row (the paper's
// Decomposition), keeps the scaled scores of that row in shared memory, and does a plain three-pass
// softmax (max, exp/sum, aggregate).  Meant for small float problems where 1e-4 parity matters more
// than speed; the bf16 tensor-core path is in attn_bf16.cu.
#include "common.cuh"

namespace gsit {

constexpr int F32_WARPS = 4;

__global__ void __launch_bounds__(F32_WARPS * 32)
attn_f32_kernel(Geometry g, const float* __restrict__ q, const float* __restrict__ k, const float* __restrict__ v,
                int64_t row_stride, float* __restrict__ out, float* __restrict__ lse, float scale, int max_keys) {
  extern __shared__ float smem_f[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float* sc = smem_f + (size_t)warp * (max_keys + g.hd);  // scores of this warp's row
  float* qs = sc + max_keys;                              // the query row

  const int64_t task = (int64_t)blockIdx.x * F32_WARPS + warp;  // (b, h, p)
  const int64_t n_tasks = (int64_t)g.batch * g.heads * g.L;
  if (task >= n_tasks) return;
  const int p = (int)(task % g.L);
  const int h = (int)((task / g.L) % g.heads);
  const int b = (int)(task / ((int64_t)g.L * g.heads));
  const int s = segment_of(g, p);
  const int hd = g.hd;
  float* o = out + ((int64_t)b * g.L + p) * g.d + (int64_t)h * hd;
  float* lse_p = lse ? lse + ((int64_t)b * g.heads + h) * g.L + p : nullptr;

  const bool real = (p - g.seg_off[s]) < valid_rows(g, b, s);
  int nkeys = 0;
  if (real)
    for (int r = 0; r < 3; ++r)
      if ((g.allowed >> (3 * s + r)) & 1u) nkeys += valid_rows(g, b, r);
  if (!real || nkeys == 0) {
    for (int e = lane; e < hd; e += 32) o[e] = 0.f;
    if (lse_p && lane == 0) *lse_p = -INFINITY;
    return;
  }

  const int64_t base = (int64_t)b * g.L * row_stride + (int64_t)h * hd;
  for (int e = lane; e < hd; e += 32) qs[e] = q[base + (int64_t)p * row_stride + e];
  __syncwarp();

  // pass 1: scaled scores of the open, real keys; running max
  float mx = -INFINITY;
  int j0 = 0;
  for (int r = 0; r < 3; ++r) {
    if (!((g.allowed >> (3 * s + r)) & 1u)) continue;
    const int nr = valid_rows(g, b, r);
    for (int j = lane; j < nr; j += 32) {
      const float* kr = k + base + (int64_t)(g.seg_off[r] + j) * row_stride;
      float acc = 0.f;
      for (int e = 0; e < hd; ++e) acc = fmaf(qs[e], kr[e], acc);
      acc *= scale;
      sc[j0 + j] = acc;
      mx = fmaxf(mx, acc);
    }
    j0 += nr;
  }
  for (int off = 16; off; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
  __syncwarp();

  // pass 2: exponentials and their sum
  float sum = 0.f;
  for (int j = lane; j < nkeys; j += 32) {
    const float e = expf(sc[j] - mx);
    sc[j] = e;
    sum += e;
  }
  for (int off = 16; off; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
  __syncwarp();
  const float inv = 1.f / sum;

  // pass 3: aggregation, lanes over the feature axis
  for (int e = lane; e < hd; e += 32) {
    float acc = 0.f;
    int jj = 0;
    for (int r = 0; r < 3; ++r) {
      if (!((g.allowed >> (3 * s + r)) & 1u)) continue;
      const int nr = valid_rows(g, b, r);
      const float* vr = v + base + (int64_t)g.seg_off[r] * row_stride + e;
      for (int j = 0; j < nr; ++j) acc = fmaf(sc[jj + j], vr[(int64_t)j * row_stride], acc);
      jj += nr;
    }
    o[e] = acc * inv;
  }
  if (lse_p && lane == 0) *lse_p = mx + logf(sum);
}

cudaError_t launch_attn_f32(const Geometry& g, const float* q, const float* k, const float* v, int64_t row_stride,
                            float* out, float* lse, float scale, cudaStream_t st) {
  const int max_keys = g.L;
  const size_t smem = (size_t)F32_WARPS * (max_keys + g.hd) * sizeof(float);
  if (smem > 200 * 1024) return cudaErrorNotSupported;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(attn_f32_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  const int64_t n_tasks = (int64_t)g.batch * g.heads * g.L;
  const int64_t blocks = (n_tasks + F32_WARPS - 1) / F32_WARPS;
  if (blocks > 0x7fffffffLL) return cudaErrorNotSupported;
  attn_f32_kernel<<<(unsigned)blocks, F32_WARPS * 32, smem, st>>>(g, q, k, v, row_stride, out, lse, scale, max_keys);
  return cudaGetLastError();
}

}  // namespace gsit
