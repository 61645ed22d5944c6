// Read-out of the fusion stack (paper, Eq. "All-Modal-In-One fusion": X_m = f(|| Split(a(G_intra))[-1])): the last real
// time step of each modality segment, concatenated, through the linear map f.  A few kilobytes per sample: one CTA per
// sample gathers the three rows into shared memory, then each warp produces output features with coalesced reads of
// the weight rows and a shuffle reduction.  float accumulation; weights float or bf16.
#include "common.cuh"

namespace gsit {
namespace {

template <typename WT>
__global__ void __launch_bounds__(256)
stack_head_kernel(const Geometry g, const float* __restrict__ c, const int64_t ldc, const int dc, const WT* __restrict__ w,
                  const float* __restrict__ bias, float* __restrict__ out, const int n_out) {
  extern __shared__ float z[];  // [3 * dc]
  const int b = blockIdx.x;
  for (int i = threadIdx.x; i < 3 * dc; i += blockDim.x) {
    const int s = i / dc, e = i - s * dc;
    const int n = valid_rows(g, b, s);
    z[i] = (n > 0) ? c[((int64_t)b * g.L + g.seg_off[s] + n - 1) * ldc + e] : 0.f;
  }
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  for (int o = warp; o < n_out; o += nwarps) {
    const WT* wr = w + (int64_t)o * 3 * dc;
    float acc = 0.f;
    for (int i = lane; i < 3 * dc; i += 32) acc = fmaf((float)wr[i], z[i], acc);
    for (int sft = 16; sft; sft >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, sft);
    if (lane == 0) out[(int64_t)b * n_out + o] = acc + (bias ? bias[o] : 0.f);
  }
}

}  // namespace

cudaError_t launch_stack_head(const Geometry& g, int dtype, const float* c, int64_t ldc, int dc, const void* w,
                              const float* bias, float* out, int n_out, cudaStream_t st) {
  const size_t smem = (size_t)3 * dc * sizeof(float);
  if (smem > 48 * 1024) return cudaErrorNotSupported;
  if (dtype == GSIT_BF16)
    stack_head_kernel<__nv_bfloat16><<<g.batch, 256, smem, st>>>(g, c, ldc, dc, static_cast<const __nv_bfloat16*>(w), bias, out, n_out);
  else
    stack_head_kernel<float><<<g.batch, 256, smem, st>>>(g, c, ldc, dc, static_cast<const float*>(w), bias, out, n_out);
  return cudaGetLastError();
}

}  // namespace gsit
