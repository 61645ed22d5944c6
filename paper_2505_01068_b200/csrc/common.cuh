// Shared device/host helpers of the IM attention library (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gsit.h"
#include "gsit_test.h"

namespace gsit {

// Problem geometry handed to every kernel by value.
struct Geometry {
  int batch, L, d, heads, hd;
  int seg_len[3];
  int seg_off[3];
  uint32_t allowed;          // bit (3*s + r): query segment s may attend key segment r
  const int32_t* valid_len;  // device [B][3] or nullptr
  unsigned int* status;      // device status word (GSIT_DEVFLAG_* bits), one per device
  // Packed row layout (nullptr = padded [B, L] layout): device int32 [3 B + 1]; entry 3 b + s is the first row of
  // segment s of sample b in a [capacity, d] matrix that holds real rows only, entry 3 B is the row after the last one.
  const int32_t* row_start;
  int capacity;              // rows of the packed matrices (host value, for the tensor maps)
};

__device__ __forceinline__ void raise_flag(const Geometry& g, unsigned int f) { atomicOr(g.status, f); }

// Real-row count of segment s in sample b, clamped to [0, seg_len[s]].
__device__ __forceinline__ int valid_rows(const Geometry& g, int b, int s) {
  if (g.valid_len == nullptr) return g.seg_len[s];
  int n = g.valid_len[3 * b + s];
  if (n < 0 || n > g.seg_len[s]) {
    raise_flag(g, GSIT_DEVFLAG_CLAMPED);
    n = n < 0 ? 0 : g.seg_len[s];
  }
  return n;
}

// First row of segment s of sample b in the activation matrices, and the range of rows that belongs to this problem.
__device__ __forceinline__ int seg_row0(const Geometry& g, int b, int s) {
  return (g.row_start != nullptr) ? g.row_start[3 * b + s] : b * g.L + g.seg_off[s];
}
__device__ __forceinline__ int rows_begin(const Geometry& g) { return (g.row_start != nullptr) ? g.row_start[0] : 0; }
__device__ __forceinline__ int rows_end(const Geometry& g) {
  return (g.row_start != nullptr) ? g.row_start[3 * g.batch] : g.batch * g.L;
}
// Rows of the activation matrices as the host knows them (bounds of the tensor maps).
inline int64_t matrix_rows(const Geometry& g) { return (g.row_start != nullptr) ? (int64_t)g.capacity : (int64_t)g.batch * g.L; }

__device__ __forceinline__ int segment_of(const Geometry& g, int p) {
  return (p >= g.seg_off[2]) ? 2 : (p >= g.seg_off[1]) ? 1 : 0;
}

// True iff row `row` of the flattened [B*L] sequence is a real (non padded) position.
__device__ __forceinline__ bool row_is_real(const Geometry& g, int64_t row) {
  const int b = (int)(row / g.L);
  const int p = (int)(row - (int64_t)b * g.L);
  const int s = segment_of(g, p);
  return (p - g.seg_off[s]) < valid_rows(g, b, s);
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}

// Per-device launch set-up (a process may drive several GPUs; kernel attributes and SM counts belong to a device):
// sets the kernel's dynamic shared-memory limit the first time `func` is launched on the current device and returns
// that device's SM count.  `func` identifies the kernel; at most 64 devices and 64 kernels are tracked.
inline cudaError_t sm_count_and_smem_once(const void* func, int smem_bytes, int* n_sm) {
  constexpr int MAX_DEV = 64, MAX_FUNC = 64;
  static int sm_count[MAX_DEV] = {};
  static const void* done[MAX_DEV][MAX_FUNC] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= MAX_DEV) return cudaErrorInvalidDevice;
  if (sm_count[dev] == 0) {
    e = cudaDeviceGetAttribute(&sm_count[dev], cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) { sm_count[dev] = 0; return e; }
  }
  if (n_sm != nullptr) *n_sm = sm_count[dev];
  if (func == nullptr) return cudaSuccess;
  int i = 0;
  while (i < MAX_FUNC && done[dev][i] != nullptr && done[dev][i] != func) ++i;
  if (i < MAX_FUNC && done[dev][i] == func) return cudaSuccess;
  e = cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
  if (e != cudaSuccess) return e;
  if (i < MAX_FUNC) done[dev][i] = func;  // beyond the table the attribute is simply set again on every launch
  return cudaSuccess;
}

// Launches `kernel` so that it may begin before the previous kernel of the stream has ended (programmatic dependent
// launch); the kernel itself waits for its predecessor with ptx::grid_dep_wait() before it touches dependent memory.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_overlapped(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// ---- host-side launch entry points of the kernel files (all asynchronous on `st`) ----
// Each returns cudaSuccess or the launch error.

// fp32 attention on CUDA cores (attn_f32.cu)
cudaError_t launch_attn_f32(const Geometry& g, const float* q, const float* k, const float* v, int64_t row_stride,
                            float* out, float* lse, float scale, cudaStream_t st);
// Operands of one bf16 attention problem; launch_attn_bf16_n serves one or two problems of the same geometry (same shape,
// valid lengths and layout; own tensors and block pattern) with one launch where the kernel family allows it.
struct AttnOperands {
  const __nv_bfloat16 *q, *k, *v;
  __nv_bfloat16* out;
  float* lse;
  uint32_t allowed;
};
cudaError_t launch_attn_bf16_n(const Geometry& g, const AttnOperands* ops, int n, int64_t row_stride, float scale, int* next_item,
                               cudaStream_t st, bool counter_cleared = false);
// bf16 attention, mma.sync tiles fed by TMA (attn_bf16.cu); returns cudaErrorNotSupported for shapes it lacks
cudaError_t launch_attn_bf16(const Geometry& g, const __nv_bfloat16* q, const __nv_bfloat16* k,
                             const __nv_bfloat16* v, int64_t row_stride, __nv_bfloat16* out, float* lse,
                             float scale, int* next_item, cudaStream_t st, bool counter_cleared = false);

// bf16 attention for head_dim 64 on tcgen05 tensor cores with TMEM accumulators (attn_tc.cu)
cudaError_t launch_attn_tc_hd64(const Geometry& g, const __nv_bfloat16* q, const __nv_bfloat16* k,
                                const __nv_bfloat16* v, int64_t row_stride, __nv_bfloat16* out, float* lse,
                                float scale, cudaStream_t st);

// bf16 attention for head_dim 8 / 16 / 32 on tcgen05 with thread-per-row softmax (attn_tcs.cu).  next_item: a device int
// the call may use as its work counter (cleared on the stream before the launch unless `counter_cleared` says that the
// kernel before this one in the stream has done so), or nullptr for a fixed assignment of work items to CTAs.
bool attn_tcs_supported(const Geometry& g);
cudaError_t launch_attn_tcs(const Geometry& g, const AttnOperands* ops, int n, int64_t row_stride, float scale, int* next_item,
                            cudaStream_t st, bool counter_cleared = false);

// Linear layers  C = act(A W^T + bias) (+ residual), rows that are padding written as zero when
// `mask_rows` is set.  A [M,K] (lda), W [N,K], C [M,N] (ldc), residual float [M,N] (ldr) or nullptr.
struct LinearArgs {
  const void* A; int64_t lda;
  const void* W;
  const float* bias;
  const float* residual; int64_t ldr;
  void* C; int64_t ldc;
  int M, N, K;
  int relu;
  int out_f32;      // bf16 path only: write float instead of bf16
  int mask_rows;    // zero the padded rows of C (uses geometry)
};
cudaError_t launch_linear_f32(const Geometry& g, const LinearArgs& a, cudaStream_t st);
// bf16 linear layer on tcgen05 tensor cores with TMEM accumulators (gemm_tc.cu): K a multiple of 64, N a multiple of 8
bool linear_tc_supported(const LinearArgs& a);
cudaError_t launch_linear_tc_bf16(const Geometry& g, const LinearArgs& a, cudaStream_t st);
cudaError_t launch_linear_bf16(const Geometry& g, const LinearArgs& a, cudaStream_t st);

// Fused halves of the layer for bf16 at d_model 64 / 128 with d_ff a multiple of 64 (fused_layer.cu):
//   qkv = LN1(x) W_qkv^T + b_qkv, and  y = y1 + relu(LN2(y1) W_1^T + b_1) W_2^T + b_2 with y1 = x + att W_o^T + b_o.
bool fused_layer_supported(const Geometry& g, int d_ff);
cudaError_t launch_ln_qkv_bf16(const Geometry& g, const float* x, int64_t ldx, const float* gamma, const float* beta,
                               float eps, const __nv_bfloat16* w_qkv, const float* b_qkv, __nv_bfloat16* qkv,
                               cudaStream_t st);
cudaError_t launch_proj_mlp_bf16(const Geometry& g, const __nv_bfloat16* att, const float* x, int64_t ldx,
                                 const __nv_bfloat16* w_o, const float* b_o, const float* gamma, const float* beta, float eps,
                                 const __nv_bfloat16* w_1, const float* b_1, const __nv_bfloat16* w_2, const float* b_2,
                                 int d_ff, float* y, int64_t ldy, cudaStream_t st);

// The same two halves at d_model 64 (d_ff <= 256) on tcgen05 tensor cores with TMEM accumulators (fused_layer_tc.cu).
// zero_word: a device int the first half clears (the work counter of the attention kernel that follows), or nullptr.
bool fused_layer_tc_supported(const Geometry& g, int d_ff);
cudaError_t launch_ln_qkv_tc(const Geometry& g, const float* x, int64_t ldx, const float* gamma, const float* beta, float eps,
                             const __nv_bfloat16* w_qkv, const float* b_qkv, __nv_bfloat16* qkv, int* zero_word, cudaStream_t st);
cudaError_t launch_proj_mlp_tc(const Geometry& g, const __nv_bfloat16* att, const float* x, int64_t ldx,
                               const __nv_bfloat16* w_o, const float* b_o, const float* gamma, const float* beta, float eps,
                               const __nv_bfloat16* w_1, const float* b_1, const __nv_bfloat16* w_2, const float* b_2, int d_ff,
                               float* y, int64_t ldy, cudaStream_t st);

// Both halves for a pair of problems of one geometry in one launch each (d_model 64): pointers of one problem.
struct FusedHalfArgs {
  const float* x; int64_t ldx;
  const float *ln1_gamma, *ln1_beta;
  const __nv_bfloat16* w_qkv; const float* b_qkv;
  __nv_bfloat16* qkv;            // written by the first half
  const __nv_bfloat16* att;      // read by the second half
  const __nv_bfloat16* w_o; const float* b_o;
  const float *ln2_gamma, *ln2_beta;
  const __nv_bfloat16* w_1; const float* b_1;
  const __nv_bfloat16* w_2; const float* b_2;
  float* y; int64_t ldy;
};
cudaError_t launch_ln_qkv_tc_pair(const Geometry& g, const FusedHalfArgs (&h)[2], float eps, int* zero_word, cudaStream_t st);
cudaError_t launch_proj_mlp_tc_pair(const Geometry& g, const FusedHalfArgs (&h)[2], float eps, int d_ff, cudaStream_t st);

// ... and at d_model 128 (d_ff <= 512), with the MLP weights streamed in chunks (fused_layer_tc128.cu)
bool fused_layer_tc128_supported(const Geometry& g, int d_ff);
cudaError_t launch_ln_qkv_tc128(const Geometry& g, const float* x, int64_t ldx, const float* gamma, const float* beta, float eps,
                                const __nv_bfloat16* w_qkv, const float* b_qkv, __nv_bfloat16* qkv, int* zero_word, cudaStream_t st);
cudaError_t launch_proj_mlp_tc128(const Geometry& g, const __nv_bfloat16* att, const float* x, int64_t ldx,
                                  const __nv_bfloat16* w_o, const float* b_o, const float* gamma, const float* beta, float eps,
                                  const __nv_bfloat16* w_1, const float* b_1, const __nv_bfloat16* w_2, const float* b_2, int d_ff,
                                  float* y, int64_t ldy, cudaStream_t st);

// Row LayerNorm of float x (row stride ldx) into float or bf16 y [rows, d]; padded rows become zero.
cudaError_t launch_layernorm(const Geometry& g, const float* x, int64_t ldx, const float* gamma, const float* beta,
                             float eps, void* y, int out_bf16, cudaStream_t st);

// Stack read-out: last real step of each segment of c [B, L, dc] (row stride ldc), concatenated, times w^T + bias.
cudaError_t launch_stack_head(const Geometry& g, int dtype, const float* c, int64_t ldc, int dc, const void* w,
                              const float* bias, float* out, int n_out, cudaStream_t st);

// packed row layout (rows.cu)
cudaError_t launch_plan_rows(const Geometry& g, int split_sample, int32_t* row_start, cudaStream_t st);
cudaError_t launch_move_rows(const Geometry& g, bool pack, const float* src, int64_t src_stride, float* dst, int64_t dst_stride,
                             int cols, cudaStream_t st);

}  // namespace gsit
