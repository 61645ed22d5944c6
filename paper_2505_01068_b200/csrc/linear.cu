// Linear layers and LayerNorm around the IM attention: C = act(A W^T + bias) (+ residual).
//   - bf16: cp.async-pipelined mma.sync.m16n8k16 tiles, float accumulate, fused bias / ReLU / residual /
//     padded-row zeroing epilogue, bf16 or float output.
//   - f32:  shared-memory tiled FMA kernel with the same epilogue (the 1e-4 parity path).
#include "common.cuh"

namespace gsit {
namespace {

// ------------------------------------------------------------------------------------------------ f32
constexpr int FT = 64, FK = 16;  // 64x64 tile, 16-deep slices, 256 threads of 4x4 outputs

__global__ void __launch_bounds__(256) linear_f32_kernel(Geometry g, LinearArgs a) {
  __shared__ float As[FK][FT + 1], Ws[FK][FT + 1];
  const float* A = static_cast<const float*>(a.A);
  const float* W = static_cast<const float*>(a.W);
  float* C = static_cast<float*>(a.C);
  const int m0 = blockIdx.y * FT, n0 = blockIdx.x * FT;
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  float acc[4][4] = {};
  for (int k0 = 0; k0 < a.K; k0 += FK) {
    for (int idx = threadIdx.x; idx < FT * FK; idx += 256) {
      const int r = idx / FK, kk = idx % FK;
      const int m = m0 + r, n = n0 + r, k = k0 + kk;
      As[kk][r] = (m < a.M && k < a.K) ? A[(int64_t)m * a.lda + k] : 0.f;
      Ws[kk][r] = (n < a.N && k < a.K) ? W[(int64_t)n * a.K + k] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < FK; ++kk) {
      float av[4], wv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { av[i] = As[kk][ty * 4 + i]; wv[i] = Ws[kk][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], wv[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= a.M) continue;
    const bool real = !a.mask_rows || row_is_real(g, m);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= a.N) continue;
      float v = acc[i][j] + (a.bias ? a.bias[n] : 0.f);
      if (a.relu) v = fmaxf(v, 0.f);
      if (a.residual) v += a.residual[(int64_t)m * a.ldr + n];
      C[(int64_t)m * a.ldc + n] = real ? v : 0.f;
    }
  }
}

// ------------------------------------------------------------------------------------------------ bf16
constexpr int BM = 128, BK = 32, GSTAGES = 3;

__device__ __forceinline__ uint32_t swz64(uint32_t off) { return off ^ (((off >> 7) & 3) << 4); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool pred) {
  const int sz = pred ? 16 : 0;  // size 0 zero-fills the 16 destination bytes
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}

template <int BN>
__global__ void __launch_bounds__(256) linear_bf16_kernel(Geometry g, LinearArgs a) {
  constexpr int WGN = (BN == 128) ? 4 : 2, WGM = 8 / WGN;
  constexpr int WTM = BM / WGM, WTN = BN / WGN;  // warp tile
  constexpr int MT = WTM / 16, NTL = WTN / 8;
  constexpr int A_BYTES = BM * BK * 2, W_BYTES = BN * BK * 2;
  __shared__ __align__(1024) uint8_t smem[GSTAGES * (A_BYTES + W_BYTES)];
  const uint32_t sA = smem_u32(smem), sW = sA + GSTAGES * A_BYTES;
  const __nv_bfloat16* A = static_cast<const __nv_bfloat16*>(a.A);
  const __nv_bfloat16* W = static_cast<const __nv_bfloat16*>(a.W);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int wm = warp / WGN, wn = warp % WGN;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  const int KT_ = (a.K + BK - 1) / BK;

  auto load_stage = [&](int kt, int st) {
    const int k0 = kt * BK;
    for (int idx = tid; idx < BM * 4; idx += 256) {  // 4 chunks of 16 B per 32-wide row
      const int r = idx >> 2, c = idx & 3;
      const bool ok = (m0 + r < a.M) && (k0 + c * 8 < a.K);
      const __nv_bfloat16* src = ok ? A + (int64_t)(m0 + r) * a.lda + k0 + c * 8 : A;
      cp_async16(sA + st * A_BYTES + swz64(r * 64 + c * 16), src, ok);
    }
    for (int idx = tid; idx < BN * 4; idx += 256) {
      const int r = idx >> 2, c = idx & 3;
      const bool ok = (n0 + r < a.N) && (k0 + c * 8 < a.K);
      const __nv_bfloat16* src = ok ? W + (int64_t)(n0 + r) * a.K + k0 + c * 8 : W;
      cp_async16(sW + st * W_BYTES + swz64(r * 64 + c * 16), src, ok);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };

  float acc[MT][NTL][4];
#pragma unroll
  for (int i = 0; i < MT; ++i)
#pragma unroll
    for (int j = 0; j < NTL; ++j) acc[i][j][0] = acc[i][j][1] = acc[i][j][2] = acc[i][j][3] = 0.f;

  for (int s = 0; s < GSTAGES - 1; ++s) {
    if (s < KT_) load_stage(s, s);
    else asm volatile("cp.async.commit_group;" ::: "memory");
  }
  for (int kt = 0; kt < KT_; ++kt) {
    asm volatile("cp.async.wait_group %0;" ::"n"(GSTAGES - 2) : "memory");
    __syncthreads();
    if (kt + GSTAGES - 1 < KT_) load_stage(kt + GSTAGES - 1, (kt + GSTAGES - 1) % GSTAGES);
    else asm volatile("cp.async.commit_group;" ::: "memory");
    const int st = kt % GSTAGES;
    const uint32_t aS = sA + st * A_BYTES, wS = sW + st * W_BYTES;
#pragma unroll
    for (int ks = 0; ks < BK / 16; ++ks) {
      uint32_t af[MT][4], bf[NTL][2];
      const int mi = lane >> 3;
#pragma unroll
      for (int i = 0; i < MT; ++i) {
        const int row = wm * WTM + i * 16 + (mi & 1) * 8 + (lane & 7);
        const uint32_t ad = aS + swz64(row * 64 + (ks * 2 + (mi >> 1)) * 16);
        asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                     : "=r"(af[i][0]), "=r"(af[i][1]), "=r"(af[i][2]), "=r"(af[i][3]) : "r"(ad));
      }
#pragma unroll
      for (int j = 0; j < NTL / 2; ++j) {
        const int row = wn * WTN + j * 16 + (mi >> 1) * 8 + (lane & 7);
        const uint32_t ad = wS + swz64(row * 64 + (ks * 2 + (mi & 1)) * 16);
        asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                     : "=r"(bf[2 * j][0]), "=r"(bf[2 * j][1]), "=r"(bf[2 * j + 1][0]), "=r"(bf[2 * j + 1][1]) : "r"(ad));
      }
#pragma unroll
      for (int i = 0; i < MT; ++i)
#pragma unroll
        for (int j = 0; j < NTL; ++j)
          asm volatile(
              "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
              : "+f"(acc[i][j][0]), "+f"(acc[i][j][1]), "+f"(acc[i][j][2]), "+f"(acc[i][j][3])
              : "r"(af[i][0]), "r"(af[i][1]), "r"(af[i][2]), "r"(af[i][3]), "r"(bf[j][0]), "r"(bf[j][1]));
    }
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");

  // ---- epilogue: bias, ReLU, residual, padded rows -> 0 ----
#pragma unroll
  for (int i = 0; i < MT; ++i)
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const int m = m0 + wm * WTM + i * 16 + (lane >> 2) + half * 8;
      if (m >= a.M) continue;
      const bool real = !a.mask_rows || row_is_real(g, m);
#pragma unroll
      for (int j = 0; j < NTL; ++j) {
        const int n = n0 + wn * WTN + j * 8 + (lane & 3) * 2;
        if (n >= a.N) continue;  // N is even, so n + 1 < N as well
        float v0 = acc[i][j][half * 2], v1 = acc[i][j][half * 2 + 1];
        if (a.bias) { v0 += a.bias[n]; v1 += a.bias[n + 1]; }
        if (a.relu) { v0 = fmaxf(v0, 0.f); v1 = fmaxf(v1, 0.f); }
        if (a.residual) {
          const float2 r = *reinterpret_cast<const float2*>(a.residual + (int64_t)m * a.ldr + n);
          v0 += r.x; v1 += r.y;
        }
        if (!real) v0 = v1 = 0.f;
        if (a.out_f32)
          *reinterpret_cast<float2*>(static_cast<float*>(a.C) + (int64_t)m * a.ldc + n) = make_float2(v0, v1);
        else
          *reinterpret_cast<__nv_bfloat162*>(static_cast<__nv_bfloat16*>(a.C) + (int64_t)m * a.ldc + n) =
              __floats2bfloat162_rn(v0, v1);
      }
    }
}

// ------------------------------------------------------------------------------------------------ LayerNorm
template <typename OutT>
__global__ void __launch_bounds__(256) layernorm_kernel(Geometry g, const float* __restrict__ x, int64_t ldx,
                                                        const float* __restrict__ gamma, const float* __restrict__ beta,
                                                        float eps, OutT* __restrict__ y, int64_t rows) {
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= rows) return;
  const int d = g.d;
  OutT* yr = y + row * d;
  if (!row_is_real(g, row)) {
    for (int e = lane; e < d; e += 32) yr[e] = OutT(0.f);
    return;
  }
  const float* xr = x + row * ldx;
  float s = 0.f;
  for (int e = lane; e < d; e += 32) s += xr[e];
  for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  const float mean = s / d;
  float vs = 0.f;
  for (int e = lane; e < d; e += 32) { const float t = xr[e] - mean; vs = fmaf(t, t, vs); }
  for (int o = 16; o; o >>= 1) vs += __shfl_xor_sync(0xffffffffu, vs, o);
  const float rstd = rsqrtf(vs / d + eps);
  for (int e = lane; e < d; e += 32) {
    const float v = (xr[e] - mean) * rstd * (gamma ? gamma[e] : 1.f) + (beta ? beta[e] : 0.f);
    yr[e] = OutT(v);
  }
}

}  // namespace

cudaError_t launch_linear_f32(const Geometry& g, const LinearArgs& a, cudaStream_t st) {
  const dim3 grid((a.N + FT - 1) / FT, (a.M + FT - 1) / FT);
  if (grid.y > 65535) return cudaErrorNotSupported;
  linear_f32_kernel<<<grid, 256, 0, st>>>(g, a);
  return cudaGetLastError();
}

extern int g_attn_variant;  // kernel selection (attn_bf16.cu): GSIT_ATTN_LEGACY keeps every bf16 kernel on the mma.sync path

cudaError_t launch_linear_bf16(const Geometry& g, const LinearArgs& a, cudaStream_t st) {
  if (g_attn_variant != GSIT_ATTN_LEGACY && linear_tc_supported(a)) return launch_linear_tc_bf16(g, a, st);
  if (a.K % 8 != 0 || a.N % 2 != 0 || a.lda % 8 != 0) return cudaErrorNotSupported;
  const bool wide = (a.N % 128 == 0) || a.N > 256;
  const int bn = wide ? 128 : 64;
  const dim3 grid((a.N + bn - 1) / bn, (a.M + BM - 1) / BM);
  if (grid.y > 65535) return cudaErrorNotSupported;
  if (wide) linear_bf16_kernel<128><<<grid, 256, 0, st>>>(g, a);
  else linear_bf16_kernel<64><<<grid, 256, 0, st>>>(g, a);
  return cudaGetLastError();
}

cudaError_t launch_layernorm(const Geometry& g, const float* x, int64_t ldx, const float* gamma, const float* beta,
                             float eps, void* y, int out_bf16, cudaStream_t st) {
  const int64_t rows = (int64_t)g.batch * g.L;
  const unsigned blocks = (unsigned)((rows + 7) / 8);
  if (out_bf16)
    layernorm_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(g, x, ldx, gamma, beta, eps, static_cast<__nv_bfloat16*>(y), rows);
  else
    layernorm_kernel<float><<<blocks, 256, 0, st>>>(g, x, ldx, gamma, beta, eps, static_cast<float*>(y), rows);
  return cudaGetLastError();
}

}  // namespace gsit
