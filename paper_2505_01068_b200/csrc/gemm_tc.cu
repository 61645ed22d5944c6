// bf16 linear layer C = act(A W^T + bias) (+ residual) on the 5th-generation tensor cores (tcgen05), for the shared
// QKV projection at large d_model (Section "Multimodal Transformers as Graphs": one W_q, W_k, W_v for the whole
// concatenated sequence) and for any other linear layer of the path whose inner width is a multiple of 64.
//
// Persistent grid, one CTA per SM, six warps:
//   warp 0      TMA producer: per 64-wide k-block one A box (128 rows x 128 B) and one W box (BN rows x 128 B), 128-byte
//               swizzle, into a ring of up to six stages
//   warp 1      allocates 512 TMEM columns and issues tcgen05.mma.kind::f16, M 128, N = BN (16..256), K 16, both operands
//               from shared memory; the accumulator is double-buffered (2 x 256 columns), so the epilogue of tile i
//               overlaps the main loop of tile i+1
//   warps 2..5  epilogue: thread = output row = TMEM lane; tcgen05.ld, bias / ReLU / residual / padded-row zeroing.
//               bf16 output without residual (the QKV projection): rows are staged in shared memory in the 128-byte
//               swizzle and written by TMA stores (64 columns x 128 rows per box), which also clip at the matrix
//               edge; other epilogues store 16 bytes per thread directly
// Tiles are numbered with the column tile fastest, so the CTAs that share an A tile run at the same time and W stays
// in L2.  Every wait is bounded (GSIT_DEVFLAG_TIMEOUT instead of a hang) and TMEM is always released.
#include <cuda.h>

#include "common.cuh"
#include "ptx.cuh"
#include "tensor_map.cuh"
#include "tmem_ldst.cuh"

namespace gsit {
namespace {

using namespace ptx;

constexpr int GM = 128, GK = 64;          // rows per tile, k-block width
constexpr int G_THREADS = 192;
constexpr int A_STAGE = GM * GK * 2;      // 16 KB
constexpr int G_MAX_STAGES = 6;
constexpr int G_BAR_BYTES = 256;
constexpr int G_MIN_SMEM = 120 * 1024;    // more than half an SM's shared memory: one CTA per SM, so 512 TMEM columns fit

struct GemmParams {
  int M, N, K;
  int bn;            // columns per tile (multiple of 16, <= 256)
  int tiles_n, n_tiles;
  int stages, stage_bytes;
  const float* bias;
  const float* residual; int64_t ldr;
  void* C; int64_t ldc;
  int relu, out_f32, mask_rows;
  int packed;        // rows are the packed layout's: only rows_begin(g) .. rows_end(g) - 1 (read on the device) are computed
                     // and written, all of them real; everything outside that range is left untouched
  int tma_store;     // bf16 output through the shared-memory staging area and TMA stores
  int staging_off;   // offset of the staging area from the aligned base
};

__global__ void __launch_bounds__(G_THREADS, 1)
linear_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW,
                 const __grid_constant__ CUtensorMap tmC, const Geometry g, const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bars = base + p.staging_off + (p.tma_store ? (p.bn / 64) * 16384 : 0);
  const uint32_t bar_full = bars, bar_empty = bars + 8 * G_MAX_STAGES, bar_accf = bars + 16 * G_MAX_STAGES,
                 bar_acce = bar_accf + 16, slot = bar_acce + 16, slot_gave_up = slot + 4;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const WaitCtx wc{g.status, slot_gave_up};
  const int kblocks = p.K / GK;

  if (tid == 0) {
    for (int i = 0; i < p.stages; ++i) { mbar_init(bar_full + 8 * i, 1); mbar_init(bar_empty + 8 * i, 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(bar_accf + 8 * i, 1); mbar_init(bar_acce + 8 * i, 4); }
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(slot_gave_up), "r"(0u) : "memory");
    mbar_init_fence();
  }
  if (warp == 1) tmem_alloc(slot, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  uint32_t tmem;
  asm volatile("ld.shared.b32 %0, [%1];" : "=r"(tmem) : "r"(slot) : "memory");
  // rows this call computes; a row tile wholly outside them is skipped by every role alike
  const int row_lo = p.packed ? rows_begin(g) : 0, row_hi = p.packed ? rows_end(g) : p.M;
  auto tile_outside = [&](int m0) { return m0 + GM <= row_lo || m0 >= row_hi; };

  if (warp == 0) {
    // ================================ TMA producer ================================
    int n = 0;  // k-blocks requested so far
    for (int t = blockIdx.x; t < p.n_tiles; t += gridDim.x) {
      const int m0 = (t / p.tiles_n) * GM, n0 = (t % p.tiles_n) * p.bn;
      if (tile_outside(m0)) continue;
      for (int kb = 0; kb < kblocks; ++kb, ++n) {
        const int st = n % p.stages, use = n / p.stages;
        if (use > 0) mbar_wait(wc, bar_empty + 8 * st, (use - 1) & 1);
        if (elect_one()) {
          const uint32_t sA = base + st * p.stage_bytes;
          mbar_expect_tx(bar_full + 8 * st, (uint32_t)(A_STAGE + p.bn * GK * 2));
          tma_load_2d(sA, &tmA, kb * GK, m0, bar_full + 8 * st);
          tma_load_2d(sA + A_STAGE, &tmW, kb * GK, n0, bar_full + 8 * st);
        }
        __syncwarp();
      }
    }
  } else if (warp == 1) {
    // ================================ MMA issuer ================================
    const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.bn >> 3) << 17) | ((uint32_t)(GM >> 4) << 24);
    int n = 0, i = 0;  // k-blocks consumed, tiles done by this CTA
    for (int t = blockIdx.x; t < p.n_tiles; t += gridDim.x) {
      if (tile_outside((t / p.tiles_n) * GM)) continue;
      const int ab = i & 1;
      if (i >= 2) mbar_wait(wc, bar_acce + 8 * ab, ((i >> 1) - 1) & 1);  // the epilogue has drained this accumulator
      tc_fence_after();
      for (int kb = 0; kb < kblocks; ++kb, ++n) {
        const int st = n % p.stages;
        mbar_wait(wc, bar_full + 8 * st, (n / p.stages) & 1);
        tc_fence_after();
        if (elect_one()) {
          const uint32_t sA = base + st * p.stage_bytes;
#pragma unroll
          for (int k = 0; k < GK / 16; ++k)
            umma_ss(tmem + ab * 256, smem_desc_sw128(sA + 32 * k), smem_desc_sw128(sA + A_STAGE + 32 * k), idesc, (kb > 0 || k > 0) ? 1u : 0u);
          umma_commit(bar_empty + 8 * st);
          if (kb + 1 == kblocks) umma_commit(bar_accf + 8 * ab);
        }
        __syncwarp();
      }
      ++i;
    }
  } else {
    // ================================ epilogue: one thread per output row ================================
    const int quarter = warp & 3;
    const uint32_t tl = tmem + ((uint32_t)(quarter << 5) << 16);
    int i = 0;
    for (int t = blockIdx.x; t < p.n_tiles; t += gridDim.x) {
      const int m0 = (t / p.tiles_n) * GM, n0 = (t % p.tiles_n) * p.bn;
      if (tile_outside(m0)) continue;
      const int ab = i & 1;
      const int64_t row = (int64_t)m0 + quarter * 32 + lane;
      const bool in_m = row >= row_lo && row < row_hi;
      const bool real = in_m && (!p.mask_rows || p.packed || row_is_real(g, row));
      mbar_wait(wc, bar_accf + 8 * ab, (i >> 1) & 1);
      tc_fence_after();
      if (p.tma_store) {
        const uint32_t stg = base + p.staging_off;
        const int r = quarter * 32 + lane;
        if (i > 0) {  // the previous tile's stores must have finished reading the staging area
          if (tid == 64) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
          asm volatile("bar.sync 1, 128;" ::: "memory");
        }
        for (int c0 = 0; c0 < p.bn; c0 += 32) {
          uint32_t v[32];
          tmem_ld32(tl + ab * 256 + c0, v);
          tmem_wait_ld();
          tmem_regs_ready(v);
          const int col0 = n0 + c0;
          uint32_t pk[16];
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            float f0 = __uint_as_float(v[e]), f1 = __uint_as_float(v[e + 1]);
            if (p.bias != nullptr && col0 + e < p.N) { f0 += p.bias[col0 + e]; f1 += p.bias[col0 + e + 1]; }
            if (p.relu) { f0 = fmaxf(f0, 0.f); f1 = fmaxf(f1, 0.f); }
            if (!real) { f0 = 0.f; f1 = 0.f; }
            pk[e >> 1] = pack_bf16(f0, f1);
          }
          // box (c0 / 64), row r, 16-byte chunks (c0 % 64) / 8 .. +3, swizzled with the row
          const uint32_t rowp = stg + (c0 >> 6) * 16384 + r * 128;
          const int ch0 = (c0 & 32) >> 3;
#pragma unroll
          for (int q = 0; q < 4; ++q)
            asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(rowp + (((ch0 + q) ^ (r & 7)) << 4)), "r"(pk[4 * q]),
                         "r"(pk[4 * q + 1]), "r"(pk[4 * q + 2]), "r"(pk[4 * q + 3]) : "memory");
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_acce + 8 * ab);  // the accumulator is in shared memory: free it
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (tid == 64) {
          for (int j = 0; j < p.bn / 64; ++j)
            if (n0 + 64 * j < p.N) tma_store_2d(&tmC, stg + j * 16384, n0 + 64 * j, m0);
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
        ++i;
        continue;
      }
      for (int c0 = 0; c0 < p.bn; c0 += 32) {
        uint32_t v[32];
        tmem_ld32(tl + ab * 256 + c0, v);
        tmem_wait_ld();
        tmem_regs_ready(v);
        const int col0 = n0 + c0;
        if (in_m && col0 < p.N) {
          float f[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) f[e] = __uint_as_float(v[e]);
          if (p.bias != nullptr) {
#pragma unroll
            for (int e = 0; e < 32; ++e)
              if (col0 + e < p.N) f[e] += p.bias[col0 + e];
          }
          if (p.relu) {
#pragma unroll
            for (int e = 0; e < 32; ++e) f[e] = fmaxf(f[e], 0.f);
          }
          if (p.residual != nullptr) {
            const float* rr = p.residual + row * p.ldr + col0;
#pragma unroll
            for (int e = 0; e < 32; e += 4)
              if (col0 + e < p.N) {  // N is a multiple of 8, so groups of 4 are all inside or all outside
                const float4 r4 = *reinterpret_cast<const float4*>(rr + e);
                f[e] += r4.x; f[e + 1] += r4.y; f[e + 2] += r4.z; f[e + 3] += r4.w;
              }
          }
          if (!real) {
#pragma unroll
            for (int e = 0; e < 32; ++e) f[e] = 0.f;
          }
          if (p.out_f32) {
            float* dst = static_cast<float*>(p.C) + row * p.ldc + col0;
#pragma unroll
            for (int e = 0; e < 32; e += 4)
              if (col0 + e < p.N) *reinterpret_cast<float4*>(dst + e) = make_float4(f[e], f[e + 1], f[e + 2], f[e + 3]);
          } else {
            __nv_bfloat16* dst = static_cast<__nv_bfloat16*>(p.C) + row * p.ldc + col0;
#pragma unroll
            for (int e = 0; e < 32; e += 8)
              if (col0 + e < p.N)
                *reinterpret_cast<uint4*>(dst + e) = make_uint4(pack_bf16(f[e], f[e + 1]), pack_bf16(f[e + 2], f[e + 3]),
                                                                pack_bf16(f[e + 4], f[e + 5]), pack_bf16(f[e + 6], f[e + 7]));
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_acce + 8 * ab);
      ++i;
    }
  }

  if (tid == 64) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");  // outstanding TMA stores of this CTA
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

}  // namespace

// Shapes the tensor-core path covers; everything else stays on the mma.sync kernel.
bool linear_tc_supported(const LinearArgs& a) {
  return a.K >= GK && a.K % GK == 0 && a.N >= 16 && a.N % 8 == 0 && a.lda % 8 == 0 && a.M >= 1 &&
         (a.out_f32 ? a.ldc % 4 == 0 : a.ldc % 8 == 0) && (a.residual == nullptr || a.ldr % 4 == 0);
}

cudaError_t launch_linear_tc_bf16(const Geometry& g, const LinearArgs& a, cudaStream_t st) {
  if (!linear_tc_supported(a)) return cudaErrorNotSupported;
  GemmParams p = {};
  p.M = a.M; p.N = a.N; p.K = a.K;
  const int nt = (a.N + 255) / 256;
  p.bn = (((a.N + nt - 1) / nt) + 15) & ~15;
  p.tiles_n = (a.N + p.bn - 1) / p.bn;
  const int64_t tiles = (int64_t)((a.M + GM - 1) / GM) * p.tiles_n;
  if (tiles > 0x7fffffffLL) return cudaErrorNotSupported;
  p.n_tiles = (int)tiles;
  p.stage_bytes = A_STAGE + ((p.bn * GK * 2 + 1023) & ~1023);
  p.bias = a.bias; p.residual = a.residual; p.ldr = a.ldr; p.C = a.C; p.ldc = a.ldc;
  p.relu = a.relu; p.out_f32 = a.out_f32; p.mask_rows = a.mask_rows;
  p.packed = (g.row_start != nullptr) ? 1 : 0;
  // TMA stores write whole tiles; in the packed layout the rows of a boundary tile that lie outside this call's range
  // belong to other samples, so there every thread stores its own row
  p.tma_store = (!p.packed && !a.out_f32 && a.residual == nullptr && p.bn % 64 == 0 && a.N % 8 == 0 &&
                 (reinterpret_cast<uintptr_t>(a.C) & 15u) == 0) ? 1 : 0;
  const int staging = p.tma_store ? (p.bn / 64) * 16384 : 0;
  const int budget = 227 * 1024 - 1024 - G_BAR_BYTES - staging;
  p.stages = budget / p.stage_bytes;
  if (p.stages > G_MAX_STAGES) p.stages = G_MAX_STAGES;
  if (p.stages < 2) return cudaErrorNotSupported;
  p.staging_off = p.stages * p.stage_bytes;
  int smem = p.staging_off + staging + G_BAR_BYTES + 1024;
  if (smem < G_MIN_SMEM) smem = G_MIN_SMEM;
  alignas(64) CUtensorMap tmA, tmW, tmC;
  if (!make_map(&tmA, a.A, a.M, a.K, a.lda, GK, GM) || !make_map(&tmW, a.W, a.N, a.K, a.K, GK, p.bn))
    return cudaErrorInvalidValue;
  if (p.tma_store) {
    if (!make_map(&tmC, a.C, a.M, a.N, a.ldc, 64, GM)) return cudaErrorInvalidValue;
  } else {
    tmC = tmA;  // unused by the kernel on this path
  }
  int n_sm = 0;
  {
    cudaError_t e = sm_count_and_smem_once(reinterpret_cast<const void*>(linear_tc_kernel), 227 * 1024, &n_sm);
    if (e != cudaSuccess) return e;
  }
  const unsigned grid = (unsigned)(p.n_tiles < n_sm ? p.n_tiles : n_sm);
  linear_tc_kernel<<<grid, G_THREADS, smem, st>>>(tmA, tmW, tmC, g, p);
  return cudaGetLastError();
}

}  // namespace gsit
