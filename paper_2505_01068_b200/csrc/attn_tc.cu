// bf16 IM attention for head_dim 64 on the 5th-generation tensor cores (tcgen05) with accumulators in tensor
// memory (TMEM), fed by TMA.
//
// Decomposition (paper, Section "Inner Decomposition for Efficiency"; Appendix A "From Set to Set Aggregation"):
// a CTA owns 128 query rows of one modality segment of one head of one sample and walks only the key tiles of
// the segment(s) the Interlaced Mask opens for that block row, up to the sample's valid length.
//
// Roles inside a CTA of 6 warps (two CTAs share an SM, so one CTA's softmax overlaps the other's MMAs):
//   warp 0, one thread   TMA producer: Q once, then K and V tiles of 128 keys into two-stage rings
//   warp 1               allocates 256 TMEM columns; one thread issues every tcgen05.mma
//                          S = Q K^T   (M 128, N 128, K 64: A and B from shared memory, 128-byte swizzle)
//                          O += P V    (M 128, N 64, K 128: A = P from TMEM, B = V tile as loaded, MN-major)
//   warps 2..5           softmax: thread = query row = TMEM lane.  Reads S with tcgen05.ld, keeps the running
//                        maximum and sum in registers, writes P (bf16 pairs) back to TMEM with tcgen05.st, rescales
//                        O in TMEM only when the maximum has grown by more than 2^8, and writes the result.
// TMEM columns: [0,128) S fp32, [128,192) P bf16x2, [192,256) O fp32.
// Every wait is bounded; when one expires GSIT_DEVFLAG_TIMEOUT is raised, all later waits give up at once and
// the CTA still releases its TMEM and returns.
#include <cuda.h>

#include "common.cuh"
#include "tensor_map.cuh"
#include "tmem_ldst.cuh"

namespace gsit {
namespace {

constexpr int TQ = 128, TK = 128, HD64 = 64;
constexpr int KV_STAGES = 2;
constexpr int TILE_BYTES = 128 * 128;  // 128 rows of 128 bytes
constexpr int TC_THREADS = 192;
constexpr int TMEM_COLS = 256, COL_S = 0, COL_P = 128, COL_O = 192;
constexpr int SPIN_LIMIT = 1 << 18;
// shared-memory map, relative to a 1024-byte aligned base
constexpr int OFF_Q = 0, OFF_K = TILE_BYTES, OFF_V = OFF_K + KV_STAGES * TILE_BYTES, OFF_BAR = OFF_V + KV_STAGES * TILE_BYTES;
constexpr int BAR_Q = 0, BAR_KFULL = 8, BAR_VFULL = 24, BAR_KEMPTY = 40, BAR_VEMPTY = 56, BAR_SFULL = 72, BAR_PFULL = 80,
              BAR_OFINAL = 88, SLOT_TMEM = 96;
constexpr int TC_SMEM = OFF_BAR + 128 + 1024 /* alignment slack */;

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Gives up after SPIN_LIMIT polls (raising the timeout flag), or as soon as another wait anywhere on
// the device has already raised it, so that a broken pipeline drains in milliseconds instead of stalling the GPU.
__device__ __forceinline__ void mbar_wait(const Geometry& g, uint32_t bar, uint32_t parity) {
  for (int it = 0; it < SPIN_LIMIT; ++it) {
    if (mbar_test(bar, parity)) return;
    if (it > 32) __nanosleep(32);
    if ((it & 255) == 255 && (*reinterpret_cast<volatile unsigned int*>(g.status) & GSIT_DEVFLAG_TIMEOUT)) return;
  }
  raise_flag(g, GSIT_DEVFLAG_TIMEOUT);
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor for tiles whose rows are 128 bytes with the 128-byte swizzle (what TMA wrote):
// groups of 8 rows are 1024 bytes apart (stride byte offset); the leading byte offset is unused for these shapes.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)(1024u >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor, kind::f16: D = f32, A = B = bf16, M = 128, N = n; b_mn_major: B is stored N-contiguous.
__host__ __device__ constexpr uint32_t idesc_bf16(int n, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(128 >> 4) << 24);
}
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
// Makes the barrier complete once every tcgen05.mma issued so far by this thread has finished.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

template <bool V> struct BoolTag { static constexpr bool value = V; };

__global__ void __launch_bounds__(TC_THREADS, 2)
attn_tc_hd64_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const Geometry g, __nv_bfloat16* __restrict__ out,
                    float* __restrict__ lse, const float sl2 /* scale * log2(e) */) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sQ = base + OFF_Q, sK = base + OFF_K, sV = base + OFF_V, bars = base + OFF_BAR;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // ---- which query tile of which block row ----
  int tile = blockIdx.x, s = 0;
#pragma unroll
  for (int ss = 0; ss < 2; ++ss) {
    const int nts = (g.seg_len[s] + TQ - 1) / TQ;
    if (tile >= nts) { tile -= nts; ++s; }
  }
  const int q0 = tile * TQ;
  const int rows_in_tile = min(TQ, g.seg_len[s] - q0);
  const int h = blockIdx.y, b = blockIdx.z;
  const int q_real_all = max(0, min(rows_in_tile, valid_rows(g, b, s) - q0));
  const int kn0 = ((g.allowed >> (3 * s + 0)) & 1u) ? valid_rows(g, b, 0) : 0;
  const int kn1 = ((g.allowed >> (3 * s + 1)) & 1u) ? valid_rows(g, b, 1) : 0;
  const int kn2 = ((g.allowed >> (3 * s + 2)) & 1u) ? valid_rows(g, b, 2) : 0;
  const int nk0 = (kn0 + TK - 1) / TK, nk1 = (kn1 + TK - 1) / TK, nk2 = (kn2 + TK - 1) / TK;
  const int T = (q_real_all > 0) ? nk0 + nk1 + nk2 : 0;  // key tiles this CTA walks
  const int q_real = (T > 0) ? q_real_all : 0;
  const int64_t grow0 = (int64_t)b * g.L + g.seg_off[s] + q0;
  const int xcol = h * HD64;
  const int off1 = g.seg_off[1], off2 = g.seg_off[2];

  auto locate = [&](int i, int& krem, int& yrow) {  // key tile i: real keys left from its start, first global row
    int t = i, r = 0;
    if (t >= nk0) { t -= nk0; r = 1; if (t >= nk1) { t -= nk1; r = 2; } }
    const int kn = (r == 0) ? kn0 : (r == 1) ? kn1 : kn2;
    const int off = (r == 0) ? 0 : (r == 1) ? off1 : off2;
    krem = kn - t * TK;
    yrow = b * g.L + off + t * TK;
  };

  if (T == 0) {  // nothing to attend (padding rows only, or an empty key set): exact zeros, lse = -inf
    if (warp >= 2) {
      const int r = ((warp & 3) << 5) + lane;
      if (r < rows_in_tile) {
        uint4* dst = reinterpret_cast<uint4*>(out + (grow0 + r) * g.d + xcol);
#pragma unroll
        for (int c = 0; c < 8; ++c) dst[c] = make_uint4(0, 0, 0, 0);
        if (lse != nullptr) lse[((int64_t)b * g.heads + h) * g.L + g.seg_off[s] + q0 + r] = -INFINITY;
      }
    }
    return;
  }

  // ---- set-up: barriers, tensor memory ----
  if (tid == 0) {
    mbar_init(bars + BAR_Q, 1);
#pragma unroll
    for (int st = 0; st < KV_STAGES; ++st) {
      mbar_init(bars + BAR_KFULL + 8 * st, 1);
      mbar_init(bars + BAR_VFULL + 8 * st, 1);
      mbar_init(bars + BAR_KEMPTY + 8 * st, 1);
      mbar_init(bars + BAR_VEMPTY + 8 * st, 1);
    }
    mbar_init(bars + BAR_SFULL, 1);
    mbar_init(bars + BAR_PFULL, 128);
    mbar_init(bars + BAR_OFINAL, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(bars + SLOT_TMEM), "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  uint32_t tmem;
  asm volatile("ld.shared.b32 %0, [%1];" : "=r"(tmem) : "r"(bars + SLOT_TMEM) : "memory");

  if (warp == 0) {
    // ================================ TMA producer ================================
    if (lane == 0) {
      mbar_expect_tx(bars + BAR_Q, TILE_BYTES);
      tma_load_2d(sQ, &tmQ, xcol, (int)grow0, bars + BAR_Q);
      for (int i = 0; i < T; ++i) {
        int krem, yrow;
        locate(i, krem, yrow);
        const int st = i % KV_STAGES, use = i / KV_STAGES;
        if (use > 0) mbar_wait(g, bars + BAR_KEMPTY + 8 * st, (use - 1) & 1);
        mbar_expect_tx(bars + BAR_KFULL + 8 * st, TILE_BYTES);
        tma_load_2d(sK + st * TILE_BYTES, &tmK, xcol, yrow, bars + BAR_KFULL + 8 * st);
        if (use > 0) mbar_wait(g, bars + BAR_VEMPTY + 8 * st, (use - 1) & 1);
        mbar_expect_tx(bars + BAR_VFULL + 8 * st, TILE_BYTES);
        tma_load_2d(sV + st * TILE_BYTES, &tmV, xcol, yrow, bars + BAR_VFULL + 8 * st);
      }
    }
  } else if (warp == 1) {
    // ================================ MMA issuer ================================
    if (lane == 0) {
      constexpr uint32_t IDESC_QK = idesc_bf16(TK, false), IDESC_PV = idesc_bf16(HD64, true);
      auto issue_qk = [&](int i) {  // S = Q K_i^T, four steps of 16 along head_dim (32 bytes inside the swizzle row)
        const int st = i % KV_STAGES;
        mbar_wait(g, bars + BAR_KFULL + 8 * st, (i / KV_STAGES) & 1);
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < HD64 / 16; ++k)
          umma_ss(tmem + COL_S, smem_desc_sw128(sQ + 32 * k), smem_desc_sw128(sK + st * TILE_BYTES + 32 * k), IDESC_QK, k > 0);
        umma_commit(bars + BAR_KEMPTY + 8 * st);
        umma_commit(bars + BAR_SFULL);
      };
      mbar_wait(g, bars + BAR_Q, 0);
      issue_qk(0);
      for (int j = 0; j < T; ++j) {
        const int st = j % KV_STAGES;
        mbar_wait(g, bars + BAR_PFULL, j & 1);  // P_j is in TMEM and S_j has been read
        mbar_wait(g, bars + BAR_VFULL + 8 * st, (j / KV_STAGES) & 1);
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < TK / 16; ++k)  // O += P V_j, eight steps of 16 keys (two 8-row groups = 2048 bytes of V)
          umma_ts(tmem + COL_O, tmem + COL_P + 8 * k, smem_desc_sw128(sV + st * TILE_BYTES + 2048 * k), IDESC_PV,
                  (j > 0 || k > 0) ? 1u : 0u);
        umma_commit(bars + BAR_VEMPTY + 8 * st);
        if (j + 1 < T) issue_qk(j + 1);
        else umma_commit(bars + BAR_OFINAL);
      }
    }
  } else {
    // ================================ softmax, one thread per query row ================================
    const int r = ((warp & 3) << 5) + lane;                    // row in the tile = TMEM lane
    const uint32_t tl = tmem + ((uint32_t)((warp & 3) << 5) << 16);  // this warp's lane quarter
    float m_used = -INFINITY, l = 0.f;

    auto tile_step = [&](auto ragged_tag, const int j, const int krem) {
      constexpr bool RAGGED = decltype(ragged_tag)::value;
      mbar_wait(g, bars + BAR_SFULL, j & 1);
      tc_fence_after();
      uint32_t sr[4][32];
#pragma unroll
      for (int c = 0; c < 4; ++c) tmem_ld32(tl + COL_S + 32 * c, sr[c]);
      tmem_wait_ld();
      float mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < 4; ++c)
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          float v = __uint_as_float(sr[c][e]);
          if (RAGGED) { if (c * 32 + e >= krem) { v = -INFINITY; sr[c][e] = __float_as_uint(v); } }
          mx = fmaxf(mx, v);
        }
      // rescale only when the maximum has grown by more than 2^8 (P stays below 256, exact enough in bf16 and f32)
      const bool grow = (j == 0) || ((mx - m_used) * sl2 > 8.f);
      if (j > 0 && __any_sync(0xffffffffu, grow)) {
        const float alpha = grow ? ex2((m_used - mx) * sl2) : 1.f;
        l *= alpha;
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          uint32_t o[32];
          tmem_ld32(tl + COL_O + 32 * c, o);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
          tmem_st32(tl + COL_O + 32 * c, o);
        }
      }
      if (grow) m_used = mx;
      const float msl = m_used * sl2;
      float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        uint32_t pr[32];
#pragma unroll
        for (int c = 0; c < 2; ++c)
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            const float p0 = ex2(fmaf(__uint_as_float(sr[2 * hh + c][e]), sl2, -msl));
            const float p1 = ex2(fmaf(__uint_as_float(sr[2 * hh + c][e + 1]), sl2, -msl));
            sum0 += p0;
            sum1 += p1;
            pr[c * 16 + e / 2] = pack_bf16(p0, p1);
          }
        tmem_st32(tl + COL_P + 32 * hh, pr);
      }
      l += sum0 + sum1;
      if (RAGGED) {
        // Rows of the V tile past the valid length hold whatever follows in memory; a zero weight times NaN or Inf
        // would still poison the accumulator, so clear them before the MMA reads the tile.
        const int st = j % KV_STAGES;
        mbar_wait(g, bars + BAR_VFULL + 8 * st, (j / KV_STAGES) & 1);
        const int row = krem + (tid - 64);
        if (row < TK) {
          const uint32_t a = sV + st * TILE_BYTES + row * 128;
#pragma unroll
          for (int c = 0; c < 8; ++c)
            asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(a + 16 * c), "r"(0) : "memory");
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(bars + BAR_PFULL);
    };

    for (int j = 0; j < T; ++j) {
      int krem, yrow;
      locate(j, krem, yrow);
      if (krem < TK) tile_step(BoolTag<true>{}, j, krem);
      else tile_step(BoolTag<false>{}, j, TK);
    }

    // ---- epilogue: O / l -> bf16, each thread its own 128-byte row; padded rows +0 ----
    mbar_wait(g, bars + BAR_OFINAL, 0);
    tc_fence_after();
    const float inv = (l > 0.f) ? 1.f / l : 0.f;
    uint4* dst = reinterpret_cast<uint4*>(out + (grow0 + r) * g.d + xcol);
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      uint32_t o[32];
      tmem_ld32(tl + COL_O + 32 * c, o);
      tmem_wait_ld();
      if (r < rows_in_tile) {
        const bool real = r < q_real;
#pragma unroll
        for (int e = 0; e < 32; e += 8) {
          uint4 v = make_uint4(0, 0, 0, 0);
          if (real) {
            v.x = pack_bf16(__uint_as_float(o[e + 0]) * inv, __uint_as_float(o[e + 1]) * inv);
            v.y = pack_bf16(__uint_as_float(o[e + 2]) * inv, __uint_as_float(o[e + 3]) * inv);
            v.z = pack_bf16(__uint_as_float(o[e + 4]) * inv, __uint_as_float(o[e + 5]) * inv);
            v.w = pack_bf16(__uint_as_float(o[e + 6]) * inv, __uint_as_float(o[e + 7]) * inv);
          }
          dst[c * 4 + e / 8] = v;
        }
      }
    }
    if (lse != nullptr && r < rows_in_tile) {
      const float ln2 = 0.6931471805599453f;
      lse[((int64_t)b * g.heads + h) * g.L + g.seg_off[s] + q0 + r] =
          (r < q_real && l > 0.f) ? (m_used * sl2 + log2f(l)) * ln2 : -INFINITY;
    }
  }

  // ---- release tensor memory once every role is done with it ----
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
  }
}

}  // namespace

cudaError_t launch_attn_tc_hd64(const Geometry& g, const __nv_bfloat16* q, const __nv_bfloat16* k,
                                const __nv_bfloat16* v, int64_t row_stride, __nv_bfloat16* out, float* lse,
                                float scale, cudaStream_t st) {
  if (g.hd != HD64 || g.batch > 65535 || g.heads > 65535) return cudaErrorNotSupported;
  const int64_t rows = (int64_t)g.batch * g.L;
  alignas(64) CUtensorMap tmQ, tmK, tmV;
  if (!make_map(&tmQ, q, rows, g.d, row_stride, HD64, TQ) || !make_map(&tmK, k, rows, g.d, row_stride, HD64, TK) ||
      !make_map(&tmV, v, rows, g.d, row_stride, HD64, TK))
    return cudaErrorInvalidValue;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(attn_tc_hd64_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  int tiles = 0;
  for (int s = 0; s < 3; ++s) tiles += (g.seg_len[s] + TQ - 1) / TQ;
  const dim3 grid((unsigned)tiles, (unsigned)g.heads, (unsigned)g.batch);
  attn_tc_hd64_kernel<<<grid, TC_THREADS, TC_SMEM, st>>>(tmQ, tmK, tmV, g, out, lse, scale * 1.4426950408889634f);
  return cudaGetLastError();
}

}  // namespace gsit
