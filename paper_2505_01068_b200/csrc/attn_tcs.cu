// bf16 IM attention for head_dim 8 / 16 / 32 on the 5th-generation tensor cores (tcgen05), scores and accumulators in
// tensor memory (TMEM), operands fed by TMA.  One thread owns one query row, so the softmax needs no shuffles, no
// fragment repacking and no shared-memory round trip: per score it costs a maximum, half a packed multiply-add, one
// exponential, half a packed add and half a conversion.
//
// Decomposition (paper, Section "Inner Decomposition for Efficiency"; Appendix A "From Set to Set Aggregation"): a work
// item is 128 query rows of one modality segment of one sample and a slice of 64 features (8 heads of 8, 4 of 16 or 2 of
// 32); it walks only the key tiles (64 keys) of the segment(s) the Interlaced Mask opens for that block row, up to the
// sample's valid length, and inside a key tile the heads of the slice one after the other.  A (key tile, head) pair is a
// "unit".
//
// The grid is persistent, two CTAs per SM.  Roles inside a CTA of 6 warps:
//   warp 0      TMA producer: the Q tile of an item, K and V tiles (64 keys x 128 bytes, 128-byte swizzle) in four-stage
//               rings, straight out of the fused qkv buffer; it also decodes the work items and hands them to the others
//   warp 1      owns 256 TMEM columns and issues every tcgen05.mma:
//                 S = Q_h K_h^T  M 128, N 64 (16 per 16-key group of a ragged tile), K 16 per step.  With head_dim 8 a
//                   K step spans a pair of heads in the K tile; the A operand is then [q_h, 0] or [0, q_h]: the Q tile is
//                   loaded head by head as 16-byte rows and the second core matrix of the step is a block of zeros,
//                   reached through the descriptor's leading byte offset, so the neighbour head contributes nothing
//                 O_h += P V_h   M 128, N 16 (32 for head_dim 32), K 16 per step; A = P from TMEM, B = the V tile as
//                   loaded (N-contiguous).  With head_dim 8, N = 16 covers the head pair; the neighbour's 8 columns of
//                   the accumulator are never read
//               S is double-buffered, so the scores of unit u+1 are computed while the softmax works on unit u
//   warps 2..5  softmax: thread = query row = TMEM lane.  tcgen05.ld of the scores, running maximum and sum per head in
//               shared memory, P (bf16 pairs) written over the scores it came from, O rescaled in TMEM only when the
//               maximum has grown by more than 2^8.  Warps whose 32 rows hold no real query skip the arithmetic.
// TMEM columns: [0,64) and [64,128) S fp32 / P bf16x2 (first 32 columns of each), [128,256) O, one block of 16 (32)
// columns per head.  Every wait is bounded; when one expires GSIT_DEVFLAG_TIMEOUT is raised, the CTA's other waits give
// up at once, and the CTA still releases its TMEM and returns.
#include <cuda.h>

#include "common.cuh"
#include "ptx.cuh"
#include "tensor_map.cuh"
#include "tmem_ldst.cuh"

namespace gsit {
namespace {

using namespace ptx;

constexpr int SQ = 128, SK = 64, SLICE = 64;
constexpr int S_STAGES = 4;
constexpr int S_KV_BYTES = SK * 128;
constexpr int S_THREADS = 192;
constexpr int S_TMEM_COLS = 256, S_COL_O = 128;
constexpr int S_ITEM_SLOTS = 4;
// barriers (8 bytes each), relative to the barrier block
constexpr int B_QFULL = 0, B_QEMPTY = 8, B_KFULL = 16, B_VFULL = 48, B_KEMPTY = 80, B_VEMPTY = 112, B_SFULL = 144,
              B_PFULL = 160, B_OFINAL = 176, B_TMEM_SLOT = 184, B_GAVE_UP = 188, B_ITEMBAR = 192, B_ITEMS = 256,
              B_STATE = 512;

template <int HD>
struct SCfg {
  static constexpr int G = SLICE / HD;             // heads per slice
  static constexpr int NPV = HD < 16 ? 16 : HD;    // N of O_h += P V
  // head_dim 8: per head pair [q_even 2 KB][zeros 2 KB][q_odd 2 KB], rows of 16 bytes; otherwise 128 rows x 128 bytes
  static constexpr int Q_BYTES = (HD == 8) ? 4 * 6144 : SQ * 128;
  static constexpr int OFF_K = Q_BYTES, OFF_V = OFF_K + S_STAGES * S_KV_BYTES, OFF_BAR = OFF_V + S_STAGES * S_KV_BYTES;
  static constexpr int SMEM = OFF_BAR + B_STATE + G * 2 * SQ * 4 + 1024 /* alignment slack */;
};

// One work item (16 ints = one 64-byte record of the hand-over ring).
struct SItem {
  int b, c, s, q0;
  int rows_in_tile;  // rows of the tile this CTA writes (padding included in the padded layout)
  int q_real;        // rows that receive a computed result
  int T;             // key tiles to walk
  int kn0, kn1, kn2, nk0, nk1;  // real keys per open key segment, key tiles of the first two
  int kb0, kb1, kb2;            // first row of each key segment in the activation matrices
  int grow0;                    // first row of the query tile in the activation matrices
};

__device__ __forceinline__ SItem decode_item(const Geometry& g, int w, int slices, int seg_order) {
  SItem it;
  it.b = w % g.batch;
  int t = w / g.batch;
  it.c = t % slices;
  int tile = t / slices, s = seg_order & 3;
#pragma unroll
  for (int rank = 0; rank < 2; ++rank) {
    const int nts = (g.seg_len[s] + SQ - 1) / SQ;
    if (tile >= nts) { tile -= nts; s = (seg_order >> (2 * rank + 2)) & 3; }
  }
  it.s = s;
  it.q0 = tile * SQ;
  const int in_seg = min(SQ, g.seg_len[s] - it.q0);
  const int q_real_all = max(0, min(in_seg, valid_rows(g, it.b, s) - it.q0));
  it.rows_in_tile = (g.row_start != nullptr) ? q_real_all : in_seg;
  it.kn0 = ((g.allowed >> (3 * s + 0)) & 1u) ? valid_rows(g, it.b, 0) : 0;
  it.kn1 = ((g.allowed >> (3 * s + 1)) & 1u) ? valid_rows(g, it.b, 1) : 0;
  it.kn2 = ((g.allowed >> (3 * s + 2)) & 1u) ? valid_rows(g, it.b, 2) : 0;
  it.nk0 = (it.kn0 + SK - 1) / SK;
  it.nk1 = (it.kn1 + SK - 1) / SK;
  const int nk2 = (it.kn2 + SK - 1) / SK;
  it.T = (q_real_all > 0) ? it.nk0 + it.nk1 + nk2 : 0;
  it.q_real = (it.T > 0) ? q_real_all : 0;
  it.kb0 = seg_row0(g, it.b, 0);
  it.kb1 = seg_row0(g, it.b, 1);
  it.kb2 = seg_row0(g, it.b, 2);
  it.grow0 = seg_row0(g, it.b, s) + it.q0;
  return it;
}

// Key tile i of an item: real keys left from its start (>= 1) and its first row in the activation matrices.
__device__ __forceinline__ void locate(const SItem& it, int i, int& krem, int& yrow) {
  int t = i, r = 0;
  if (t >= it.nk0) { t -= it.nk0; r = 1; if (t >= it.nk1) { t -= it.nk1; r = 2; } }
  const int kn = (r == 0) ? it.kn0 : (r == 1) ? it.kn1 : it.kn2;
  krem = kn - t * SK;
  yrow = ((r == 0) ? it.kb0 : (r == 1) ? it.kb1 : it.kb2) + t * SK;
}

__device__ __forceinline__ void publish_item(uint32_t bars, const SItem& it, int k, int lane) {
  if (lane == 0) {
    const uint32_t a = bars + B_ITEMS + 64 * (k % S_ITEM_SLOTS);
    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(it.b), "r"(it.c), "r"(it.s), "r"(it.q0) : "memory");
    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(a + 16), "r"(it.rows_in_tile), "r"(it.q_real), "r"(it.T), "r"(it.kn0) : "memory");
    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(a + 32), "r"(it.kn1), "r"(it.kn2), "r"(it.nk0), "r"(it.nk1) : "memory");
    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(a + 48), "r"(it.kb0), "r"(it.kb1), "r"(it.kb2), "r"(it.grow0) : "memory");
    mbar_arrive(bars + B_ITEMBAR + 8 * (k % S_ITEM_SLOTS));
  }
  __syncwarp();
}
__device__ __forceinline__ SItem fetch_item(const WaitCtx& wc, uint32_t bars, int k, int lane) {
  const int slot = k % S_ITEM_SLOTS;
  mbar_wait(wc, bars + B_ITEMBAR + 8 * slot, (k / S_ITEM_SLOTS) & 1);
  const uint32_t a = bars + B_ITEMS + 64 * slot;
  SItem it;
  asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(it.b), "=r"(it.c), "=r"(it.s), "=r"(it.q0) : "r"(a) : "memory");
  asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(it.rows_in_tile), "=r"(it.q_real), "=r"(it.T), "=r"(it.kn0) : "r"(a + 16) : "memory");
  asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(it.kn1), "=r"(it.kn2), "=r"(it.nk0), "=r"(it.nk1) : "r"(a + 32) : "memory");
  asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(it.kb0), "=r"(it.kb1), "=r"(it.kb2), "=r"(it.grow0) : "r"(a + 48) : "memory");
  __syncwarp();
  if (lane == 0) mbar_arrive(bars + B_ITEMBAR + 8 * S_ITEM_SLOTS + 8 * slot);
  return it;
}

template <int V> struct IntTag { static constexpr int value = V; };
template <bool V> struct BoolTag { static constexpr bool value = V; };

template <int HD>
__global__ void __launch_bounds__(S_THREADS, 2)
attn_tcs_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, const Geometry g, __nv_bfloat16* __restrict__ out,
                float* __restrict__ lse, const float sl2 /* scale * log2(e) */, const int slices, const int seg_order,
                const int n_items) {
  using C = SCfg<HD>;
  constexpr int G = C::G, NPV = C::NPV;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sQ = base, sK = base + C::OFF_K, sV = base + C::OFF_V, bars = base + C::OFF_BAR;
  const uint32_t sState = bars + B_STATE;  // running maximum and sum: float [G][2][128]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const WaitCtx wc{g.status, bars + B_GAVE_UP};

  // ---- set-up, once per CTA: barriers, the zero blocks of the Q layout, tensor memory ----
  if (tid == 0) {
    mbar_init(bars + B_QFULL, 1);
    mbar_init(bars + B_QEMPTY, 1);
#pragma unroll
    for (int i = 0; i < S_STAGES; ++i) {
      mbar_init(bars + B_KFULL + 8 * i, 1);
      mbar_init(bars + B_VFULL + 8 * i, 1);
      mbar_init(bars + B_KEMPTY + 8 * i, 1);
      mbar_init(bars + B_VEMPTY + 8 * i, 1);
    }
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      mbar_init(bars + B_SFULL + 8 * i, 1);
      mbar_init(bars + B_PFULL + 8 * i, 4);  // one arrival per softmax warp
    }
    mbar_init(bars + B_OFINAL, 1);
    for (int i = 0; i < S_ITEM_SLOTS; ++i) {
      mbar_init(bars + B_ITEMBAR + 8 * i, 1);                     // record written (producer)
      mbar_init(bars + B_ITEMBAR + 8 * S_ITEM_SLOTS + 8 * i, 5);  // record read (MMA warp + four softmax warps)
    }
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(bars + B_GAVE_UP), "r"(0u) : "memory");
    mbar_init_fence();
  }
  if constexpr (HD == 8) {
    for (int i = tid; i < 4 * 128; i += S_THREADS)  // 4 pairs x 2 KB of zeros, 16 bytes per step
      st_shared_v4(sQ + (i >> 7) * 6144 + 2048 + (i & 127) * 16, 0, 0, 0, 0);
    fence_async_smem();
  }
  if (warp == 1) tmem_alloc(bars + B_TMEM_SLOT, S_TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  uint32_t tmem;
  asm volatile("ld.shared.b32 %0, [%1];" : "=r"(tmem) : "r"(bars + B_TMEM_SLOT) : "memory");

  if (warp == 0) {
    // ================================ TMA producer ================================
    int n_q = 0, n_kv = 0, k = 0;
    for (int w = blockIdx.x; w < n_items; w += gridDim.x, ++k) {
      const SItem it = decode_item(g, w, slices, seg_order);
      if (k >= S_ITEM_SLOTS)
        mbar_wait(wc, bars + B_ITEMBAR + 8 * S_ITEM_SLOTS + 8 * (k % S_ITEM_SLOTS), ((k / S_ITEM_SLOTS) - 1) & 1);
      publish_item(bars, it, k, lane);
      if (it.T == 0) continue;
      if (n_q > 0) mbar_wait(wc, bars + B_QEMPTY, (n_q - 1) & 1);
      if (elect_one()) {
        mbar_expect_tx(bars + B_QFULL, SQ * 128);
        if constexpr (HD == 8) {
#pragma unroll
          for (int h = 0; h < 8; ++h)
            tma_load_2d(sQ + (h >> 1) * 6144 + (h & 1) * 4096, &tmQ, it.c * SLICE + h * 8, it.grow0, bars + B_QFULL);
        } else {
          tma_load_2d(sQ, &tmQ, it.c * SLICE, it.grow0, bars + B_QFULL);
        }
      }
      ++n_q;
      for (int i = 0; i < it.T; ++i, ++n_kv) {
        int krem, yrow;
        locate(it, i, krem, yrow);
        const int st = n_kv % S_STAGES, use = n_kv / S_STAGES;
        if (use > 0) mbar_wait(wc, bars + B_KEMPTY + 8 * st, (use - 1) & 1);
        if (elect_one()) {
          mbar_expect_tx(bars + B_KFULL + 8 * st, S_KV_BYTES);
          tma_load_2d(sK + st * S_KV_BYTES, &tmK, it.c * SLICE, yrow, bars + B_KFULL + 8 * st);
        }
        if (use > 0) mbar_wait(wc, bars + B_VEMPTY + 8 * st, (use - 1) & 1);
        if (elect_one()) {
          mbar_expect_tx(bars + B_VFULL + 8 * st, S_KV_BYTES);
          tma_load_2d(sV + st * S_KV_BYTES, &tmV, it.c * SLICE, yrow, bars + B_VFULL + 8 * st);
        }
      }
    }
  } else if (warp == 1) {
    // ================================ MMA issuer ================================
    constexpr uint32_t IDESC_PV = idesc_bf16(NPV, true);
    int n_q = 0, n_kv = 0, n_u = 0, k = 0;  // Q tiles, key tiles and units consumed so far
    for (int w = blockIdx.x; w < n_items; w += gridDim.x, ++k) {
      const SItem it = fetch_item(wc, bars, k, lane);
      if (it.T == 0) continue;
      const int U = it.T * G;
      // S[nu & 1] = Q_h K_h^T for unit u of the item.  The buffer was last read (as P) by the P V of unit u - 2, which
      // this thread has issued before; tcgen05.mma instructions of one thread execute in issue order.
      auto issue_qk = [&](int u) {
        const int j = u / G, h = u - j * G, n = n_kv + j, st = n % S_STAGES, nu = n_u + u;
        if (h == 0) mbar_wait(wc, bars + B_KFULL + 8 * st, (n / S_STAGES) & 1);
        int krem, yrow;
        locate(it, j, krem, yrow);
        const int ncols = (krem >= SK) ? SK : ((krem + 15) >> 4) << 4;
        tc_fence_after();
        if (elect_one()) {
          const uint32_t d = tmem + 64 * (nu & 1), idesc = idesc_bf16(ncols, false);
          const uint32_t kt = sK + st * S_KV_BYTES;
          if constexpr (HD == 8) {
            // [q_h, 0] for an even head, [0, q_h] for an odd one: start at q_even or at the zeros, 2 KB to the other half
            const uint64_t a = smem_desc_plain(sQ + (h >> 1) * 6144 + (h & 1) * 2048, 2048, 128);
            umma_ss(d, a, smem_desc_sw128(kt + 32 * (h >> 1)), idesc, 0);
          } else {
#pragma unroll
            for (int ks = 0; ks < HD / 16; ++ks)
              umma_ss(d, smem_desc_sw128(sQ + 2 * HD * h + 32 * ks), smem_desc_sw128(kt + 2 * HD * h + 32 * ks), idesc, ks > 0);
          }
          if (h == G - 1) umma_commit(bars + B_KEMPTY + 8 * st);
          if (u == U - 1) umma_commit(bars + B_QEMPTY);
          umma_commit(bars + B_SFULL + 8 * (nu & 1));
        }
        __syncwarp();
      };
      mbar_wait(wc, bars + B_QFULL, n_q & 1);
      issue_qk(0);
      for (int u = 0; u < U; ++u) {
        if (u + 1 < U) issue_qk(u + 1);  // scores of the next unit, ahead of this unit's P V
        const int j = u / G, h = u - j * G, n = n_kv + j, st = n % S_STAGES, nu = n_u + u;
        int krem, yrow;
        locate(it, j, krem, yrow);
        const int ksteps = (krem >= SK) ? SK / 16 : (krem + 15) >> 4;
        // P of this unit is in TMEM (and, for the first unit of an item, the previous item's O has been read)
        mbar_wait(wc, bars + B_PFULL + 8 * (nu & 1), (nu >> 1) & 1);
        if (h == 0) mbar_wait(wc, bars + B_VFULL + 8 * st, (n / S_STAGES) & 1);
        tc_fence_after();
        if (elect_one()) {
          const uint32_t vt = sV + st * S_KV_BYTES + ((HD == 8) ? 32 * (h >> 1) : 2 * HD * h);
          for (int kk = 0; kk < ksteps; ++kk)  // 16 keys per step: two 8-row groups = 2048 bytes of the V tile
            umma_ts(tmem + S_COL_O + NPV * h, tmem + 64 * (nu & 1) + 8 * kk, smem_desc_sw128(vt + 2048 * kk), IDESC_PV,
                    (j > 0 || kk > 0) ? 1u : 0u);
          if (h == G - 1) umma_commit(bars + B_VEMPTY + 8 * st);  // also: O holds key tiles 0..j of every head
          if (u == U - 1) umma_commit(bars + B_OFINAL);
        }
        __syncwarp();
      }
      n_kv += it.T;
      n_u += U;
      ++n_q;
    }
  } else {
    // ================================ softmax, one thread per query row ================================
    const int wq = warp & 3;                               // TMEM lane quarter this warp may access
    const int r = (wq << 5) + lane;                        // row in the tile = TMEM lane
    const uint32_t tl = tmem + ((uint32_t)(wq << 5) << 16);
    const float2 sl2v = make_float2(sl2, sl2);
    const uint32_t my_state = sState + r * 4;              // + (2 h + {0: maximum, 1: sum}) * 512
    int n_kv = 0, n_u = 0, n_items_done = 0, k = 0;

    for (int w = blockIdx.x; w < n_items; w += gridDim.x, ++k) {
      const SItem it = fetch_item(wc, bars, k, lane);
      const int64_t grow = (int64_t)it.grow0 + r;
      uint4* dst = reinterpret_cast<uint4*>(out + grow * g.d + it.c * SLICE);
      float* lse_row = (lse != nullptr) ? lse + ((int64_t)it.b * g.heads + it.c * G) * g.L + g.seg_off[it.s] + it.q0 + r : nullptr;
      if (it.T == 0) {  // nothing to attend (padding rows only, or an empty key set): exact zeros, lse = -inf
        if (r < it.rows_in_tile) {
#pragma unroll
          for (int c = 0; c < 8; ++c) dst[c] = make_uint4(0, 0, 0, 0);
          if (lse_row != nullptr)
            for (int h = 0; h < G; ++h) lse_row[(int64_t)h * g.L] = -INFINITY;
        }
        continue;
      }
      const bool warp_active = (wq << 5) < it.q_real;  // some row of this warp receives a result

      // One unit: NCH = 16-key groups of the tile that hold real keys (4 = all), MASKED = the last group is partly padding.
      auto unit = [&](auto nch_tag, auto masked_tag, const int j, const int h, const int n, const int nu, const int krem) {
        constexpr int NCH = decltype(nch_tag)::value;
        constexpr bool MASKED = decltype(masked_tag)::value;
        const int sb = nu & 1;
        const uint32_t tS = tl + 64 * sb;
        uint32_t sr[NCH][16];
#pragma unroll
        for (int c = 0; c < NCH; ++c) tmem_ld16(tS + 16 * c, sr[c]);
        float m_used = -INFINITY, l = 0.f;
        if (j > 0) {
          asm volatile("ld.shared.f32 %0, [%1];" : "=f"(m_used) : "r"(my_state + (2 * h) * 512) : "memory");
          asm volatile("ld.shared.f32 %0, [%1];" : "=f"(l) : "r"(my_state + (2 * h + 1) * 512) : "memory");
        }
        tmem_wait_ld();
        if constexpr (MASKED) {  // keys past the valid length get weight exactly zero
#pragma unroll
          for (int e = 0; e < 16; ++e)
            if ((NCH - 1) * 16 + e >= krem) sr[NCH - 1][e] = 0xff800000u;  // -inf
        }
        float mx4[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) mx4[i] = -INFINITY;
#pragma unroll
        for (int c = 0; c < NCH; ++c)
#pragma unroll
          for (int e = 0; e < 16; e += 2)
            mx4[(e >> 1) & 3] = fmax3(mx4[(e >> 1) & 3], __uint_as_float(sr[c][e]), __uint_as_float(sr[c][e + 1]));
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        // rescale only when the maximum has grown by more than 2^8 (P stays below 256: exact enough in bf16 and f32)
        const bool grow_m = (j == 0) || ((mx - m_used) * sl2 > 8.f);
        if (j > 0 && __any_sync(0xffffffffu, grow_m)) {
          const float alpha = grow_m ? ex2((m_used - mx) * sl2) : 1.f;
          l *= alpha;
          // O_h must hold every earlier key tile before it is rescaled: wait for the last P V of key tile n - 1
          mbar_wait(wc, bars + B_VEMPTY + 8 * ((n - 1) % S_STAGES), ((n - 1) / S_STAGES) & 1);
          tc_fence_after();
          const uint32_t tO = tl + S_COL_O + NPV * h + ((HD == 8) ? 8 * (h & 1) : 0);
#pragma unroll
          for (int c = 0; c < HD / 8; ++c) {
            uint32_t o[8];
            tmem_ld8(tO + 8 * c, o);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 8; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
            tmem_st8(tO + 8 * c, o);
          }
        }
        if (grow_m) m_used = mx;
        const float nm = -m_used * sl2;
        const float2 nmv = make_float2(nm, nm);
        float2 sum[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
          uint32_t pr[8];
#pragma unroll
          for (int e = 0; e < 16; e += 2) {
            const float2 x = __ffma2_rn(make_float2(__uint_as_float(sr[c][e]), __uint_as_float(sr[c][e + 1])), sl2v, nmv);
            const float2 p = make_float2(ex2(x.x), ex2(x.y));
            sum[(e >> 1) & 1] = __fadd2_rn(sum[(e >> 1) & 1], p);
            pr[e >> 1] = pack_bf16(p.x, p.y);
          }
          tmem_st8(tS + 8 * c, pr);
        }
        const float2 s01 = __fadd2_rn(sum[0], sum[1]);
        l += s01.x + s01.y;
        asm volatile("st.shared.f32 [%0], %1;" ::"r"(my_state + (2 * h) * 512), "f"(m_used) : "memory");
        asm volatile("st.shared.f32 [%0], %1;" ::"r"(my_state + (2 * h + 1) * 512), "f"(l) : "memory");
        tmem_wait_st();
      };

      const int U = it.T * G;
      for (int u = 0; u < U; ++u) {
        const int j = u / G, h = u - j * G, n = n_kv + j, nu = n_u + u;
        int krem, yrow;
        locate(it, j, krem, yrow);
        mbar_wait(wc, bars + B_SFULL + 8 * (nu & 1), (nu >> 1) & 1);
        tc_fence_after();
        if (krem < SK && h == 0) {
          // Rows of the V tile past the valid length hold whatever follows in memory; a zero weight times NaN or Inf
          // would still poison the accumulator, so clear them (up to the end of the last 16-key group that is
          // multiplied) before the first P V of the tile reads them.
          const int st = n % S_STAGES;
          mbar_wait(wc, bars + B_VFULL + 8 * st, (n / S_STAGES) & 1);
          const int row = krem + r;
          if (row < (((krem + 15) >> 4) << 4)) {
            const uint32_t a = sV + st * S_KV_BYTES + row * 128;
#pragma unroll
            for (int c = 0; c < 8; ++c) st_shared_v4(a + 16 * c, 0, 0, 0, 0);
          }
          fence_async_smem();
        }
        if (warp_active) {
          if (krem >= SK) unit(IntTag<4>{}, BoolTag<false>{}, j, h, n, nu, SK);
          else if (krem > 48) unit(IntTag<4>{}, BoolTag<true>{}, j, h, n, nu, krem);
          else if (krem > 32) unit(IntTag<3>{}, BoolTag<true>{}, j, h, n, nu, krem);
          else if (krem > 16) unit(IntTag<2>{}, BoolTag<true>{}, j, h, n, nu, krem);
          else unit(IntTag<1>{}, BoolTag<true>{}, j, h, n, nu, krem);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bars + B_PFULL + 8 * (nu & 1));
      }
      n_kv += it.T;
      n_u += U;

      // ---- epilogue: O_h / l_h -> bf16, each thread its own 128-byte row of the slice; padded rows +0 ----
      mbar_wait(wc, bars + B_OFINAL, n_items_done & 1);
      ++n_items_done;
      tc_fence_after();
      const bool real = r < it.q_real;
      if (warp_active) {
        uint32_t orow[32];
#pragma unroll
        for (int h = 0; h < G; ++h) {
          float m_used, l;
          asm volatile("ld.shared.f32 %0, [%1];" : "=f"(m_used) : "r"(my_state + (2 * h) * 512) : "memory");
          asm volatile("ld.shared.f32 %0, [%1];" : "=f"(l) : "r"(my_state + (2 * h + 1) * 512) : "memory");
          const float inv = (l > 0.f) ? 1.f / l : 0.f;
          const uint32_t tO = tl + S_COL_O + NPV * h + ((HD == 8) ? 8 * (h & 1) : 0);
#pragma unroll
          for (int c = 0; c < HD / 8; ++c) {
            uint32_t o[8];
            tmem_ld8(tO + 8 * c, o);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 8; e += 2)
              orow[(h * HD + c * 8 + e) >> 1] = pack_bf16(__uint_as_float(o[e]) * inv, __uint_as_float(o[e + 1]) * inv);
          }
          if (lse_row != nullptr && r < it.rows_in_tile) {
            const float ln2 = 0.6931471805599453f;
            lse_row[(int64_t)h * g.L] = (real && l > 0.f) ? (m_used * sl2 + log2f(l)) * ln2 : -INFINITY;
          }
        }
        if (r < it.rows_in_tile) {
#pragma unroll
          for (int c = 0; c < 8; ++c)
            dst[c] = real ? make_uint4(orow[4 * c], orow[4 * c + 1], orow[4 * c + 2], orow[4 * c + 3]) : make_uint4(0, 0, 0, 0);
        }
      } else if (r < it.rows_in_tile) {
#pragma unroll
        for (int c = 0; c < 8; ++c) dst[c] = make_uint4(0, 0, 0, 0);
        if (lse_row != nullptr)
          for (int h = 0; h < G; ++h) lse_row[(int64_t)h * g.L] = -INFINITY;
      }
    }
  }

  // ---- release tensor memory once every role is done with it ----
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, S_TMEM_COLS);
  }
}

constexpr int MAX_DEVICES = 64;

template <int HD>
cudaError_t launch_tcs(const Geometry& g, const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v,
                       int64_t row_stride, __nv_bfloat16* out, float* lse, float scale, cudaStream_t st) {
  using C = SCfg<HD>;
  const int64_t rows = matrix_rows(g);
  alignas(64) CUtensorMap tmQ, tmK, tmV;
  const bool okq = (HD == 8) ? make_map(&tmQ, q, rows, g.d, row_stride, 8, SQ, true)
                             : make_map(&tmQ, q, rows, g.d, row_stride, SLICE, SQ);
  if (!okq || !make_map(&tmK, k, rows, g.d, row_stride, SLICE, SK) || !make_map(&tmV, v, rows, g.d, row_stride, SLICE, SK))
    return cudaErrorInvalidValue;
  static int n_sm[MAX_DEVICES] = {};  // per device: SM count, and whether the kernel's shared-memory size has been set
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
  if (n_sm[dev] == 0) {
    int n = 0;
    e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(attn_tcs_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM);
    if (e != cudaSuccess) return e;
    n_sm[dev] = n;
  }
  int tiles = 0;
  for (int s = 0; s < 3; ++s) tiles += (g.seg_len[s] + SQ - 1) / SQ;
  const int slices = g.d / SLICE;
  const int64_t n_items = (int64_t)tiles * slices * g.batch;
  if (n_items > 0x7fffffffLL) return cudaErrorNotSupported;
  // query segments in descending order of the keys their tiles walk (longest work first)
  int cost[3], ord[3] = {0, 1, 2};
  for (int s = 0; s < 3; ++s) {
    cost[s] = 0;
    for (int r = 0; r < 3; ++r)
      if ((g.allowed >> (3 * s + r)) & 1u) cost[s] += g.seg_len[r];
  }
  for (int i = 0; i < 3; ++i)
    for (int j = i + 1; j < 3; ++j)
      if (cost[ord[j]] > cost[ord[i]]) { const int t = ord[i]; ord[i] = ord[j]; ord[j] = t; }
  const int seg_order = ord[0] | (ord[1] << 2) | (ord[2] << 4);
  const unsigned grid = (unsigned)((n_items < 2 * n_sm[dev]) ? n_items : 2 * n_sm[dev]);  // two resident CTAs per SM
  attn_tcs_kernel<HD><<<grid, S_THREADS, C::SMEM, st>>>(tmQ, tmK, tmV, g, out, lse, scale * 1.4426950408889634f, slices,
                                                         seg_order, (int)n_items);
  return cudaGetLastError();
}

}  // namespace

bool attn_tcs_supported(const Geometry& g) { return g.d % SLICE == 0 && (g.hd == 8 || g.hd == 16 || g.hd == 32); }

cudaError_t launch_attn_tcs(const Geometry& g, const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v,
                            int64_t row_stride, __nv_bfloat16* out, float* lse, float scale, cudaStream_t st) {
  if (!attn_tcs_supported(g)) return cudaErrorNotSupported;
  if (g.hd == 8) return launch_tcs<8>(g, q, k, v, row_stride, out, lse, scale, st);
  if (g.hd == 16) return launch_tcs<16>(g, q, k, v, row_stride, out, lse, scale, st);
  return launch_tcs<32>(g, q, k, v, row_stride, out, lse, scale, st);
}

}  // namespace gsit
