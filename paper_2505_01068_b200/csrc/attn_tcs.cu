// bf16 IM attention for head_dim 8 / 16 / 32 on the 5th-generation tensor cores (tcgen05), scores and accumulators in
// tensor memory (TMEM), operands fed by TMA.  One thread owns one query row of one head, so the softmax needs no
// shuffles, no fragment repacking and no shared-memory round trip: per score it costs a third of a three-way maximum,
// half a packed multiply-add, one exponential, half a packed add and half a byte permute.
//
// Decomposition (paper, Section "Inner Decomposition for Efficiency"; Appendix A "From Set to Set Aggregation"): a work
// item is 128 query rows of one modality segment of one sample and a PAIR OF HEADS (32, 64 or 128 bytes of every row for
// head_dim 8, 16, 32).  It walks only the key tiles (64 keys) of the segment(s) the Interlaced Mask opens for that block
// row, up to the sample's valid length.  Items are small (at most 16 head-tiles at the MOSEI shape) and are handed out
// through an atomic counter, longest first, so that all SMs finish together although the valid lengths differ.
//
// The two heads of an item are two independent chains: each has its own score buffer, weight buffer and accumulator
// in tensor memory and its own group of four softmax warps.  While one group waits for the round trip
// weights -> P V and next Q K^T -> scores (some 450 clocks through the MMA warp), the other computes, and with two CTAs
// per SM every scheduler holds four softmax warps: what keeps the exponential unit and the issue slots busy is the
// number of independent softmax warps, not a deep pipeline behind one.
//
// The grid is persistent, two CTAs per SM.  Roles inside a CTA of 10 warps:
//   warp 0      takes the next item from the counter, decodes it and hands it to the other warps through a ring of records;
//               TMA producer: the Q tile of an item (two buffers), K and V tiles of 64 keys in four-stage rings
//   warp 1      owns 256 TMEM columns and issues every tcgen05.mma, alternating between the two heads:
//                 S_h = Q_h K_h^T  M 128, N 64 (16 per 16-key group of a ragged tile), K 16 per step.  With head_dim 8 a
//                   K step spans the pair of heads in the K tile; the A operand is then [q_h, 0] or [0, q_h]: the Q tile is
//                   loaded head by head as 16-byte rows and the other core matrix of the step is a block of zeros,
//                   reached through the descriptor's leading byte offset, so the neighbour head contributes nothing
//                 O_h += P_h V     M 128, N 16 (32), K 16 per step; A = P_h from TMEM, B = the V tile as loaded
//                   (N-contiguous).  With head_dim 8, N = 16 covers the head pair; the neighbour's 8 columns of each
//                   head's accumulator are never read
//   warps 2..5  softmax of head 0, warps 6..9 of head 1: thread = query row = TMEM lane.  Two passes over the scores in
//               groups of 16 columns (maximum, then weights), running maximum and sum in registers, O_h rescaled in TMEM
//               only when the maximum has grown by more than 2^8.  Warps whose 32 rows hold no real query skip the
//               arithmetic.
// TMEM columns: [0,64) S_0, [64,128) S_1 fp32; [128,160) P_0, [160,192) P_1 bf16x2; [192,224) O_0, [224,256) O_1.
// Every wait is bounded; when one expires GSIT_DEVFLAG_TIMEOUT is raised, the CTA's other waits give up at once, and the
// CTA still releases its TMEM and returns.
#include <cuda.h>

#include "common.cuh"
#include "ptx.cuh"
#include "tensor_map.cuh"
#include "tmem_ldst.cuh"

namespace gsit {
namespace {

using namespace ptx;

constexpr int SQ = 128, SK = 64;
constexpr int S_THREADS = 320;
constexpr int S_TMEM_COLS = 256, S_COL_P = 128, S_COL_O = 192;
constexpr int S_CTAS_PER_SM = 2;
constexpr int S_ITEM_SLOTS = 4;
constexpr int S_QBUF = 16384;  // bytes reserved per Q buffer
#ifndef GSIT_POLY_PAIRS
#define GSIT_POLY_PAIRS 0x11
#endif
// The weights are cut to bf16 by dropping the low 16 bits (one byte permute on the integer pipe per pair; the rounding
// conversion would occupy the special-function unit as long as an exponential).  Dropping bits loses on average
// 0.72 * 2^-9 of a value whose mantissa is spread like that of an exponential, so every weight is raised by that factor
// beforehand (it is one constant added to the exponent) and the row sum, which is taken of the raised values in float, is
// lowered by it at the end: the weights are then unbiased, with the same spread as round-to-nearest.
constexpr float TRUNC_GAIN = 1.0f + 0.72f / 512.0f;
constexpr float TRUNC_LOG2 = 0.0020273f;  // log2(TRUNC_GAIN)
constexpr unsigned POLY_PAIRS = GSIT_POLY_PAIRS;  // bit i: pair i of every 16-key group takes the polynomial 2^x
// barriers (8 bytes each), relative to the barrier block
constexpr int B_QFULL = 0, B_QEMPTY = 16, B_SFULL = 32, B_PFULL = 48, B_OFINAL = 64, B_TMEM_SLOT = 72, B_GAVE_UP = 76,
              B_ITEMBAR = 80, B_ITEMS = 256, B_KFULL = 512, B_VFULL = 576, B_KVEMPTY = 640, B_END = 704;

template <int HD>
struct SCfg {
  static constexpr int SLW = 2 * HD;                 // features per slice: a pair of heads
  static constexpr int ROWB = SLW * 2;               // bytes per tile row: 32, 64, 128
  static constexpr int NPV = (HD == 8) ? 16 : HD;    // N of O_h += P_h V
  static constexpr uint32_t SWZ = (ROWB == 32) ? 6u : (ROWB == 64) ? 4u : 2u;  // descriptor code of the 32 / 64 / 128-byte swizzle
  static constexpr uint32_t SBO = 8 * ROWB;          // bytes between groups of 8 rows
  static constexpr int KV_BYTES = SK * ROWB;
  static constexpr int STAGES = 4;
  static constexpr int Q_TX = SQ * ROWB;             // bytes TMA delivers per Q tile
  static constexpr int OFF_K = 2 * S_QBUF, OFF_V = OFF_K + STAGES * KV_BYTES, OFF_BAR = OFF_V + STAGES * KV_BYTES;
  static constexpr int SMEM = OFF_BAR + B_END + 1024 /* alignment slack */;
};

// Descriptor of a swizzled tile as TMA wrote it (rows of 32, 64 or 128 bytes): groups of 8 rows `sbo` bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw(uint32_t addr, uint32_t sbo, uint32_t code) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)(sbo >> 4) << 32) | (1ull << 46) | ((uint64_t)code << 61);
}

// One work item (16 ints = one 64-byte record of the hand-over ring).
struct SItem {
  int b, c, s, q0;
  int rows_in_tile;  // rows of the tile this CTA writes (padding included in the padded layout)
  int q_real;        // rows that receive a computed result
  int T;             // key tiles to walk; -1 = no more items
  int kn0, kn1, kn2, nk0, nk1;  // real keys per open key segment, key tiles of the first two
  int kb0, kb1, kb2;            // first row of each key segment in the activation matrices
  int grow0;                    // first row of the query tile in the activation matrices
};

// What distinguishes one problem of a launch from the other (a launch serves one or two problems of the same geometry).
struct SProblem {
  CUtensorMap tmQ, tmK, tmV;
  __nv_bfloat16* out;
  float* lse;
  uint32_t allowed;
  int seg_order;
};
constexpr int WHICH_SHIFT = 30;  // the problem index rides in bit 30 of the item's slice field

__device__ __forceinline__ SItem decode_item(const Geometry& g, int w, int slices, int seg_order, int which) {
  SItem it;
  it.b = w % g.batch;
  int t = w / g.batch;
  it.c = (t % slices) | (which << WHICH_SHIFT);
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
// Copies record `slot` to registers and releases the slot (one arrival per warp).
__device__ __forceinline__ SItem read_item(uint32_t bars, int slot, int lane) {
  const uint32_t a = bars + B_ITEMS + 64 * slot;
  SItem it;
  asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(it.b), "=r"(it.c), "=r"(it.s), "=r"(it.q0) : "r"(a) : "memory");
  asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(it.rows_in_tile), "=r"(it.q_real), "=r"(it.T), "=r"(it.kn0) : "r"(a + 16) : "memory");
  asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(it.kn1), "=r"(it.kn2), "=r"(it.nk0), "=r"(it.nk1) : "r"(a + 32) : "memory");
  asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(it.kb0), "=r"(it.kb1), "=r"(it.kb2), "=r"(it.grow0) : "r"(a + 48) : "memory");
  fence_reads_before_release();
  __syncwarp();
  if (lane == 0) mbar_arrive(bars + B_ITEMBAR + 8 * S_ITEM_SLOTS + 8 * slot);
  return it;
}
__device__ __forceinline__ SItem fetch_item(const WaitCtx& wc, uint32_t bars, int k, int lane) {
  const int slot = k % S_ITEM_SLOTS;
  const bool ok = mbar_wait(wc, bars + B_ITEMBAR + 8 * slot, (k / S_ITEM_SLOTS) & 1);
  SItem it = read_item(bars, slot, lane);
  if (!ok) it.T = -1;  // the hand-over itself timed out: stop (the flag has been raised)
  return it;
}

template <int HD>
__global__ void __launch_bounds__(S_THREADS, S_CTAS_PER_SM)
attn_tcs_kernel(const __grid_constant__ SProblem prob0, const __grid_constant__ SProblem prob1, const Geometry g0,
                const float sl2 /* scale * log2(e) */, const int slices, const int n_items /* of all problems */,
                const int problems, int* __restrict__ next_item /* zeroed counter, or nullptr = static round robin */) {
  using C = SCfg<HD>;
  constexpr int NPV = C::NPV, STAGES = C::STAGES, KVB = C::KV_BYTES, ROWB = C::ROWB;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sQ = base, sK = base + C::OFF_K, sV = base + C::OFF_V, bars = base + C::OFF_BAR;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const Geometry& g = g0;
  const WaitCtx wc{g.status, bars + B_GAVE_UP};

  // ---- set-up, once per CTA: barriers, the zero blocks of the Q layout, tensor memory ----
  if (tid == 0) {
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      mbar_init(bars + B_QFULL + 8 * i, 1);
      mbar_init(bars + B_QEMPTY + 8 * i, 1);
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      mbar_init(bars + B_SFULL + 8 * h, 1);
      mbar_init(bars + B_PFULL + 8 * h, 4);  // one arrival per softmax warp of the head
    }
#pragma unroll
    for (int i = 0; i < STAGES; ++i) {
      mbar_init(bars + B_KFULL + 8 * i, 1);
      mbar_init(bars + B_VFULL + 8 * i, 1);
      mbar_init(bars + B_KVEMPTY + 8 * i, 1);
    }
    mbar_init(bars + B_OFINAL, 1);
    for (int i = 0; i < S_ITEM_SLOTS; ++i) {
      mbar_init(bars + B_ITEMBAR + 8 * i, 1);                     // record written (producer)
      mbar_init(bars + B_ITEMBAR + 8 * S_ITEM_SLOTS + 8 * i, 9);  // record read (MMA warp + eight softmax warps)
    }
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(bars + B_GAVE_UP), "r"(0u) : "memory");
    mbar_init_fence();
  }
  if constexpr (HD == 8) {
    // Q buffer: [q_even 2 KB][zeros 2 KB][q_odd 2 KB], rows of 16 bytes
    for (int i = tid; i < 2 * 128; i += S_THREADS) st_shared_v4(sQ + (i >> 7) * S_QBUF + 2048 + (i & 127) * 16, 0, 0, 0, 0);
    fence_async_smem();
  }
  if (warp == 1) tmem_alloc(bars + B_TMEM_SLOT, S_TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  uint32_t tmem;
  asm volatile("ld.shared.b32 %0, [%1];" : "=r"(tmem) : "r"(bars + B_TMEM_SLOT) : "memory");
  grid_dep_wait();
  grid_dep_launch();

  if (warp == 0) {
    // ================================ scheduler and TMA producer ================================
    int n_q = 0, n_kv = 0;
    for (int k = 0;; ++k) {
      int w;
      if (next_item != nullptr) {
        w = (lane == 0) ? atomicAdd(next_item, 1) : 0;
        w = __shfl_sync(0xffffffffu, w, 0);
      } else {
        w = blockIdx.x + k * gridDim.x;
      }
      if (k >= S_ITEM_SLOTS)
        mbar_wait(wc, bars + B_ITEMBAR + 8 * S_ITEM_SLOTS + 8 * (k % S_ITEM_SLOTS), ((k / S_ITEM_SLOTS) - 1) & 1);
      if (w >= n_items || cta_gave_up(wc)) {
        SItem end = {};
        end.T = -1;
        publish_item(bars, end, k, lane);
        break;
      }
      const int which = (problems == 2) ? (w & 1) : 0;
      const SProblem& prob = which ? prob1 : prob0;
      Geometry g = g0;
      g.allowed = prob.allowed;
      SItem it = decode_item(g, (problems == 2) ? (w >> 1) : w, slices, prob.seg_order, which);
      publish_item(bars, it, k, lane);
      if (it.T == 0) continue;
      it.c &= (1 << WHICH_SHIFT) - 1;
      const CUtensorMap &tmQ = prob.tmQ, &tmK = prob.tmK, &tmV = prob.tmV;
      const int qb = n_q & 1;
      if (n_q >= 2) mbar_wait(wc, bars + B_QEMPTY + 8 * qb, ((n_q >> 1) - 1) & 1);
      if (elect_one()) {
        mbar_expect_tx(bars + B_QFULL + 8 * qb, C::Q_TX);
        if constexpr (HD == 8) {
          tma_load_2d(sQ + qb * S_QBUF, &tmQ, it.c * 16, it.grow0, bars + B_QFULL + 8 * qb);
          tma_load_2d(sQ + qb * S_QBUF + 4096, &tmQ, it.c * 16 + 8, it.grow0, bars + B_QFULL + 8 * qb);
        } else {
          tma_load_2d(sQ + qb * S_QBUF, &tmQ, it.c * C::SLW, it.grow0, bars + B_QFULL + 8 * qb);
        }
      }
      ++n_q;
      for (int i = 0; i < it.T; ++i, ++n_kv) {
        int krem, yrow;
        locate(it, i, krem, yrow);
        const int st = n_kv % STAGES, use = n_kv / STAGES;
        if (use > 0) mbar_wait(wc, bars + B_KVEMPTY + 8 * st, (use - 1) & 1);
        if (elect_one()) {
          mbar_expect_tx(bars + B_KFULL + 8 * st, KVB);
          tma_load_2d(sK + st * KVB, &tmK, it.c * C::SLW, yrow, bars + B_KFULL + 8 * st);
          mbar_expect_tx(bars + B_VFULL + 8 * st, KVB);
          tma_load_2d(sV + st * KVB, &tmV, it.c * C::SLW, yrow, bars + B_VFULL + 8 * st);
        }
      }
    }
  } else if (warp == 1) {
    // ================================ MMA issuer ================================
    constexpr uint32_t IDESC_PV = idesc_bf16(NPV, true);
    int n_q = 0, n_kv = 0;  // Q tiles and key tiles consumed so far; key tile n is also phase n of the heads' S / P barriers
    for (int k = 0;; ++k) {
      const SItem it = fetch_item(wc, bars, k, lane);
      if (it.T < 0) break;
      if (it.T == 0) continue;
      const int qb = n_q & 1;
      const uint32_t sQb = sQ + qb * S_QBUF;
      mbar_wait(wc, bars + B_QFULL + 8 * qb, (n_q >> 1) & 1);
      // Round (j, h): the P V of key tile j - 1 of head h (once its weights are in TMEM), then the scores of key tile j of
      // head h.  The softmax warps of the head have finished reading S_h before they release P_h, so S_h may be
      // overwritten then; tcgen05.mma instructions of one thread execute in issue order, so P_h is read by the P V
      // before the head's next softmax (which waits for the scores issued after it) writes it again.  The other head's
      // softmax runs meanwhile.
      int krem_prev = 0;
#pragma unroll 1
      for (int j = 0; j <= it.T; ++j) {
        const int n = n_kv + j, st = n % STAGES, pst = (n - 1) % STAGES;
        int krem = 0;
        if (j < it.T) {
          int yrow;
          locate(it, j, krem, yrow);
          mbar_wait(wc, bars + B_KFULL + 8 * st, (n / STAGES) & 1);
        }
        if (j > 0) mbar_wait(wc, bars + B_VFULL + 8 * pst, ((n - 1) / STAGES) & 1);
        const int ncols = (krem >= SK) ? SK : ((krem + 15) >> 4) << 4;
        const int ksteps = (krem_prev >= SK) ? SK / 16 : (krem_prev + 15) >> 4;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          // P_h of key tile j - 1 is in TMEM (and, for the first tile of an item, the previous item's O_h has been read)
          if (j > 0) mbar_wait(wc, bars + B_PFULL + 8 * h, (n - 1) & 1);
          tc_fence_after();
          if (elect_one()) {
            if (j > 0) {
              const uint32_t vt = sV + pst * KVB + ((HD == 8) ? 0 : 2 * HD * h);
              for (int kk = 0; kk < ksteps; ++kk)  // 16 keys per step: two groups of 8 rows of the V tile
                umma_ts(tmem + S_COL_O + 32 * h, tmem + S_COL_P + 32 * h + 8 * kk, smem_desc_sw(vt + 2 * C::SBO * kk, C::SBO, C::SWZ),
                        IDESC_PV, (j > 1 || kk > 0) ? 1u : 0u);
              if (h == 1) umma_commit(bars + B_KVEMPTY + 8 * pst);  // both tiles of the stage are read
              if (j == it.T && h == 1) umma_commit(bars + B_OFINAL);
            }
            if (j < it.T) {
              const uint32_t idesc = idesc_bf16(ncols, false), kt = sK + st * KVB, d = tmem + 64 * h;
              if constexpr (HD == 8) {
                // [q_h, 0] for the even head, [0, q_h] for the odd one: start at q_even or at the zeros, 2 KB to the other half
                umma_ss(d, smem_desc_plain(sQb + h * 2048, 2048, 128), smem_desc_sw(kt, C::SBO, C::SWZ), idesc, 0);
              } else {
#pragma unroll
                for (int ks = 0; ks < HD / 16; ++ks)
                  umma_ss(d, smem_desc_sw(sQb + 2 * HD * h + 32 * ks, C::SBO, C::SWZ), smem_desc_sw(kt + 2 * HD * h + 32 * ks, C::SBO, C::SWZ),
                          idesc, ks > 0);
              }
              if (j == it.T - 1 && h == 1) umma_commit(bars + B_QEMPTY + 8 * qb);
              umma_commit(bars + B_SFULL + 8 * h);
            }
          }
          __syncwarp();
        }
        krem_prev = krem;
      }
      n_kv += it.T;
      ++n_q;
    }
  } else {
    // ================================ softmax: thread = (query row = TMEM lane, head of the pair) ================================
    const int wq = warp & 3;                               // TMEM lane quarter this warp may access
    const int h = (warp - 2) >> 2;                         // head of the pair this warp group works for
    const int r = (wq << 5) + lane;                        // row in the tile = TMEM lane
    const uint32_t tl = tmem + ((uint32_t)(wq << 5) << 16);
    const uint32_t tS = tl + 64 * h, tP = tl + S_COL_P + 32 * h, tO = tl + S_COL_O + 32 * h + ((HD == 8) ? 8 * h : 0);
    const float2 sl2v = make_float2(sl2, sl2);
    int n_kv = 0, n_items_done = 0;

    for (int k = 0;; ++k) {
      const SItem it = fetch_item(wc, bars, k, lane);
      if (it.T < 0) break;
      const int64_t grow = (int64_t)it.grow0 + r;
      const SProblem& prob = (it.c >> WHICH_SHIFT) ? prob1 : prob0;
      const int slice = it.c & ((1 << WHICH_SHIFT) - 1);
      __nv_bfloat16* __restrict__ out = prob.out;
      float* __restrict__ lse = prob.lse;
      uint4* dst = reinterpret_cast<uint4*>(out + grow * g.d + slice * C::SLW + h * HD);
      float* lse_row = (lse != nullptr) ? lse + ((int64_t)it.b * g.heads + slice * 2 + h) * g.L + g.seg_off[it.s] + it.q0 + r : nullptr;
      const bool warp_active = (wq << 5) < it.q_real;  // some row of this warp receives a result
      if (it.T == 0 || !warp_active) {
        // nothing to compute for these rows (padding only, or an empty key set): exact zeros, lse = -inf.  A warp without
        // a real row leaves the item here: the head's first warp (rows 0..31, which always hold a real row when any does)
        // arrives on the weights barrier for it as well, so it neither polls nor arrives during the key walk.
        if (r < it.rows_in_tile) {
#pragma unroll
          for (int c = 0; c < HD / 8; ++c) dst[c] = make_uint4(0, 0, 0, 0);
          if (lse_row != nullptr) *lse_row = -INFINITY;
        }
        if (it.T > 0) {
          // ... but it may not run ahead into the next item: a barrier phase is told from the one two phases later only
          // by the order of events, so every warp stays within one item of the others
          mbar_wait(wc, bars + B_OFINAL, n_items_done & 1);
          n_kv += it.T;
          ++n_items_done;
        }
        continue;
      }
      const uint32_t arrivals = (wq == 0) ? 1u + (uint32_t)(4 - min(4, (it.q_real + 31) >> 5)) : 1u;  // own + the idle warps' 
      float mu = -INFINITY, lsum = 0.f;  // running maximum (the one the weights are taken against) and sum of this row and head
#pragma unroll 1
      for (int j = 0; j < it.T; ++j) {
        const int n = n_kv + j;
        int krem, yrow;
        locate(it, j, krem, yrow);
        mbar_wait(wc, bars + B_SFULL + 8 * h, n & 1);
        tc_fence_after();
        if (krem < SK && h == 0) {
          // Rows of the V tile past the valid length hold whatever follows in memory; a zero weight times NaN or Inf
          // would still poison the accumulator, so clear them (up to the end of the last 16-key group that is
          // multiplied) before the first P V of the tile reads them: the MMA warp issues head 0's product first, after
          // this group's release of P_0.
          const int st = n % STAGES;
          mbar_wait(wc, bars + B_VFULL + 8 * st, (n / STAGES) & 1);
          const int row = krem + r;
          if (row < (((krem + 15) >> 4) << 4)) {
            const uint32_t a = sV + st * KVB + row * ROWB;
#pragma unroll
            for (int c = 0; c < ROWB / 16; ++c) st_shared_v4(a + 16 * c, 0, 0, 0, 0);
          }
          fence_async_smem();
        }
        if (warp_active) {
          // One key tile of this head, in four groups of 16 keys; groups without a real key are skipped (the branches are
          // uniform over the CTA), the group that straddles the valid length is masked element by element.  Two register
          // buffers of 16 scores: a group is requested from TMEM while the one before it is being worked on.
          uint32_t sa[16], sb[16];
          auto fix = [&](uint32_t (&a)[16], const int c) {  // keys past the valid length get weight exactly zero
            if (krem < 16 * c + 16) {
#pragma unroll
              for (int e = 0; e < 16; ++e)
                if (16 * c + e >= krem) a[e] = 0xff800000u;  // -inf
            }
          };
          // ---- pass 1: row maximum ----
          float mx4[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) mx4[i] = -INFINITY;
          auto maxc = [&](const uint32_t (&a)[16]) {
#pragma unroll
            for (int e = 0; e < 16; e += 2)
              mx4[(e >> 1) & 3] = fmax3(mx4[(e >> 1) & 3], __uint_as_float(a[e]), __uint_as_float(a[e + 1]));
          };
          tmem_ld16(tS + 0, sa);
          if (16 < krem) tmem_ld16(tS + 16, sb);
          tmem_wait_ld();
          fix(sa, 0);
          maxc(sa);
          if (16 < krem) { fix(sb, 1); maxc(sb); }
          if (32 < krem) {
            tmem_ld16(tS + 32, sa);
            if (48 < krem) tmem_ld16(tS + 48, sb);
            tmem_wait_ld();
            fix(sa, 2);
            maxc(sa);
            if (48 < krem) { fix(sb, 3); maxc(sb); }
          }
          const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
          // rescale only when the maximum has grown by more than 2^8 (P stays below 256: exact enough in bf16 and f32)
          const bool grow_m = (j == 0) || ((mx - mu) * sl2 > 8.f);
          if (j > 0 && __any_sync(0xffffffffu, grow_m)) {
            const float alpha = grow_m ? ex2((mu - mx) * sl2) : 1.f;
            lsum *= alpha;
            // O_h holds every earlier key tile: the P V of tile j - 1 was issued before the scores this thread has just
            // waited for, and the tensor pipe runs in issue order
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
          if (grow_m) mu = mx;
          // ---- pass 2: weights.  Groups 2 and 3 are still in registers when the tile has them; 0 and 1 are read again. ----
          const float nm = fmaf(-mu, sl2, TRUNC_LOG2);
          const float2 nmv = make_float2(nm, nm);
          float2 sum[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
          auto weights = [&](const uint32_t (&a)[16], const int c) {
            uint32_t pr[8];
#pragma unroll
            for (int e = 0; e < 16; e += 2) {
              const float2 x = __ffma2_rn(make_float2(__uint_as_float(a[e]), __uint_as_float(a[e + 1])), sl2v, nmv);
              // a fixed share of the exponentials goes to the FMA pipe, so that it and the special-function unit finish together
              const float2 p = ((POLY_PAIRS >> (e >> 1)) & 1) ? ex2_poly2(x) : make_float2(ex2(x.x), ex2(x.y));
              sum[(e >> 1) & 1] = __fadd2_rn(sum[(e >> 1) & 1], p);
              pr[e >> 1] = __byte_perm(__float_as_uint(p.x), __float_as_uint(p.y), 0x7632);  // upper halves: bf16 pair
            }
            tmem_st8(tP + 8 * c, pr);
          };
          if (32 < krem) {
            weights(sa, 2);
            tmem_ld16(tS + 0, sa);
            if (48 < krem) weights(sb, 3);
            tmem_wait_ld();
            tmem_ld16(tS + 16, sb);
            weights(sa, 0);
            tmem_wait_ld();
            weights(sb, 1);
          } else {
            // at most two groups: both are still in registers from pass 1 (masked already)
            weights(sa, 0);
            if (16 < krem) weights(sb, 1);
          }
          const float2 s01 = __fadd2_rn(sum[0], sum[1]);
          lsum += s01.x + s01.y;
          tmem_wait_st();
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_n(bars + B_PFULL + 8 * h, arrivals);
      }
      n_kv += it.T;

      // ---- epilogue: O_h / l -> bf16, each thread the 16 (32, 64) bytes of its row and head; padded rows +0 ----
      mbar_wait(wc, bars + B_OFINAL, n_items_done & 1);
      ++n_items_done;
      tc_fence_after();
      if (warp_active) {
        const bool real = r < it.q_real;
        const float inv = (lsum > 0.f) ? TRUNC_GAIN / lsum : 0.f;
        uint32_t orow[HD / 2];
#pragma unroll
        for (int c = 0; c < HD / 8; ++c) {
          uint32_t o[8];
          tmem_ld8(tO + 8 * c, o);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 8; e += 2)
            orow[(c * 8 + e) >> 1] = pack_bf16(__uint_as_float(o[e]) * inv, __uint_as_float(o[e + 1]) * inv);
        }
        if (r < it.rows_in_tile) {
          if (lse_row != nullptr) {
            const float ln2 = 0.6931471805599453f;
            *lse_row = (real && lsum > 0.f) ? (mu * sl2 + log2f(lsum) - TRUNC_LOG2) * ln2 : -INFINITY;
          }
#pragma unroll
          for (int c = 0; c < HD / 8; ++c)
            dst[c] = real ? make_uint4(orow[4 * c], orow[4 * c + 1], orow[4 * c + 2], orow[4 * c + 3]) : make_uint4(0, 0, 0, 0);
        }
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

template <int HD>
cudaError_t launch_tcs(const Geometry& g, const AttnOperands* ops, int n, int64_t row_stride, float scale, int* next_item,
                       cudaStream_t st, bool counter_cleared) {
  using C = SCfg<HD>;
  const int64_t rows = matrix_rows(g);
  alignas(64) SProblem pr[2];
  for (int i = 0; i < n; ++i) {
    const bool okq = (HD == 8) ? make_map(&pr[i].tmQ, ops[i].q, rows, g.d, row_stride, 8, SQ, true)
                               : make_map(&pr[i].tmQ, ops[i].q, rows, g.d, row_stride, C::SLW, SQ);
    if (!okq || !make_map(&pr[i].tmK, ops[i].k, rows, g.d, row_stride, C::SLW, SK) ||
        !make_map(&pr[i].tmV, ops[i].v, rows, g.d, row_stride, C::SLW, SK))
      return cudaErrorInvalidValue;
    pr[i].out = ops[i].out;
    pr[i].lse = ops[i].lse;
    pr[i].allowed = ops[i].allowed;
    // query segments in descending order of the keys their tiles walk (longest work first)
    int cost[3], ord[3] = {0, 1, 2};
    for (int s = 0; s < 3; ++s) {
      cost[s] = 0;
      for (int r = 0; r < 3; ++r)
        if ((ops[i].allowed >> (3 * s + r)) & 1u) cost[s] += g.seg_len[r];
    }
    for (int a = 0; a < 3; ++a)
      for (int b = a + 1; b < 3; ++b)
        if (cost[ord[b]] > cost[ord[a]]) { const int t = ord[a]; ord[a] = ord[b]; ord[b] = t; }
    pr[i].seg_order = ord[0] | (ord[1] << 2) | (ord[2] << 4);
  }
  if (n == 1) pr[1] = pr[0];
  int n_sm = 0;
  cudaError_t e = sm_count_and_smem_once(reinterpret_cast<const void*>(attn_tcs_kernel<HD>), C::SMEM, &n_sm);
  if (e != cudaSuccess) return e;
  int tiles = 0;
  for (int s = 0; s < 3; ++s) tiles += (g.seg_len[s] + SQ - 1) / SQ;
  const int slices = g.d / C::SLW;
  const int64_t n_items = (int64_t)tiles * slices * g.batch * n;
  if (n_items > 0x3fffffffLL || slices >= (1 << WHICH_SHIFT)) return cudaErrorNotSupported;
  const int64_t resident = (int64_t)S_CTAS_PER_SM * n_sm;
  const unsigned grid = (unsigned)((n_items < resident) ? n_items : resident);
  if (next_item != nullptr && !counter_cleared) {
    e = cudaMemsetAsync(next_item, 0, sizeof(int), st);
    if (e != cudaSuccess) return e;
  }
  return launch_overlapped(attn_tcs_kernel<HD>, dim3(grid), dim3(S_THREADS), C::SMEM, st, pr[0], pr[1], g,
                           scale * 1.4426950408889634f, slices, (int)n_items, n, next_item);
}

}  // namespace

bool attn_tcs_supported(const Geometry& g) {  // the kernel works on pairs of heads
  return (g.hd == 8 || g.hd == 16 || g.hd == 32) && g.heads % 2 == 0;
}

cudaError_t launch_attn_tcs(const Geometry& g, const AttnOperands* ops, int n, int64_t row_stride, float scale, int* next_item,
                            cudaStream_t st, bool counter_cleared) {
  if (!attn_tcs_supported(g) || n < 1 || n > 2) return cudaErrorNotSupported;
  if (g.hd == 8) return launch_tcs<8>(g, ops, n, row_stride, scale, next_item, st, counter_cleared);
  if (g.hd == 16) return launch_tcs<16>(g, ops, n, row_stride, scale, next_item, st, counter_cleared);
  return launch_tcs<32>(g, ops, n, row_stride, scale, next_item, st, counter_cleared);
}

}  // namespace gsit
