// bf16 IM attention for head_dim 64 on the 5th-generation tensor cores (tcgen05) with accumulators in tensor
// memory (TMEM), fed by TMA.
//
// Decomposition (paper, Section "Inner Decomposition for Efficiency"; Appendix A "From Set to Set Aggregation"):
// a work item is 128 query rows of one modality segment of one head of one sample; it walks only the key tiles of
// the segment(s) the Interlaced Mask opens for that block row, up to the sample's valid length.
//
// The grid is persistent: two CTAs per SM, each striding over the work items, so tensor memory, barriers and the
// tensor maps are set up once and the loads of the next item start while the current one is still being reduced.
// Roles inside a CTA of 6 warps:
//   warp 0, one thread   TMA producer: Q (two buffers), K and V tiles of 64 keys (four-stage rings)
//   warp 1               allocates 256 TMEM columns; one thread issues every tcgen05.mma
//                          S = Q K^T   (M 128, N 64, K 64: A and B from shared memory, 128-byte swizzle)
//                          O += P V    (M 128, N 64, K 64: A = P from TMEM, B = V tile as loaded, MN-major)
//                        S and P are double-buffered: the scores of key tile j+1 are computed while the softmax
//                        warps still work on tile j, so the exponential pipe never waits for the tensor pipe.
//   warps 2..5           softmax: thread = query row = TMEM lane.  Reads S with tcgen05.ld, keeps the running
//                        maximum and sum in registers, writes P (bf16 pairs) back to TMEM with tcgen05.st, rescales
//                        O in TMEM only when the maximum has grown by more than 2^8, and writes the result.
// TMEM columns: [0,64) and [64,128) S fp32, [128,160) and [160,192) P bf16x2, [192,256) O fp32.
// Every wait is bounded; when one expires GSIT_DEVFLAG_TIMEOUT is raised, the CTA's later waits give up at once and
// the CTA still releases its TMEM and returns.
#include <cuda.h>

#include "common.cuh"
#include "ptx.cuh"
#include "tensor_map.cuh"
#include "tmem_ldst.cuh"

namespace gsit {
namespace {

using namespace ptx;

constexpr int TQ = 128, TK = 64, HD64 = 64;
constexpr int KV_STAGES = 4, Q_BUFS = 2;
constexpr int Q_BYTES = TQ * 128, KV_BYTES = TK * 128;  // rows of 128 bytes (64 bf16)
constexpr int TC_THREADS = 192;
constexpr int TMEM_COLS = 256, COL_S = 0, COL_P = 128, COL_O = 192;  // S: 2 x 64, P: 2 x 32, O: 64 columns
// shared-memory map, relative to a 1024-byte aligned base
constexpr int OFF_Q = 0, OFF_K = OFF_Q + Q_BUFS * Q_BYTES, OFF_V = OFF_K + KV_STAGES * KV_BYTES,
              OFF_BAR = OFF_V + KV_STAGES * KV_BYTES;
constexpr int BAR_QFULL = 0, BAR_QEMPTY = 16, BAR_KFULL = 32, BAR_VFULL = 64, BAR_KEMPTY = 96, BAR_VEMPTY = 128,
              BAR_SFULL = 160, BAR_PFULL = 176, BAR_OFINAL = 192, SLOT_TMEM = 200, SLOT_GAVE_UP = 204;
// Work items are decoded once, by the producer warp, and handed to the other roles through a ring of records in
// shared memory (the decode needs the sample's valid lengths from global memory and two integer divisions).
constexpr int ITEM_SLOTS = 8;
constexpr int OFF_ITEMBAR = OFF_BAR + 256;                      // ITEM_SLOTS "record written" + ITEM_SLOTS "record read" barriers
constexpr int OFF_ITEMS = OFF_ITEMBAR + 16 * ITEM_SLOTS;        // ITEM_SLOTS records of 16 ints
constexpr int TC_SMEM = OFF_ITEMS + 64 * ITEM_SLOTS + 1024 /* alignment slack */;

template <bool V> struct BoolTag { static constexpr bool value = V; };

// One work item: a tile of query rows of one block row, one head, one sample.
struct Item {
  int b, h, s, q0;
  int rows_in_tile;  // rows of the tile that belong to the segment (the rest belongs to whatever follows)
  int q_real;        // rows that receive a computed result; the remaining rows_in_tile - q_real are written as +0
  int T;             // key tiles to walk
  int kn0, kn1, kn2, nk0, nk1;  // real keys per open key segment, key tiles of the first two
  int kb0, kb1, kb2;            // first row of each key segment in the activation matrices (padded or packed layout)
  int grow0;                    // first row of the query tile in the activation matrices
};

__device__ __forceinline__ Item decode_item(const Geometry& g, int w, int tiles_per_sample) {
  Item it;
  const int bh = w / tiles_per_sample;
  int tile = w - bh * tiles_per_sample;
  it.b = bh / g.heads;
  it.h = bh - it.b * g.heads;
  int s = 0;
#pragma unroll
  for (int ss = 0; ss < 2; ++ss) {
    const int nts = (g.seg_len[s] + TQ - 1) / TQ;
    if (tile >= nts) { tile -= nts; ++s; }
  }
  it.s = s;
  it.q0 = tile * TQ;
  const int in_seg = min(TQ, g.seg_len[s] - it.q0);
  const int q_real_all = max(0, min(in_seg, valid_rows(g, it.b, s) - it.q0));
  // rows of the tile this CTA writes: in the padded layout all that belong to the segment (padding as +0); in the packed
  // layout only the real ones exist -- what follows them in memory is another segment
  it.rows_in_tile = (g.row_start != nullptr) ? q_real_all : in_seg;
  it.kb0 = seg_row0(g, it.b, 0);
  it.kb1 = seg_row0(g, it.b, 1);
  it.kb2 = seg_row0(g, it.b, 2);
  it.grow0 = seg_row0(g, it.b, s) + it.q0;
  it.kn0 = ((g.allowed >> (3 * s + 0)) & 1u) ? valid_rows(g, it.b, 0) : 0;
  it.kn1 = ((g.allowed >> (3 * s + 1)) & 1u) ? valid_rows(g, it.b, 1) : 0;
  it.kn2 = ((g.allowed >> (3 * s + 2)) & 1u) ? valid_rows(g, it.b, 2) : 0;
  it.nk0 = (it.kn0 + TK - 1) / TK;
  it.nk1 = (it.kn1 + TK - 1) / TK;
  const int nk2 = (it.kn2 + TK - 1) / TK;
  it.T = (q_real_all > 0) ? it.nk0 + it.nk1 + nk2 : 0;
  it.q_real = (it.T > 0) ? q_real_all : 0;
  return it;
}

// Key tile i of an item: real keys left from its start (>= 1), first row in the flattened [B*L] sequence.
__device__ __forceinline__ void locate(const Geometry& g, const Item& it, int i, int& krem, int& yrow) {
  int t = i, r = 0;
  if (t >= it.nk0) { t -= it.nk0; r = 1; if (t >= it.nk1) { t -= it.nk1; r = 2; } }
  const int kn = (r == 0) ? it.kn0 : (r == 1) ? it.kn1 : it.kn2;
  krem = kn - t * TK;
  yrow = ((r == 0) ? it.kb0 : (r == 1) ? it.kb1 : it.kb2) + t * TK;
}

// Producer side: lane 0 writes record k of this CTA, then the slot's "written" barrier is released.
__device__ __forceinline__ void publish_item(uint32_t base, const Item& it, int k, int lane) {
  if (lane == 0) {
    const uint32_t a = base + OFF_ITEMS + 64 * (k % ITEM_SLOTS);
    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(it.b), "r"(it.h), "r"(it.s), "r"(it.q0) : "memory");
    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(a + 16), "r"(it.rows_in_tile), "r"(it.q_real), "r"(it.T), "r"(it.kn0) : "memory");
    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(a + 32), "r"(it.kn1), "r"(it.kn2), "r"(it.nk0), "r"(it.nk1) : "memory");
    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(a + 48), "r"(it.kb0), "r"(it.kb1), "r"(it.kb2), "r"(it.grow0) : "memory");
    mbar_arrive(base + OFF_ITEMBAR + 8 * (k % ITEM_SLOTS));
  }
  __syncwarp();
}
// Consumer side (whole warp): waits for record k, copies it to registers and releases the slot (one arrival per warp).
__device__ __forceinline__ Item fetch_item(const WaitCtx& wc, uint32_t base, int k, int lane) {
  const int slot = k % ITEM_SLOTS;
  mbar_wait(wc, base + OFF_ITEMBAR + 8 * slot, (k / ITEM_SLOTS) & 1);
  const uint32_t a = base + OFF_ITEMS + 64 * slot;
  Item it;
  asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(it.b), "=r"(it.h), "=r"(it.s), "=r"(it.q0) : "r"(a) : "memory");
  asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(it.rows_in_tile), "=r"(it.q_real), "=r"(it.T), "=r"(it.kn0) : "r"(a + 16) : "memory");
  asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(it.kn1), "=r"(it.kn2), "=r"(it.nk0), "=r"(it.nk1) : "r"(a + 32) : "memory");
  asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(it.kb0), "=r"(it.kb1), "=r"(it.kb2), "=r"(it.grow0) : "r"(a + 48) : "memory");
  fence_reads_before_release();
  __syncwarp();
  if (lane == 0) mbar_arrive(base + OFF_ITEMBAR + 8 * ITEM_SLOTS + 8 * slot);
  return it;
}

__global__ void __launch_bounds__(TC_THREADS, 2)
attn_tc_hd64_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const Geometry g, __nv_bfloat16* __restrict__ out,
                    float* __restrict__ lse, const float sl2 /* scale * log2(e) */, const int tiles_per_sample,
                    const int n_items) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sQ = base + OFF_Q, sK = base + OFF_K, sV = base + OFF_V, bars = base + OFF_BAR;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const WaitCtx wc{g.status, bars + SLOT_GAVE_UP};

  // ---- set-up, once per CTA: barriers, tensor memory ----
  if (tid == 0) {
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(bars + SLOT_GAVE_UP), "r"(0u) : "memory");
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      mbar_init(bars + BAR_QFULL + 8 * i, 1);
      mbar_init(bars + BAR_QEMPTY + 8 * i, 1);
      mbar_init(bars + BAR_SFULL + 8 * i, 1);
      mbar_init(bars + BAR_PFULL + 8 * i, 128);
    }
#pragma unroll
    for (int i = 0; i < KV_STAGES; ++i) {
      mbar_init(bars + BAR_KFULL + 8 * i, 1);
      mbar_init(bars + BAR_VFULL + 8 * i, 1);
      mbar_init(bars + BAR_KEMPTY + 8 * i, 1);
      mbar_init(bars + BAR_VEMPTY + 8 * i, 1);
    }
    mbar_init(bars + BAR_OFINAL, 1);
    for (int i = 0; i < ITEM_SLOTS; ++i) {
      mbar_init(base + OFF_ITEMBAR + 8 * i, 1);                   // record written (producer)
      mbar_init(base + OFF_ITEMBAR + 8 * ITEM_SLOTS + 8 * i, 5);  // record read (MMA warp + four softmax warps)
    }
    mbar_init_fence();
  }
  if (warp == 1) tmem_alloc(bars + SLOT_TMEM, TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  uint32_t tmem;
  asm volatile("ld.shared.b32 %0, [%1];" : "=r"(tmem) : "r"(bars + SLOT_TMEM) : "memory");

  if (warp == 0) {
    // ================================ TMA producer ================================
    {
      int n_q = 0, n_kv = 0;  // Q tiles and K/V tiles requested so far (ring positions and phases follow from them)
      int k = 0;              // items of this CTA so far
      for (int w = blockIdx.x; w < n_items; w += gridDim.x, ++k) {
        const Item it = decode_item(g, w, tiles_per_sample);
        if (k >= ITEM_SLOTS) mbar_wait(wc, base + OFF_ITEMBAR + 8 * ITEM_SLOTS + 8 * (k % ITEM_SLOTS), ((k / ITEM_SLOTS) - 1) & 1);
        publish_item(base, it, k, lane);
        if (it.T == 0) continue;
        const int qb = n_q & 1, quse = n_q >> 1;
        if (quse > 0) mbar_wait(wc, bars + BAR_QEMPTY + 8 * qb, (quse - 1) & 1);
        if (elect_one()) {
          mbar_expect_tx(bars + BAR_QFULL + 8 * qb, Q_BYTES);
          tma_load_2d(sQ + qb * Q_BYTES, &tmQ, it.h * HD64, it.grow0, bars + BAR_QFULL + 8 * qb);
        }
        ++n_q;
        for (int i = 0; i < it.T; ++i, ++n_kv) {
          int krem, yrow;
          locate(g, it, i, krem, yrow);
          const int st = n_kv % KV_STAGES, use = n_kv / KV_STAGES;
          if (use > 0) mbar_wait(wc, bars + BAR_KEMPTY + 8 * st, (use - 1) & 1);
          if (elect_one()) {
            mbar_expect_tx(bars + BAR_KFULL + 8 * st, KV_BYTES);
            tma_load_2d(sK + st * KV_BYTES, &tmK, it.h * HD64, yrow, bars + BAR_KFULL + 8 * st);
          }
          if (use > 0) mbar_wait(wc, bars + BAR_VEMPTY + 8 * st, (use - 1) & 1);
          if (elect_one()) {
            mbar_expect_tx(bars + BAR_VFULL + 8 * st, KV_BYTES);
            tma_load_2d(sV + st * KV_BYTES, &tmV, it.h * HD64, yrow, bars + BAR_VFULL + 8 * st);
          }
        }
      }
    }
  } else if (warp == 1) {
    // ================================ MMA issuer ================================
    {
      constexpr uint32_t IDESC_QK = idesc_bf16(TK, false), IDESC_PV = idesc_bf16(HD64, true);
      int n_q = 0, n_kv = 0;  // Q tiles / key tiles consumed so far.  Key tile n uses S and P buffer n & 1 (phase
                              // (n >> 1) & 1 of their barriers) and ring stage n % KV_STAGES
      int k = 0;
      for (int w = blockIdx.x; w < n_items; w += gridDim.x, ++k) {
        const Item it = fetch_item(wc, base, k, lane);
        if (it.T == 0) continue;
        const int qb = n_q & 1;
        const uint32_t sQb = sQ + qb * Q_BYTES;
        // S[n & 1] = Q K_n^T: four steps of 16 along head_dim (32 bytes inside the swizzled row).  The buffer was last
        // read by the softmax of key tile n - 2, whose P this thread has already waited for.
        auto issue_qk = [&](int n, bool last) {
          const int st = n % KV_STAGES;
          mbar_wait(wc, bars + BAR_KFULL + 8 * st, (n / KV_STAGES) & 1);
          tc_fence_after();
          if (elect_one()) {
#pragma unroll
            for (int k = 0; k < HD64 / 16; ++k)
              umma_ss(tmem + COL_S + 64 * (n & 1), smem_desc_sw128(sQb + 32 * k),
                      smem_desc_sw128(sK + st * KV_BYTES + 32 * k), IDESC_QK, k > 0);
            umma_commit(bars + BAR_KEMPTY + 8 * st);
            if (last) umma_commit(bars + BAR_QEMPTY + 8 * qb);
            umma_commit(bars + BAR_SFULL + 8 * (n & 1));
          }
          __syncwarp();
        };
        mbar_wait(wc, bars + BAR_QFULL + 8 * qb, (n_q >> 1) & 1);
        issue_qk(n_kv, it.T == 1);
        for (int j = 0; j < it.T; ++j) {
          const int n = n_kv + j, st = n % KV_STAGES;
          if (j + 1 < it.T) issue_qk(n + 1, j + 2 == it.T);  // scores of the next tile, ahead of this tile's P V
          // P[n & 1] is in TMEM (and, for the first tile of an item, the previous item's O has been read)
          mbar_wait(wc, bars + BAR_PFULL + 8 * (n & 1), (n >> 1) & 1);
          mbar_wait(wc, bars + BAR_VFULL + 8 * st, (n / KV_STAGES) & 1);
          tc_fence_after();
          if (elect_one()) {
#pragma unroll
            for (int k = 0; k < TK / 16; ++k)  // O += P V: four steps of 16 keys (two 8-row groups = 2048 bytes of V)
              umma_ts(tmem + COL_O, tmem + COL_P + 32 * (n & 1) + 8 * k, smem_desc_sw128(sV + st * KV_BYTES + 2048 * k),
                      IDESC_PV, (j > 0 || k > 0) ? 1u : 0u);
            umma_commit(bars + BAR_VEMPTY + 8 * st);  // also tells the softmax warps that O holds tiles 0..j
            if (j + 1 == it.T) umma_commit(bars + BAR_OFINAL);
          }
          __syncwarp();
        }
        n_kv += it.T;
        ++n_q;
      }
    }
  } else {
    // ================================ softmax, one thread per query row ================================
    const int r = ((warp & 3) << 5) + lane;                          // row in the tile = TMEM lane
    const uint32_t tl = tmem + ((uint32_t)((warp & 3) << 5) << 16);  // this warp's lane quarter
    const float2 sl2v = make_float2(sl2, sl2);
    int n_kv = 0, n_items_done = 0;

    int k = 0;
    for (int w = blockIdx.x; w < n_items; w += gridDim.x, ++k) {
      const Item it = fetch_item(wc, base, k, lane);
      const int64_t grow = (int64_t)it.grow0 + r;
      uint4* dst = reinterpret_cast<uint4*>(out + grow * g.d + it.h * HD64);
      float* lse_row = (lse != nullptr) ? lse + ((int64_t)it.b * g.heads + it.h) * g.L + g.seg_off[it.s] + it.q0 + r : nullptr;
      if (it.T == 0) {  // nothing to attend (padding rows only, or an empty key set): exact zeros, lse = -inf
        if (r < it.rows_in_tile) {
#pragma unroll
          for (int c = 0; c < 8; ++c) dst[c] = make_uint4(0, 0, 0, 0);
          if (lse_row != nullptr) *lse_row = -INFINITY;
        }
        continue;
      }
      float m_used = -INFINITY, l = 0.f;

      auto tile_step = [&](auto ragged_tag, const int j, const int n, const int krem) {
        constexpr bool RAGGED = decltype(ragged_tag)::value;
        const int sb = n & 1;
        mbar_wait(wc, bars + BAR_SFULL + 8 * sb, (n >> 1) & 1);
        tc_fence_after();
        uint32_t sr[2][32];
#pragma unroll
        for (int c = 0; c < 2; ++c) tmem_ld32(tl + COL_S + 64 * sb + 32 * c, sr[c]);
        tmem_wait_ld();
        if (RAGGED) {  // keys past the valid length get weight exactly zero
#pragma unroll
          for (int c = 0; c < 2; ++c)
#pragma unroll
            for (int e = 0; e < 32; ++e)
              if (c * 32 + e >= krem) sr[c][e] = 0xff800000u;  // -inf
        }
        float mx8[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) mx8[i] = -INFINITY;
#pragma unroll
        for (int c = 0; c < 2; ++c)
#pragma unroll
          for (int e = 0; e < 32; e += 2)
            mx8[(e >> 1) & 7] = fmaxf(mx8[(e >> 1) & 7], fmaxf(__uint_as_float(sr[c][e]), __uint_as_float(sr[c][e + 1])));
        const float mx = fmaxf(fmaxf(fmaxf(mx8[0], mx8[1]), fmaxf(mx8[2], mx8[3])),
                               fmaxf(fmaxf(mx8[4], mx8[5]), fmaxf(mx8[6], mx8[7])));
        // rescale only when the maximum has grown by more than 2^8 (P stays below 256: exact enough in bf16 and f32)
        const bool grow_m = (j == 0) || ((mx - m_used) * sl2 > 8.f);
        if (j > 0 && __any_sync(0xffffffffu, grow_m)) {
          const float alpha = grow_m ? ex2((m_used - mx) * sl2) : 1.f;
          l *= alpha;
          // O must hold every earlier tile of the item before it is rescaled: wait for the P V of tile n - 1
          mbar_wait(wc, bars + BAR_VEMPTY + 8 * ((n - 1) % KV_STAGES), ((n - 1) / KV_STAGES) & 1);
          tc_fence_after();
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            uint32_t o[16];
            tmem_ld16(tl + COL_O + 16 * c, o);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 16; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
            tmem_st16(tl + COL_O + 16 * c, o);
          }
        }
        if (grow_m) m_used = mx;
        const float nm = -m_used * sl2;
        const float2 nmv = make_float2(nm, nm);
        float2 sum[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) sum[i] = make_float2(0.f, 0.f);
        uint32_t pr[32];
#pragma unroll
        for (int c = 0; c < 2; ++c)
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            const float2 x = __ffma2_rn(make_float2(__uint_as_float(sr[c][e]), __uint_as_float(sr[c][e + 1])), sl2v, nmv);
            const float2 p = make_float2(ex2(x.x), ex2(x.y));
            sum[(e >> 1) & 3] = __fadd2_rn(sum[(e >> 1) & 3], p);
            pr[c * 16 + (e >> 1)] = pack_bf16(p.x, p.y);
          }
        tmem_st32(tl + COL_P + 32 * sb, pr);
        const float2 s01 = __fadd2_rn(__fadd2_rn(sum[0], sum[1]), __fadd2_rn(sum[2], sum[3]));
        l += s01.x + s01.y;
        if (RAGGED) {
          // Rows of the V tile past the valid length hold whatever follows in memory; a zero weight times NaN or Inf
          // would still poison the accumulator, so clear them before the MMA reads the tile.
          const int st = n % KV_STAGES;
          mbar_wait(wc, bars + BAR_VFULL + 8 * st, (n / KV_STAGES) & 1);
          const int row = krem + (tid - 64);
          if (row < TK) {
            const uint32_t a = sV + st * KV_BYTES + row * 128;
#pragma unroll
            for (int c = 0; c < 8; ++c)
              st_shared_v4(a + 16 * c, 0, 0, 0, 0);
          }
          fence_async_smem();
        }
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bars + BAR_PFULL + 8 * sb);
      };

      for (int j = 0; j < it.T; ++j) {
        int krem, yrow;
        locate(g, it, j, krem, yrow);
        if (krem < TK) tile_step(BoolTag<true>{}, j, n_kv + j, krem);
        else tile_step(BoolTag<false>{}, j, n_kv + j, TK);
      }
      n_kv += it.T;

      // ---- epilogue: O / l -> bf16, each thread its own 128-byte row; padded rows +0 ----
      mbar_wait(wc, bars + BAR_OFINAL, n_items_done & 1);
      ++n_items_done;
      tc_fence_after();
      const float inv = (l > 0.f) ? 1.f / l : 0.f;
      const bool real = r < it.q_real;
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t o[32];
        tmem_ld32(tl + COL_O + 32 * c, o);
        tmem_wait_ld();
        if (r < it.rows_in_tile) {
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
      if (lse_row != nullptr && r < it.rows_in_tile) {
        const float ln2 = 0.6931471805599453f;
        *lse_row = (real && l > 0.f) ? (m_used * sl2 + log2f(l)) * ln2 : -INFINITY;
      }
    }
  }

  // ---- release tensor memory once every role is done with it ----
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, TMEM_COLS);
  }
}

}  // namespace

cudaError_t launch_attn_tc_hd64(const Geometry& g, const __nv_bfloat16* q, const __nv_bfloat16* k,
                                const __nv_bfloat16* v, int64_t row_stride, __nv_bfloat16* out, float* lse,
                                float scale, cudaStream_t st) {
  if (g.hd != HD64) return cudaErrorNotSupported;
  const int64_t rows = matrix_rows(g);
  alignas(64) CUtensorMap tmQ, tmK, tmV;
  if (!make_map(&tmQ, q, rows, g.d, row_stride, HD64, TQ) || !make_map(&tmK, k, rows, g.d, row_stride, HD64, TK) ||
      !make_map(&tmV, v, rows, g.d, row_stride, HD64, TK))
    return cudaErrorInvalidValue;
  int n_sm = 0;
  {
    cudaError_t e = sm_count_and_smem_once(reinterpret_cast<const void*>(attn_tc_hd64_kernel), TC_SMEM, &n_sm);
    if (e != cudaSuccess) return e;
  }
  int tiles = 0;
  for (int s = 0; s < 3; ++s) tiles += (g.seg_len[s] + TQ - 1) / TQ;
  const int64_t n_items = (int64_t)tiles * g.heads * g.batch;
  if (n_items > 0x7fffffffLL) return cudaErrorNotSupported;
  const unsigned grid = (unsigned)((n_items < 2 * n_sm) ? n_items : 2 * n_sm);  // two resident CTAs per SM
  attn_tc_hd64_kernel<<<grid, TC_THREADS, TC_SMEM, st>>>(tmQ, tmK, tmV, g, out, lse, scale * 1.4426950408889634f, tiles,
                                                          (int)n_items);
  return cudaGetLastError();
}

}  // namespace gsit
