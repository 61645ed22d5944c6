// Kernel body of the bf16 IM attention (included by attn_bf16.cu only).
#pragma once

namespace gsit {
namespace {

template <bool V> struct BoolTag { static constexpr bool value = V; };
template <int V> struct IntTag { static constexpr int value = V; };

// What distinguishes one attention problem of a launch from the other: its tensors, its block pattern and the order in
// which its query segments are launched.
struct AttnProblem {
  CUtensorMap tmQ, tmK, tmV;
  __nv_bfloat16* out;
  float* lse;
  uint32_t allowed;
  int seg_order;
};

#ifndef GSIT_MS_POLY
#define GSIT_MS_POLY 0
#endif
constexpr unsigned MS_POLY = GSIT_MS_POLY;  // bit i: score n-tile i of a step takes the polynomial 2^x

template <typename C>
__global__ void __launch_bounds__(NTHREADS, C::MINB)
attn_bf16_kernel(const __grid_constant__ AttnProblem prob0, const __grid_constant__ AttnProblem prob1, const Geometry g0,
                 const float sl2 /* scale * log2(e) */, const int problems) {
  // One launch can serve two problems of the same geometry that differ in their tensors and block pattern (the forward
  // and the backward ring of one encoder depth); the problem index varies fastest over the grid, so both keep the
  // longest-first launch order.
  const int which = (problems == 2) ? (int)(blockIdx.x & 1u) : 0;
  const int bx = (problems == 2) ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const AttnProblem& prob = which ? prob1 : prob0;
  const CUtensorMap &tmQ = prob.tmQ, &tmK = prob.tmK, &tmV = prob.tmV;
  __nv_bfloat16* __restrict__ out = prob.out;
  float* __restrict__ lse = prob.lse;
  const int seg_order = prob.seg_order;
  Geometry g = g0;
  g.allowed = prob.allowed;
  constexpr int HD = C::HD, CW = C::CW, G = C::G, R = C::R, QT = C::QT, PITCH = C::PITCH, SWZ = C::SWZ,
                KSTEP = C::KSTEP, NT = C::NT, KSQ = C::KSQ, NTO = C::NTO, CPR = CW / 8 /* 16-byte chunks per row */;
  constexpr bool HOIST = (R > 1);  // several query slabs per warp reuse the K/V fragments of a step

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t sQ = (raw + 1023u) & ~1023u;
  const uint32_t sK = sQ + ((C::Q_BYTES + 1023) / 1024) * 1024;
  const uint32_t sV = sK + STAGES * C::KV_BYTES;
  const uint32_t bar_full = sV + STAGES * C::KV_BYTES;  // STAGES barriers of 8 bytes: TMA bytes have landed
  const uint32_t bar_empty = bar_full + 8 * STAGES;     // STAGES barriers: all 8 warps are done with the stage
  const uint32_t bar_q = bar_empty + 8 * STAGES;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int head_in_slice = warp % G, sg = warp / G;
  grid_dep_wait();  // q, k, v come from the kernel before this one
  grid_dep_launch();
  const int cb = head_in_slice * (HD / 8);  // first 16-byte chunk of this warp's head inside a tile row

  // ---- which tile of which block row.  blockIdx.x = (tile in cost order) * batch + sample: the query segments with
  // the most keys to walk are launched first (seg_order packs the three segment indices, two bits each), and CTAs that
  // run together work on the same tile of different samples, so the last wave is short and made of the cheapest tiles.
  const int b = bx % g.batch;
  int tile = bx / g.batch, s = seg_order & 3;
#pragma unroll
  for (int rank = 0; rank < 2; ++rank) {
    const int nts = (g.seg_len[s] + QT - 1) / QT;
    if (tile >= nts) { tile -= nts; s = (seg_order >> (2 * rank + 2)) & 3; }
  }
  const int q0 = tile * QT;
  const int cs = blockIdx.y;
  const int q_real_all = max(0, min(min(QT, g.seg_len[s] - q0), valid_rows(g, b, s) - q0));
  // rows of the tile this CTA writes: in the padded layout all that belong to the segment (padding as +0); in the packed
  // layout only the real ones exist -- what follows them in memory is another segment
  const bool packed = g.row_start != nullptr;
  const int rows_in_tile = packed ? q_real_all : min(QT, g.seg_len[s] - q0);
  const int kn0 = ((g.allowed >> (3 * s + 0)) & 1u) ? valid_rows(g, b, 0) : 0;
  const int kn1 = ((g.allowed >> (3 * s + 1)) & 1u) ? valid_rows(g, b, 1) : 0;
  const int kn2 = ((g.allowed >> (3 * s + 2)) & 1u) ? valid_rows(g, b, 2) : 0;
  const int nk0 = (kn0 + KT - 1) / KT, nk1 = (kn1 + KT - 1) / KT, nk2 = (kn2 + KT - 1) / KT;
  const int T = (q_real_all > 0) ? nk0 + nk1 + nk2 : 0;  // key tiles this CTA walks
  const int q_real = (T > 0) ? q_real_all : 0;           // rows that receive a computed result
  const int64_t grow0 = (int64_t)seg_row0(g, b, s) + q0;  // first row of the tile in the activation matrices
  const int xcol = cs * CW;
  const int kbase0 = seg_row0(g, b, 0), kbase1 = seg_row0(g, b, 1), kbase2 = seg_row0(g, b, 2);

  auto locate = [&](int i, int& krem, int& yrow) {
    int t = i, r = 0;
    if (t >= nk0) { t -= nk0; r = 1; if (t >= nk1) { t -= nk1; r = 2; } }
    const int kn = (r == 0) ? kn0 : (r == 1) ? kn1 : kn2;
    krem = kn - t * KT;
    yrow = ((r == 0) ? kbase0 : (r == 1) ? kbase1 : kbase2) + t * KT;
  };
  auto issue = [&](int i) {  // one thread: TMA loads of key tile i into its stage
    int krem, yrow;
    locate(i, krem, yrow);
    const int st = i % STAGES;
    mbar_expect_tx(bar_full + 8 * st, 2 * C::KV_BYTES);
    tma_load_2d(sK + st * C::KV_BYTES, &tmK, xcol, yrow, bar_full + 8 * st);
    tma_load_2d(sV + st * C::KV_BYTES, &tmV, xcol, yrow, bar_full + 8 * st);
  };

  float O[R][NTO][4];
  float m[R][2], l[R][4];  // l: accumulator tile of P 1 (elements 0 and 2 are the sums of rows g and g + 8)
#pragma unroll
  for (int r_ = 0; r_ < R; ++r_) {
    m[r_][0] = m[r_][1] = -INFINITY;
    l[r_][0] = l[r_][1] = l[r_][2] = l[r_][3] = 0.f;
#pragma unroll
    for (int n = 0; n < NTO; ++n) O[r_][n][0] = O[r_][n][1] = O[r_][n][2] = O[r_][n][3] = 0.f;
  }

  if (T > 0) {
    if (tid == 0) {
#pragma unroll
      for (int st = 0; st < STAGES; ++st) {
        mbar_init(bar_full + 8 * st, 1);
        mbar_init(bar_empty + 8 * st, NTHREADS / 32);
      }
      mbar_init(bar_q, 1);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    int next_issue = 0;  // meaningful in thread 0 only: next key tile to request
    if (tid == 0) {
      mbar_expect_tx(bar_q, C::Q_BYTES);
      tma_load_2d(sQ, &tmQ, xcol, (int)grow0, bar_q);
      for (; next_issue < STAGES && next_issue < T; ++next_issue) issue(next_issue);
    }

    // ---- query fragments, kept in registers for the whole key walk ----
    uint32_t QF[R][KSQ][4];
    mbar_wait(g, bar_q, 0);
#pragma unroll
    for (int r_ = 0; r_ < R; ++r_) {
      const int row0 = (sg * R + r_) * 16;
      if constexpr (HD == 8) {
        const int row = row0 + (lane & 15);
        ldsm_x2(sQ + swz<SWZ>(row * PITCH + cb * 16), QF[r_][0][0], QF[r_][0][1]);
        QF[r_][0][2] = QF[r_][0][3] = 0;
      } else {
        const int mi = lane >> 3;
        const int row = row0 + (mi & 1) * 8 + (lane & 7);
#pragma unroll
        for (int ks = 0; ks < KSQ; ++ks)
          ldsm_x4(sQ + swz<SWZ>(row * PITCH + (cb + ks * 2 + (mi >> 1)) * 16), QF[r_][ks][0], QF[r_][ks][1],
                  QF[r_][ks][2], QF[r_][ks][3]);
      }
    }

    // One pipeline stage (KT keys) for all query slabs of this warp.  RAGGED: the stage holds fewer than KT real keys;
    // the instantiation then covers only the first NTV score n-tiles (8 keys each, NTV even: whole 16-key groups of
    // P V), so that a tile with few real keys costs proportionally less, and only its last two n-tiles are masked
    // element by element.  Everything stays straight-line code inside an instantiation.
    auto process = [&](auto ragged_tag, auto ntv_tag, const uint32_t sKs, const uint32_t sVs, const int krem) {
      constexpr bool RAGGED = decltype(ragged_tag)::value;
      constexpr int NTV = decltype(ntv_tag)::value;  // n-tiles computed (== NT for a full tile)
      static_assert(NTV % 2 == 0 && NTV >= 2 && NTV <= NT && (KT == KSTEP || !RAGGED || NTV == NT), "n-tile count");
      if constexpr (RAGGED) {
        // Rows past the valid length hold whatever follows in memory: clear this head's part of them in V so that a
        // zero weight times a NaN/Inf value cannot poison the accumulator (their scores become -inf below).  Warps
        // sharing the head write the same zeros.
        constexpr int KROWS = (KT == KSTEP) ? NTV * 8 : KT;  // key rows of the stage that the products read
        for (int idx = lane; idx < (KROWS - krem) * (HD / 8); idx += 32) {
          const int row = krem + idx / (HD / 8), ch = cb + idx % (HD / 8);
          asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(sVs + swz<SWZ>(row * PITCH + ch * 16)), "r"(0) : "memory");
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
      }
#pragma unroll
      for (int stp = 0; stp < KT / KSTEP; ++stp) {
        const int kb = stp * KSTEP;
        if (RAGGED && kb >= krem) break;
        uint32_t KF[NT][KSQ][2];
        uint32_t VF[KSTEP / 16][NTO][2];

        auto load_k_pair = [&](int p) {  // K fragments of score n-tiles 2p, 2p+1 (HD >= 16)
          const int mi = lane >> 3;
          const int key = kb + p * 16 + (mi >> 1) * 8 + (lane & 7);
#pragma unroll
          for (int ks = 0; ks < KSQ; ++ks)
            ldsm_x4(sKs + swz<SWZ>(key * PITCH + (cb + ks * 2 + (mi & 1)) * 16), KF[2 * p][ks][0], KF[2 * p][ks][1],
                    KF[2 * p + 1][ks][0], KF[2 * p + 1][ks][1]);
        };
        auto load_v_pair = [&](int kk, int np) {  // V fragments of key step kk, output n-tiles 2np, 2np+1 (HD >= 16)
          const int mi = lane >> 3;
          const int key = kb + kk * 16 + (mi & 1) * 8 + (lane & 7);
          ldsm_x4_t(sVs + swz<SWZ>(key * PITCH + (cb + np * 2 + (mi >> 1)) * 16), VF[kk][2 * np][0], VF[kk][2 * np][1],
                    VF[kk][2 * np + 1][0], VF[kk][2 * np + 1][1]);
        };
        auto load_k8 = [&](int j) {  // HD == 8: K fragments of n-tiles 4j .. 4j+3 (32 keys)
          ldsm_x4(sKs + swz<SWZ>((kb + j * 32 + lane) * PITCH + cb * 16), KF[4 * j][0][0], KF[4 * j + 1][0][0],
                  KF[4 * j + 2][0][0], KF[4 * j + 3][0][0]);
        };
        auto load_v8 = [&](int j) {  // HD == 8: V fragments of key steps 2j, 2j+1 (32 keys)
          ldsm_x4_t(sVs + swz<SWZ>((kb + j * 32 + lane) * PITCH + cb * 16), VF[2 * j][0][0], VF[2 * j][0][1],
                    VF[2 * j + 1][0][0], VF[2 * j + 1][0][1]);
        };

        if constexpr (HOIST) {
          if constexpr (HD == 8) {
#pragma unroll
            for (int j = 0; j < (NTV + 3) / 4; ++j) { load_k8(j); load_v8(j); }
          } else {
#pragma unroll
            for (int p = 0; p < NTV / 2; ++p) load_k_pair(p);
#pragma unroll
            for (int kk = 0; kk < NTV / 2; ++kk)
#pragma unroll
              for (int np = 0; np < NTO / 2; ++np) load_v_pair(kk, np);
          }
        }

#pragma unroll
        for (int r_ = 0; r_ < R; ++r_) {
          const int row0 = (sg * R + r_) * 16;
          if (row0 >= q_real) continue;  // slab of padding rows only
          float S[NT][4];
#pragma unroll
          for (int n = 0; n < NT; ++n) S[n][0] = S[n][1] = S[n][2] = S[n][3] = 0.f;

          // ---- S = Q K^T (raw dot products) ----
          if constexpr (HD == 8) {
#pragma unroll
            for (int j = 0; j < (NTV + 3) / 4; ++j) {
              if constexpr (!HOIST) load_k8(j);
#pragma unroll
              for (int n = 4 * j; n < 4 * j + 4; ++n)
                if (n < NTV) mma_k8(S[n], QF[r_][0][0], QF[r_][0][1], KF[n][0][0]);
            }
          } else {
#pragma unroll
            for (int p = 0; p < NTV / 2; ++p) {
              if constexpr (!HOIST) load_k_pair(p);
#pragma unroll
              for (int ks = 0; ks < KSQ; ++ks) {
                mma_k16(S[2 * p], QF[r_][ks][0], QF[r_][ks][1], QF[r_][ks][2], QF[r_][ks][3], KF[2 * p][ks][0],
                        KF[2 * p][ks][1]);
                mma_k16(S[2 * p + 1], QF[r_][ks][0], QF[r_][ks][1], QF[r_][ks][2], QF[r_][ks][3], KF[2 * p + 1][ks][0],
                        KF[2 * p + 1][ks][1]);
              }
            }
          }
          // ---- keys past the valid length get weight exactly zero ----
          if constexpr (RAGGED) {
            const int c0 = kb + (lane & 3) * 2;
#pragma unroll
            for (int n = (KT == KSTEP ? NTV - 2 : 0); n < NTV; ++n) {  // the invalid keys are a suffix of the last 16-key group
              if (c0 + n * 8 >= krem) S[n][0] = S[n][2] = -INFINITY;
              if (c0 + n * 8 + 1 >= krem) S[n][1] = S[n][3] = -INFINITY;
            }
          }
          // ---- online softmax (base 2, scale folded into sl2); pairwise trees keep dependency chains short ----
          float t0[NTV], t1[NTV];
#pragma unroll
          for (int n = 0; n < NTV; ++n) { t0[n] = fmaxf(S[n][0], S[n][1]); t1[n] = fmaxf(S[n][2], S[n][3]); }
#pragma unroll
          for (int cnt = NTV; cnt > 1; cnt = (cnt + 1) / 2)  // pairwise tree over any count
#pragma unroll
            for (int n = 0; n < cnt / 2; ++n) {
              t0[n] = fmaxf(t0[n], t0[n + (cnt + 1) / 2]);
              t1[n] = fmaxf(t1[n], t1[n + (cnt + 1) / 2]);
            }
          float mx0 = t0[0], mx1 = t1[0];
          mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
          mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
          mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
          mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
          const float mn0 = fmaxf(m[r_][0], mx0), mn1 = fmaxf(m[r_][1], mx1);
          // every key tile that is walked holds at least one real key, so the new maximum is finite (only the old one can
          // be -inf, on the first tile, where the factor below becomes exp2(-inf) = 0)
          const float ms0 = mn0 * sl2, ms1 = mn1 * sl2;
          const float al0 = ex2(fmaf(m[r_][0], sl2, -ms0)), al1 = ex2(fmaf(m[r_][1], sl2, -ms1));
          m[r_][0] = mn0;
          m[r_][1] = mn1;
          // One packed FMA forms s * sl2 - m * sl2 for a pair of scores (both <= 0); each gets its own f32 ex2 (the
          // packed bf16 form of ex2 issues two special-function operations as well, plus unpacking), and the pair is
          // rounded once into the bf16x2 layout of the A operand of P V.  The row sum is taken by the tensor core from
          // those same bf16 weights (a column of ones appended to V), so numerator and denominator of the softmax see
          // identical values.
          const float2 sl2v = make_float2(sl2, sl2), nm0 = make_float2(-ms0, -ms0), nm1 = make_float2(-ms1, -ms1);
          uint32_t P[NTV][2];
#pragma unroll
          for (int n = 0; n < NTV; ++n) {
            const float2 x0 = __ffma2_rn(make_float2(S[n][0], S[n][1]), sl2v, nm0);
            const float2 x1 = __ffma2_rn(make_float2(S[n][2], S[n][3]), sl2v, nm1);
            if ((MS_POLY >> (n & 7)) & 1) {
              const float2 p0 = ptx::ex2_poly2(x0), p1 = ptx::ex2_poly2(x1);
              P[n][0] = __byte_perm(__float_as_uint(p0.x), __float_as_uint(p0.y), 0x7632);
              P[n][1] = __byte_perm(__float_as_uint(p1.x), __float_as_uint(p1.y), 0x7632);
            } else {
              P[n][0] = __byte_perm(__float_as_uint(ex2(x0.x)), __float_as_uint(ex2(x0.y)), 0x7632);
              P[n][1] = __byte_perm(__float_as_uint(ex2(x1.x)), __float_as_uint(ex2(x1.y)), 0x7632);
            }
          }
          l[r_][0] *= al0;
          l[r_][2] *= al1;
#pragma unroll
          for (int n = 0; n < NTO; ++n) {
            O[r_][n][0] *= al0; O[r_][n][1] *= al0;
            O[r_][n][2] *= al1; O[r_][n][3] *= al1;
          }
          // ---- O += P V and l += P 1, the weights being the A operand ----
#pragma unroll
          for (int kk = 0; kk < NTV / 2; ++kk) {
            const uint32_t a0 = P[2 * kk][0], a1 = P[2 * kk][1], a2 = P[2 * kk + 1][0], a3 = P[2 * kk + 1][1];
            mma_k16(l[r_], a0, a1, a2, a3, 0x3F803F80u, 0x3F803F80u);  // B = ones: every column of the result is the row sum
            if constexpr (HD == 8) {
              if constexpr (!HOIST) { if ((kk & 1) == 0) load_v8(kk / 2); }
              mma_k16(O[r_][0], a0, a1, a2, a3, VF[kk][0][0], VF[kk][0][1]);
            } else {
#pragma unroll
              for (int np = 0; np < NTO / 2; ++np) {
                if constexpr (!HOIST) load_v_pair(kk, np);
                mma_k16(O[r_][2 * np], a0, a1, a2, a3, VF[kk][2 * np][0], VF[kk][2 * np][1]);
                mma_k16(O[r_][2 * np + 1], a0, a1, a2, a3, VF[kk][2 * np + 1][0], VF[kk][2 * np + 1][1]);
              }
            }
          }
        }  // slabs
      }    // steps
    };

    for (int i = 0; i < T; ++i) {
      const int st = i % STAGES;
      if (tid == 0) {
        // request further key tiles whose stage every warp has released; never block unless tile i itself is missing
        while (next_issue < T) {
          const uint32_t eb = bar_empty + 8 * (next_issue % STAGES);
          const uint32_t par = ((next_issue / STAGES) - 1) & 1;
          if (next_issue <= i) mbar_wait(g, eb, par);
          else if (!mbar_test(eb, par)) break;
          issue(next_issue);
          ++next_issue;
        }
      }
      __syncwarp();
      mbar_wait(g, bar_full + 8 * st, (i / STAGES) & 1);
      int krem, yrow;
      locate(i, krem, yrow);
      const uint32_t sKs = sK + st * C::KV_BYTES, sVs = sV + st * C::KV_BYTES;
      if (krem >= KT) {
        process(BoolTag<false>{}, IntTag<NT>{}, sKs, sVs, KT);
      } else if constexpr (KT == KSTEP && NT == 8) {  // as many 16-key groups as hold real keys
        if (krem <= 16) process(BoolTag<true>{}, IntTag<2>{}, sKs, sVs, krem);
        else if (krem <= 32) process(BoolTag<true>{}, IntTag<4>{}, sKs, sVs, krem);
        else if (krem <= 48) process(BoolTag<true>{}, IntTag<6>{}, sKs, sVs, krem);
        else process(BoolTag<true>{}, IntTag<8>{}, sKs, sVs, krem);
      } else {
        process(BoolTag<true>{}, IntTag<NT>{}, sKs, sVs, krem);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_empty + 8 * st);  // this warp is done with the stage
    }

    // ---- normalise and stage the tile in shared memory.  A warp overwrites only the Q bytes it alone read. ----
#pragma unroll
    for (int r_ = 0; r_ < R; ++r_) {
      const int row0 = (sg * R + r_) * 16;
      if (row0 >= q_real) continue;
      const float l0 = l[r_][0], l1 = l[r_][2];
      const float inv0 = l0 > 0.f ? 1.f / l0 : 0.f, inv1 = l1 > 0.f ? 1.f / l1 : 0.f;
      const int rowA = row0 + (lane >> 2), rowB = rowA + 8;
#pragma unroll
      for (int n = 0; n < NTO; ++n) {
        const int colb = (head_in_slice * HD + n * 8 + (lane & 3) * 2) * 2;  // byte column in the tile row
        const uint32_t vA = pack_bf16(O[r_][n][0] * inv0, O[r_][n][1] * inv0);
        const uint32_t vB = pack_bf16(O[r_][n][2] * inv1, O[r_][n][3] * inv1);
        asm volatile("st.shared.b32 [%0], %1;" ::"r"(sQ + swz<SWZ>(rowA * PITCH + colb)), "r"(vA) : "memory");
        asm volatile("st.shared.b32 [%0], %1;" ::"r"(sQ + swz<SWZ>(rowB * PITCH + colb)), "r"(vB) : "memory");
      }
      if (lse != nullptr && (lane & 3) == 0) {
        const int head = cs * G + head_in_slice;
        float* lp = lse + ((int64_t)b * g.heads + head) * g.L + g.seg_off[s] + q0;
        const float ln2 = 0.6931471805599453f;
        if (rowA < q_real) lp[rowA] = l0 > 0.f ? (m[r_][0] * sl2 + log2f(l0)) * ln2 : -INFINITY;
        if (rowB < q_real) lp[rowB] = l1 > 0.f ? (m[r_][1] * sl2 + log2f(l1)) * ln2 : -INFINITY;
      }
    }
    __syncthreads();
  }  // T > 0

  // ---- coalesced 16-byte stores; padded rows are written as +0, rows of the next segment are left alone ----
  for (int idx = tid; idx < rows_in_tile * CPR; idx += NTHREADS) {
    const int row = idx / CPR, ch = idx % CPR;
    uint32_t v0 = 0, v1 = 0, v2 = 0, v3 = 0;
    if (row < q_real)
      asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];"
                   : "=r"(v0), "=r"(v1), "=r"(v2), "=r"(v3) : "r"(sQ + swz<SWZ>(row * PITCH + ch * 16)) : "memory");
    uint4* dst = reinterpret_cast<uint4*>(out + (grow0 + row) * g.d + xcol + ch * 8);
    *dst = make_uint4(v0, v1, v2, v3);
  }
  if (lse != nullptr) {
    const int npad = rows_in_tile - q_real;
    for (int idx = tid; idx < npad * G; idx += NTHREADS) {
      const int row = q_real + idx / G, head = cs * G + idx % G;
      lse[((int64_t)b * g.heads + head) * g.L + g.seg_off[s] + q0 + row] = -INFINITY;
    }
  }
}

}  // namespace
}  // namespace gsit
