// The fused halves of the IM encoder layer at d_model 128 (the intra-modal encoder on the feature concat of the two
// ring encoders) on tcgen05 / TMEM.  Same structure as fused_layer_tc.cu (one CTA per SM, 128-row tiles, two threads per
// row for LayerNorm and epilogues -- warps w and w + 4 own the same TMEM lanes and half of the columns each --, operands
// in the 128-byte swizzle); what differs is the budget: rows are two k-blocks of
// 64 features wide, the 384 QKV columns need two MMA groups (N 256 + N 128), and the MLP weights (2 x 128 KB at
// d_ff 512) no longer fit in shared memory, so W_1 / W_2 stream through a two-stage TMA ring in chunks of 64 hidden
// units while the hidden accumulator is double-buffered in TMEM.
#include "fused_tc_common.cuh"

namespace gsit {
namespace {

constexpr int D2 = 128;  // d_model

// Reads the thread's half of float row r (64 values: two boxes of a four-box swizzled float tile).
__device__ __forceinline__ void load_half_row128(uint32_t boxes, int r, float (&v)[64]) {
#pragma unroll
  for (int j = 0; j < 2; ++j)
#pragma unroll
    for (int ch = 0; ch < 8; ++ch) {
      const float4 t = ld_v4f(sw128(boxes + j * XBOX, r, ch));
      const int e = 32 * j + 4 * ch;
      v[e] = t.x; v[e + 1] = t.y; v[e + 2] = t.z; v[e + 3] = t.w;
    }
}

// ------------------------------------------------------------------------------------------------ LN1 + shared QKV
namespace qk2 {
constexpr int NQ = 3 * D2;                        // 384 output columns
constexpr int OFF_W = 0;                          // W_qkv: 2 k-blocks x 384 rows x 128 B
constexpr int OFF_X = OFF_W + 2 * NQ * 128;       // float input tile (4 boxes), refilled as soon as it is in registers
constexpr int OFF_OUT = OFF_X + 4 * XBOX;         // 3 boxes of 64 columns: the output leaves in two passes
constexpr int OFF_H = OFF_OUT;                    // normalised rows (2 k-blocks): the first two boxes, free while the MMA runs
constexpr int OFF_P = OFF_OUT + 3 * XBOX;         // gamma[128], beta[128], bias[384]
constexpr int OFF_STAT = OFF_P + (2 * D2 + NQ) * 4;  // LayerNorm statistics exchanged by the two threads of a row
constexpr int OFF_BAR = OFF_STAT + 2 * TM * 8;
constexpr int B_W = 0, B_XFULL = 8, B_XFREE = 16, B_HREADY = 24, B_ACCFULL = 32, B_ACCFREE = 40, SLOT = 48;
constexpr int SMEM = OFF_BAR + 64 + 1024;
constexpr int TMEM_COLS = 512;
static_assert(SMEM <= 227 * 1024, "shared memory budget");
}  // namespace qk2

__global__ void __launch_bounds__(T_THREADS8, 1)
ln_qkv_tc128_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX,
                    const __grid_constant__ CUtensorMap tmOut, const Geometry g, const float* __restrict__ gamma,
                    const float* __restrict__ beta, const float eps, const float* __restrict__ bias, int* const zero_word) {
  using namespace qk2;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bars = base + OFF_BAR;
  const WaitCtx wc{g.status, bars + SLOT + 4};
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  float* prm = reinterpret_cast<float*>(base_ptr + OFF_P);
  stage_vector(prm, gamma, D2, 1.f, tid, T_THREADS8);
  stage_vector(prm + D2, beta, D2, 0.f, tid, T_THREADS8);
  stage_vector(prm + 2 * D2, bias, NQ, 0.f, tid, T_THREADS8);
  if (tid == 0) {
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(bars + SLOT + 4), "r"(0u) : "memory");
    mbar_init(bars + B_W, 1);
    mbar_init(bars + B_XFULL, 1);
    mbar_init(bars + B_XFREE, 8);
    mbar_init(bars + B_HREADY, 8);
    mbar_init(bars + B_ACCFULL, 1);
    mbar_init(bars + B_ACCFREE, 8);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(bars + SLOT), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  uint32_t tmem;
  asm volatile("ld.shared.b32 %0, [%1];" : "=r"(tmem) : "r"(bars + SLOT) : "memory");
  if (warp == 0) {  // the weights do not depend on the kernel before this one
    if (elect_one()) {
      mbar_expect_tx(bars + B_W, 2 * NQ * 128);
      for (int kb = 0; kb < 2; ++kb)
        for (int j = 0; j < 3; ++j)  // boxes of 128 weight rows
          tma_load_2d(base + OFF_W + kb * NQ * 128 + j * XBOX, &tmW, 64 * kb, 128 * j, bars + B_W);
    }
    __syncwarp();
  }
  grid_dep_wait();
  grid_dep_launch();
  const int row_base = rows_begin(g), rows = rows_end(g);  // this problem's rows of the activation matrices
  const int ntiles = (rows - row_base + TM - 1) / TM;
  if (zero_word != nullptr && blockIdx.x == 0 && tid == 0) *zero_word = 0;  // work counter of the attention kernel that follows

  if (warp == 0) {
    // ================================ producer ================================
    int i = 0;
    for (int t = blockIdx.x; t < ntiles; t += gridDim.x, ++i) {
      if (i > 0) mbar_wait(wc, bars + B_XFREE, (i - 1) & 1);  // the row warps hold the previous tile in registers
      if (elect_one()) {
        mbar_expect_tx(bars + B_XFULL, 4 * XBOX);
        for (int j = 0; j < 4; ++j) tma_load_2d(base + OFF_X + j * XBOX, &tmX, 32 * j, row_base + t * TM, bars + B_XFULL);
      }
      __syncwarp();
    }
  } else if (warp == 1) {
    // ================================ MMA issuer ================================
    constexpr uint32_t IDESC_256 = idesc_bf16(256, false), IDESC_128 = idesc_bf16(128, false);
    mbar_wait(wc, bars + B_W, 0);
    int i = 0;
    for (int t = blockIdx.x; t < ntiles; t += gridDim.x, ++i) {
      mbar_wait(wc, bars + B_HREADY, i & 1);
      if (i > 0) mbar_wait(wc, bars + B_ACCFREE, (i - 1) & 1);
      tc_fence_after();
      if (elect_one()) {
#pragma unroll
        for (int kb = 0; kb < 2; ++kb)
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const uint64_t a = smem_desc_sw128(base + OFF_H + kb * XBOX + 32 * k);
            const uint32_t w = base + OFF_W + kb * NQ * 128 + 32 * k;
            umma_ss(tmem, a, smem_desc_sw128(w), IDESC_256, (kb > 0 || k > 0) ? 1u : 0u);                    // columns 0..255
            umma_ss(tmem + 256, a, smem_desc_sw128(w + 256 * 128), IDESC_128, (kb > 0 || k > 0) ? 1u : 0u);  // columns 256..383
          }
        umma_commit(bars + B_ACCFULL);
      }
      __syncwarp();
    }
  } else {
    // ================================ two threads per sequence row ================================
    const int r = ((warp & 3) << 5) + lane, hf = (warp - 2) >> 2;  // row = TMEM lane; which half of the columns
    const uint32_t tl = tmem + ((uint32_t)((warp & 3) << 5) << 16);
    const uint32_t s_gamma = base + OFF_P, s_beta = s_gamma + D2 * 4, s_bias = s_beta + D2 * 4;
    int i = 0;
    bool real = row_real32(g, row_base + (int)blockIdx.x * TM + r, rows);
    for (int t = blockIdx.x; t < ntiles; t += gridDim.x, ++i) {
      const int row0 = row_base + t * TM;
      mbar_wait(wc, bars + B_XFULL, i & 1);
      float v[64];
      if (real) {
        load_half_row128(base + OFF_X + 2 * hf * XBOX, r, v);
      } else {  // padded input rows may hold anything (NaN included): never read them
#pragma unroll
        for (int e = 0; e < 64; ++e) v[e] = 0.f;
      }
      fence_reads_before_release();
      __syncwarp();
      if (lane == 0) mbar_arrive(bars + B_XFREE);
      if (i > 0 && tid == 64) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
      // the barrier inside: the previous tile's stores have finished reading the staging rows the normalised rows overlay
      float mean, rstd;
      split_row_stats<64>(v, base + OFF_STAT, r, hf, eps, real, mean, rstd);
      normalise_to_tile<64>(v, mean, rstd, real, s_gamma, s_beta, 64 * hf, base + OFF_H + hf * XBOX, r, 0);
      fence_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(bars + B_HREADY);
      const bool real_next = row_real32(g, row_base + (t + (int)gridDim.x) * TM + r, rows);  // overlaps the MMA

      mbar_wait(wc, bars + B_ACCFULL, i & 1);  // the MMA has also finished reading the normalised rows
      tc_fence_after();
#pragma unroll 1
      for (int pass = 0; pass < 2; ++pass) {
        if (pass > 0) {  // the first pass's stores must have finished reading the staging rows
          if (tid == 64) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
          t_bar_rows8();
        }
#pragma unroll 1
        for (int c0 = 32 * hf; c0 < NQ / 2; c0 += 64) {  // alternate groups of 32 output columns
          const int col = pass * (NQ / 2) + c0;
          uint32_t a[32];
          tmem_ld32(tl + col, a);
          tmem_wait_ld();
          tmem_regs_ready(a);
          uint32_t pk[16];
#pragma unroll
          for (int e = 0; e < 32; e += 4) {
            const float4 bb = ld_v4f(s_bias + (col + e) * 4);
            const float2 h0 = __fadd2_rn(make_float2(__uint_as_float(a[e]), __uint_as_float(a[e + 1])), make_float2(bb.x, bb.y));
            const float2 h1 = __fadd2_rn(make_float2(__uint_as_float(a[e + 2]), __uint_as_float(a[e + 3])), make_float2(bb.z, bb.w));
            pk[e >> 1] = real ? pack_bf16(h0.x, h0.y) : 0u;
            pk[(e >> 1) + 1] = real ? pack_bf16(h1.x, h1.y) : 0u;
          }
          const uint32_t box = base + OFF_OUT + (c0 >> 6) * XBOX;
          const int ch0 = (c0 & 32) >> 3;
#pragma unroll
          for (int q = 0; q < 4; ++q) st_shared_v4(sw128(box, r, ch0 + q), pk[4 * q], pk[4 * q + 1], pk[4 * q + 2], pk[4 * q + 3]);
        }
        if (pass == 1) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bars + B_ACCFREE);
        }
        fence_async_smem();
        t_bar_rows8();
        if (tid == 64) {
#pragma unroll
          for (int j = 0; j < 3; ++j) tma_store_2d(&tmOut, base + OFF_OUT + j * XBOX, pass * (NQ / 2) + 64 * j, row0);
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
      }
      real = real_next;
    }
    if (tid == 64) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
  }
}

// ------------------------------------------------------------------------------------------------ out-proj + MLP
namespace pm2 {
constexpr int OFF_WO = 0;                          // W_o: 2 k-blocks x 128 rows x 128 B
constexpr int OFF_ATT = OFF_WO + 2 * XBOX;         // attention tile (2 k-blocks); LN2 output overlays it
constexpr int OFF_X = OFF_ATT + 2 * XBOX;          // float residual input tile (4 boxes)
constexpr int WC_STAGE = 2 * 64 * 128 + XBOX;      // W_1 chunk: 2 k-blocks x 64 rows; W_2 chunk: 128 rows x 128 B
constexpr int OFF_WC = OFF_X + 4 * XBOX;           // 2 stages
constexpr int OFF_F = OFF_WC + 2 * WC_STAGE;       // hidden chunk: 128 rows x 64 units, bf16
constexpr int OFF_P = OFF_F + XBOX;                // b_o[128], gamma[128], beta[128], b_2[128], b_1[512]
constexpr int OFF_STAT = OFF_P + (4 * D2 + 512) * 4;  // LayerNorm statistics exchanged by the two threads of a row
constexpr int OFF_BAR = OFF_STAT + 2 * TM * 8;
constexpr int B_WO = 0, B_ATTFULL = 8, B_ATTFREE = 16, B_XFULL = 24, B_XFREE = 32, B_ACC1 = 40, B_HREADY = 48,
              B_W1FULL = 56, B_W1FREE = 72, B_ACCF = 88, B_FREADY = 104, B_FFREE = 112, B_ACCY = 120, B_W2FULL = 128,
              B_W2FREE = 144, SLOT = 160;
constexpr int SMEM = OFF_BAR + 176 + 1024;
constexpr int COL_1 = 0, COL_F = 128, COL_Y = 256, TMEM_COLS = 512;
static_assert(SMEM <= 227 * 1024, "shared memory budget");
}  // namespace pm2

__global__ void __launch_bounds__(T_THREADS8, 1)
proj_mlp_tc128_kernel(const __grid_constant__ CUtensorMap tmAtt, const __grid_constant__ CUtensorMap tmX,
                      const __grid_constant__ CUtensorMap tmWo, const __grid_constant__ CUtensorMap tmW1,
                      const __grid_constant__ CUtensorMap tmW2, const Geometry g, const float* __restrict__ bo,
                      const float* __restrict__ gamma, const float* __restrict__ beta, const float eps,
                      const float* __restrict__ b1, const float* __restrict__ b2, const int d_ff, float* __restrict__ y,
                      const int64_t ldy) {
  using namespace pm2;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bars = base + OFF_BAR;
  const WaitCtx wc{g.status, bars + SLOT + 4};
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nc = d_ff / 64;  // chunks of 64 hidden units

  float* prm = reinterpret_cast<float*>(base_ptr + OFF_P);
  stage_vector(prm, bo, D2, 0.f, tid, T_THREADS8);
  stage_vector(prm + D2, gamma, D2, 1.f, tid, T_THREADS8);
  stage_vector(prm + 2 * D2, beta, D2, 0.f, tid, T_THREADS8);
  stage_vector(prm + 3 * D2, b2, D2, 0.f, tid, T_THREADS8);
  stage_vector(prm + 4 * D2, b1, d_ff, 0.f, tid, T_THREADS8);
  if (tid == 0) {
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(bars + SLOT + 4), "r"(0u) : "memory");
    mbar_init(bars + B_WO, 1);
    mbar_init(bars + B_ATTFULL, 1);
    mbar_init(bars + B_ATTFREE, 1);
    mbar_init(bars + B_XFULL, 1);
    mbar_init(bars + B_XFREE, 8);
    mbar_init(bars + B_ACC1, 1);
    mbar_init(bars + B_HREADY, 8);
    for (int i = 0; i < 2; ++i) {
      mbar_init(bars + B_W1FULL + 8 * i, 1);
      mbar_init(bars + B_W1FREE + 8 * i, 1);
      mbar_init(bars + B_W2FULL + 8 * i, 1);
      mbar_init(bars + B_W2FREE + 8 * i, 1);
      mbar_init(bars + B_ACCF + 8 * i, 1);
    }
    mbar_init(bars + B_FREADY, 8);
    mbar_init(bars + B_FFREE, 1);
    mbar_init(bars + B_ACCY, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(bars + SLOT), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  uint32_t tmem;
  asm volatile("ld.shared.b32 %0, [%1];" : "=r"(tmem) : "r"(bars + SLOT) : "memory");
  if (warp == 0) {  // the weights do not depend on the kernel before this one
    if (elect_one()) {
      mbar_expect_tx(bars + B_WO, 2 * XBOX);
      for (int kb = 0; kb < 2; ++kb) tma_load_2d(base + OFF_WO + kb * XBOX, &tmWo, 64 * kb, 0, bars + B_WO);
    }
    __syncwarp();
  }
  grid_dep_wait();
  grid_dep_launch();
  const int row_base = rows_begin(g), rows = rows_end(g);  // this problem's rows of the activation matrices
  const int ntiles = (rows - row_base + TM - 1) / TM;

  if (warp == 0) {
    // ================================ producer ================================
    // The two halves of a weight chunk have their own rings: the W_1 half of a stage is free once the chunk's first product
    // has completed, the W_2 half only after its second product, two hand-overs later.  Requests are made in the order in
    // which their stages come free -- W_1(n), then W_2(n - 1) -- so that no wait holds back a load that could already go.
    int i = 0, n = 0;  // tiles, weight chunks whose W_1 half has been requested
    auto request_w1 = [&](int m) {
      const int st = m & 1, use = m >> 1, c = m % nc;
      if (use > 0) mbar_wait(wc, bars + B_W1FREE + 8 * st, (use - 1) & 1);
      if (elect_one()) {
        const uint32_t dst = base + OFF_WC + st * WC_STAGE;
        mbar_expect_tx(bars + B_W1FULL + 8 * st, 2 * 64 * 128);
        tma_load_2d(dst, &tmW1, 0, 64 * c, bars + B_W1FULL + 8 * st);              // W_1[64c .. 64c+63, 0..63]
        tma_load_2d(dst + 64 * 128, &tmW1, 64, 64 * c, bars + B_W1FULL + 8 * st);  // W_1[64c .. 64c+63, 64..127]
      }
      __syncwarp();
    };
    auto request_w2 = [&](int m) {
      const int st = m & 1, use = m >> 1, c = m % nc;
      if (use > 0) mbar_wait(wc, bars + B_W2FREE + 8 * st, (use - 1) & 1);
      if (elect_one()) {
        const uint32_t dst = base + OFF_WC + st * WC_STAGE + 2 * 64 * 128;
        mbar_expect_tx(bars + B_W2FULL + 8 * st, XBOX);
        tma_load_2d(dst, &tmW2, 64 * c, 0, bars + B_W2FULL + 8 * st);              // W_2[0..127, 64c .. 64c+63]
      }
      __syncwarp();
    };
    for (int t = blockIdx.x; t < ntiles; t += gridDim.x, ++i) {
      const int row0 = row_base + t * TM;
      for (int c = 0; c < nc; ++c, ++n) {
        request_w1(n);
        if (n > 0) request_w2(n - 1);
        if (c == 0) {
          // the attention buffer also holds the LN2 rows of the previous tile until its last first-MLP product is done
          if (i > 0) mbar_wait(wc, bars + B_ATTFREE, (i - 1) & 1);
          if (elect_one()) {
            mbar_expect_tx(bars + B_ATTFULL, 2 * XBOX);
            for (int kb = 0; kb < 2; ++kb) tma_load_2d(base + OFF_ATT + kb * XBOX, &tmAtt, 64 * kb, row0, bars + B_ATTFULL);
          }
          __syncwarp();
          if (i > 0) mbar_wait(wc, bars + B_XFREE, (i - 1) & 1);
          if (elect_one()) {
            mbar_expect_tx(bars + B_XFULL, 4 * XBOX);
            for (int j = 0; j < 4; ++j) tma_load_2d(base + OFF_X + j * XBOX, &tmX, 32 * j, row0, bars + B_XFULL);
          }
          __syncwarp();
        }
      }
    }
    if (n > 0) request_w2(n - 1);
  } else if (warp == 1) {
    // ================================ MMA issuer ================================
    constexpr uint32_t IDESC_128 = idesc_bf16(128, false), IDESC_64 = idesc_bf16(64, false);
    mbar_wait(wc, bars + B_WO, 0);
    int i = 0, n = 0;  // tiles done, chunks whose first product has been issued
    for (int t = blockIdx.x; t < ntiles; t += gridDim.x, ++i) {
      // y1 accumulator = att W_o^T
      mbar_wait(wc, bars + B_ATTFULL, i & 1);
      tc_fence_after();
      if (elect_one()) {
#pragma unroll
        for (int kb = 0; kb < 2; ++kb)
#pragma unroll
          for (int k = 0; k < 4; ++k)
            umma_ss(tmem + COL_1, smem_desc_sw128(base + OFF_ATT + kb * XBOX + 32 * k), smem_desc_sw128(base + OFF_WO + kb * XBOX + 32 * k),
                   IDESC_128, (kb > 0 || k > 0) ? 1u : 0u);
        umma_commit(bars + B_ACC1);
      }
      __syncwarp();
      mbar_wait(wc, bars + B_HREADY, i & 1);
      // first product of chunk m (global index): hidden accumulator (m & 1) = LN2(y1) W_1c^T
      auto first = [&](int m, bool last_of_tile) {
        const int st = m & 1;
        mbar_wait(wc, bars + B_W1FULL + 8 * st, (m >> 1) & 1);
        tc_fence_after();
        if (elect_one()) {
          const uint32_t w1 = base + OFF_WC + st * WC_STAGE;
#pragma unroll
          for (int kb = 0; kb < 2; ++kb)
#pragma unroll
            for (int k = 0; k < 4; ++k)
              umma_ss(tmem + COL_F + 64 * st, smem_desc_sw128(base + OFF_ATT + kb * XBOX + 32 * k), smem_desc_sw128(w1 + kb * 64 * 128 + 32 * k),
                     IDESC_64, (kb > 0 || k > 0) ? 1u : 0u);
          umma_commit(bars + B_ACCF + 8 * st);
          umma_commit(bars + B_W1FREE + 8 * st);
          if (last_of_tile) umma_commit(bars + B_ATTFREE);  // LN2 rows no longer needed: the next attention tile may land
        }
        __syncwarp();
      };
      // second product of chunk m: accY += relu-hidden(m) W_2c^T
      auto second = [&](int m, bool first_of_tile, bool last_of_tile) {
        mbar_wait(wc, bars + B_FREADY, m & 1);
        mbar_wait(wc, bars + B_W2FULL + 8 * (m & 1), (m >> 1) & 1);
        tc_fence_after();
        if (elect_one()) {
          const uint32_t w2 = base + OFF_WC + (m & 1) * WC_STAGE + 2 * 64 * 128;
#pragma unroll
          for (int k = 0; k < 4; ++k)
            umma_ss(tmem + COL_Y, smem_desc_sw128(base + OFF_F + 32 * k), smem_desc_sw128(w2 + 32 * k), IDESC_128, (!first_of_tile || k > 0) ? 1u : 0u);
          umma_commit(bars + B_W2FREE + 8 * (m & 1));
          umma_commit(bars + B_FFREE);
          if (last_of_tile) umma_commit(bars + B_ACCY);
        }
        __syncwarp();
      };
      // The second product of chunk c sits on the critical chain (hidden buffer free -> next ReLU rows -> next second
      // product); the first product of chunk c + 2 only has to be ready by the time the row warps come back for it.  So
      // the first products run two chunks ahead and each is issued right behind a second product.
      first(n, nc == 1);
      if (nc > 1) first(n + 1, nc == 2);
      for (int c = 0; c < nc; ++c) {
        second(n + c, c == 0, c + 1 == nc);  // (its wait covers the rows' reads of hidden accumulator c & 1)
        if (c + 2 < nc) first(n + c + 2, c + 3 == nc);
      }
      n += nc;
    }
  } else {
    // ================================ two threads per sequence row ================================
    const int r = ((warp & 3) << 5) + lane, hf = (warp - 2) >> 2;  // row = TMEM lane; which half of the columns
    const uint32_t tl = tmem + ((uint32_t)((warp & 3) << 5) << 16);
    const uint32_t s_bo = base + OFF_P, s_gamma = s_bo + D2 * 4, s_beta = s_gamma + D2 * 4, s_b2 = s_beta + D2 * 4,
                   s_b1 = s_b2 + D2 * 4;
    int i = 0, n = 0;
    bool real = row_real32(g, row_base + (int)blockIdx.x * TM + r, rows);
    for (int t = blockIdx.x; t < ntiles; t += gridDim.x, ++i) {
      const int row0 = row_base + t * TM;
      // ---- y1 = x + att W_o^T + b_o (this thread's 64 columns, in registers) ----
      mbar_wait(wc, bars + B_XFULL, i & 1);
      float v[64];
      if (real) {
        load_half_row128(base + OFF_X + 2 * hf * XBOX, r, v);
      } else {
#pragma unroll
        for (int e = 0; e < 64; ++e) v[e] = 0.f;
      }
      fence_reads_before_release();
      __syncwarp();
      if (lane == 0) mbar_arrive(bars + B_XFREE);
      mbar_wait(wc, bars + B_ACC1, i & 1);
      tc_fence_after();
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t a[32];
        tmem_ld32(tl + COL_1 + 64 * hf + 32 * c, a);
        tmem_wait_ld();
        tmem_regs_ready(a);
#pragma unroll
        for (int e = 0; e < 32; e += 4) {
          const float4 bb = ld_v4f(s_bo + (64 * hf + 32 * c + e) * 4);
          v[32 * c + e] += __uint_as_float(a[e]) + bb.x;
          v[32 * c + e + 1] += __uint_as_float(a[e + 1]) + bb.y;
          v[32 * c + e + 2] += __uint_as_float(a[e + 2]) + bb.z;
          v[32 * c + e + 3] += __uint_as_float(a[e + 3]) + bb.w;
        }
      }
      // ---- h = LN2(y1) over the attention tile (its product has completed); this thread's columns are k-block hf ----
      float mean, rstd;
      split_row_stats<64>(v, base + OFF_STAT, r, hf, eps, real, mean, rstd);
      normalise_to_tile<64>(v, mean, rstd, real, s_gamma, s_beta, 64 * hf, base + OFF_ATT + hf * XBOX, r, 0);
      fence_async_smem();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bars + B_HREADY);
      const bool real_next = row_real32(g, row_base + (t + (int)gridDim.x) * TM + r, rows);
      // ---- hidden chunks: f = relu(h W_1c^T + b_1c) -> A operand of the second product (32 of the 64 units each) ----
#pragma unroll 1
      for (int c = 0; c < nc; ++c, ++n) {
        mbar_wait(wc, bars + B_ACCF + 8 * (n & 1), (n >> 1) & 1);
        tc_fence_after();
        uint32_t pk[16];
        {
          uint32_t a[32];
          tmem_ld32(tl + COL_F + 64 * (n & 1) + 32 * hf, a);
          tmem_wait_ld();
          tmem_regs_ready(a);
#pragma unroll
          for (int e = 0; e < 32; e += 4) {
            const float4 bb = ld_v4f(s_b1 + (64 * c + 32 * hf + e) * 4);
            const float2 h0 = __fadd2_rn(make_float2(__uint_as_float(a[e]), __uint_as_float(a[e + 1])), make_float2(bb.x, bb.y));
            const float2 h1 = __fadd2_rn(make_float2(__uint_as_float(a[e + 2]), __uint_as_float(a[e + 3])), make_float2(bb.z, bb.w));
            pk[e >> 1] = pack_bf16_relu(h0.x, h0.y);
            pk[(e >> 1) + 1] = pack_bf16_relu(h1.x, h1.y);
          }
        }
        if (n > 0) mbar_wait(wc, bars + B_FFREE, (n - 1) & 1);  // the previous second product has read the hidden chunk
#pragma unroll
        for (int q = 0; q < 4; ++q) st_shared_v4(sw128(base + OFF_F, r, 4 * hf + q), pk[4 * q], pk[4 * q + 1], pk[4 * q + 2], pk[4 * q + 3]);
        fence_async_smem();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bars + B_FREADY);
      }
      // ---- y = y1 + f W_2^T + b_2; padded rows +0 ----
      mbar_wait(wc, bars + B_ACCY, i & 1);
      tc_fence_after();
      // The rows leave through a per-warp transpose in shared memory (2 KB of the hidden-chunk buffer per warp, which
      // nothing reads between the last second product and the next tile's first chunk): a thread owns a row, but a store
      // instruction that writes 16 bytes to each of 32 rows touches half of 32 sectors, so 16 columns at a time are
      // written swizzled and read back with four lanes per row -- each store then covers 8 rows x 64 contiguous bytes.
      const uint32_t scr = base + OFF_F + (uint32_t)(warp - 2) * 2048u;
      const int jj = lane & 3, rr0 = lane >> 2;
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t a[32];
        tmem_ld32(tl + COL_Y + 64 * hf + 32 * c, a);
        tmem_wait_ld();
        tmem_regs_ready(a);
#pragma unroll
        for (int sub = 0; sub < 2; ++sub) {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int e = 16 * sub + 4 * q, ve = 32 * c + e;
            const float4 bb = ld_v4f(s_b2 + (64 * hf + ve) * 4);
            float4 o = make_float4(v[ve] + __uint_as_float(a[e]) + bb.x, v[ve + 1] + __uint_as_float(a[e + 1]) + bb.y,
                                   v[ve + 2] + __uint_as_float(a[e + 2]) + bb.z, v[ve + 3] + __uint_as_float(a[e + 3]) + bb.w);
            if (!real) o = make_float4(0.f, 0.f, 0.f, 0.f);
            st_shared_v4(scr + lane * 64 + ((q ^ ((lane >> 1) & 3)) << 4), __float_as_uint(o.x), __float_as_uint(o.y), __float_as_uint(o.z),
                         __float_as_uint(o.w));
          }
          __syncwarp();
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const int rr = 8 * k + rr0;
            const float4 o = ld_v4f(scr + rr * 64 + ((jj ^ ((rr >> 1) & 3)) << 4));
            const int grow = row0 + ((warp & 3) << 5) + rr;
            if (grow < rows) *reinterpret_cast<float4*>(y + (int64_t)grow * ldy + 64 * hf + 32 * c + 16 * sub + 4 * jj) = o;
          }
          __syncwarp();
        }
      }
      tc_fence_before();  // orders these TMEM reads before the next tile's products (which wait for this thread's arrivals)
      real = real_next;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
  }
}

}  // namespace

bool fused_layer_tc128_supported(const Geometry& g, int d_ff) { return g.d == D2 && d_ff >= 64 && d_ff <= 512 && d_ff % 64 == 0; }

cudaError_t launch_ln_qkv_tc128(const Geometry& g, const float* x, int64_t ldx, const float* gamma, const float* beta, float eps,
                                const __nv_bfloat16* w_qkv, const float* b_qkv, __nv_bfloat16* qkv, int* zero_word, cudaStream_t st) {
  if (g.d != D2) return cudaErrorNotSupported;
  const int64_t rows = matrix_rows(g);  // bounds of the tensor maps; the kernel takes its own row range from the geometry
  const int ntiles = (int)((rows + TM - 1) / TM), nsm = t_sm_count();
  if (nsm == 0) return cudaErrorUnknown;
  alignas(64) CUtensorMap tmW, tmX, tmOut;
  if (!make_map(&tmW, w_qkv, 3 * D2, D2, D2, 64, 128) || !make_map_f32(&tmX, x, rows, D2, ldx, TM) ||
      !make_map(&tmOut, qkv, rows, 3 * D2, 3 * D2, 64, TM))
    return cudaErrorInvalidValue;
  {
    cudaError_t e = sm_count_and_smem_once(reinterpret_cast<const void*>(ln_qkv_tc128_kernel), qk2::SMEM, nullptr);
    if (e != cudaSuccess) return e;
  }
  return launch_overlapped(ln_qkv_tc128_kernel, dim3(min(ntiles, nsm)), dim3(T_THREADS8), qk2::SMEM, st, tmW, tmX, tmOut, g, gamma, beta,
                           eps, b_qkv, zero_word);
}

cudaError_t launch_proj_mlp_tc128(const Geometry& g, const __nv_bfloat16* att, const float* x, int64_t ldx,
                                  const __nv_bfloat16* w_o, const float* b_o, const float* gamma, const float* beta, float eps,
                                  const __nv_bfloat16* w_1, const float* b_1, const __nv_bfloat16* w_2, const float* b_2, int d_ff,
                                  float* y, int64_t ldy, cudaStream_t st) {
  if (!fused_layer_tc128_supported(g, d_ff)) return cudaErrorNotSupported;
  const int64_t rows = matrix_rows(g);  // bounds of the tensor maps; the kernel takes its own row range from the geometry
  const int ntiles = (int)((rows + TM - 1) / TM), nsm = t_sm_count();
  if (nsm == 0) return cudaErrorUnknown;
  alignas(64) CUtensorMap tmAtt, tmX, tmWo, tmW1, tmW2;
  if (!make_map(&tmAtt, att, rows, D2, D2, 64, TM) || !make_map_f32(&tmX, x, rows, D2, ldx, TM) ||
      !make_map(&tmWo, w_o, D2, D2, D2, 64, D2) || !make_map(&tmW1, w_1, d_ff, D2, D2, 64, 64) ||
      !make_map(&tmW2, w_2, D2, d_ff, d_ff, 64, D2))
    return cudaErrorInvalidValue;
  {
    cudaError_t e = sm_count_and_smem_once(reinterpret_cast<const void*>(proj_mlp_tc128_kernel), pm2::SMEM, nullptr);
    if (e != cudaSuccess) return e;
  }
  return launch_overlapped(proj_mlp_tc128_kernel, dim3(min(ntiles, nsm)), dim3(T_THREADS8), pm2::SMEM, st, tmAtt, tmX, tmWo, tmW1, tmW2,
                           g, b_o, gamma, beta, eps, b_1, b_2, d_ff, y, ldy);
}

}  // namespace gsit
