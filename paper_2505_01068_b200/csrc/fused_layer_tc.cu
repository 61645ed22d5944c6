// The two fused halves of the IM encoder layer at d_model 64 on the 5th-generation tensor cores (tcgen05 / TMEM):
//
//   ln_qkv_tc_kernel     qkv = LN1(x) W_qkv^T + b_qkv          (the shared projection of the concatenated sequence)
//   proj_mlp_tc_kernel   y1 = x + att W_o^T + b_o ;  y = y1 + relu(LN2(y1) W_1^T + b_1) W_2^T + b_2   (d_ff <= 256)
//
// Persistent (the first half two CTAs per SM, the second one), tiles of 128 sequence rows:
//   warp 0      producer: weights once (TMA, 128-byte swizzle, resident for the whole kernel), then per tile the x rows
//               (TMA, two boxes of 32 floats) and the attention tile (TMA)
//   warp 1      owns the TMEM columns and issues every tcgen05.mma (M 128, K 16, operands from shared memory)
//   row warps   thread = sequence row = TMEM lane.  LayerNorm needs no shuffles.  Rows are written back to shared memory
//               as bf16 in the 128-byte swizzle the MMA expects (the A operand of the next product), so the normalised
//               rows, the float residual y1 (registers) and the 256 hidden units per row never leave the SM.  Outputs
//               leave through swizzled staging rows and TMA stores.
//               First half: four row warps, a thread holds its whole row.  Second half: eight row warps, two threads per
//               row -- warps w and w + 4 own the same 32 lanes and half of the columns each (of the input row, and
//               alternate groups of 32 accumulator columns); the pair exchanges a mean and a centred sum of squares
//               through shared memory for LN2.
// Every wait is bounded (GSIT_DEVFLAG_TIMEOUT instead of a hang) and TMEM is always released.
#include "fused_tc_common.cuh"

namespace gsit {
namespace {

constexpr int TD = 64;            // d_model

// Reads the thread's half of float row r (32 values: one box of a two-box swizzled float tile).
__device__ __forceinline__ void load_half_row(uint32_t box, int r, float (&v)[32]) {
#pragma unroll
  for (int ch = 0; ch < 8; ++ch) {
    const float4 t = ld_v4f(sw128(box, r, ch));
    v[4 * ch] = t.x; v[4 * ch + 1] = t.y; v[4 * ch + 2] = t.z; v[4 * ch + 3] = t.w;
  }
}

// Reads the thread's float row r (64 values) from a two-box swizzled float tile.
__device__ __forceinline__ void load_row64(uint32_t tile, int r, float (&v)[TD]) {
#pragma unroll
  for (int j = 0; j < 2; ++j)
#pragma unroll
    for (int ch = 0; ch < 8; ++ch) {
      const float4 t = ld_v4f(sw128(tile + j * XBOX, r, ch));
      const int e = 32 * j + 4 * ch;
      v[e] = t.x; v[e + 1] = t.y; v[e + 2] = t.z; v[e + 3] = t.w;
    }
}
// LayerNorm of one row held by one thread -> bf16 row r of a swizzled 128-byte-row tile (zeros when !real).
__device__ __forceinline__ void layernorm_row_to_tile(const float (&v)[TD], bool real, uint32_t s_gamma, uint32_t s_beta,
                                                      float eps, uint32_t tile, int r) {
  float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
  for (int e = 0; e < TD; e += 4) { s0 += v[e]; s1 += v[e + 1]; s2 += v[e + 2]; s3 += v[e + 3]; }
  const float mean = ((s0 + s1) + (s2 + s3)) * (1.f / TD);
  float q0 = 0.f, q1 = 0.f, q2 = 0.f, q3 = 0.f;
#pragma unroll
  for (int e = 0; e < TD; e += 4) {
    const float a = v[e] - mean, b = v[e + 1] - mean, c = v[e + 2] - mean, d = v[e + 3] - mean;
    q0 = fmaf(a, a, q0); q1 = fmaf(b, b, q1); q2 = fmaf(c, c, q2); q3 = fmaf(d, d, q3);
  }
  const float rstd = real ? rsqrtf(((q0 + q1) + (q2 + q3)) * (1.f / TD) + eps) : 0.f;
#pragma unroll
  for (int ch = 0; ch < 8; ++ch) {
    const float4 g0 = ld_v4f(s_gamma + ch * 32), g1 = ld_v4f(s_gamma + ch * 32 + 16);
    const float4 b0 = ld_v4f(s_beta + ch * 32), b1 = ld_v4f(s_beta + ch * 32 + 16);
    const float gm[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
    const float bt[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
    uint32_t pk[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int e = ch * 8 + 2 * k;
      float a = fmaf((v[e] - mean) * rstd, gm[2 * k], bt[2 * k]), b = fmaf((v[e + 1] - mean) * rstd, gm[2 * k + 1], bt[2 * k + 1]);
      if (!real) { a = 0.f; b = 0.f; }
      pk[k] = pack_bf16(a, b);
    }
    st_shared_v4(sw128(tile, r, ch), pk[0], pk[1], pk[2], pk[3]);
  }
}

// ------------------------------------------------------------------------------------------------ LN1 + shared QKV
namespace qk {
constexpr int NQ = 3 * TD;                       // 192 output columns
constexpr int OFF_W = 0;                         // W_qkv: 192 rows x 128 B, swizzled
constexpr int OFF_OUT = OFF_W + NQ * 128;        // 3 boxes of 64 columns x 128 rows
constexpr int OFF_H = OFF_OUT;                   // normalised rows (A operand): the first box, free while the MMA runs
constexpr int OFF_X = OFF_OUT + 3 * TM * 128;    // one float input tile (2 boxes), refilled as soon as it is in registers
constexpr int OFF_P = OFF_X + 2 * XBOX;          // gamma[64], beta[64], bias[192] as floats
constexpr int OFF_BAR = OFF_P + (2 * TD + NQ) * 4;
constexpr int B_W = 0, B_XFULL = 8, B_XFREE = 24, B_HREADY = 40, B_ACCFULL = 48, B_ACCFREE = 56, SLOT = 64;
constexpr int SMEM = OFF_BAR + 80 + 1024;
constexpr int TMEM_COLS = 256;
static_assert(2 * (SMEM + 1024) <= 227 * 1024, "two CTAs per SM");
}  // namespace qk

// Per-problem arguments of the LN1 + QKV kernel.  One launch can serve two problems of the same geometry (the forward-
// ring and the backward-ring encoder layers of the same depth, Eq. "All-Modal-In-One fusion": they share nothing but
// their shape): CTAs with an even index take the first, odd ones the second, each with its own weights resident.
struct LnQkvArgs {
  CUtensorMap tmW, tmX, tmOut;
  const float *gamma, *beta, *bias;
};

__global__ void __launch_bounds__(T_THREADS, 2)
ln_qkv_tc_kernel(const __grid_constant__ LnQkvArgs arg0, const __grid_constant__ LnQkvArgs arg1, const Geometry g,
                 const float eps, const int problems, int* const zero_word) {
  using namespace qk;
  const int which = (problems == 2) ? (int)(blockIdx.x & 1u) : 0;
  const int cta = (problems == 2) ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;       // index among the CTAs of this problem
  const int ctas = (problems == 2) ? (int)((gridDim.x + 1 - which) >> 1) : (int)gridDim.x;
  const LnQkvArgs& arg = which ? arg1 : arg0;
  const CUtensorMap &tmW = arg.tmW, &tmX = arg.tmX, &tmOut = arg.tmOut;
  const float *gamma = arg.gamma, *beta = arg.beta, *bias = arg.bias;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bars = base + OFF_BAR;
  const WaitCtx wc{g.status, bars + SLOT + 4};
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  float* prm = reinterpret_cast<float*>(base_ptr + OFF_P);
  stage_vector(prm, gamma, TD, 1.f, tid, T_THREADS);
  stage_vector(prm + TD, beta, TD, 0.f, tid, T_THREADS);
  stage_vector(prm + 2 * TD, bias, NQ, 0.f, tid, T_THREADS);
  if (tid == 0) {
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(bars + SLOT + 4), "r"(0u) : "memory");
    mbar_init(bars + B_W, 1);
    mbar_init(bars + B_XFULL, 1);
    mbar_init(bars + B_XFREE, 4);
    mbar_init(bars + B_HREADY, 4);
    mbar_init(bars + B_ACCFULL, 1);
    mbar_init(bars + B_ACCFREE, 4);
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
      mbar_expect_tx(bars + B_W, NQ * 128);
      tma_load_2d(base + OFF_W, &tmW, 0, 0, bars + B_W);
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
    for (int t = cta; t < ntiles; t += ctas, ++i) {
      if (i >= 1) mbar_wait(wc, bars + B_XFREE, (i - 1) & 1);  // the row warps hold the previous tile in registers
      if (elect_one()) {
        mbar_expect_tx(bars + B_XFULL, 2 * XBOX);
        tma_load_2d(base + OFF_X, &tmX, 0, row_base + t * TM, bars + B_XFULL);
        tma_load_2d(base + OFF_X + XBOX, &tmX, 32, row_base + t * TM, bars + B_XFULL);
      }
      __syncwarp();
    }
  } else if (warp == 1) {
    // ================================ MMA issuer ================================
    constexpr uint32_t IDESC = idesc_bf16(NQ, false);
    mbar_wait(wc, bars + B_W, 0);
    int i = 0;
    for (int t = cta; t < ntiles; t += ctas, ++i) {
      mbar_wait(wc, bars + B_HREADY, i & 1);
      if (i > 0) mbar_wait(wc, bars + B_ACCFREE, (i - 1) & 1);
      tc_fence_after();
      if (elect_one()) {
#pragma unroll
        for (int k = 0; k < TD / 16; ++k)
          umma_ss(tmem, smem_desc_sw128(base + OFF_H + 32 * k), smem_desc_sw128(base + OFF_W + 32 * k), IDESC, k > 0);
        umma_commit(bars + B_ACCFULL);
      }
      __syncwarp();
    }
  } else {
    // ================================ one thread per sequence row ================================
    const int r = ((warp & 3) << 5) + lane;
    const uint32_t tl = tmem + ((uint32_t)((warp & 3) << 5) << 16);
    const uint32_t s_gamma = base + OFF_P, s_beta = s_gamma + TD * 4, s_bias = s_beta + TD * 4;
    int i = 0;
    bool real = row_real32(g, row_base + cta * TM + r, rows);
    for (int t = cta; t < ntiles; t += ctas, ++i) {
      const int row0 = row_base + t * TM;
      mbar_wait(wc, bars + B_XFULL, i & 1);
      float v[TD];
      if (real) {
        load_row64(base + OFF_X, r, v);
      } else {  // padded input rows may hold anything (NaN included): never read them
#pragma unroll
        for (int e = 0; e < TD; ++e) v[e] = 0.f;
      }
      fence_reads_before_release();
      __syncwarp();
      if (lane == 0) mbar_arrive(bars + B_XFREE);
      if (i > 0) {  // the previous tile's stores must have finished reading the staging rows (the normalised rows overlay them)
        if (tid == 64) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        t_bar_rows();
      }
      layernorm_row_to_tile(v, real, s_gamma, s_beta, eps, base + OFF_H, r);
      fence_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(bars + B_HREADY);
      const bool real_next = row_real32(g, row_base + (t + ctas) * TM + r, rows);  // overlaps the MMA

      mbar_wait(wc, bars + B_ACCFULL, i & 1);  // the MMA has also finished reading the normalised rows
      tc_fence_after();
#pragma unroll 1
      for (int c0 = 0; c0 < NQ; c0 += 32) {
        uint32_t a[32];
        tmem_ld32(tl + c0, a);
        tmem_wait_ld();
        tmem_regs_ready(a);
        uint32_t pk[16];
#pragma unroll
        for (int e = 0; e < 32; e += 4) {
          const float4 bb = ld_v4f(s_bias + (c0 + e) * 4);
          const float2 h0 = __fadd2_rn(make_float2(__uint_as_float(a[e]), __uint_as_float(a[e + 1])), make_float2(bb.x, bb.y));
          const float2 h1 = __fadd2_rn(make_float2(__uint_as_float(a[e + 2]), __uint_as_float(a[e + 3])), make_float2(bb.z, bb.w));
          pk[e >> 1] = real ? pack_bf16(h0.x, h0.y) : 0u;
          pk[(e >> 1) + 1] = real ? pack_bf16(h1.x, h1.y) : 0u;
        }
        const uint32_t box = base + OFF_OUT + (c0 >> 6) * (TM * 128);
        const int ch0 = (c0 & 32) >> 3;
#pragma unroll
        for (int q = 0; q < 4; ++q) st_shared_v4(sw128(box, r, ch0 + q), pk[4 * q], pk[4 * q + 1], pk[4 * q + 2], pk[4 * q + 3]);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bars + B_ACCFREE);
      fence_async_smem();
      t_bar_rows();
      if (tid == 64) {
#pragma unroll
        for (int j = 0; j < 3; ++j) tma_store_2d(&tmOut, base + OFF_OUT + j * (TM * 128), 64 * j, row0);
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
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
namespace pm {
constexpr int OFF_WO = 0;                          // W_o: 64 rows x 128 B
constexpr int OFF_W1 = OFF_WO + TD * 128;          // W_1: up to 256 rows x 128 B
constexpr int OFF_W2 = OFF_W1 + 256 * 128;         // W_2: up to 4 k-blocks of 64 rows x 128 B
constexpr int OFF_ATT = OFF_W2 + 4 * TD * 128;     // 2 attention tiles
constexpr int OFF_H = OFF_ATT + 2 * TM * 128;      // LN2 output
constexpr int OFF_F = OFF_H + TM * 128;            // hidden units: up to 4 k-blocks of 128 rows x 128 B; later the y staging
constexpr int OFF_X = OFF_F + 4 * TM * 128;        // float residual input tile (2 boxes)
constexpr int OFF_P = OFF_X + 2 * XBOX;            // b_o[64], gamma[64], beta[64], b_2[64], b_1[256] as floats
constexpr int OFF_STAT = OFF_P + (4 * TD + 256) * 4;  // LayerNorm statistics exchanged by the two threads of a row
constexpr int OFF_BAR = OFF_STAT + 2 * TM * 8;
constexpr int B_W = 0, B_ATTFULL = 8, B_ATTFREE = 24, B_XFULL = 40, B_XFREE = 48, B_ACC1 = 56, B_HREADY = 64, B_ACCF = 72,
              B_FREADY = 80, B_ACCY = 88, SLOT = 96;
constexpr int SMEM = OFF_BAR + 112 + 1024;
constexpr int COL_1 = 0, COL_F = 64, COL_Y = 320, TMEM_COLS = 512;
static_assert(SMEM <= 227 * 1024, "shared memory budget");
}  // namespace pm

// Per-problem arguments of the out-projection + MLP kernel (two problems per launch as for LnQkvArgs).
struct ProjMlpArgs {
  CUtensorMap tmAtt, tmX, tmWo, tmW1, tmW2, tmY;
  const float *bo, *gamma, *beta, *b1, *b2;
};

__global__ void __launch_bounds__(T_THREADS8, 1)
proj_mlp_tc_kernel(const __grid_constant__ ProjMlpArgs arg0, const __grid_constant__ ProjMlpArgs arg1, const Geometry g,
                   const float eps, const int d_ff, const int problems) {
  using namespace pm;
  const int which = (problems == 2) ? (int)(blockIdx.x & 1u) : 0;
  const int cta = (problems == 2) ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int ctas = (problems == 2) ? (int)((gridDim.x + 1 - which) >> 1) : (int)gridDim.x;
  const ProjMlpArgs& arg = which ? arg1 : arg0;
  const CUtensorMap &tmAtt = arg.tmAtt, &tmX = arg.tmX, &tmWo = arg.tmWo, &tmW1 = arg.tmW1, &tmW2 = arg.tmW2, &tmY = arg.tmY;
  const float *bo = arg.bo, *gamma = arg.gamma, *beta = arg.beta, *b1 = arg.b1, *b2 = arg.b2;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bars = base + OFF_BAR;
  const WaitCtx wc{g.status, bars + SLOT + 4};
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nh = d_ff / 64;  // k-blocks of hidden units

  float* prm = reinterpret_cast<float*>(base_ptr + OFF_P);
  stage_vector(prm, bo, TD, 0.f, tid, T_THREADS8);
  stage_vector(prm + TD, gamma, TD, 1.f, tid, T_THREADS8);
  stage_vector(prm + 2 * TD, beta, TD, 0.f, tid, T_THREADS8);
  stage_vector(prm + 3 * TD, b2, TD, 0.f, tid, T_THREADS8);
  stage_vector(prm + 4 * TD, b1, d_ff, 0.f, tid, T_THREADS8);
  if (tid == 0) {
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(bars + SLOT + 4), "r"(0u) : "memory");
    mbar_init(bars + B_W, 1);
    for (int i = 0; i < 2; ++i) { mbar_init(bars + B_ATTFULL + 8 * i, 1); mbar_init(bars + B_ATTFREE + 8 * i, 1); }
    mbar_init(bars + B_XFULL, 1);
    mbar_init(bars + B_XFREE, 8);
    mbar_init(bars + B_ACC1, 1);
    mbar_init(bars + B_HREADY, 8);
    mbar_init(bars + B_ACCF, 1);
    mbar_init(bars + B_FREADY, 8);
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
      mbar_expect_tx(bars + B_W, (uint32_t)(TD * 128 + d_ff * 128 + nh * TD * 128));
      tma_load_2d(base + OFF_WO, &tmWo, 0, 0, bars + B_W);
      tma_load_2d(base + OFF_W1, &tmW1, 0, 0, bars + B_W);
      for (int kb = 0; kb < nh; ++kb) tma_load_2d(base + OFF_W2 + kb * TD * 128, &tmW2, 64 * kb, 0, bars + B_W);
    }
    __syncwarp();
  }
  grid_dep_wait();
  grid_dep_launch();
  const int row_base = rows_begin(g), rows = rows_end(g);  // this problem's rows of the activation matrices
  const int ntiles = (rows - row_base + TM - 1) / TM;

  if (warp == 0) {
    // ================================ producer ================================
    int i = 0;
    for (int t = cta; t < ntiles; t += ctas, ++i) {
      const int row0 = row_base + t * TM;
      const int b = i & 1;
      if (i >= 2) mbar_wait(wc, bars + B_ATTFREE + 8 * b, ((i >> 1) - 1) & 1);
      if (elect_one()) {
        mbar_expect_tx(bars + B_ATTFULL + 8 * b, TM * 128);
        tma_load_2d(base + OFF_ATT + b * TM * 128, &tmAtt, 0, row0, bars + B_ATTFULL + 8 * b);
      }
      __syncwarp();
      if (i > 0) mbar_wait(wc, bars + B_XFREE, (i - 1) & 1);
      if (elect_one()) {
        mbar_expect_tx(bars + B_XFULL, 2 * XBOX);
        tma_load_2d(base + OFF_X, &tmX, 0, row0, bars + B_XFULL);
        tma_load_2d(base + OFF_X + XBOX, &tmX, 32, row0, bars + B_XFULL);
      }
      __syncwarp();
    }
  } else if (warp == 1) {
    // ================================ MMA issuer ================================
    constexpr uint32_t IDESC_D = idesc_bf16(TD, false);
    const uint32_t idesc_f = idesc_bf16(d_ff, false);
    mbar_wait(wc, bars + B_W, 0);
    // y1 accumulator of tile number i_ = att W_o^T
    auto out_proj = [&](int i_) {
      const int b = i_ & 1;
      mbar_wait(wc, bars + B_ATTFULL + 8 * b, (i_ >> 1) & 1);
      tc_fence_after();
      if (elect_one()) {
#pragma unroll
        for (int k = 0; k < 4; ++k)
          umma_ss(tmem + COL_1, smem_desc_sw128(base + OFF_ATT + b * TM * 128 + 32 * k), smem_desc_sw128(base + OFF_WO + 32 * k), IDESC_D, k > 0);
        umma_commit(bars + B_ATTFREE + 8 * b);
        umma_commit(bars + B_ACC1);
      }
      __syncwarp();
    };
    // The row warps work one tile ahead with the first part of a tile (y1 and LN2) while the tensor core finishes the
    // tile before it, so the products are issued in that order: W_1 of tile i, W_o of tile i + 1, W_2 of tile i.
    int i = 0;
    if (cta < ntiles) out_proj(0);
    for (int t = cta; t < ntiles; t += ctas, ++i) {
      // hidden accumulator = LN2(y1) W_1^T
      mbar_wait(wc, bars + B_HREADY, i & 1);  // (the rows have also read the y1 accumulator of this tile)
      tc_fence_after();
      if (elect_one()) {
#pragma unroll
        for (int k = 0; k < 4; ++k)
          umma_ss(tmem + COL_F, smem_desc_sw128(base + OFF_H + 32 * k), smem_desc_sw128(base + OFF_W1 + 32 * k), idesc_f, k > 0);
        umma_commit(bars + B_ACCF);
      }
      __syncwarp();
      if (t + ctas < ntiles) out_proj(i + 1);
      // output accumulator = relu(hidden) W_2^T
      mbar_wait(wc, bars + B_FREADY, i & 1);
      tc_fence_after();
      if (elect_one()) {
        for (int kb = 0; kb < nh; ++kb)
#pragma unroll
          for (int k = 0; k < 4; ++k)
            umma_ss(tmem + COL_Y, smem_desc_sw128(base + OFF_F + kb * TM * 128 + 32 * k), smem_desc_sw128(base + OFF_W2 + kb * TD * 128 + 32 * k),
                   IDESC_D, (kb > 0 || k > 0) ? 1u : 0u);
        umma_commit(bars + B_ACCY);
      }
      __syncwarp();
    }
  } else {
    // ================================ two threads per sequence row ================================
    const int r = ((warp & 3) << 5) + lane, hf = (warp - 2) >> 2;  // row = TMEM lane; which half of the columns
    const uint32_t tl = tmem + ((uint32_t)((warp & 3) << 5) << 16);
    const uint32_t s_bo = base + OFF_P, s_gamma = s_bo + TD * 4, s_beta = s_gamma + TD * 4, s_b2 = s_beta + TD * 4,
                   s_b1 = s_b2 + TD * 4;
    // First part of tile number i_: y1 = x + att W_o^T + b_o (this thread's 32 columns, kept in v_) and h = LN2(y1), the
    // A operand of the first MLP product.  It runs one tile ahead of the rest, while the tensor core is still busy with
    // the tile before (whose first MLP product has completed, so the LN2 buffer is free).
    auto first_part = [&](int i_, bool real_, float (&v_)[32]) {
      mbar_wait(wc, bars + B_XFULL, i_ & 1);
      if (real_) {
        load_half_row(base + OFF_X + hf * XBOX, r, v_);
      } else {
#pragma unroll
        for (int e = 0; e < 32; ++e) v_[e] = 0.f;
      }
      fence_reads_before_release();
      __syncwarp();
      if (lane == 0) mbar_arrive(bars + B_XFREE);
      mbar_wait(wc, bars + B_ACC1, i_ & 1);
      tc_fence_after();
      {
        uint32_t a[32];
        tmem_ld32(tl + COL_1 + 32 * hf, a);
        tmem_wait_ld();
        tmem_regs_ready(a);
#pragma unroll
        for (int e = 0; e < 32; e += 4) {
          const float4 bb = ld_v4f(s_bo + (32 * hf + e) * 4);
          v_[e] += __uint_as_float(a[e]) + bb.x;
          v_[e + 1] += __uint_as_float(a[e + 1]) + bb.y;
          v_[e + 2] += __uint_as_float(a[e + 2]) + bb.z;
          v_[e + 3] += __uint_as_float(a[e + 3]) + bb.w;
        }
      }
      float mean, rstd;
      split_row_stats<32>(v_, base + OFF_STAT, r, hf, eps, real_, mean, rstd);
      normalise_to_tile<32>(v_, mean, rstd, real_, s_gamma, s_beta, 32 * hf, base + OFF_H, r, 4 * hf);
      fence_async_smem();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bars + B_HREADY);
    };
    int i = 0;
    bool real = row_real32(g, row_base + cta * TM + r, rows);
    float v[32];
    if (cta < ntiles) first_part(0, real, v);
    for (int t = cta; t < ntiles; t += ctas, ++i) {
      const int row0 = row_base + t * TM;
      const bool has_next = t + ctas < ntiles;
      const bool real_next = row_real32(g, row_base + (t + ctas) * TM + r, rows);
      // ---- f = relu(h W_1^T + b_1) -> A operand of the second MLP product ----
      mbar_wait(wc, bars + B_ACCF, i & 1);
      tc_fence_after();
      if (i > 0) {  // the previous tile's output stores must have finished reading the staging rows (they overlay f)
        if (tid == 64) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        t_bar_rows8();
      }
#pragma unroll 1
      for (int c0 = 32 * hf; c0 < d_ff; c0 += 64) {  // alternate groups of 32 hidden units
        uint32_t a[32];
        tmem_ld32(tl + COL_F + c0, a);
        tmem_wait_ld();
        tmem_regs_ready(a);
        uint32_t pk[16];
#pragma unroll
        for (int e = 0; e < 32; e += 4) {
          const float4 bb = ld_v4f(s_b1 + (c0 + e) * 4);
          const float2 h0 = __fadd2_rn(make_float2(__uint_as_float(a[e]), __uint_as_float(a[e + 1])), make_float2(bb.x, bb.y));
          const float2 h1 = __fadd2_rn(make_float2(__uint_as_float(a[e + 2]), __uint_as_float(a[e + 3])), make_float2(bb.z, bb.w));
          pk[e >> 1] = pack_bf16_relu(h0.x, h0.y);
          pk[(e >> 1) + 1] = pack_bf16_relu(h1.x, h1.y);
        }
        const uint32_t blk = base + OFF_F + (c0 >> 6) * (TM * 128);
        const int ch0 = (c0 & 32) >> 3;
#pragma unroll
        for (int q = 0; q < 4; ++q) st_shared_v4(sw128(blk, r, ch0 + q), pk[4 * q], pk[4 * q + 1], pk[4 * q + 2], pk[4 * q + 3]);
      }
      fence_async_smem();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bars + B_FREADY);
      // ---- the next tile's first part, while the second MLP product of this one runs ----
      float vn[32];
      if (has_next) first_part(i + 1, real_next, vn);
      // ---- y = y1 + f W_2^T + b_2 -> staging rows (this thread's box of 32 floats) -> TMA stores; padded rows +0 ----
      mbar_wait(wc, bars + B_ACCY, i & 1);
      tc_fence_after();
      {
        uint32_t a[32];
        tmem_ld32(tl + COL_Y + 32 * hf, a);
        tmem_wait_ld();
        tmem_regs_ready(a);
        const uint32_t box = base + OFF_F + hf * (TM * 128);
#pragma unroll
        for (int ch = 0; ch < 8; ++ch) {
          const int e = 4 * ch;
          const float4 bb = ld_v4f(s_b2 + (32 * hf + e) * 4);
          float o0 = v[e] + __uint_as_float(a[e]) + bb.x, o1 = v[e + 1] + __uint_as_float(a[e + 1]) + bb.y;
          float o2 = v[e + 2] + __uint_as_float(a[e + 2]) + bb.z, o3 = v[e + 3] + __uint_as_float(a[e + 3]) + bb.w;
          if (!real) { o0 = 0.f; o1 = 0.f; o2 = 0.f; o3 = 0.f; }
          st_shared_v4(sw128(box, r, ch), __float_as_uint(o0), __float_as_uint(o1), __float_as_uint(o2), __float_as_uint(o3));
        }
      }
      tc_fence_before();
      fence_async_smem();
      t_bar_rows8();
      if (tid == 64) {
        tma_store_2d(&tmY, base + OFF_F, 0, row0);
        tma_store_2d(&tmY, base + OFF_F + TM * 128, 32, row0);
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
      }
      real = real_next;
      if (has_next) {
#pragma unroll
        for (int e = 0; e < 32; ++e) v[e] = vn[e];
      }
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

}  // namespace

bool fused_layer_tc_supported(const Geometry& g, int d_ff) { return g.d == TD && d_ff >= 64 && d_ff <= 256 && d_ff % 64 == 0; }

namespace {

bool fill_ln_qkv(LnQkvArgs* a, int64_t rows, const float* x, int64_t ldx, const float* gamma, const float* beta,
                 const __nv_bfloat16* w_qkv, const float* b_qkv, __nv_bfloat16* qkv) {
  a->gamma = gamma; a->beta = beta; a->bias = b_qkv;
  return make_map(&a->tmW, w_qkv, 3 * TD, TD, TD, 64, 3 * TD) && make_map_f32(&a->tmX, x, rows, TD, ldx, TM) &&
         make_map(&a->tmOut, qkv, rows, 3 * TD, 3 * TD, 64, TM);
}

bool fill_proj_mlp(ProjMlpArgs* a, int64_t rows, const __nv_bfloat16* att, const float* x, int64_t ldx, const __nv_bfloat16* w_o,
                   const float* b_o, const float* gamma, const float* beta, const __nv_bfloat16* w_1, const float* b_1,
                   const __nv_bfloat16* w_2, const float* b_2, int d_ff, float* y, int64_t ldy) {
  a->bo = b_o; a->gamma = gamma; a->beta = beta; a->b1 = b_1; a->b2 = b_2;
  return make_map(&a->tmAtt, att, rows, TD, TD, 64, TM) && make_map_f32(&a->tmX, x, rows, TD, ldx, TM) &&
         make_map(&a->tmWo, w_o, TD, TD, TD, 64, TD) && make_map(&a->tmW1, w_1, d_ff, TD, TD, 64, d_ff) &&
         make_map(&a->tmW2, w_2, TD, d_ff, d_ff, 64, TD) && make_map_f32(&a->tmY, y, rows, TD, ldy, TM);
}

}  // namespace

cudaError_t launch_ln_qkv_tc(const Geometry& g, const float* x, int64_t ldx, const float* gamma, const float* beta, float eps,
                             const __nv_bfloat16* w_qkv, const float* b_qkv, __nv_bfloat16* qkv, int* zero_word, cudaStream_t st) {
  if (g.d != TD) return cudaErrorNotSupported;
  const int64_t rows = matrix_rows(g);  // bounds of the tensor maps; the kernel takes its own row range from the geometry
  const int ntiles = (int)((rows + TM - 1) / TM), nsm = t_sm_count();
  if (nsm == 0) return cudaErrorUnknown;
  alignas(64) LnQkvArgs a;
  if (!fill_ln_qkv(&a, rows, x, ldx, gamma, beta, w_qkv, b_qkv, qkv)) return cudaErrorInvalidValue;
  cudaError_t e = sm_count_and_smem_once(reinterpret_cast<const void*>(ln_qkv_tc_kernel), qk::SMEM, nullptr);
  if (e != cudaSuccess) return e;
  return launch_overlapped(ln_qkv_tc_kernel, dim3(min(ntiles, 2 * nsm)), dim3(T_THREADS), qk::SMEM, st, a, a, g, eps, 1, zero_word);
}

cudaError_t launch_proj_mlp_tc(const Geometry& g, const __nv_bfloat16* att, const float* x, int64_t ldx,
                               const __nv_bfloat16* w_o, const float* b_o, const float* gamma, const float* beta, float eps,
                               const __nv_bfloat16* w_1, const float* b_1, const __nv_bfloat16* w_2, const float* b_2, int d_ff,
                               float* y, int64_t ldy, cudaStream_t st) {
  if (!fused_layer_tc_supported(g, d_ff)) return cudaErrorNotSupported;
  const int64_t rows = matrix_rows(g);  // bounds of the tensor maps; the kernel takes its own row range from the geometry
  const int ntiles = (int)((rows + TM - 1) / TM), nsm = t_sm_count();
  if (nsm == 0) return cudaErrorUnknown;
  alignas(64) ProjMlpArgs a;
  if (!fill_proj_mlp(&a, rows, att, x, ldx, w_o, b_o, gamma, beta, w_1, b_1, w_2, b_2, d_ff, y, ldy)) return cudaErrorInvalidValue;
  cudaError_t e = sm_count_and_smem_once(reinterpret_cast<const void*>(proj_mlp_tc_kernel), pm::SMEM, nullptr);
  if (e != cudaSuccess) return e;
  return launch_overlapped(proj_mlp_tc_kernel, dim3(min(ntiles, nsm)), dim3(T_THREADS8), pm::SMEM, st, a, a, g, eps, d_ff, 1);
}

// The same two halves for a PAIR of problems of one geometry in one launch each (the two ring encoders' layers of equal
// depth): CTAs alternate between the problems, so each problem has half the SMs for the whole launch and one tail is paid
// instead of two.
cudaError_t launch_ln_qkv_tc_pair(const Geometry& g, const FusedHalfArgs (&h)[2], float eps, int* zero_word, cudaStream_t st) {
  if (g.d != TD) return cudaErrorNotSupported;
  const int64_t rows = matrix_rows(g);
  const int ntiles = (int)((rows + TM - 1) / TM), nsm = t_sm_count();
  if (nsm < 2) return cudaErrorUnknown;
  alignas(64) LnQkvArgs a[2];
  for (int i = 0; i < 2; ++i)
    if (!fill_ln_qkv(&a[i], rows, h[i].x, h[i].ldx, h[i].ln1_gamma, h[i].ln1_beta, h[i].w_qkv, h[i].b_qkv, h[i].qkv))
      return cudaErrorInvalidValue;
  cudaError_t e = sm_count_and_smem_once(reinterpret_cast<const void*>(ln_qkv_tc_kernel), qk::SMEM, nullptr);
  if (e != cudaSuccess) return e;
  return launch_overlapped(ln_qkv_tc_kernel, dim3(min(2 * ntiles, 2 * nsm)), dim3(T_THREADS), qk::SMEM, st, a[0], a[1], g, eps, 2, zero_word);
}

cudaError_t launch_proj_mlp_tc_pair(const Geometry& g, const FusedHalfArgs (&h)[2], float eps, int d_ff, cudaStream_t st) {
  if (!fused_layer_tc_supported(g, d_ff)) return cudaErrorNotSupported;
  const int64_t rows = matrix_rows(g);
  const int ntiles = (int)((rows + TM - 1) / TM), nsm = t_sm_count();
  if (nsm < 2) return cudaErrorUnknown;
  alignas(64) ProjMlpArgs a[2];
  for (int i = 0; i < 2; ++i)
    if (!fill_proj_mlp(&a[i], rows, h[i].att, h[i].x, h[i].ldx, h[i].w_o, h[i].b_o, h[i].ln2_gamma, h[i].ln2_beta, h[i].w_1, h[i].b_1,
                       h[i].w_2, h[i].b_2, d_ff, h[i].y, h[i].ldy))
      return cudaErrorInvalidValue;
  cudaError_t e = sm_count_and_smem_once(reinterpret_cast<const void*>(proj_mlp_tc_kernel), pm::SMEM, nullptr);
  if (e != cudaSuccess) return e;
  return launch_overlapped(proj_mlp_tc_kernel, dim3(min(2 * ntiles, nsm & ~1)), dim3(T_THREADS8), pm::SMEM, st, a[0], a[1], g, eps, d_ff, 2);
}

}  // namespace gsit
