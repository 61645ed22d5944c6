// Fused halves of the IM encoder layer around the attention (bf16 operands, fp32 accumulation and residual stream),
// for d_model 64 and 128 -- the widths at which separate LayerNorm and linear kernels are bound by HBM round trips of
// their intermediates, not by arithmetic.
//
//   ln_qkv_kernel     qkv = LN1(x) W_qkv^T + b_qkv            (shared projection of the whole concatenated sequence)
//   proj_mlp_kernel   y1 = x + att W_o^T + b_o ;  y = y1 + relu(LN2(y1) W_1^T + b_1) W_2^T + b_2
//
// Both are persistent over tiles of 64 sequence rows.  A tile's activations stay in shared memory from the first
// read of x / att to the last write of qkv / y: the normalised rows, the float residual y1 and the MLP hidden units
// (produced and consumed 64 at a time) never travel to HBM.  The input rows of the next tile are fetched with bulk
// asynchronous copies (completion on an mbarrier) while the current tile is being computed.  Matrix products run on
// mma.sync.m16n8k16 tiles fed by ldmatrix from padded shared-memory rows; W_qkv and W_o stay resident in shared
// memory, W_1 / W_2 stream through a double-buffered cp.async ring (they are L2-resident).  Padded rows are +0.
#include "common.cuh"

namespace gsit {
namespace {

constexpr int FM = 64;         // rows per tile
constexpr int FTHREADS = 256;  // 8 warps: 2 along rows x 4 along columns
constexpr int HC = 64;         // hidden units per MLP chunk

__device__ __forceinline__ void ldsm4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void cp16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ uint32_t bf2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// ---- bulk asynchronous copies of whole rows, completing on an mbarrier (input tiles are fetched one tile ahead) ----
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// Bounded wait for a phase of the tile barrier; raises GSIT_DEVFLAG_TIMEOUT instead of hanging.
__device__ __forceinline__ void mbar_wait(const Geometry& g, uint32_t bar, uint32_t parity) {
  for (int it = 0; it < (1 << 16); ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    if (ok) return;
    if ((it & 63) == 63 && (*reinterpret_cast<volatile unsigned int*>(g.status) & GSIT_DEVFLAG_TIMEOUT)) return;
  }
  raise_flag(g, GSIT_DEVFLAG_TIMEOUT);
}
// One copy per row: threads 0..nrows-1 each request `row_bytes` bytes (a multiple of 16, 16-byte aligned on both
// sides).  The byte total must have been posted on `bar` by mbar_expect_tx.
__device__ __forceinline__ void fetch_rows(uint32_t bar, uint32_t dst, int dst_pitch, const uint8_t* src, int64_t src_pitch,
                                           int nrows, int row_bytes, int tid) {
  if (tid < nrows) bulk_g2s(dst + tid * dst_pitch, src + tid * src_pitch, (uint32_t)row_bytes, bar);
}

// acc[MT][NT] (16x8 tiles) += A[m0 .. m0+16*MT, 0..K) * W[n0 .. n0+8*NT, 0..K)^T.
// A and W are bf16 rows in shared memory with pitches lda / ldw BYTES (pitch = row bytes + 16, so that the eight rows
// of an ldmatrix land in different banks).  NT is even.
template <int MT, int NT>
__device__ __forceinline__ void warp_gemm(float (&acc)[MT][NT][4], uint32_t sA, int lda, int m0, uint32_t sW, int ldw,
                                          int n0, int K, int lane) {
  const int mi = lane >> 3, l7 = lane & 7;
  for (int k0 = 0; k0 < K; k0 += 16) {
    uint32_t a[MT][4];
#pragma unroll
    for (int i = 0; i < MT; ++i)
      ldsm4(sA + (m0 + i * 16 + (mi & 1) * 8 + l7) * lda + (k0 + (mi >> 1) * 8) * 2, a[i][0], a[i][1], a[i][2], a[i][3]);
#pragma unroll
    for (int j = 0; j < NT / 2; ++j) {
      uint32_t b0, b1, b2, b3;  // (n-tile 2j: k lo, k hi), (n-tile 2j+1: k lo, k hi)
      ldsm4(sW + (n0 + j * 16 + (mi >> 1) * 8 + l7) * ldw + (k0 + (mi & 1) * 8) * 2, b0, b1, b2, b3);
#pragma unroll
      for (int i = 0; i < MT; ++i) {
        mma16816(acc[i][2 * j], a[i], b0, b1);
        mma16816(acc[i][2 * j + 1], a[i], b2, b3);
      }
    }
  }
}

// Copies `rows` rows of `row_bytes` bytes (multiple of 16) from global (pitch src_pitch bytes) into shared memory
// (pitch dst_pitch bytes) with cp.async; the caller commits and waits.
__device__ __forceinline__ void stage_rows(uint32_t dst, int dst_pitch, const uint8_t* src, int64_t src_pitch, int rows,
                                           int row_bytes, int tid) {
  const int cpr = row_bytes >> 4;
  for (int idx = tid; idx < rows * cpr; idx += FTHREADS) {
    const int r = idx / cpr, c = idx - r * cpr;
    cp16(dst + r * dst_pitch + c * 16, src + r * src_pitch + c * 16);
  }
}

// LayerNorm of the 8 rows a warp owns in a tile: float rows in shared memory -> bf16 rows in shared memory.
// D / 32 consecutive features per lane.  Rows flagged as padding are written as zeros (their input is not read).
template <int D>
__device__ __forceinline__ void warp_layernorm8(uint32_t s_src, int src_pitch, const uint8_t* real, const float* gamma,
                                                const float* beta, float eps, uint32_t s_dst, int dst_pitch, int warp,
                                                int lane) {
  constexpr int E = D / 32;
  float gm[E], bt[E];
#pragma unroll
  for (int e = 0; e < E; ++e) {
    gm[e] = gamma ? gamma[lane * E + e] : 1.f;
    bt[e] = beta ? beta[lane * E + e] : 0.f;
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int r = warp * 8 + i;
    float v[E];
    if (real[r]) {
#pragma unroll
      for (int e = 0; e < E; ++e)
        asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v[e]) : "r"(s_src + r * src_pitch + (lane * E + e) * 4));
      float s = 0.f;
#pragma unroll
      for (int e = 0; e < E; ++e) s += v[e];
#pragma unroll
      for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      const float mean = s * (1.f / D);
      float q = 0.f;
#pragma unroll
      for (int e = 0; e < E; ++e) { v[e] -= mean; q = fmaf(v[e], v[e], q); }
#pragma unroll
      for (int o = 16; o; o >>= 1) q += __shfl_xor_sync(0xffffffffu, q, o);
      const float rstd = rsqrtf(q * (1.f / D) + eps);
#pragma unroll
      for (int e = 0; e < E; ++e) v[e] = fmaf(v[e] * rstd, gm[e], bt[e]);
    } else {
#pragma unroll
      for (int e = 0; e < E; ++e) v[e] = 0.f;
    }
    const uint32_t d = s_dst + r * dst_pitch + lane * E * 2;
    if (E == 2) asm volatile("st.shared.b32 [%0], %1;" ::"r"(d), "r"(bf2(v[0], v[1])) : "memory");
    else asm volatile("st.shared.v2.b32 [%0], {%1,%2};" ::"r"(d), "r"(bf2(v[0], v[1])), "r"(bf2(v[E - 2], v[E - 1])) : "memory");
  }
}

// Marks which of the tile's FM rows are real (inside the matrix and not padding).  Done by the last two warps, so
// that it overlaps with the copies the first two warps issue.
__device__ __forceinline__ void flag_rows(const Geometry& g, int64_t row0, int64_t rows, uint8_t* real, int tid) {
  if (tid >= FTHREADS - FM) {
    const int r = tid - (FTHREADS - FM);
    real[r] = (row0 + r < rows) && row_is_real(g, row0 + r);
  }
}

// ------------------------------------------------------------------------------------------------ LN1 + shared QKV
template <int D>
struct QkvSmem {
  static constexpr int WP = D * 2 + 16;             // pitch of a weight / normalised row (bytes)
  static constexpr int CP = 3 * D * 2 + 16;         // pitch of an output row
  static constexpr int XP = D * 4 + 16;             // pitch of a float input row
  static constexpr int OFF_W = 0;                   // [3D][WP]
  static constexpr int OFF_A = OFF_W + 3 * D * WP;  // [FM][WP]
  static constexpr int OFF_C = OFF_A + FM * WP;     // [FM][CP]
  static constexpr int OFF_X = OFF_C + FM * CP;     // [FM][XP] input tile, fetched one tile ahead
  static constexpr int OFF_F = OFF_X + FM * XP;     // 2 x [FM] row flags
  static constexpr int OFF_B = OFF_F + 2 * FM;      // tile barrier
  static constexpr int BYTES = OFF_B + 16;
};

template <int D>
__global__ void __launch_bounds__(FTHREADS)
ln_qkv_kernel(const Geometry g, const float* __restrict__ x, const int64_t ldx, const float* __restrict__ gamma,
              const float* __restrict__ beta, const float eps, const __nv_bfloat16* __restrict__ w,
              const float* __restrict__ bias, __nv_bfloat16* __restrict__ qkv) {
  using S = QkvSmem<D>;
  extern __shared__ __align__(16) uint8_t smem[];
  const uint32_t sb = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int wm = warp >> 2, wn = warp & 3;
  const int64_t rows = (int64_t)g.batch * g.L;
  const int ntiles = (int)((rows + FM - 1) / FM);
  constexpr int NT = 3 * D / 4 / 8;  // n-tiles per warp: a quarter of the 3D output columns

  stage_rows(sb + S::OFF_W, S::WP, reinterpret_cast<const uint8_t*>(w), D * 2, 3 * D, D * 2, tid);
  cp_commit();
  const uint32_t bar = sb + S::OFF_B;
  if (tid == 0) {
    mbar_init(bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  auto fetch_tile = [&](int tile) {  // x rows of a tile -> shared memory (asynchronous)
    const int64_t row0 = (int64_t)tile * FM;
    const int nrows = (int)min((int64_t)FM, rows - row0);
    if (tid == 0) mbar_expect_tx(bar, (uint32_t)(nrows * D * 4));
    fetch_rows(bar, sb + S::OFF_X, S::XP, reinterpret_cast<const uint8_t*>(x + row0 * ldx), ldx * 4, nrows, D * 4, tid);
  };
  if ((int)blockIdx.x < ntiles) fetch_tile(blockIdx.x);

  int it = 0;
  for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++it) {
    const int64_t row0 = (int64_t)tile * FM;
    uint8_t* real = smem + S::OFF_F + (it & 1) * FM;
    flag_rows(g, row0, rows, real, tid);
    mbar_wait(g, bar, it & 1);
    __syncthreads();  // flags visible; the previous tile's staged output has been stored
    warp_layernorm8<D>(sb + S::OFF_X, S::XP, real, gamma, beta, eps, sb + S::OFF_A, S::WP, warp, lane);
    cp_wait<0>();
    __syncthreads();  // normalised rows complete, input tile consumed
    if (tile + (int)gridDim.x < ntiles) fetch_tile(tile + gridDim.x);

    float acc[2][NT][4];
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int j = 0; j < NT; ++j) acc[i][j][0] = acc[i][j][1] = acc[i][j][2] = acc[i][j][3] = 0.f;
    warp_gemm<2, NT>(acc, sb + S::OFF_A, S::WP, wm * 32, sb + S::OFF_W, S::WP, wn * (3 * D / 4), D, lane);

    // bias, bf16, into the staging rows
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int j = 0; j < NT; ++j) {
        const int col = wn * (3 * D / 4) + j * 8 + (lane & 3) * 2;
        const float b0 = bias ? bias[col] : 0.f, b1 = bias ? bias[col + 1] : 0.f;
        const int r0 = wm * 32 + i * 16 + (lane >> 2);
        asm volatile("st.shared.b32 [%0], %1;" ::"r"(sb + S::OFF_C + r0 * S::CP + col * 2),
                     "r"(bf2(acc[i][j][0] + b0, acc[i][j][1] + b1)) : "memory");
        asm volatile("st.shared.b32 [%0], %1;" ::"r"(sb + S::OFF_C + (r0 + 8) * S::CP + col * 2),
                     "r"(bf2(acc[i][j][2] + b0, acc[i][j][3] + b1)) : "memory");
      }
    __syncthreads();
    // coalesced 16-byte stores; padded rows are written as +0
    constexpr int CPR = 3 * D * 2 / 16;
    const int nrows = (int)min((int64_t)FM, rows - row0);
    for (int idx = tid; idx < nrows * CPR; idx += FTHREADS) {
      const int r = idx / CPR, c = idx - r * CPR;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (real[r])
        asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                     : "r"(sb + S::OFF_C + r * S::CP + c * 16));
      *reinterpret_cast<uint4*>(reinterpret_cast<uint8_t*>(qkv) + (row0 + r) * (int64_t)(3 * D * 2) + c * 16) = v;
    }
  }
  cp_wait<0>();
}

// ------------------------------------------------------------------------------------------------ out-proj + MLP
template <int D>
struct MlpSmem {
  static constexpr int AP = D * 2 + 16;    // pitch of a bf16 row of D features (att, LN2 output, W_o, W_1 chunk)
  static constexpr int YP = D * 4 + 16;    // pitch of a float row of D features (x, then y1, then y)
  static constexpr int FP = HC * 2 + 16;   // pitch of a bf16 row of HC hidden units (hidden chunk, W_2 chunk)
  static constexpr int OFF_A = 0;                       // [FM][AP] attention tile, fetched one tile ahead
  static constexpr int OFF_H = OFF_A + FM * AP;         // [FM][AP] LN2 output
  static constexpr int OFF_Y = OFF_H + FM * AP;         // 2 x [FM][YP]; the other buffer receives the next tile's x
  static constexpr int OFF_WO = OFF_Y + 2 * FM * YP;    // [D][AP]
  static constexpr int OFF_F = OFF_WO + D * AP;         // [FM][FP]
  static constexpr int OFF_W1 = OFF_F + FM * FP;        // 2 x [HC][AP]
  static constexpr int OFF_W2 = OFF_W1 + 2 * HC * AP;   // 2 x [D][FP]
  static constexpr int OFF_FL = OFF_W2 + 2 * D * FP;    // 2 x [FM] row flags
  static constexpr int OFF_B = OFF_FL + 2 * FM;         // tile barrier
  static constexpr int BYTES = OFF_B + 16;
};

template <int D>
__global__ void __launch_bounds__(FTHREADS)
proj_mlp_kernel(const Geometry g, const __nv_bfloat16* __restrict__ att, const float* __restrict__ x, const int64_t ldx,
                const __nv_bfloat16* __restrict__ wo, const float* __restrict__ bo, const float* __restrict__ gamma,
                const float* __restrict__ beta, const float eps, const __nv_bfloat16* __restrict__ w1,
                const float* __restrict__ b1, const __nv_bfloat16* __restrict__ w2, const float* __restrict__ b2,
                const int d_ff, float* __restrict__ y, const int64_t ldy) {
  using S = MlpSmem<D>;
  extern __shared__ __align__(16) uint8_t smem[];
  const uint32_t sb = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int wm = warp >> 2, wn = warp & 3;
  const int64_t rows = (int64_t)g.batch * g.L;
  const int ntiles = (int)((rows + FM - 1) / FM);
  const int nch = d_ff / HC;
  constexpr int NTD = D / 4 / 8;  // n-tiles per warp over D output columns
  const int fr = lane >> 2, fc = (lane & 3) * 2;  // fragment row / column inside a 16x8 tile

  auto stage_chunk = [&](int c, int buf) {  // hidden units [c*HC, (c+1)*HC): rows of W_1, columns of W_2
    stage_rows(sb + S::OFF_W1 + buf * HC * S::AP, S::AP, reinterpret_cast<const uint8_t*>(w1 + (int64_t)c * HC * D), D * 2,
               HC, D * 2, tid);
    stage_rows(sb + S::OFF_W2 + buf * D * S::FP, S::FP, reinterpret_cast<const uint8_t*>(w2 + (int64_t)c * HC),
               (int64_t)d_ff * 2, D, HC * 2, tid);
  };
  const uint32_t bar = sb + S::OFF_B;
  if (tid == 0) {
    mbar_init(bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  auto fetch_tile = [&](int tile, int ybuf) {  // att and x rows of a tile -> shared memory (asynchronous)
    const int64_t row0 = (int64_t)tile * FM;
    const int nrows = (int)min((int64_t)FM, rows - row0);
    if (tid == 0) mbar_expect_tx(bar, (uint32_t)(nrows * (D * 2 + D * 4)));
    fetch_rows(bar, sb + S::OFF_A, S::AP, reinterpret_cast<const uint8_t*>(att + row0 * D), D * 2, nrows, D * 2, tid);
    fetch_rows(bar, sb + S::OFF_Y + ybuf * FM * S::YP, S::YP, reinterpret_cast<const uint8_t*>(x + row0 * ldx), ldx * 4,
               nrows, D * 4, tid);
  };
  if ((int)blockIdx.x < ntiles) fetch_tile(blockIdx.x, 0);
  stage_rows(sb + S::OFF_WO, S::AP, reinterpret_cast<const uint8_t*>(wo), D * 2, D, D * 2, tid);  // joins the first group

  int it = 0;
  for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x, ++it) {
    const int64_t row0 = (int64_t)tile * FM;
    const int nrows = (int)min((int64_t)FM, rows - row0);
    const int cur = it & 1;
    uint8_t* real = smem + S::OFF_FL + cur * FM;
    uint8_t* yt = smem + S::OFF_Y + cur * FM * S::YP;  // this tile's float rows
    flag_rows(g, row0, rows, real, tid);
    stage_chunk(0, 0);
    cp_commit();
    mbar_wait(g, bar, it & 1);
    cp_wait<0>();
    __syncthreads();

    // ---- y1 = x + att W_o^T + b_o, in place in the float tile ----
    {
      float acc[2][NTD][4];
#pragma unroll
      for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int j = 0; j < NTD; ++j) acc[i][j][0] = acc[i][j][1] = acc[i][j][2] = acc[i][j][3] = 0.f;
      warp_gemm<2, NTD>(acc, sb + S::OFF_A, S::AP, wm * 32, sb + S::OFF_WO, S::AP, wn * (D / 4), D, lane);
#pragma unroll
      for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int j = 0; j < NTD; ++j) {
          const int col = wn * (D / 4) + j * 8 + fc;
          const float c0 = bo ? bo[col] : 0.f, c1 = bo ? bo[col + 1] : 0.f;
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            float2* p = reinterpret_cast<float2*>(yt + (wm * 32 + i * 16 + fr + hh * 8) * S::YP + col * 4);
            float2 v = *p;
            v.x += acc[i][j][2 * hh] + c0;
            v.y += acc[i][j][2 * hh + 1] + c1;
            *p = v;
          }
        }
    }
    __syncthreads();  // y1 complete; the attention tile is no longer needed
    if (tile + (int)gridDim.x < ntiles) fetch_tile(tile + gridDim.x, cur ^ 1);
    // ---- h = LN2(y1) as bf16 ----
    warp_layernorm8<D>(sb + S::OFF_Y + cur * FM * S::YP, S::YP, real, gamma, beta, eps, sb + S::OFF_H, S::AP, warp, lane);
    __syncthreads();

    // ---- MLP, 64 hidden units at a time: f = relu(h W_1c^T + b_1c);  acc += f W_2c^T ----
    float acc2[2][NTD][4];
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int j = 0; j < NTD; ++j) acc2[i][j][0] = acc2[i][j][1] = acc2[i][j][2] = acc2[i][j][3] = 0.f;
    for (int c = 0; c < nch; ++c) {
      const int buf = c & 1;
      if (c + 1 < nch) {
        stage_chunk(c + 1, buf ^ 1);
        cp_commit();
        cp_wait<1>();
      } else {
        cp_wait<0>();
      }
      __syncthreads();
      {
        float af[2][2][4];
#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
          for (int j = 0; j < 2; ++j) af[i][j][0] = af[i][j][1] = af[i][j][2] = af[i][j][3] = 0.f;
        warp_gemm<2, 2>(af, sb + S::OFF_H, S::AP, wm * 32, sb + S::OFF_W1 + buf * HC * S::AP, S::AP, wn * 16, D, lane);
#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const int col = wn * 16 + j * 8 + fc;
            const float c0 = b1 ? b1[c * HC + col] : 0.f, c1 = b1 ? b1[c * HC + col + 1] : 0.f;
#pragma unroll
            for (int hh = 0; hh < 2; ++hh)
              asm volatile("st.shared.b32 [%0], %1;" ::"r"(sb + S::OFF_F + (wm * 32 + i * 16 + fr + hh * 8) * S::FP + col * 2),
                           "r"(bf2(fmaxf(af[i][j][2 * hh] + c0, 0.f), fmaxf(af[i][j][2 * hh + 1] + c1, 0.f))) : "memory");
          }
      }
      __syncthreads();
      warp_gemm<2, NTD>(acc2, sb + S::OFF_F, S::FP, wm * 32, sb + S::OFF_W2 + buf * D * S::FP, S::FP, wn * (D / 4), HC, lane);
      __syncthreads();  // the hidden chunk and this weight buffer may be overwritten
    }

    // ---- y = y1 + acc + b_2, staged in the float tile, then coalesced 16-byte stores; padded rows +0 ----
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int j = 0; j < NTD; ++j) {
        const int col = wn * (D / 4) + j * 8 + fc;
        const float c0 = b2 ? b2[col] : 0.f, c1 = b2 ? b2[col + 1] : 0.f;
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          float2* p = reinterpret_cast<float2*>(yt + (wm * 32 + i * 16 + fr + hh * 8) * S::YP + col * 4);
          float2 v = *p;
          v.x += acc2[i][j][2 * hh] + c0;
          v.y += acc2[i][j][2 * hh + 1] + c1;
          *p = v;
        }
      }
    __syncthreads();
    constexpr int CPR = D * 4 / 16;
    for (int idx = tid; idx < nrows * CPR; idx += FTHREADS) {
      const int r = idx / CPR, c = idx - r * CPR;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (real[r]) v = *reinterpret_cast<const float4*>(yt + r * S::YP + c * 16);
      *reinterpret_cast<float4*>(y + (row0 + r) * ldy + c * 4) = v;
    }
  }
  cp_wait<0>();
}

template <typename K>
cudaError_t set_smem(K kernel, int bytes) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
}
int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) n = 0;
  }
  return n;
}

}  // namespace

bool fused_layer_supported(const Geometry& g, int d_ff) { return (g.d == 64 || g.d == 128) && d_ff >= HC && d_ff % HC == 0; }

cudaError_t launch_ln_qkv_bf16(const Geometry& g, const float* x, int64_t ldx, const float* gamma, const float* beta,
                               float eps, const __nv_bfloat16* w_qkv, const float* b_qkv, __nv_bfloat16* qkv,
                               cudaStream_t st) {
  const int64_t rows = (int64_t)g.batch * g.L;
  const int ntiles = (int)((rows + FM - 1) / FM), nsm = sm_count();
  if (nsm == 0) return cudaErrorUnknown;
  cudaError_t e;
  if (g.d == 64) {
    static bool done = false;
    if (!done) { if ((e = set_smem(ln_qkv_kernel<64>, QkvSmem<64>::BYTES)) != cudaSuccess) return e; done = true; }
    ln_qkv_kernel<64><<<min(ntiles, 2 * nsm), FTHREADS, QkvSmem<64>::BYTES, st>>>(g, x, ldx, gamma, beta, eps, w_qkv, b_qkv, qkv);
  } else if (g.d == 128) {
    static bool done = false;
    if (!done) { if ((e = set_smem(ln_qkv_kernel<128>, QkvSmem<128>::BYTES)) != cudaSuccess) return e; done = true; }
    ln_qkv_kernel<128><<<min(ntiles, nsm), FTHREADS, QkvSmem<128>::BYTES, st>>>(g, x, ldx, gamma, beta, eps, w_qkv, b_qkv, qkv);
  } else {
    return cudaErrorNotSupported;
  }
  return cudaGetLastError();
}

cudaError_t launch_proj_mlp_bf16(const Geometry& g, const __nv_bfloat16* att, const float* x, int64_t ldx,
                                 const __nv_bfloat16* w_o, const float* b_o, const float* gamma, const float* beta, float eps,
                                 const __nv_bfloat16* w_1, const float* b_1, const __nv_bfloat16* w_2, const float* b_2,
                                 int d_ff, float* y, int64_t ldy, cudaStream_t st) {
  if (!fused_layer_supported(g, d_ff)) return cudaErrorNotSupported;
  const int64_t rows = (int64_t)g.batch * g.L;
  const int ntiles = (int)((rows + FM - 1) / FM), nsm = sm_count();
  if (nsm == 0) return cudaErrorUnknown;
  cudaError_t e;
  if (g.d == 64) {
    static bool done = false;
    if (!done) { if ((e = set_smem(proj_mlp_kernel<64>, MlpSmem<64>::BYTES)) != cudaSuccess) return e; done = true; }
    proj_mlp_kernel<64><<<min(ntiles, 2 * nsm), FTHREADS, MlpSmem<64>::BYTES, st>>>(g, att, x, ldx, w_o, b_o, gamma, beta, eps,
                                                                                   w_1, b_1, w_2, b_2, d_ff, y, ldy);
  } else {
    static bool done = false;
    if (!done) { if ((e = set_smem(proj_mlp_kernel<128>, MlpSmem<128>::BYTES)) != cudaSuccess) return e; done = true; }
    proj_mlp_kernel<128><<<min(ntiles, nsm), FTHREADS, MlpSmem<128>::BYTES, st>>>(g, att, x, ldx, w_o, b_o, gamma, beta, eps,
                                                                                 w_1, b_1, w_2, b_2, d_ff, y, ldy);
  }
  return cudaGetLastError();
}

}  // namespace gsit
