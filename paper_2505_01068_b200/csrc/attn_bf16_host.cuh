// Host side of the bf16 IM attention: tensor maps and launch (included by attn_bf16.cu only).
#pragma once

namespace gsit {
namespace {

// Query segments in descending order of the keys their tiles walk (longest work first), two bits per segment index.
int segment_order(const Geometry& g, uint32_t allowed) {
  int cost[3], ord[3] = {0, 1, 2};
  for (int s = 0; s < 3; ++s) {
    cost[s] = 0;
    for (int r = 0; r < 3; ++r)
      if ((allowed >> (3 * s + r)) & 1u) cost[s] += g.seg_len[r];
  }
  for (int i = 0; i < 3; ++i)
    for (int j = i + 1; j < 3; ++j)
      if (cost[ord[j]] > cost[ord[i]]) { const int t = ord[i]; ord[i] = ord[j]; ord[j] = t; }
  return ord[0] | (ord[1] << 2) | (ord[2] << 4);
}

// n = 1 or 2 problems of the geometry g (g.allowed is ignored: every problem brings its own pattern).
template <typename C>
cudaError_t launch_one(const Geometry& g, const AttnOperands* ops, int n, int64_t row_stride, float scale, cudaStream_t st) {
  constexpr int CW = C::CW;
  const int64_t rows = matrix_rows(g);
  alignas(64) AttnProblem pr[2];
  for (int i = 0; i < n; ++i) {
    if (!make_map(&pr[i].tmQ, ops[i].q, rows, g.d, row_stride, CW, C::QT) || !make_map(&pr[i].tmK, ops[i].k, rows, g.d, row_stride, CW, KT) ||
        !make_map(&pr[i].tmV, ops[i].v, rows, g.d, row_stride, CW, KT))
      return cudaErrorInvalidValue;
    pr[i].out = ops[i].out;
    pr[i].lse = ops[i].lse;
    pr[i].allowed = ops[i].allowed;
    pr[i].seg_order = segment_order(g, ops[i].allowed);
  }
  if (n == 1) pr[1] = pr[0];
  {
    cudaError_t e = sm_count_and_smem_once(reinterpret_cast<const void*>(attn_bf16_kernel<C>), C::SMEM, nullptr);
    if (e != cudaSuccess) return e;
  }
  int tiles = 0;
  for (int s = 0; s < 3; ++s) tiles += (g.seg_len[s] + C::QT - 1) / C::QT;
  if ((int64_t)tiles * g.batch * n > 0x7fffffffLL) return cudaErrorNotSupported;
  const dim3 grid((unsigned)(tiles * g.batch * n), (unsigned)(g.d / CW), 1u);
  const float sl2 = scale * 1.4426950408889634f;
  return launch_overlapped(attn_bf16_kernel<C>, grid, dim3(NTHREADS), C::SMEM, st, pr[0], pr[1], g, sl2, n);
}

}  // namespace

int g_attn_variant = 0;  // gsit_kernel_choice, or 1..7 = alternative tile configurations of the mma.sync attention

cudaError_t launch_attn_bf16_n(const Geometry& g, const AttnOperands* ops, int n, int64_t row_stride, float scale, int* next_item,
                               cudaStream_t st, bool counter_cleared) {
  if (n < 1 || n > 2) return cudaErrorInvalidValue;
  if (g.batch > 65535 || g.d % 16 != 0) return cudaErrorNotSupported;
  const int cw = (g.d % 64 == 0) ? 64 : (g.d % 32 == 0) ? 32 : 16;
  const int var = g_attn_variant;
  // head_dim 64 is a dense contraction: tcgen05 / TMEM kernel (GSIT_ATTN_LEGACY keeps the mma.sync kernel for comparison)
  if (g.hd == 64 && var != GSIT_ATTN_LEGACY) {
    for (int i = 0; i < n; ++i) {  // one launch per problem
      Geometry gi = g;
      gi.allowed = ops[i].allowed;
      cudaError_t e = launch_attn_tc_hd64(gi, ops[i].q, ops[i].k, ops[i].v, row_stride, ops[i].out, ops[i].lse, scale, st);
      if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
  }
  // head_dim 16 / 32: thread-per-row softmax on tensor-memory tiles.  At head_dim 8 that kernel measures slower than the
  // mma.sync kernel below (61 against 46 us at the MOSEI cross shape: a tcgen05 hand-over per 64 keys of one head costs
  // more than the 8192 exponentials it feeds), so there it is selected by the knob only.
  if (attn_tcs_supported(g) && (var == GSIT_ATTN_TMEM || (var == 0 && g.hd >= 16)))
    return launch_attn_tcs(g, ops, n, row_stride, scale, next_item, st, counter_cleared);
#define GSIT_CASE(VAR_, HD_, CW_, R_, KS_, MB_)         \
  if (g.hd == HD_ && cw == CW_ && (var == VAR_ || VAR_ == 0)) \
    return launch_one<Cfg<HD_, CW_, R_, KS_, MB_>>(g, ops, n, row_stride, scale, st);
  // alternatives first (selected only by the knob), then the defaults (VAR_ == 0 matches any knob value)
  GSIT_CASE(1, 8, 64, 4, 64, 2) GSIT_CASE(2, 8, 64, 4, 32, 2) GSIT_CASE(3, 8, 64, 2, 64, 2)
  GSIT_CASE(4, 8, 64, 2, 32, 3) GSIT_CASE(5, 8, 64, 2, 64, 3) GSIT_CASE(6, 8, 64, 1, 64, 3)
  GSIT_CASE(7, 8, 64, 1, 32, 4)
  GSIT_CASE(1, 16, 64, 2, 64, 2) GSIT_CASE(2, 16, 64, 2, 32, 2) GSIT_CASE(3, 16, 64, 1, 64, 2)
  GSIT_CASE(4, 16, 64, 1, 32, 3)
  GSIT_CASE(0, 8, 64, 4, 64, 2) GSIT_CASE(0, 16, 64, 2, 64, 2) GSIT_CASE(0, 32, 64, 1, 32, 2)
  GSIT_CASE(0, 64, 64, 1, 32, 2)
  GSIT_CASE(0, 8, 32, 2, 64, 2) GSIT_CASE(0, 16, 32, 1, 64, 2) GSIT_CASE(0, 32, 32, 1, 32, 2)
  GSIT_CASE(0, 8, 16, 1, 64, 2) GSIT_CASE(0, 16, 16, 1, 64, 2)
#undef GSIT_CASE
  return cudaErrorNotSupported;
}

cudaError_t launch_attn_bf16(const Geometry& g, const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v,
                             int64_t row_stride, __nv_bfloat16* out, float* lse, float scale, int* next_item, cudaStream_t st,
                             bool counter_cleared) {
  const AttnOperands op = {q, k, v, out, lse, g.allowed};
  return launch_attn_bf16_n(g, &op, 1, row_stride, scale, next_item, st, counter_cleared);
}

}  // namespace gsit
