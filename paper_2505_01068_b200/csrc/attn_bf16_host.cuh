// Host side of the bf16 IM attention: tensor maps and launch (included by attn_bf16.cu only).
#pragma once

namespace gsit {
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// 2-D map over a [rows, d] bf16 view with row pitch `row_stride` elements; box = [CW columns, box_rows rows],
// shared-memory swizzle matched to the box width.  Out-of-range rows read as zero.
bool make_map(CUtensorMap* tm, const void* base, int64_t rows, int d, int64_t row_stride, int cw, int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (fn == nullptr) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)row_stride * 2};
  const cuuint32_t box[2] = {(cuuint32_t)cw, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUtensorMapSwizzle sw = (cw == 64) ? CU_TENSOR_MAP_SWIZZLE_128B
                                : (cw == 32) ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <typename C>
cudaError_t launch_one(const Geometry& g, const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v,
                       int64_t row_stride, __nv_bfloat16* out, float* lse, float scale, cudaStream_t st) {
  constexpr int CW = C::CW;
  const int64_t rows = (int64_t)g.batch * g.L;
  alignas(64) CUtensorMap tmQ, tmK, tmV;
  if (!make_map(&tmQ, q, rows, g.d, row_stride, CW, C::QT) || !make_map(&tmK, k, rows, g.d, row_stride, CW, KT) ||
      !make_map(&tmV, v, rows, g.d, row_stride, CW, KT))
    return cudaErrorInvalidValue;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(attn_bf16_kernel<C>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  int tiles = 0;
  for (int s = 0; s < 3; ++s) tiles += (g.seg_len[s] + C::QT - 1) / C::QT;
  const dim3 grid((unsigned)tiles, (unsigned)(g.d / CW), (unsigned)g.batch);
  const float sl2 = scale * 1.4426950408889634f;
  attn_bf16_kernel<C><<<grid, NTHREADS, C::SMEM, st>>>(tmQ, tmK, tmV, g, out, lse, sl2);
  return cudaGetLastError();
}

}  // namespace

int g_attn_variant = 0;  // 0 = default tile configuration per shape; 1.. = alternatives (tuning knob)

cudaError_t launch_attn_bf16(const Geometry& g, const __nv_bfloat16* q, const __nv_bfloat16* k,
                             const __nv_bfloat16* v, int64_t row_stride, __nv_bfloat16* out, float* lse,
                             float scale, cudaStream_t st) {
  if (g.batch > 65535 || g.d % 16 != 0) return cudaErrorNotSupported;
  const int cw = (g.d % 64 == 0) ? 64 : (g.d % 32 == 0) ? 32 : 16;
  const int var = g_attn_variant;
#define GSIT_CASE(VAR_, HD_, CW_, R_, KS_, MB_)         \
  if (g.hd == HD_ && cw == CW_ && (var == VAR_ || VAR_ == 0)) \
    return launch_one<Cfg<HD_, CW_, R_, KS_, MB_>>(g, q, k, v, row_stride, out, lse, scale, st);
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

}  // namespace gsit
