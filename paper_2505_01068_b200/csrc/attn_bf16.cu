// bf16 IM attention for sm_100a: TMA-fed, register-resident online softmax on mma.sync tiles.
//
// Decomposition (paper, Section "Inner Decomposition for Efficiency"): a CTA owns one tile of query
// rows of one modality segment of one sample and walks only the key tiles of the segment(s) the
// Interlaced Mask opens for that block row, and only up to the sample's valid length.  Closed blocks
// and padded keys are never loaded, multiplied or exponentiated.
//
// Layout: a CTA covers a column slice of CW features (= CW/HD heads) so that one TMA box row is a whole
// 128-byte (or 64/32-byte) line shared by all heads of the slice; warp w works on head (w % G).  With
// head_dim 8 the tensor-core shapes fit exactly: S = Q K^T is mma.m16n8k8 (K = head_dim) and O += P V is
// mma.m16n8k16 (N = head_dim); the score accumulators are reused in registers as the A operand of P V.
#include <cuda.h>

#include "common.cuh"
#include "ptx.cuh"
#include "tensor_map.cuh"

namespace gsit {
namespace {

using namespace ptx;

constexpr int KT = 64;          // keys per pipeline stage
constexpr int STAGES = 3;
constexpr int NTHREADS = 256;   // 8 warps
constexpr int WAIT_SPINS = 1 << 20;

// HD = head_dim, CW = features per CTA column slice, R_ = 16-row query slabs per warp, KSTEP_ = keys per softmax
// step, MINB_ = CTAs per SM the register allocation must allow.
template <int HD_, int CW_, int R_, int KSTEP_, int MINB_>
struct Cfg {
  static constexpr int HD = HD_, CW = CW_, R = R_, KSTEP = KSTEP_, MINB = MINB_;
  static constexpr int G = CW / HD;                 // heads per column slice
  static constexpr int NSG = 8 / G;                 // slab groups (warps per head)
  static constexpr int QT = 16 * R * NSG;           // query rows per CTA
  static constexpr int PITCH = CW * 2;              // bytes per tile row
  static constexpr int SWZ = (CW == 64) ? 7 : (CW == 32) ? 3 : 1;  // swizzle mask (128B / 64B / 32B modes)
  static constexpr int NT = KSTEP / 8;              // score n-tiles per step
  static constexpr int KSQ = (HD == 8) ? 1 : HD / 16;  // k-steps of Q K^T
  static constexpr int NTO = HD / 8;                // output n-tiles
  static constexpr int Q_BYTES = QT * PITCH;
  static constexpr int KV_BYTES = KT * PITCH;
  static constexpr int SMEM = ((Q_BYTES + 1023) / 1024) * 1024 + 2 * STAGES * KV_BYTES + 1024 /*align slack*/ + 64 /*barriers*/;
  static_assert(G >= 1 && G <= 8 && QT <= 256 && (KSTEP == 32 || KSTEP == 64), "unsupported tile configuration");
};

// TMA shared-memory swizzle: 16-byte chunk index bits [4, 4+B) are XORed with address bits [7, 7+B).
template <int SWZ>
__device__ __forceinline__ uint32_t swz(uint32_t off) { return off ^ (((off >> 7) & SWZ) << 4); }

// Bounded wait: gives up after WAIT_SPINS polls, raises GSIT_DEVFLAG_TIMEOUT and lets the CTA run on
// (its results are then invalid, but nothing hangs).
__device__ __forceinline__ void mbar_wait(const Geometry& g, uint32_t bar, uint32_t parity) {
  for (int it = 0; it < WAIT_SPINS; ++it) {
    if (mbar_test(bar, parity)) return;
    if (it > 64) __nanosleep(64);
  }
  raise_flag(g, GSIT_DEVFLAG_TIMEOUT);
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x2(uint32_t addr, uint32_t& r0, uint32_t& r1) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_k16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                        uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_k8(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t b0) {
  asm("mma.sync.aligned.m16n8k8.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(b0));
}

}  // namespace
}  // namespace gsit

#include "attn_bf16_kernel.cuh"
#include "attn_bf16_host.cuh"
