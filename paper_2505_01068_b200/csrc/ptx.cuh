// Thin wrappers around the sm_100a PTX that the TMA / tcgen05 kernels of this library share: mbarriers with bounded
// waits, bulk tensor copies, tcgen05.mma with shared-memory and tensor-memory operands, descriptors, small conversions.
#pragma once
#include <cuda.h>
#include <stdint.h>

#include "gsit.h"

namespace gsit {
namespace ptx {

// ---------------------------------------------------------------- mbarriers
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_init_fence() {  // makes freshly initialised barriers visible to the async proxy
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// One poll of a phase; the hardware may park the thread for a short, bounded time before answering.
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// One poll that lets the hardware park the thread for up to `ns` nanoseconds (it wakes as soon as the phase completes):
// for roles that wait long, so that their polling does not take issue slots from the warps that compute.
__device__ __forceinline__ bool mbar_try_park(uint32_t bar, uint32_t parity, uint32_t ns) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity), "r"(ns) : "memory");
  return ok != 0;
}
// One poll that never parks the thread.
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}

// Where a CTA records that one of its waits has run out: the device-wide status word (read by the host) and a word in the
// CTA's own shared memory (read by the CTA's other waits, so that a broken pipeline drains in a few polls per wait instead
// of one full limit per wait).  The shared word is cleared at kernel start, so a flag left in the device-wide word by an
// earlier launch cannot make a healthy launch give up.
struct WaitCtx {
  unsigned int* status;  // device status word (GSIT_DEVFLAG_* bits)
  uint32_t gave_up;      // shared-memory address of the CTA's "a wait expired" word
};
__device__ __forceinline__ bool cta_gave_up(const WaitCtx& w) {
  uint32_t v;
  asm volatile("ld.volatile.shared.u32 %0, [%1];" : "=r"(v) : "r"(w.gave_up) : "memory");
  return v != 0;
}
// Bounded wait on a barrier phase.  Returns true when the phase completed; false after `limit` polls (the timeout flag is
// raised) or as soon as another wait of this CTA has expired.  The caller carries on either way and must still release
// whatever it holds.
__device__ __forceinline__ bool mbar_wait(const WaitCtx& w, uint32_t bar, uint32_t parity, int limit = 1 << 16) {
  for (int it = 0; it < limit; ++it) {
    if (mbar_try(bar, parity)) return true;
    if ((it & 63) == 63 && cta_gave_up(w)) return false;
  }
  asm volatile("st.volatile.shared.u32 [%0], %1;" ::"r"(w.gave_up), "r"(1u) : "memory");
  atomicOr(w.status, GSIT_DEVFLAG_TIMEOUT);
  return false;
}

// The same with parked polls of up to ten microseconds each (2^15 of them at most: a third of a second).
__device__ __forceinline__ bool mbar_wait_parked(const WaitCtx& w, uint32_t bar, uint32_t parity, int limit = 1 << 15) {
  for (int it = 0; it < limit; ++it) {
    if (mbar_try_park(bar, parity, 10000u)) return true;
    if ((it & 15) == 15 && cta_gave_up(w)) return false;
  }
  asm volatile("st.volatile.shared.u32 [%0], %1;" ::"r"(w.gave_up), "r"(1u) : "memory");
  atomicOr(w.status, GSIT_DEVFLAG_TIMEOUT);
  return false;
}

// Bounded wait that sleeps between polls.  A try_wait that fails comes back within tens of clocks, so a warp that waits
// by polling alone keeps issuing instructions; with several waiting warps per scheduler that takes most of the issue
// slots from the warps that compute.  Here a poll never parks (test_wait) and is followed by a sleep of about `ns`
// nanoseconds during which the warp issues nothing.  Gives up after `limit` polls like mbar_wait.
__device__ __forceinline__ bool mbar_wait_sleep(const WaitCtx& w, uint32_t bar, uint32_t parity, unsigned ns, int limit = 1 << 17) {
  for (int it = 0; it < limit; ++it) {
    if (mbar_test(bar, parity)) return true;
    if (ns) __nanosleep(ns);
    if ((it & 63) == 63 && cta_gave_up(w)) return false;
  }
  asm volatile("st.volatile.shared.u32 [%0], %1;" ::"r"(w.gave_up), "r"(1u) : "memory");
  atomicOr(w.status, GSIT_DEVFLAG_TIMEOUT);
  return false;
}

// Arrival that counts for `count` participants (a warp arriving on behalf of warps that have nothing to contribute).
__device__ __forceinline__ void mbar_arrive_n(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
// Bounded wait that spins on non-parking polls: the shortest hand-over latency, at the price of issue slots.
__device__ __forceinline__ bool mbar_wait_spin(const WaitCtx& w, uint32_t bar, uint32_t parity, int limit = 1 << 22) {
  for (int it = 0; it < limit; ++it) {
    if (mbar_test(bar, parity)) return true;
    if ((it & 1023) == 1023 && cta_gave_up(w)) return false;
  }
  asm volatile("st.volatile.shared.u32 [%0], %1;" ::"r"(w.gave_up), "r"(1u) : "memory");
  atomicOr(w.status, GSIT_DEVFLAG_TIMEOUT);
  return false;
}

// ---------------------------------------------------------------- TMA
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* tm, uint32_t src, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
               ::"l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(src) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// True in exactly one lane of a converged warp.  Whole warps run the producer / issuer loops so that addresses,
// descriptors and barrier phases stay warp-uniform; only the asynchronous instruction itself is issued by one lane.
// Between reading a shared-memory buffer into registers and releasing that buffer for an asynchronous refill.  The
// loaded values need not be used before the release, and nothing else keeps the loads from being performed after it (the
// release is one lane's mbarrier arrive behind a warp barrier); measured: without this fence the last 16-byte load of a
// row was served from the refilled buffer in about 3 % of repeated full-batch runs of the pipelined out-projection + MLP.
__device__ __forceinline__ void fence_reads_before_release() { asm volatile("fence.acq_rel.cta;" ::: "memory"); }

// Programmatic dependent launch.  A kernel launched with the "programmatic stream serialization" attribute may start
// while the kernel before it in the stream is still running; grid_dep_wait() blocks until that kernel has completed and
// its writes are visible (a no-op for an ordinary launch), so everything above it -- barrier set-up, TMEM allocation,
// loads of weights -- overlaps the predecessor's tail.  Every kernel launched that way calls it, in every thread, before
// its first access to memory an earlier kernel of the stream wrote or read: completion then chains through the stream.
// grid_dep_launch() lets the next kernel's CTAs be placed as soon as every CTA of this one has called it (or exited).
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred != 0;
}

// ---------------------------------------------------------------- tcgen05
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor for tiles whose rows are 128 bytes with the 128-byte swizzle (what TMA wrote):
// groups of 8 rows are 1024 bytes apart (stride byte offset); the leading byte offset is unused for these shapes.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)(1024u >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// Descriptor of a K-major operand without swizzle: 8-row x 16-byte core matrices of 128 contiguous bytes; `sbo` bytes
// between core matrices along the rows, `lbo` bytes between the two core matrices that make up one K step of 16.
__device__ __forceinline__ uint64_t smem_desc_plain(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)((sbo >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}
// Instruction descriptor, kind::f16: D = f32, A = B = bf16, M = 128, N = n; b_mn_major: B is stored N-contiguous.
__host__ __device__ constexpr uint32_t idesc_bf16(int n, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(128 >> 4) << 24);
}
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
// Makes the barrier complete once every tcgen05.mma issued so far by this thread has finished.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem, uint32_t cols) {  // whole warp
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t tmem, uint32_t cols) {  // whole warp
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(cols) : "memory");
}

// ---------------------------------------------------------------- arithmetic
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// 2^x for a pair of arguments on the FMA and integer pipes instead of the special-function unit: x = n + f with n the
// nearest integer (taken from the low mantissa bits of x + 1.5 * 2^23) and |f| <= 1/2, 2^f by a cubic with relative
// error 7.6e-5 (well below the 2^-9 of the bf16 rounding that follows), n added into the exponent field.  Arguments
// are clamped at -126 (the result then flushes towards 2^-126 instead of wrapping); valid up to x < 128.
__device__ __forceinline__ float2 ex2_poly2(float2 x) {
  x.x = fmaxf(x.x, -126.f);
  x.y = fmaxf(x.y, -126.f);
  const float2 t = __fadd2_rn(x, make_float2(12582912.f, 12582912.f));
  const float2 n = __fadd2_rn(t, make_float2(-12582912.f, -12582912.f));
  const float2 f = __ffma2_rn(n, make_float2(-1.f, -1.f), x);
  float2 p = __ffma2_rn(make_float2(0.055205505f, 0.055205505f), f, make_float2(0.24261397f, 0.24261397f));
  p = __ffma2_rn(p, f, make_float2(0.69325477f, 0.69325477f));
  p = __ffma2_rn(p, f, make_float2(0.9999277f, 0.9999277f));
  return make_float2(__int_as_float(__float_as_int(p.x) + (__float_as_int(t.x) << 23)),
                     __int_as_float(__float_as_int(p.y) + (__float_as_int(t.y) << 23)));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
// The same conversion with negative values clamped to zero first (ReLU for free in the pack instruction).
__device__ __forceinline__ uint32_t pack_bf16_relu(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.relu.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float y;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(y) : "f"(a), "f"(b), "f"(c));
  return y;
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

}  // namespace ptx
}  // namespace gsit
