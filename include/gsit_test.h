/*
 * gsit_test.h -- hooks of libgsit.so for its tests, its benchmark and profilers.  None of them belongs to the method
 * (the paper has no counterpart for any of them): they select between kernel families that compute the same thing,
 * time the library's launches, and exercise the error path of the bounded device-side waits.  Host state only; a
 * program that uses the library for its results needs nothing from this header.
 */
#ifndef GSIT_TEST_H_
#define GSIT_TEST_H_

#include "gsit.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Kernel selection (process-wide host state; 0 restores the defaults).  Every choice computes the same result up to
 * floating-point summation order.
 *   GSIT_ATTN_DEFAULT   head_dim 64, 32, 16: tcgen05 / tensor-memory attention; head_dim 8: mma.sync attention;
 *                       layer at d_model 64 / 128: fused tcgen05 halves; linear layers: tcgen05 GEMM where it applies
 *   1 .. 7              the mma.sync attention with its n-th alternative tile configuration (where the shape has one)
 *   GSIT_ATTN_UNFUSED   the layer as separate LayerNorm / linear / attention kernels (padded layout only)
 *   GSIT_ATTN_LEGACY    the mma.sync family everywhere: attention, fused layer halves, linear layers (padded layout only)
 *   GSIT_ATTN_TMEM      the tensor-memory attention also at head_dim 8 */
typedef enum { GSIT_ATTN_DEFAULT = 0, GSIT_ATTN_UNFUSED = 8, GSIT_ATTN_LEGACY = 9, GSIT_ATTN_TMEM = 10 } gsit_kernel_choice;
gsit_status gsit_tune_attention(int choice);

/* Event timing of the library's launches (off by default).  While enabled, every kernel launch of the library is
 * bracketed by a pair of CUDA events on the launching stream (up to 8192 launches are kept; later ones go unrecorded).
 * Do not enable it while a stream is being captured into a CUDA graph. */
typedef enum { GSIT_KERNEL_ATTENTION = 0, GSIT_KERNEL_LINEAR = 1, GSIT_KERNEL_LAYERNORM = 2 } gsit_kernel_kind;
gsit_status gsit_trace_enable(int on);
/* Waits for the recorded events, returns the summed device time (ms) and launch count of one kernel kind since the
 * last gsit_trace_reset(); both outputs are HOST pointers. */
gsit_status gsit_trace_read(int kernel_kind, float* total_ms, int32_t* launches);
/* Per-launch device times (ms) of one kernel kind, in launch order, into out_ms[0..capacity); *launches receives
 * the number written.  HOST pointers. */
gsit_status gsit_trace_launches(int kernel_kind, float* out_ms, int32_t capacity, int32_t* launches);
gsit_status gsit_trace_reset(void);

/* Runs a one-CTA kernel whose only action is a bounded wait (the same routine the tcgen05 kernels wait with, limited to
 * 4096 polls) on a barrier that nothing will ever complete.  The wait runs out, the kernel raises GSIT_DEVFLAG_TIMEOUT
 * and returns normally: nothing traps, faults or spins without limit, and the context stays usable.  Afterwards
 * gsit_last_device_status() answers GSIT_ERR_TIMEOUT once and clears the flag.  Asynchronous on `stream`. */
gsit_status gsit_test_expire_wait(gsit_stream stream);

#ifdef __cplusplus
}
#endif
#endif /* GSIT_TEST_H_ */
