/*
 * gsit.h -- C ABI of the Interlaced-Mask (IM) attention library for NVIDIA B200 (sm_100a).
 *
 * The library computes the attention of GsiT (arXiv 2505.01068): one set of query/key/value weights
 * is applied to the concatenation V_m = [V_0; V_1; V_2] of three modality sequences (Section
 * "Multimodal Transformers as Graphs"), and a 3x3 pattern of modality blocks -- the Interlaced Mask
 * of Section "All-Modal-In-One Fusion", Eq. IFM / IEM -- decides which query block may attend which
 * key block.  Only the open blocks are ever computed and the softmax runs over just their keys
 * (Section "Inner Decomposition for Efficiency"); a dense masked L x L product is never formed.
 *
 * General conventions
 *   - Segments are positional: s = 0,1,2 in the order the caller concatenated them, lengths
 *     seg_len[s], L = seg_len[0]+seg_len[1]+seg_len[2].
 *   - valid_len (DEVICE pointer, int32 [batch][3], or NULL = no padding) gives, per sample and segment,
 *     the number of real rows at the start of the segment; the rest of the segment is padding.
 *     Values outside [0, seg_len[s]] are clamped on the device and GSIT_DEVFLAG_CLAMPED is raised.
 *   - Padded rows of every output are exactly +0.0 (lse: -inf).  A real query whose open blocks hold no
 *     real key also yields +0.0 / -inf.  Contents of padded input rows (NaN and Inf included) never
 *     influence a real output row.
 *   - All tensors are row-major and live in DEVICE memory unless stated otherwise; the caller owns every
 *     buffer; the library allocates nothing, keeps no pointer after a call returns and launches all work
 *     asynchronously on the given stream without synchronising the host.
 *   - dtype GSIT_F32: activations and weights are float.  dtype GSIT_BF16: activations and weights are
 *     bfloat16, accumulation is float.  Biases, LayerNorm parameters, lse and the residual stream
 *     x / y of gsit_im_layer_fwd are float in both cases.
 *   - Errors are reported by return code only; nothing aborts, throws or traps.  Problems visible on the
 *     host (NULL pointers, bad sizes, unsupported shapes, misalignment, short workspace) are rejected
 *     before any launch.  There is no CPU fallback.
 *   - GSIT_BF16 needs: d_model % 16 == 0, head_dim in {8,16,32,64}, every row stride a multiple of 8
 *     elements, pointers 16-byte aligned.  GSIT_F32 needs head_dim <= 256.
 */
#ifndef GSIT_H_
#define GSIT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  GSIT_OK = 0,
  GSIT_ERR_INVALID_ARG = 1,  /* NULL pointer, non-positive size, d_model % heads != 0, bad enum, misalignment */
  GSIT_ERR_UNSUPPORTED = 2,  /* shape or dtype outside what the kernels cover */
  GSIT_ERR_WORKSPACE = 3,    /* workspace NULL or smaller than gsit_workspace_bytes() */
  GSIT_ERR_CUDA = 4,         /* a CUDA runtime / driver call failed */
  GSIT_ERR_TIMEOUT = 5       /* a bounded device-side wait expired (see gsit_last_device_status) */
} gsit_status;

typedef enum { GSIT_F32 = 0, GSIT_BF16 = 1 } gsit_dtype;

/* Which blocks are open.  Rows = query segment s, columns = key segment r.
 *   INTER_FWD: s attends (s+1)%3   -- M_inter^forward of Eq. IFM  (J O J / J J O / O J J)
 *   INTER_BWD: s attends (s+2)%3   -- M_inter^backward of Eq. IFM (J J O / O J J / J O J)
 *   INTRA:     s attends s         -- M_intra, the IEM            (O J J / J O J / J J O)
 *   CUSTOM:    bit (3*s + r) of custom_mask set = block open (ablation structures of Appendix
 *              "Graph Structures", the unmasked naive graph 0x1FF, ...).  With several open blocks in a
 *              block row the softmax runs over the union of their real keys. */
typedef enum {
  GSIT_PHASE_INTER_FWD = 0,
  GSIT_PHASE_INTER_BWD = 1,
  GSIT_PHASE_INTRA = 2,
  GSIT_PHASE_CUSTOM = 3
} gsit_phase;

/* Problem description shared by all calls.  HOST struct, passed by pointer, read during the call only. */
typedef struct gsit_shape {
  int32_t batch;            /* B >= 1 */
  int32_t seg_len[3];       /* each >= 0, sum >= 1 */
  int32_t d_model;          /* d = heads * head_dim */
  int32_t heads;            /* H */
  const int32_t* valid_len; /* DEVICE int32 [B][3] or NULL */
  int32_t dtype;            /* gsit_dtype */
  int32_t phase;            /* gsit_phase */
  uint32_t custom_mask;     /* used when phase == GSIT_PHASE_CUSTOM */
  float scale;              /* score scale; <= 0 selects 1/sqrt(head_dim) */
  /* Packed row layout (optional; NULL selects the padded [B, L] layout described with each call).  The paper's
   * Decomposition drops padded positions from the computation; in the packed layout they do not exist in memory
   * either: activations are [packed_capacity, d] matrices of real rows, segment s of sample b at rows
   * row_start[3 b + s] .. + valid_len[b][s] - 1.  row_start is a DEVICE int32 array of 3 B + 1 entries written by
   * gsit_plan_rows (entry 3 B = the row after the last one); valid_len must be given.  Accepted by
   * gsit_im_attention_fwd (bf16, every head_dim), gsit_im_layer_fwd (bf16, d_model 64 or 128) and gsit_im_qkv_proj
   * (bf16, d_model a multiple of 64); other calls and shapes answer GSIT_ERR_UNSUPPORTED.  A call on samples
   * b0 .. b1 - 1 passes valid_len + 3 b0 and row_start + 3 b0 with the same matrices (rows are absolute) and reads
   * and writes the rows of those samples only. */
  const int32_t* row_start;
  int32_t packed_capacity;  /* rows of the packed matrices (>= the plan's last entry rounded up to 128) */
} gsit_shape;

/* Weights of one IM encoder layer (HOST struct of DEVICE pointers).  Matrices are [out_features,
 * in_features] row-major in shape->dtype; y = x W^T.  Biases and LayerNorm vectors are float and may be
 * NULL (bias 0, gamma 1, beta 0). */
typedef struct gsit_layer_weights {
  const float* ln1_gamma; const float* ln1_beta;   /* [d] */
  const void* w_qkv;  const float* b_qkv;          /* [3d, d] rows = (W_q; W_k; W_v), [3d] */
  const void* w_o;    const float* b_o;            /* [d, d], [d] */
  const float* ln2_gamma; const float* ln2_beta;   /* [d] */
  const void* w_1;    const float* b_1;            /* [d_ff, d], [d_ff] */
  const void* w_2;    const float* b_2;            /* [d, d_ff], [d] */
  int32_t d_ff;                                    /* width of the MLP (the paper's d^p >= d^f) */
  float ln_eps;                                    /* <= 0 selects 1e-5 */
} gsit_layer_weights;

typedef void* gsit_stream; /* a cudaStream_t; NULL = the legacy default stream */

/* Shared QKV projection (Section "Multimodal Transformers as Graphs"; Appendix A, Eq. adjmat_all:
 * A = (W_q V_m)(W_k V_m)^T, i.e. one W_q, W_k, W_v for the whole concatenated sequence).
 *   x     [B, L, d]  row stride x_row_stride elements (>= d)
 *   w_qkv [3d, d], b_qkv float [3d] or NULL
 *   qkv   [B, L, 3, H, hd] contiguous: qkv[b,p,0] = q, [b,p,1] = k, [b,p,2] = v; padded rows = 0. */
gsit_status gsit_im_qkv_proj(const gsit_shape* shape, const void* x, int64_t x_row_stride, const void* w_qkv,
                             const float* b_qkv, void* qkv, gsit_stream stream);

/* IM attention (Eq. "All-Modal-In-One fusion": G = softmax(MHSA_1(V_m) + M), aggregation MHSA_2; computed
 * block-wise as Section "Inner Decomposition" and Appendix A "From Set to Set Aggregation" describe).
 *   q, k, v  [B, L, H, hd] views with a common row stride (elements) between sequence positions:
 *            d for three separate tensors, 3d for the fused buffer written by gsit_im_qkv_proj
 *   out      [B, L, d] contiguous, heads concatenated along features
 *   lse      float [B, H, L] or NULL: natural-log-sum-exp of the scaled scores of each row
 *   workspace / workspace_bytes: gsit_workspace_bytes(shape, GSIT_CALL_ATTENTION, 0) bytes, 4-byte aligned, or NULL / 0.
 *            Optional: given the scratch, the bf16 kernels hand their work items to the SMs through a counter kept there
 *            (cleared on `stream` by the call itself), which balances samples of different valid lengths; without it
 *            the items are assigned in a fixed round-robin order.  The result is the same either way.  Calls that may
 *            overlap in time need separate scratch. */
gsit_status gsit_im_attention_fwd(const gsit_shape* shape, const void* q, const void* k, const void* v,
                                  int64_t row_stride, void* out, float* lse, void* workspace,
                                  size_t workspace_bytes, gsit_stream stream);

/* One IM encoder layer, a = MLP o MHSA_2 (Eq. 1 / Eq. "All-Modal-In-One fusion"), in the pre-LayerNorm
 * form with residuals:   h = LN1(x); O = IM-attention(h W_qkv^T + b_qkv);
 *                        y1 = x + O W_o^T + b_o;   y = y1 + relu(LN2(y1) W_1^T + b_1) W_2^T + b_2.
 *   x  float [B, L, d] with row stride x_row_stride;  y  float [B, L, d] with row stride y_row_stride
 *      (strides let two encoders write the halves of one [B, L, 2d] buffer -- the feature concat of the
 *      fusion encoder pair).  x and y must not overlap.
 *   workspace: gsit_workspace_bytes(shape, GSIT_CALL_LAYER, d_ff) bytes, 256-byte aligned. */
gsit_status gsit_im_layer_fwd(const gsit_shape* shape, const gsit_layer_weights* weights, const float* x,
                              int64_t x_row_stride, float* y, int64_t y_row_stride, void* workspace,
                              size_t workspace_bytes, gsit_stream stream);

/* Two IM encoder layers of the same geometry in one call (Eq. "All-Modal-In-One fusion": the forward-ring and the
 * backward-ring fusion encoders have their own weights and share nothing until their outputs are put side by side, so
 * their layers of equal depth are two independent problems of one shape).  Computes exactly what two gsit_im_layer_fwd
 * calls compute, bit for bit; for bf16 at d_model 64 (d_ff <= 256) each of the layer's three kernels is launched once
 * for both problems -- every SM works for one of the two, one launch tail is paid instead of two and the result does not
 * depend on how two streams happen to interleave.  Other shapes run the two layers one after the other.
 *   shape_a / shape_b  must agree in everything (sizes, dtype, valid_len and row_start pointers, scale) except phase and
 *                      custom_mask; the two weight sets must have the same d_ff and ln_eps
 *   x_*, y_*           as for gsit_im_layer_fwd, one pair per problem (x_a and x_b may be the same tensor); no y may
 *                      overlap any x or the other y
 *   workspace          2 * gsit_workspace_bytes(shape_a, GSIT_CALL_LAYER, d_ff) bytes, 256-byte aligned */
gsit_status gsit_im_layer_pair_fwd(const gsit_shape* shape_a, const gsit_shape* shape_b, const gsit_layer_weights* weights_a,
                                   const gsit_layer_weights* weights_b, const float* x_a, int64_t x_a_row_stride, const float* x_b,
                                   int64_t x_b_row_stride, float* y_a, int64_t y_a_row_stride, float* y_b, int64_t y_b_row_stride,
                                   void* workspace, size_t workspace_bytes, gsit_stream stream);

/* Packed row layout, the three helpers (Section "Inner Decomposition for Efficiency": padded positions take no part in
 * the computation; here they take no memory either).  All run on the device, asynchronously on `stream`, and need no
 * host knowledge of the lengths, so a captured sequence of calls stays valid when valid_len changes.
 *
 * gsit_plan_rows: row_start[3 b + s] = running sum of the (clamped) valid lengths in the order (b, s), row_start[3 B] =
 *   their total.  If 0 < split_sample < B, the first row of sample split_sample is rounded up to a multiple of 128, so that
 *   the samples before and after it can be processed by separate calls (shape->batch and the valid_len / row_start
 *   pointers advanced) whose 128-row tiles do not touch each other's rows.
 *   shape: batch, seg_len, valid_len (required) are read.  row_start: DEVICE int32 [3 B + 1].
 * gsit_pack_rows: x_packed[row_start[3 b + s] + i, :] = x[b, seg_off[s] + i, :] for i < valid_len[b][s].
 * gsit_unpack_rows: the inverse; padded positions of y are written as +0.
 *   x / y float [B, L, cols] with the given row strides (elements); the packed matrices are float [capacity, cols].
 * A capacity of B * L + 128 rows always suffices. */
gsit_status gsit_plan_rows(const gsit_shape* shape, int32_t split_sample, int32_t* row_start, gsit_stream stream);
gsit_status gsit_pack_rows(const gsit_shape* shape, const float* x, int64_t x_row_stride, float* x_packed,
                           int64_t packed_row_stride, int32_t cols, gsit_stream stream);
gsit_status gsit_unpack_rows(const gsit_shape* shape, const float* y_packed, int64_t packed_row_stride, float* y,
                             int64_t y_row_stride, int32_t cols, gsit_stream stream);

/* Read-out of the fusion stack (Eq. "All-Modal-In-One fusion": X_m = f(|| Split(a(G_intra))[-1])): the encoder output is
 * split by the original modality lengths, the last time step of each modality is taken (with right padding inside a
 * segment: its last real step; an empty segment contributes zeros), the three vectors are concatenated and the linear
 * map f is applied.
 *   shape   batch, seg_len, valid_len and dtype are read (dtype = type of w_f); d_model, heads and phase are ignored
 *   c       float [B, L, d_c] with row stride c_row_stride elements (>= d_c): the intra encoder's output, d_c = 2 d
 *   w_f     [out_features, 3 * d_c] row-major in shape->dtype;  b_f float [out_features] or NULL
 *   out     float [B, out_features] contiguous
 * Needs 3 * d_c * 4 <= 48 KiB.  Errors as for the other calls. */
gsit_status gsit_stack_head_fwd(const gsit_shape* shape, const float* c, int64_t c_row_stride, int32_t d_c, const void* w_f,
                                const float* b_f, float* out, int32_t out_features, gsit_stream stream);

/* gsit_im_layer_fwd for callers that cannot allocate device memory (no counterpart in the paper; it computes
 * exactly what gsit_im_layer_fwd computes).  A host that lives inside someone else's memory budget, that must not
 * risk the implicit device synchronisation of an allocation in a latency-critical loop, or that runs after its
 * application has frozen all pools, cannot create the workspace gsit_im_layer_fwd asks for.  This variant takes
 * none: its scratch is a fixed array of GSIT_STATIC_SCRATCH_BYTES inside the library image, held by every GPU
 * that loads the library until the process exits.  The call itself allocates and frees nothing.
 *   - Arguments as for gsit_im_layer_fwd, without workspace / workspace_bytes; x, y and all weights are still the
 *     caller's device buffers.
 *   - Limit: gsit_workspace_bytes(shape, GSIT_CALL_LAYER, d_ff) must not exceed GSIT_STATIC_SCRATCH_BYTES;
 *     larger problems are rejected with GSIT_ERR_WORKSPACE before anything is launched (split the batch).
 *   - The first call on each GPU looks up the array's device address (that GPU must be current); make that
 *     first call before starting any stream capture.  The CUDA driver loads device arrays lazily, so it is also at
 *     this first call that the GPU's free memory drops by the array's size, once; later calls leave it unchanged.
 *   - All calls on a GPU share the one array, and it keeps the previous call's intermediates.  The layer
 *     writes every scratch row that contributes to a real output row before reading it, so nothing needs clearing
 *     (stale rows past the last real one may be read by a row tile; what is computed from them is discarded) -- but
 *     two calls that
 *     overlap in time on the same GPU (different streams, or different host threads) race on it and both
 *     results are then undefined.  Order them on one stream or with events. */
#define GSIT_STATIC_SCRATCH_BYTES (4u << 20)
gsit_status gsit_im_layer_fwd_static(const gsit_shape* shape, const gsit_layer_weights* weights, const float* x,
                                     int64_t x_row_stride, float* y, int64_t y_row_stride, gsit_stream stream);

typedef enum { GSIT_CALL_QKV_PROJ = 0, GSIT_CALL_ATTENTION = 1, GSIT_CALL_LAYER = 2 } gsit_call;

/* Scratch bytes the given call needs for this shape (d_ff is read for GSIT_CALL_LAYER only).
 * Returns 0 for calls that need none and (size_t)-1 for an invalid shape. */
size_t gsit_workspace_bytes(const gsit_shape* shape, int which_call, int32_t d_ff);

/* Device status flags, accumulated by kernels of this library on the current device. */
#define GSIT_DEVFLAG_CLAMPED 1u  /* a valid_len value was outside [0, seg_len] and was clamped */
#define GSIT_DEVFLAG_TIMEOUT 2u  /* a bounded wait on an asynchronous copy expired; results are invalid */

/* Synchronises `stream`, reads and clears the device status flags into *flags (HOST, may be NULL).
 * Returns GSIT_ERR_TIMEOUT if GSIT_DEVFLAG_TIMEOUT was set, GSIT_ERR_CUDA on a CUDA error, else GSIT_OK. */
gsit_status gsit_last_device_status(gsit_stream stream, uint32_t* flags);

const char* gsit_status_string(gsit_status status);
int gsit_version(void);

#ifdef __cplusplus
}
#endif
#endif /* GSIT_H_ */
