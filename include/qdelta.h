/*
 * qdelta.h -- C ABI of the B200 (sm_100a) Q-Delta library.
 *
 * Q-Delta (arXiv 2606.08804) evolves a d_k x d_v associative state per (batch, head):
 *
 *     x_t = k_t + lambda_t q_t                                   (Section 3.3.2, definition of x_t)
 *     S_t = alpha_t S_{t-1} (I - beta_t x_t k_t^T) + beta_t v_t k_t^T      (Section 3.3.1, final rule)
 *     o_t = S_t q_t
 *
 * This library keeps the state transposed, h_t = S_t^T in R^{d_k x d_v}, row-major, fp32:
 *
 *     h_t = alpha_t h_{t-1} + k_t (beta_t (v_t - alpha_t h_{t-1}^T x_t))^T ,   o_t = h_t^T q_t .
 *
 * Conventions that hold for every entry point
 *   - All tensor pointers are DEVICE pointers, dense and contiguous, token-major:
 *       q, k            [B, T, H, dk]          v, o, dO          [B, T, H, dv]
 *       beta, alpha, lambda (and their gradients) [B, T, H]
 *       states h0, hT, dhT, dh0                 [B, H, dk, dv]  fp32 always
 *     q,k,v,o,dO,dq,dk,dv,beta,alpha,lambda are stored in `dtype` (fp32 or bf16);
 *     dbeta,dalpha,dlambda and every state are fp32.
 *   - The caller owns every buffer, including the workspace whose size it queries.  The library
 *     never allocates, frees or synchronises; all work is enqueued on `stream`.
 *   - Ordering: a call reads its inputs only after everything enqueued on `stream` before the call has
 *     completed, and everything enqueued on `stream` after the call sees its outputs complete -- ordinary
 *     stream order.  (Internally the kernels of one call overlap their set-up with the tail of the kernel
 *     before them; none of them touches caller data, or workspace contents it depends on, before that
 *     kernel has completed.)  Work on OTHER streams needs events as usual.
 *   - Inputs are read-only.  Outputs are fully overwritten.  q,k,v,o,dO,dq,dk,dv, the
 *     states and the workspace must be 16-byte aligned; coefficient tensors (and the decode step's o)
 *     need only the alignment of their element type.
 *   - Coefficient domains: beta, lambda in [0,1], alpha in (0,1] (Section 3.3.1); not checked on device.
 *   - Return value: QD_OK, or an error code reported synchronously.  After a validation error (every code but
 *     QD_ERR_CUDA) nothing was enqueued; QD_ERR_CUDA means a CUDA call failed part-way, earlier kernels of the call may run.
 *     Conditions found on the device (a bounded wait that ran out) are written to the first
 *     32-bit word of the workspace and can be read with qdelta_workspace_status after the
 *     caller has synchronised the stream.
 *   - Supported shapes: chunk = 64, any T >= 1, dk and dv in {64, 128}.  A sequence length that is not a
 *     multiple of the chunk is completed, inside the library, with tokens that leave the recurrence
 *     untouched (beta = 0, alpha = 1); tensors are never read or written beyond their T rows.
 *     bf16 with dk = dv = 128 runs on the tensor cores (tcgen05); fp32, and bf16 with another head
 *     dimension, run on plain fp32 FMA kernels (qdelta_chunk_path tells which).
 */
#ifndef QDELTA_H_
#define QDELTA_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    QD_OK = 0,
    QD_ERR_INVALID_ARG = 1,   /* null required pointer, non-positive size, misaligned pointer, unknown flag */
    QD_ERR_UNSUPPORTED = 2,   /* (dk, dv, chunk, dtype) outside the supported set */
    QD_ERR_WORKSPACE = 3,     /* workspace null or smaller than qdelta_chunk_workspace_bytes */
    QD_ERR_CUDA = 4,          /* a CUDA runtime call (launch, attribute) failed */
    QD_ERR_TIMEOUT = 5,       /* device side: a bounded wait expired (see qdelta_workspace_status) */
    QD_ERR_STATIC_SCRATCH = 6 /* qdelta_chunk_fwd_static: the shape needs more than QDELTA_STATIC_SCRATCH_BYTES */
} qd_status;

typedef enum { QD_F32 = 0, QD_BF16 = 1 } qd_dtype;

/* flags of qdelta_chunk_fwd / qdelta_chunk_bwd */
enum {
    QD_FWD_SAVE_FOR_BWD = 1,  /* fwd: also keep the per-chunk states etc. in a backward-sized workspace */
    QD_BWD_REUSE_FWD = 2,     /* bwd: the workspace still holds what a QD_FWD_SAVE_FOR_BWD forward of the
                                 SAME inputs (and the same QD_COEF_LOGITS setting) left there; skip the recomputation */
    QD_COEF_LOGITS = 4,       /* fwd, bwd, qdelta_recurrent_steps: beta, alpha and lambda hold the pre-activation
                                 logits z of sigmoid gates (Appendix B: lambda = sigmoid(W h + b)); the kernels use
                                 sigmoid(z), computed in fp32, and the backward writes dbeta, dalpha, dlambda as
                                 derivatives with respect to the logits.  NULL alpha / lambda still mean 1 / 0. */
    QD_NORM_QK = 8,           /* fwd, bwd, qdelta_recurrent_steps: q and k are given un-normalised; the kernels use
                                 q / sqrt(|q|^2 + 1e-6) and k / sqrt(|k|^2 + 1e-6), per token and head (the L2
                                 normalisation that otherwise precedes the call), and the backward writes dq, dk as
                                 derivatives with respect to the un-normalised q, k.  A QD_BWD_REUSE_FWD backward must
                                 carry the same setting as its forward. */
    QD_STATE_BF16 = 16        /* qdelta_recurrent_steps only: `state` points to bf16 [B,H,dk,dv] instead of fp32 (half the
                                 bytes of a decode step).  The state is widened to fp32 when read, the S tokens of the
                                 call are applied in fp32, and it is rounded to bf16 once when written back.  This is
                                 a reduced-precision OPTION, not the method's fp32 state: every call adds a rounding of
                                 relative size 2^-9 to the state, which the forget gate damps by alpha per token; with
                                 alpha == 1 (no forgetting) the error grows like sqrt(calls) * 2^-9. */
};

typedef struct {
    int B, T, H;      /* batch, tokens per sequence, heads */
    int dk, dv;       /* key/query and value head dimensions */
    int chunk;        /* chunk length C of the chunkwise form; 64 */
    int dtype;        /* qd_dtype of q,k,v,beta,alpha,lambda,o,dO,dq,dk,dv */
} qd_shape;

typedef struct CUstream_st *qd_stream;   /* a cudaStream_t */

/* Which kernels serve `shape` (the paper has no counterpart; a query for tests and benchmarks):
 * 1 = tensor-core kernels, 0 = fp32 FMA kernels, -1 = invalid or unsupported shape. */
int qdelta_chunk_path(const qd_shape *shape);

/* Bytes of device workspace the chunkwise calls need for this shape (0 on invalid shape).
 * for_backward != 0: the size qdelta_chunk_bwd (and a QD_FWD_SAVE_FOR_BWD forward) needs. */
size_t qdelta_chunk_workspace_bytes(const qd_shape *shape, int for_backward);

/*
 * Chunkwise-parallel forward (Section 3.3.2: chunk expansion, extended WY representation,
 * UT transform, chunk-level state update and output).  The result equals the token-by-token
 * recurrence of Section 3.3.1 up to rounding:
 *     o   [B,T,H,dv]   o_t = h_t^T q_t           (read-out from the post-update state)
 *     hT  [B,H,dk,dv]  final state, fp32         (NULL: not returned)
 * alpha NULL means alpha == 1 (no forgetting); lambda NULL means lambda == 0 (the gated delta rule);
 * h0 NULL means a zero initial state.
 */
int qdelta_chunk_fwd(const qd_shape *shape,
                     const void *q, const void *k, const void *v,
                     const void *beta, const void *alpha, const void *lambda,
                     const float *h0, void *o, float *hT,
                     void *workspace, size_t workspace_bytes, unsigned flags, qd_stream stream);

/*
 * Backward of qdelta_chunk_fwd for the scalar  L = sum_t <o_t, dO_t> + <h_T, dhT>_F.
 * The paper prints no backward pass; this is the exact gradient of the chunk equations of
 * Section 3.3.2 (equivalently of the recurrence of Section 3.3.1).
 *     dq, dk [B,T,H,dk], dv [B,T,H,dv] in `dtype`;  dbeta, dalpha, dlambda [B,T,H] fp32;
 *     dh0 [B,H,dk,dv] fp32 (NULL: skipped).  dalpha is the derivative with respect to alpha itself.
 * dhT NULL means zero.  alpha / lambda / h0 NULL as in the forward (dalpha / dlambda are still
 * written when their pointers are non-NULL; they may be NULL only if the input was NULL).
 */
int qdelta_chunk_bwd(const qd_shape *shape,
                     const void *q, const void *k, const void *v,
                     const void *beta, const void *alpha, const void *lambda,
                     const float *h0, const void *dO, const float *dhT,
                     void *dq, void *dk, void *dv,
                     float *dbeta, float *dalpha, float *dlambda, float *dh0,
                     void *workspace, size_t workspace_bytes, unsigned flags, qd_stream stream);

/*
 * One token of the recurrence of Section 3.3.1 for B*H independent states, in place:
 *     state [B,H,dk,dv] fp32  h <- alpha h + k (beta (v - alpha h^T (k + lambda q)))^T
 *     o     [B,H,dv]          o = h_new^T q
 * q,k [B,H,dk], v [B,H,dv], beta/alpha/lambda [B,H] in `dtype` (alpha, lambda may be NULL).
 * `state` is the only in/out buffer.  Needs no workspace.
 */
int qdelta_recurrent_step(int B, int H, int dk, int dv, int dtype,
                          const void *q, const void *k, const void *v,
                          const void *beta, const void *alpha, const void *lambda,
                          float *state, void *o, qd_stream stream);

/*
 * S consecutive tokens of the same recurrence (Section 3.3.1) per call, for multi-token / speculative decoding: the
 * state is read once and written once for all S tokens instead of once per token.  Token tensors are token-major like
 * those of the chunkwise calls:
 *     q,k [B,S,H,dk]   v,o [B,S,H,dv]   beta/alpha/lambda [B,S,H]   (alpha, lambda may be NULL)
 *     state [B,H,dk,dv] fp32 (bf16 with QD_STATE_BF16), UPDATED IN PLACE to the state after the S-th token;
 *     o_s is read out after token s.
 * With an fp32 state the result is bit-identical to S calls of qdelta_recurrent_step.
 * flags: any of QD_COEF_LOGITS, QD_NORM_QK, QD_STATE_BF16.  S >= 1; for long runs of tokens (a prompt) use
 * qdelta_chunk_fwd with h0 / hT, which runs on the tensor cores.  Needs no workspace.
 */
int qdelta_recurrent_steps(int B, int S, int H, int dk, int dv, int dtype,
                           const void *q, const void *k, const void *v,
                           const void *beta, const void *alpha, const void *lambda,
                           void *state, void *o, unsigned flags, qd_stream stream);

/* Copies the device status word of `workspace` to *status_out (a qd_status) with a blocking
 * 4-byte device-to-host copy on `stream`.  Returns QD_OK or QD_ERR_CUDA / QD_ERR_INVALID_ARG. */
int qdelta_workspace_status(const void *workspace, int *status_out, qd_stream stream);

/*
 * Per-kernel timing aid for benchmarks (the paper has no counterpart).  While enabled, every kernel
 * the entry points enqueue is bracketed by two CUDA events recorded on the caller's stream;
 * qdelta_profile_read waits for the recorded events, adds their elapsed times to per-stage totals and
 * returns the total milliseconds and number of launches of `stage` (reset != 0 clears that total).
 * Stages are numbered 0 .. qdelta_profile_stage_count()-1; qdelta_profile_stage_name names them.
 * Events are created on first use and reused.  Not thread-safe; off by default.
 */
int qdelta_profile_enable(int on);
int qdelta_profile_stage_count(void);
const char *qdelta_profile_stage_name(int stage);
int qdelta_profile_read(int stage, double *total_ms, long long *launches, int reset);

/* Human-readable name of a qd_status. */
const char *qdelta_status_string(int status);

/* Size of the scratch array built into the library's device image for qdelta_chunk_fwd_static:
 * 32 MiB, enough for B*T*H <= 32768 token-heads at d_k = d_v = 128 in bf16 (one 2048-token prompt
 * with 16 heads). */
#define QDELTA_STATIC_SCRATCH_BYTES ((size_t)32 << 20)

/* Forward without a caller workspace and without any allocation.  The paper has no counterpart to
 * this call: it is a deployment convenience of this library, not part of the method.
 *
 * Computes exactly what qdelta_chunk_fwd computes with flags = 0 (same arguments, same layouts,
 * same kernels; o and hT as there), using a fixed scratch array of QDELTA_STATIC_SCRATCH_BYTES
 * that is part of the library's device image instead of a workspace.  Meant for callers that cannot
 * allocate device memory where the call is made (all HBM already handed to the caller's own pool,
 * or an allocation's device-wide synchronisation is not acceptable there).
 *
 *  - Performs no cudaMalloc/cudaFree and calls no allocating library routine.  Keep the timing aid
 *    (qdelta_profile_enable) off: it creates events.
 *  - The first call on each device looks up the array's address (and the driver may load the
 *    module then): make that first call, with that device current, before any stream capture.
 *  - Every call on a device shares the one array.  Calls that overlap in time race on it; issue
 *    them on one stream or otherwise serialise them.  The call itself clears the status word, the
 *    only part of the array that must start at zero.
 *  - Shapes whose forward workspace (qdelta_chunk_workspace_bytes(shape, 0)) exceeds
 *    QDELTA_STATIC_SCRATCH_BYTES are rejected with QD_ERR_STATIC_SCRATCH before anything is enqueued.
 *  - status_out: optional DEVICE pointer to one 32-bit word (4-byte aligned); after the kernels, the
 *    device status word (0, or QD_ERR_TIMEOUT if a bounded wait ran out) is copied there on `stream`.
 *  - All other pointers are device pointers with the meaning, layout and ownership documented at
 *    qdelta_chunk_fwd; errors as there.  Not saved for backward: use qdelta_chunk_fwd for training. */
int qdelta_chunk_fwd_static(const qd_shape *shape, const void *q, const void *k, const void *v,
                            const void *beta, const void *alpha, const void *lambda, const float *h0,
                            void *o, float *hT, unsigned *status_out, qd_stream stream);

#ifdef __cplusplus
}
#endif
#endif /* QDELTA_H_ */
