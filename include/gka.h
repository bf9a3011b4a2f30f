/*
 * gka.h — C ABI of the B200 (sm_100a) Gated KalmaNet hot path.
 *
 * The library computes the chunk-wise gated online ridge regression of the GKA layer:
 * for every (batch, head) pair and token t
 *
 *     H_t = gamma_t H_{t-1} + k_t k_t^T          U_t = gamma_t U_{t-1} + v_t k_t^T
 *     x_t = CH(H_t + lambda_t I, q_t, n_iter)    o_t = U_t x_t
 *
 * (forward recurrence, eq. (CH), Section 4.1), where CH is the Chebyshev Iteration of
 * Algorithm 1 run for exactly n_iter matrix-vector products with eigenvalue bounds
 * L = ||H_t||_F + lambda_t, mu = lambda_t (Section 4.1, "Adaptive Regularization").
 * ||H_t||_F is evaluated per token inside each chunk from the chunk-initial state
 * (Section 4.2.1).  (Descriptions of the layer that speak of a memory M_t mean the paper's U_t.)
 * Optional per-token inputs in the descriptor: write strengths beta_t (beta_t k k^T, beta_t v k^T)
 * and alpha-connection weights alpha_t (o_t = U_t (alpha_t x_t + (1 - alpha_t) q_t)).
 *
 * Conventions shared by every call
 *   - All data pointers are DEVICE pointers, contiguous row-major; q, k, v, out and the states are 16-byte
 *     aligned, the per-token scalars (gate, lam, fro_out, beta, alpha) 4-byte aligned.
 *     The descriptor itself is a host struct.
 *   - q, k : [B, T, heads, d_k];  v, out : [B, T, heads, d_v];  gate, lam : [B, T, heads] float32.
 *     gate holds gamma_t in (0, 1]; lam holds lambda_t > 0 (absolute), or, with
 *     GKA_FLAG_ADAPTIVE_LAMBDA, the constant a of lambda_t = a ||H_t||_F (Section 4.1).
 *   - state / state_in / state_out : [B, heads, d_k*d_k + d_v*d_k] float32; per head first
 *     H (d_k x d_k, row-major) then U (d_v x d_k, row-major, U[i][j] = sum v_i k_j).
 *   - The caller owns every buffer.  The library allocates no device memory, keeps no state
 *     between calls apart from cached device attributes (and, for gka_fwd_chunked_host, two helper
 *     streams and a few events per device), and never synchronises: work is enqueued on
 *     desc->stream and the call returns.
 *   - Argument errors are reported by the return value before anything is launched.  Nothing
 *     throws or aborts.  Device-side waits are bounded; if one runs out the kernel stores
 *     GKA_ERR_TIMEOUT into *desc->device_status (when given), stops waiting and returns; the outputs
 *     and the states written by that call are then undefined (partly updated), the device stays usable.
 *   - Supported: d_k == d_v in {16, 32, 64, 128}; chunk == 64; any T >= 1 (a sequence is ceil(T / chunk) chunks, the
 *     last one holds the remaining T mod chunk tokens); n_iter >= 0.
 *   - bf16 I/O with GKA_PREC_NATIVE and T >= 16 runs on the tensor cores (tiles of 128 tokens x 128 channels; head
 *     dimension 64 is zero-extended on chip and skips the zero channels in the contractions over the channels, about
 *     0.83 of the time of 128); f32 I/O, GKA_PREC_HIGH, T < 16 and head dimensions 16 and
 *     32 run in fp32 arithmetic on the CUDA cores (16 and 32 zero-extended to 64 on chip in the chunked calls; the
 *     decode calls handle them with one warp per (sequence, head) pair).
 */
#ifndef GKA_H_
#define GKA_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    GKA_OK = 0,
    GKA_ERR_NULL = 1,        /* a required pointer is NULL                                   */
    GKA_ERR_SHAPE = 2,       /* non-positive size, d_k != d_v                                */
    GKA_ERR_DTYPE = 3,       /* unknown io_dtype / precision value                           */
    GKA_ERR_UNSUPPORTED = 4, /* a shape or mode outside the supported set                    */
    GKA_ERR_WORKSPACE = 5,   /* workspace missing, misaligned or smaller than required       */
    GKA_ERR_DOMAIN = 6,      /* written to *device_status by the validation pass (GKA_FLAG_VALIDATE): a gate outside
                                (0, 1], a lambda (or a) that is not positive, a negative beta, a non-finite value */
    GKA_ERR_CUDA = 7,        /* a CUDA runtime / driver call failed (launch, attribute, map) */
    GKA_ERR_TIMEOUT = 8,     /* written to *device_status by a kernel whose bounded wait ran out */
    GKA_ERR_ALIGN = 9        /* a data pointer is not aligned as required                    */
} gka_status;

typedef enum { GKA_F32 = 0, GKA_BF16 = 1 } gka_dtype;

typedef enum {
    GKA_PREC_NATIVE = 0, /* bf16 I/O: bf16 tensor-core operands, fp32 accumulation and masters;
                            f32 I/O: fp32 arithmetic throughout                               */
    GKA_PREC_HIGH = 1    /* fp32 arithmetic throughout, whatever the I/O dtype                */
} gka_precision;

enum {
    GKA_FLAG_ADAPTIVE_LAMBDA = 1u, /* lam[] holds a; lambda_t = a * ||H_t||_F (Section 4.1, eq. (4)) */
    GKA_FLAG_VALIDATE = 2u         /* one extra pass over gate, lam (beta, alpha) before the kernels: gamma_t in (0, 1]
                                      (Section 4.1, "Adaptive Weighting"), lambda_t > 0 so that L >= mu > 0 (input
                                      condition of Algorithm 1), beta_t >= 0, all finite; a violation stores
                                      GKA_ERR_DOMAIN into *device_status (which must be given and hold GKA_OK); the
                                      kernels run all the same */
};

typedef struct {
    int B;               /* batch (chunked forward) or number of sequences (decode)          */
    int T;               /* tokens per sequence; ignored by gka_decode_step                  */
    int heads;
    int d_k, d_v;
    int io_dtype;        /* gka_dtype of q, k, v, out                                         */
    int precision;       /* gka_precision                                                     */
    unsigned flags;      /* GKA_FLAG_*                                                        */
    void *stream;        /* cudaStream_t, caller-owned; NULL = default stream                 */
    void *workspace;     /* device scratch, >= gka_fwd_workspace_bytes(), 256-byte aligned    */
    size_t workspace_bytes;
    const float *state_in; /* optional initial state of the chunked forward; NULL = zero state */
    int *device_status;  /* optional device int, set by kernels on a bounded-wait timeout     */
    float *fro_out;      /* optional [B, T, heads] float32: ||H_t||_F per token (debug output) */
    void *profile_start; /* optional cudaEvent_t pair recorded on the stream right before and right after the    */
    void *profile_stop;  /* dominant kernel of the call (solve kernel / decode kernel): a forward call is several
                            kernels, so events of the caller cannot bracket one of them                          */
    const float *beta;   /* optional write strengths beta_t (device pointer): [B, T, heads] for the chunked
                            calls, [B, heads] for the decode step; H_t = gamma_t H_{t-1} + beta_t k_t k_t^T,
                            U_t = gamma_t U_{t-1} + beta_t v_t k_t^T (Remark "canonical beta_t-augmented
                            variant", Section 4.1).  NULL = 1, the recurrence of eq. (CH).  Must be >= 0. */
    const float *alpha;  /* optional alpha-connection weights alpha_t (device pointer, same shapes as beta): the
                            read becomes out_t = U_t (alpha_t x_t + (1 - alpha_t) q_t) (Section 4.3, "Architectural
                            Consideration").  NULL = 1.
                            Ignored by gka_solve_chunked.                                                     */
} gka_desc;

/*
 * Scratch the chunked forward needs for this descriptor: segment summaries and segment start
 * states of the cross-chunk state scan (one fp32 state per work segment) and, on the bf16
 * tensor-core path, the bf16 copies of the initial H and U of every 128-token tile plus its
 * ||H||_F^2 (64 KB + 4 B per tile; Section 4.2.1 stores the initial state of every chunk as well).
 * The fp32 path carries the states on chip and stores none per chunk.
 * Returns 0 if the descriptor is invalid.  Pure host arithmetic; no CUDA call.
 */
size_t gka_fwd_workspace_bytes(const gka_desc *desc, int chunk);

/*
 * Chunk-wise forward (eq. (CH) evaluated chunk by chunk, Section 4.2.1; Algorithm 1 on whole
 * chunks; chunk-wise Frobenius norms).  Writes out[B,T,heads,d_v] in io_dtype and, when
 * state_out != NULL, the final (H_T, U_T) of every (batch, head) pair.  out and state_out must
 * not alias any input.  Uses desc->workspace.  Returns GKA_OK once all kernels are enqueued.
 */
gka_status gka_fwd_chunked(const gka_desc *desc, const void *q, const void *k, const void *v,
                           const float *gate, const float *lam, int n_iter, int chunk,
                           void *out, float *state_out);

/*
 * The solve alone, chunk-wise: x_out[b,t,h,:] = CH(H_t + lambda_t I, rhs_t, n_iter) with H_t, lambda_t and the
 * bounds L, mu as in gka_fwd_chunked (Algorithm 1; H_t from k and gate only).  With rhs = q it returns the
 * iterate x_t that gka_fwd_chunked multiplies by U_t; with rhs = dL/dx_t it returns dL/dq_t, the first
 * step of the backward pass: the fixed-iteration Chebyshev map is linear in its right-hand side and
 * self-adjoint, so the gradient is the same solve with a different right-hand side (Section 4.2.2,
 * "Backward Pass", implicit differentiation, Lemma 2).  rhs, k, x_out : [B, T, heads, d_k] (d_v is ignored and must
 * equal d_k in the descriptor); gate, lam : [B, T, heads].  Same dtype rules, workspace, state_in (H part
 * used), flags and error behaviour as gka_fwd_chunked; no state is written.
 */
gka_status gka_solve_chunked(const gka_desc *desc, const void *rhs, const void *k, const float *gate,
                             const float *lam, int n_iter, int chunk, void *x_out);

/*
 * Recurrent single-token step (eq. (CH) applied once): state is read, decayed by gate, updated
 * with k k^T / v k^T and written back in place; out[B,heads,d_v] = U_t CH(H_t + lambda_t I, q_t).
 * q, k : [B, heads, d_k]; v, out : [B, heads, d_v]; gate, lam : [B, heads].  Needs no workspace.
 * The state written by gka_fwd_chunked(state_out) is a valid input here.
 */
gka_status gka_decode_step(const gka_desc *desc, float *state, const void *q, const void *k,
                           const void *v, const float *gate, const float *lam, int n_iter,
                           void *out);

/*
 * The recurrent step over desc->T >= 1 consecutive tokens per sequence (multi-token / speculative decoding):
 * token after token, exactly what desc->T calls of gka_decode_step compute (eq. (CH) per token), but the
 * state is read from and written to device memory once per call instead of once per token.
 * q, k : [B, T, heads, d_k]; v, out : [B, T, heads, d_v]; gate, lam (and desc->beta, desc->alpha when
 * given) : [B, T, heads]; state : [B, heads, 2*d*d] fp32, updated in place to the state after the last
 * token.  Needs no workspace.  Same dtype rules, flags and error behaviour as gka_decode_step.
 */
gka_status gka_decode_tokens(const gka_desc *desc, float *state, const void *q, const void *k,
                             const void *v, const float *gate, const float *lam, int n_iter,
                             void *out);

/*
 * Host-buffer form of the chunked forward (same operation, eq. (CH) chunk-wise): q, k, v, gate, lam,
 * out and state_out (nullable) are HOST pointers, preferably page-locked so that the copies are truly
 * asynchronous.  `staging` is caller-owned DEVICE memory of at least gka_fwd_host_staging_bytes()
 * bytes, 256-byte aligned; desc->workspace is required as for gka_fwd_chunked, desc->state_in (if
 * any, as well as beta / alpha) stays a device pointer.  The call enqueues host-to-device copies of the
 * five inputs, the forward kernels and device-to-host copies of out (and state_out), and does not
 * synchronise.  Sequences being independent, the batch is cut into up to 8 slices (and the sequences of the last
 * slice into two pieces of whole 128-token tiles, whose state is carried on the device, so that little work is
 * left when the last input byte has arrived) that pass through the
 * three stages on three streams (copies in and out on two helper streams the library creates once per
 * device, kernels on desc->stream), so both copy directions and the kernels overlap; work already on
 * desc->stream is waited for, and desc->stream waits for the last copy, so stream order is as if
 * everything ran on desc->stream.  The host buffers must stay valid and unmodified until the stream has
 * passed the call.
 */
size_t gka_fwd_host_staging_bytes(const gka_desc *desc);
gka_status gka_fwd_chunked_host(const gka_desc *desc, void *staging, const void *q, const void *k,
                                const void *v, const float *gate, const float *lam, int n_iter,
                                int chunk, void *out, float *state_out);

/*
 * Self-test of the bounded device-side waits (no counterpart in the paper; failure detection): one thread block polls,
 * at most `polls` times (1 .. 2^20), an mbarrier that nothing arrives at, with no copy or product outstanding, then
 * stores GKA_ERR_TIMEOUT into *desc->device_status (required) and returns.  Uses desc->stream and desc->device_status
 * only.  The device and the library stay fully usable afterwards.
 */
gka_status gka_selftest_bounded_wait(const gka_desc *desc, int polls);

/* Static, human-readable name of a status code. */
const char *gka_status_string(int status);

/*
 * Detail of the last GKA_ERR_CUDA returned to the calling thread (CUDA error name and text, and
 * which call raised it); an empty string if there was none.  The pointer stays valid for the thread.
 */
const char *gka_last_error_detail(void);

/*
 * Work decomposition of the chunked forward, for callers that size buffers or report launch
 * counts: number of work items (contiguous ranges of the flat chunk list) of the state pass for this
 * descriptor on the current device, or a negative gka_status.  Normally one per SM (fewer for small problems).
 * On the tensor-core path it is pairs / k for a small divisor k of the number of (sequence, head) pairs
 * (k = 1 with fewer pairs than SMs) whenever carrying whole sequences is cheaper than cutting them: no range then
 * starts or ends inside a sequence and no summary or scan kernel runs; with at most half as many work items as
 * SMs the state kernel then runs two thread blocks per work item, one per state matrix.
 */
int gka_fwd_num_work_items(const gka_desc *desc, int chunk);

/*
 * Introspection of the work decomposition (pure host arithmetic, no CUDA call): the flat list of
 * B*heads*ceil(T/chunk) chunks is split into num_items contiguous ranges; item `item` owns chunks
 * [*first_chunk, *end_chunk).  Range sizes differ by at most one chunk; when ceil(T/chunk) is even and
 * there are at least two chunks per item the boundaries are kept at even chunk offsets (the
 * tensor-core kernel works on pairs of chunks) and sizes differ by at most two.  *cut_in / *cut_out
 * tell whether the range starts / ends inside a sequence (then its start state comes from the
 * cross-item scan / its last run is summarised).  Returns GKA_OK or an argument error.
 */
gka_status gka_fwd_work_range(const gka_desc *desc, int chunk, int num_items, int item,
                              long long *first_chunk, long long *end_chunk, int *cut_in,
                              int *cut_out);

/*
 * Chunked forward without a caller workspace (the paper has no counterpart: this is a packaging
 * variant of gka_fwd_chunked for callers that cannot allocate).  Same arguments, same results and
 * same kernels as gka_fwd_chunked, but desc->workspace / workspace_bytes are ignored: the scratch of
 * the cross-chunk state scan is a fixed array of GKA_NOALLOC_SCRATCH_BYTES inside the library image
 * (resident in every CUDA context that loads the library until the context ends).
 *   - Calls no cudaMalloc / cudaFree and no allocating library routine.
 *   - Problems whose scan needs more than the array (gka_fwd_workspace_bytes(desc, chunk) >
 *     gka_noalloc_scratch_bytes()) are rejected with GKA_ERR_WORKSPACE before anything is launched:
 *     fp32 arithmetic: d_k <= 64 fits up to 170 chunks in total (B * heads * ceil(T / chunk)), d_k = 128 up to 42;
 *     bf16 tensor-core path (d_k = 64 or 128): up to 51 tiles of 128 tokens in total (B * heads * ceil(T / 128)).
 *   - The first call on a device looks up the array's device address (cudaGetSymbolAddress) with
 *     that device current; make that first call before any stream capture.
 *   - All calls on one device share the array.  Calls that overlap on the GPU race, whatever their
 *     streams; serialise them.  No part of the array has to be cleared between calls.
 */
#define GKA_NOALLOC_SCRATCH_BYTES (16u << 20)
gka_status gka_fwd_chunked_noalloc(const gka_desc *desc, const void *q, const void *k, const void *v,
                                   const float *gate, const float *lam, int n_iter, int chunk,
                                   void *out, float *state_out);
size_t gka_noalloc_scratch_bytes(void);

#ifdef __cplusplus
}
#endif
#endif /* GKA_H_ */
