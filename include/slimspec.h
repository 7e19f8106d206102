/*
 * slimspec.h -- C ABI of the B200 (sm_100a) SlimSpec draft LM-head library.
 *
 * The operation is the low-rank draft LM-head of the SlimSpec paper, Section 4.1:
 *     logits = W_up W_down h          (standard head: logits = W_full h)
 * written here with row vectors and the transposed weights
 *     A = W_down^T (d x r),  B = W_up^T (r x V),  W = W_full^T (d x V):
 *     z = h A   (rank-r code),   logits = z B          |   logits = h W
 * followed by the full-vocabulary softmax that Section 3.2 names, in its stable
 * logarithmic form, and the selection of the k most probable tokens per row:
 *     lse = max_v logit + log sum_v exp(logit - max),   logprob = logit - lse
 *     top-k ordered by (logit descending, token id ascending).
 *
 * Common conventions
 *   - Every matrix is dense, contiguous, row-major; weights and activations are bf16
 *     (passed as const void*), all accumulation is fp32, outputs are int32 / fp32.
 *       h[M][d]   A[d][r]   B[r][V]   W[d][V]   out_ids[M][k]   out_logprobs[M][k]
 *   - Unless a parameter says "host", pointers are DEVICE pointers on the device that was
 *     current when the context was created.  The caller owns every buffer; the library
 *     neither frees nor keeps them after the call's work has run.
 *   - Calls enqueue work on `stream` (a cudaStream_t passed as void*, NULL = the default
 *     stream) and return without synchronising, except where stated.  Calls on one
 *     context must not overlap on the GPU: a context owns one set of scratch buffers.
 *   - Stream order, and the one exception to it.  The activations h may be produced by
 *     whatever precedes the call in `stream`, the kernel directly before it included, and
 *     the outputs are complete for whatever follows it.  The WEIGHTS A, B, W must be final
 *     and visible to the device before the call is made: written by work that has completed
 *     (a stream or event synchronisation, or work in the stream that is not still running
 *     when the call's first kernel starts -- anything but the last kernel before the call
 *     qualifies, and so does a memcpy).  The kernels are launched with programmatic dependent
 *     launch and start reading weights while the kernel before the call may still be
 *     running; a kernel that rewrites weights directly before a call (a dequantisation, a
 *     weight swap) must be followed by an event or stream synchronisation.
 *   - The generic path (shapes the fast kernels do not take, or forced) keeps an M x V fp32
 *     buffer in the context for its top-k call and grows it on demand: such a call may
 *     allocate and synchronise the device.  The fast paths never do.
 *   - Return value: SLIMSPEC_OK or a negative status; nothing is launched on an argument
 *     error.  There is no CPU fallback: every step runs in CUDA kernels.
 *   - 1 <= k <= min(V, SLIMSPEC_MAX_K).  Inputs holding NaN or infinity give unspecified
 *     (but terminating) results.
 */
#ifndef SLIMSPEC_H
#define SLIMSPEC_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SLIMSPEC_MAX_K 64

/* status codes */
#define SLIMSPEC_OK 0
#define SLIMSPEC_ERR_NULL (-1)      /* a required pointer is NULL                              */
#define SLIMSPEC_ERR_DIM (-2)       /* a dimension is <= 0, k out of range, or beyond the ctx  */
#define SLIMSPEC_ERR_ALIGN (-3)     /* the forced path cannot take these shapes / alignments   */
#define SLIMSPEC_ERR_CUDA (-4)      /* a CUDA runtime call or a launch failed                  */
#define SLIMSPEC_ERR_TIMEOUT (-5)   /* a bounded device-side wait ran out (see last_error)     */
#define SLIMSPEC_ERR_NOMEM (-6)     /* device memory for scratch could not be allocated        */
#define SLIMSPEC_ERR_STATIC_LIMIT (-7) /* beyond the fixed scratch of slimspec_head_topk_static */

/* execution paths (slimspec_force_path) */
#define SLIMSPEC_PATH_AUTO 0        /* chosen per (M, shapes) from measured timings            */
#define SLIMSPEC_PATH_GENERIC 1     /* any shape; one thread per logit; slow                   */
#define SLIMSPEC_PATH_STREAM 2      /* split-V weight-streaming kernels (M <= 16 per launch)   */
#define SLIMSPEC_PATH_TENSOR 3      /* tcgen05 / TMEM tensor-core kernels (large M)            */

typedef struct slimspec_ctx slimspec_ctx;

/*
 * Create a context on the current device.  It owns the scratch the kernels need (the
 * fp32 code z, split-V partial max / sum-exp / top-k records, tickets, an error word),
 * sized for calls with M <= max_M, d and r <= max_d, V <= max_V, k <= max_k.
 * Allocates device memory (synchronising).  *out receives the context.
 */
int slimspec_create(slimspec_ctx** out, int max_M, int max_d, int max_V, int max_k);

/* Free the context's scratch.  Synchronises the device.  NULL is allowed. */
void slimspec_destroy(slimspec_ctx* ctx);

/* Force one execution path for later calls on this context (SLIMSPEC_PATH_*). */
int slimspec_force_path(slimspec_ctx* ctx, int path);

/* The path (SLIMSPEC_PATH_*, never AUTO) the last *_topk / *_logits call on ctx took. */
int slimspec_last_path(const slimspec_ctx* ctx);

/*
 * Low-rank draft head with fused log-softmax and top-k (Section 4.1, low-rank form;
 * softmax of Section 3.2).  The M x V logits are never written to memory.
 *   out_ids[m][j]      id of the j-th most probable token of row m (ties: lower id first)
 *   out_logprobs[m][j] its log-probability, logit - lse
 */
int slimspec_head_topk(slimspec_ctx* ctx, const void* h, const void* A, const void* B,
                       int M, int d, int r, int V, int k,
                       int32_t* out_ids, float* out_logprobs, void* stream);

/*
 * Same computation with host-side activations and results: copies h (M x d bf16, host;
 * pinned memory makes the copy asynchronous) to the device, runs slimspec_head_topk,
 * copies ids and log-probs back to the host buffers and waits for `stream`.
 * A and B stay device pointers: weights are resident.
 */
int slimspec_head_topk_host(slimspec_ctx* ctx, const void* h_host, const void* A, const void* B,
                            int M, int d, int r, int V, int k,
                            int32_t* out_ids_host, float* out_logprobs_host, void* stream);

/*
 * Low-rank draft head, raw logits (Section 4.1): out_logits[M][V] fp32 = (h A) B.
 */
int slimspec_head_logits(slimspec_ctx* ctx, const void* h, const void* A, const void* B,
                         int M, int d, int r, int V, float* out_logits, void* stream);

/*
 * Standard full-rank head (Section 4.1, logits = W_full h) with the same fused
 * log-softmax and top-k: the baseline every relative head cost in the paper is
 * normalised to.
 */
int fullhead_topk(slimspec_ctx* ctx, const void* h, const void* W,
                  int M, int d, int V, int k,
                  int32_t* out_ids, float* out_logprobs, void* stream);

/*
 * Synchronise the device and return the context's device-side error word:
 * SLIMSPEC_OK, or SLIMSPEC_ERR_TIMEOUT if a bounded wait inside a kernel gave up
 * (the outputs of that call are then invalid).  Clears the word.  Meant for tests.
 */
int slimspec_last_error(slimspec_ctx* ctx);

/* Number of kernels the library has launched on this context since it was created. */
long long slimspec_launch_count(const slimspec_ctx* ctx);

/*
 * Device timing of the dominant kernel (the one that streams B or W, on the streaming and
 * on the tensor-core path), for roofline reports.  While enabled, each *_topk / *_logits
 * call records a CUDA event on its stream directly before and after that kernel; the events
 * also keep it from overlapping its neighbours, so the figure is the kernel alone and calls
 * are slightly slower than with timing off.  Enabling resets the totals.
 * At most 256 launches are pending at a time; the call that records the 257th first waits
 * for the earlier ones.
 */
int slimspec_kernel_timing(slimspec_ctx* ctx, int enable);

/*
 * Wait for the timed kernels recorded so far and return their summed duration in
 * milliseconds and their number (both host pointers, both required).
 */
int slimspec_kernel_timing_read(slimspec_ctx* ctx, double* total_ms, long long* launches);

/*
 * The low-rank head with fused log-softmax / top-k for callers that cannot allocate device
 * memory.  (The paper has no counterpart: this entry point exists for deployment only; it
 * computes exactly what slimspec_head_topk computes on its streaming path.)
 *
 * Who needs it: code that runs where cudaMalloc / cudaFree are off limits -- inside a serving
 * loop whose memory pool already owns the whole device, in a plugin whose host runtime forbids
 * driver allocations on its worker threads, or in a latency-critical section that cannot take
 * the device-wide synchronisation an allocation implies.  This call needs no context and calls
 * no allocating routine: its scratch (the fp32 code z, the per-slab records, a ticket and an
 * error word, about 1.5 MB) is a fixed device array inside the library image, held by every
 * GPU that loads the library until the process exits.
 *
 * Limits, because that array has a fixed size: M <= SLIMSPEC_STATIC_MAX_M,
 * r <= SLIMSPEC_STATIC_MAX_R, k <= SLIMSPEC_STATIC_MAX_K; larger values return
 * SLIMSPEC_ERR_STATIC_LIMIT and launch nothing.  Shapes the streaming kernels do not take
 * (V not a multiple of 8, r not a multiple of 16, pointers not 16-byte aligned) return
 * SLIMSPEC_ERR_ALIGN.  h, A, B, out_ids, out_logprobs are device pointers with the layouts of
 * slimspec_head_topk; the work is enqueued on `stream` without synchronising.
 *
 * The first call on a device looks up the device address of the array and loads the kernels
 * (once per device, with that device current; loading is what may allocate, so it is done
 * there and not on later calls); make that first call before any stream capture begins.
 * All calls on a device share the one array, and it keeps the previous call's contents (the
 * call clears the words that must start at zero).  Two calls whose kernels overlap on the GPU
 * -- different streams, or several host threads -- race on it: serialise them.
 */
#define SLIMSPEC_STATIC_MAX_M 8
#define SLIMSPEC_STATIC_MAX_R 8192
#define SLIMSPEC_STATIC_MAX_K 32
int slimspec_head_topk_static(const void* h, const void* A, const void* B,
                              int M, int d, int r, int V, int k,
                              int32_t* out_ids, float* out_logprobs, void* stream);

/* Static description of a status code. */
const char* slimspec_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* SLIMSPEC_H */
