// Internal launch interface between the C-ABI layer (api.cu) and the kernel files.
// Every launcher only enqueues work on `st` and returns the cudaError_t of its launches.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace slimspec {

typedef __nv_bfloat16 bf16;

// One split-V partial record per (row, slab): running max, sum of exp(logit - max), and the
// slab's k best (logit, id) pairs in (logit desc, id asc) order.
// Layout in the context's scratch: float pm[P], ps[P], pv[P][k]; int pi[P][k] per row.
struct Scratch {
    float* z;            // fp32 code (or widened h): generic path [M][K]; one- and two-row streaming path: partial sums [splits][K][mt]
    uint32_t* zfrag;     // streaming path: the code, as fp32 or as tensor-core fragments (see stream.cu)
    bf16* zb;            // bf16 code [M][r] for the tensor-core path
    bf16* zb_lo;         // its rounding remainder (z - zb), bf16: used while the call is HBM-bound
    float* zpart;        // K-split partial tiles of the tensor-core down-projection
    size_t zpart_elems;
    uint32_t* smax;      // tensor path: per-row maxima of the sample tiles [64][M padded to 128]
    size_t smax_elems;
    uint32_t* thr0;      // tensor path: per-row starting bound of the top-k lists
    float* part;         // split-V partial records
    size_t part_elems;
    unsigned int* tickets;  // arrival counter: it only counts up
    unsigned int* ticket_base_host;   // host: what the counter will read when the next call starts; a launcher that takes tickets adds its CTAs
    uint2* zq;              // one- and two-row path: the code as published (value, call number) words; no other path writes here
    int* err;            // device error word
    float* logits;       // generic path only: M x V fp32, grown on demand
    size_t logits_elems;
    int max_parts;       // capacity of `part` in slabs per row
};

// ---- generic path (any shape) -------------------------------------------------------
cudaError_t generic_downproj(const bf16* h, const bf16* A, int M, int d, int r, float* z, cudaStream_t st);
cudaError_t generic_widen(const bf16* h, int n, float* z, cudaStream_t st);
cudaError_t generic_upproj(const float* z, const bf16* B, int M, int r, int V, float* logits, cudaStream_t st);
cudaError_t generic_softmax_topk(const float* logits, int M, int V, int k, int32_t* ids, float* logprobs,
                                 cudaStream_t st);

// ---- streaming path, one or two rows (stream_fma.cu) ------------------------------------
struct FmaPlan {
    int ok;          // 0: shapes not supported by this kernel
    int mt;          // rows per launch (1, 2 or 4)
    int ncta;        // V slabs = CTAs
    int launches;    // kernels per call
};
// r = 0: the full-rank head (the streamed matrix has d rows).
FmaPlan fma_plan(int M, int d, int r, int V, int k, int sm_count);
cudaError_t fma_prepare();
// The whole head for M <= 2 rows in one launch: z = h A (A null: z = h), logits = z B streamed once;
// mode 0: fused log-softmax/top-k into ids/logprobs, mode 1: raw logits out.  Uses s.zq
// (fma_code_words(max r) 8-byte words, zero before the first call, written by nothing else) and a call
// number `epoch` that differs from every earlier call's on this scratch and is never 0.
inline size_t fma_code_words(int max_r) { return (size_t)4 * max_r > 8192 ? (size_t)4 * max_r : 8192; }
cudaError_t fma_head(const bf16* h, const bf16* A, const bf16* B, int M, int mt, int d, int r, int V, int k, int mode,
                     int32_t* ids, float* logprobs, float* logits, const Scratch& s, unsigned int epoch, int sm_count,
                     cudaStream_t st);

// ---- streaming path, three to sixteen rows (stream.cu) -----------------------------------
struct StreamPlan {
    int ok;          // 0: shapes not supported by the streaming kernels
    int mt;          // rows the kernel keeps per launch (8 or 16)
    int ncta;        // V slabs = CTAs
    int parts;       // records per row the head kernel writes (slabs x column passes)
    int launches;    // kernels per row tile (for the launch counter)
};
// Once per device, before the first launch: loads the kernels and sets their shared-memory limits.
cudaError_t stream_prepare();
// K: contraction length of the streamed matrix (r, or d for the full-rank head).
StreamPlan stream_plan(int M, int K, int V, int k, int sm_count);
// Bytes of the code fragments for a streamed matrix of K rows (two parts: value and remainder).
size_t stream_code_bytes(int K);
// code = h A for M <= 16 rows, in the form the head kernel for these shapes reads; d even, r a multiple of 16.
cudaError_t stream_code(const bf16* h, const bf16* A, int M, int d, int r, int V, int k, uint32_t* code, int sm_count,
                        cudaStream_t st);
// z (bf16, [M][r]) = h A and, if z_lo is not null, its rounding remainder, for any M, on the same kernel:
// what the tensor-core path uses for small batches instead of a K-split tcgen05 product and a reduction.
cudaError_t stream_code_rows(const bf16* h, const bf16* A, int M, int d, int r, bf16* z, bf16* z_lo, int sm_count, cudaStream_t st);
// code = h itself (full-rank head: no down-projection).
cudaError_t stream_widen(const bf16* h, int M, int d, int V, int k, uint32_t* code, int sm_count, cudaStream_t st);
// logits = z B streamed once (M <= 16); mode 0: fused log-softmax/top-k into ids/logprobs, mode 1: raw logits out.
cudaError_t stream_head(const uint32_t* code, bool lowrank, const bf16* B, int M, int K, int V, int k, int mode,
                        int32_t* ids, float* logprobs, float* logits, const Scratch& s, int sm_count,
                        bool after_producer_kernel, int* launches, cudaStream_t st);

// ---- the merge of split-V records as a kernel of its own (tensor path; streaming path with many rows)
cudaError_t merge_records(const float* part, int M, int P, int RW, int k, int32_t* ids, float* logprobs, cudaStream_t st);

// ---- tensor-core path (larger M) ------------------------------------------------------
// Shapes the tcgen05 kernels take: K a multiple of 64, N a multiple of 8 and >= 64, k <= 32 in top-k mode.
bool tensor_ok(int M, int K, int N, int k, int mode);
// z (bf16 [M][r], in s.zb) = h A; with_low_part also writes s.zb_lo = bf16(z - zb).
cudaError_t tensor_downproj(const bf16* h, const bf16* A, int M, int d, int r, bool with_low_part, const Scratch& s,
                            int sm_count, int* launches, cudaStream_t st);
// X W with X bf16 [M][K], W bf16 [K][N]; mode 0: fused log-softmax / top-k, mode 1: raw fp32 logits.
// Xlo, if not null, is added to X inside the contraction (two MMAs per step).
// ev0 / ev1, if not null, are recorded directly before / after the kernel that streams W.
// tensor_records_fit: does the context's record scratch take this call?
bool tensor_records_fit(int M, int N, int k, const Scratch& s, int sm_count);
cudaError_t tensor_head(const bf16* X, const bf16* Xlo, const bf16* W, int M, int K, int N, int k, int mode, int32_t* ids,
                        float* logprobs, float* logits, const Scratch& s, int sm_count, int* launches,
                        cudaEvent_t ev0, cudaEvent_t ev1, cudaStream_t st);

}  // namespace slimspec
