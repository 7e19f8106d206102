// C-ABI layer: context, argument checks, path choice.  See include/slimspec.h for the contract.
#include "../../include/slimspec.h"
#include "kernels.h"
#include <new>
#include <stdlib.h>
#include <string.h>

using namespace slimspec;

struct slimspec_ctx {
    int device;
    int sm_count;
    int max_M, max_d, max_V, max_k;
    int forced_path;
    int last_path;
    long long launches;
    unsigned int ticket_base;   // what the arrival counter will read when the next call starts
    unsigned int epoch;   // number of the last one- or two-row call (the code it publishes carries it)
    Scratch s;
    bf16* h_stage;        // device copy of host activations (head_topk_host)
    // Results of head_topk_host: pinned host memory mapped into the device, so the kernels write
    // them straight to the host (80 bytes at M = 1) and no device-to-host copy is enqueued.
    void* res_host;       // host address of the mapping: ids, then log-probs
    size_t res_half;      // bytes from the ids to the log-probs
    int32_t* ids_stage;   // device addresses of the same memory
    float* lp_stage;
    // optional device timing of the kernel that streams the weight matrix
    int timing_on;
    int timing_used;                 // event pairs recorded and not yet read
    cudaEvent_t* ev0;
    cudaEvent_t* ev1;
    double timing_ms;                // accumulated
    long long timing_launches;
};
static const int kTimingEvents = 256;

static const int kMaxParts = 320;      // most split-V records any kernel writes per row
static const int kStreamMaxRows = 16;  // largest M the streaming path is chosen for
static const int kSplitCodeRows = 256;  // tensor path: z carried as hi + lo bf16 parts while the call is HBM-bound (up to this many rows)
static const int kRowPad = 8;          // rows of the generic path's fp32 code are padded to this
static const int kStreamTile = 16;     // rows one launch of the streaming kernels takes
static const int kCodeByStreamRows = 32;   // tensor path: up to this many rows z comes from the streaming path's down-projection

static int round_up(int x, int m) { return (x + m - 1) / m * m; }

extern "C" const char* slimspec_strerror(int status)
{
    switch (status) {
    case SLIMSPEC_OK: return "ok";
    case SLIMSPEC_ERR_NULL: return "null pointer argument";
    case SLIMSPEC_ERR_DIM: return "dimension out of range (<= 0, k > min(V, 64), or beyond the context's limits)";
    case SLIMSPEC_ERR_ALIGN: return "forced path does not support these shapes or alignments";
    case SLIMSPEC_ERR_CUDA: return "CUDA runtime or launch error";
    case SLIMSPEC_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case SLIMSPEC_ERR_NOMEM: return "out of device memory for scratch";
    case SLIMSPEC_ERR_STATIC_LIMIT: return "M, r or k beyond the fixed scratch of slimspec_head_topk_static (8 rows, r 8192, k 32)";
    default: return "unknown status";
    }
}

extern "C" int slimspec_create(slimspec_ctx** out, int max_M, int max_d, int max_V, int max_k)
{
    if (!out) return SLIMSPEC_ERR_NULL;
    *out = nullptr;
    if (max_M <= 0 || max_d <= 0 || max_V <= 0 || max_k <= 0 || max_k > SLIMSPEC_MAX_K) return SLIMSPEC_ERR_DIM;
    slimspec_ctx* c = new (std::nothrow) slimspec_ctx;
    if (!c) return SLIMSPEC_ERR_NOMEM;
    memset(c, 0, sizeof(*c));
    cudaDeviceProp prop;
    if (cudaGetDevice(&c->device) != cudaSuccess || cudaGetDeviceProperties(&prop, c->device) != cudaSuccess) {
        delete c;
        return SLIMSPEC_ERR_CUDA;
    }
    c->sm_count = prop.multiProcessorCount;
    c->max_M = max_M; c->max_d = max_d; c->max_V = max_V; c->max_k = max_k;
    c->s.max_parts = kMaxParts;
    c->s.ticket_base_host = &c->ticket_base;
    const size_t mpad = (size_t)round_up(max_M, kRowPad);
    const size_t z_elems = mpad * (size_t)max_d;
    // split-V records, padded to 16 bytes: the streaming path writes <= 16 rows x 320 records, the
    // tensor path 128 * nrb rows x (SMs / nrb) slabs
    const int rec_k = max_k < 32 ? max_k : 32;
    const size_t mpad128 = (size_t)round_up(max_M, 128);
    const size_t part_elems = ((size_t)kStreamTile * kMaxParts + (size_t)(c->sm_count + 12) * 256 + 2 * mpad128) *
                              (size_t)round_up(2 + 2 * rec_k, 4);
    // K-split partial tiles of the tensor-core down-projection: one 128 x 128 fp32 tile per SM, or one split
    size_t zpart_elems = (size_t)(c->sm_count + 12) * 128 * 128;
    if (zpart_elems < mpad128 * (size_t)max_d) zpart_elems = mpad128 * (size_t)max_d;
    bool ok = true;
    ok = ok && cudaMalloc(&c->s.z, z_elems * sizeof(float)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->s.part, part_elems * sizeof(float)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->s.zfrag, stream_code_bytes(max_d)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->s.zq, fma_code_words(max_d) * sizeof(uint2)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->s.zpart, zpart_elems * sizeof(float)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->s.zb, 2 * mpad128 * (size_t)max_d * sizeof(bf16)) == cudaSuccess;
    if (ok) c->s.zb_lo = c->s.zb + mpad128 * (size_t)max_d;
    ok = ok && cudaMalloc(&c->s.smax, 64 * mpad128 * sizeof(uint32_t)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->s.thr0, mpad128 * sizeof(uint32_t)) == cudaSuccess;
    c->s.smax_elems = 64 * mpad128;
    c->s.part_elems = part_elems;
    c->s.zpart_elems = zpart_elems;
    ok = ok && cudaMalloc(&c->s.tickets, 4096 * sizeof(unsigned int)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->s.err, sizeof(int)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->h_stage, (size_t)max_M * max_d * sizeof(bf16)) == cudaSuccess;
    {
        const size_t half = ((size_t)max_M * max_k * sizeof(int32_t) + 255) / 256 * 256;
        void* dev_view = nullptr;
        ok = ok && cudaHostAlloc(&c->res_host, 2 * half, cudaHostAllocMapped) == cudaSuccess;
        ok = ok && cudaHostGetDevicePointer(&dev_view, c->res_host, 0) == cudaSuccess;
        if (ok) {
            c->ids_stage = reinterpret_cast<int32_t*>(dev_view);
            c->lp_stage = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(dev_view) + half);
            c->res_half = half;
        }
    }
    ok = ok && cudaMemset(c->s.tickets, 0, 4096 * sizeof(unsigned int)) == cudaSuccess;
    ok = ok && cudaMemset(c->s.err, 0, sizeof(int)) == cudaSuccess;
    ok = ok && cudaMemset(c->s.zq, 0, fma_code_words(max_d) * sizeof(uint2)) == cudaSuccess;
    ok = ok && cudaMemset(c->s.z, 0, z_elems * sizeof(float)) == cudaSuccess;
    ok = ok && stream_prepare() == cudaSuccess && fma_prepare() == cudaSuccess;
    ok = ok && cudaDeviceSynchronize() == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        slimspec_destroy(c);
        return SLIMSPEC_ERR_NOMEM;
    }
    *out = c;
    return SLIMSPEC_OK;
}

extern "C" void slimspec_destroy(slimspec_ctx* c)
{
    if (!c) return;
    cudaDeviceSynchronize();
    cudaFree(c->s.z); cudaFree(c->s.zfrag); cudaFree(c->s.zq); cudaFree(c->s.part); cudaFree(c->s.zpart); cudaFree(c->s.zb); cudaFree(c->s.smax); cudaFree(c->s.thr0); cudaFree(c->s.tickets); cudaFree(c->s.err);
    cudaFree(c->s.logits); cudaFree(c->h_stage);
    if (c->res_host) cudaFreeHost(c->res_host);
    if (c->ev0) {
        for (int i = 0; i < kTimingEvents; ++i) { cudaEventDestroy(c->ev0[i]); cudaEventDestroy(c->ev1[i]); }
        delete[] c->ev0;
        delete[] c->ev1;
    }
    delete c;
}

extern "C" int slimspec_force_path(slimspec_ctx* c, int path)
{
    if (!c) return SLIMSPEC_ERR_NULL;
    if (path < SLIMSPEC_PATH_AUTO || path > SLIMSPEC_PATH_TENSOR) return SLIMSPEC_ERR_DIM;
    c->forced_path = path;
    return SLIMSPEC_OK;
}

extern "C" int slimspec_last_path(const slimspec_ctx* c) { return c ? c->last_path : SLIMSPEC_ERR_NULL; }

extern "C" long long slimspec_launch_count(const slimspec_ctx* c) { return c ? c->launches : 0; }

extern "C" int slimspec_last_error(slimspec_ctx* c)
{
    if (!c) return SLIMSPEC_ERR_NULL;
    int e = 0;
    if (cudaDeviceSynchronize() != cudaSuccess) return SLIMSPEC_ERR_CUDA;
    if (cudaMemcpy(&e, c->s.err, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return SLIMSPEC_ERR_CUDA;
    if (e != 0) {
        cudaMemset(c->s.err, 0, sizeof(int));
        // tickets may have been left mid-count by the kernel that gave up
        cudaMemset(c->s.tickets, 0, 4096 * sizeof(unsigned int));
        c->ticket_base = 0;
        return SLIMSPEC_ERR_TIMEOUT;
    }
    return SLIMSPEC_OK;
}

// Fold the recorded event pairs into the totals; waits for the last recorded kernel.
static int timing_drain(slimspec_ctx* c)
{
    for (int i = 0; i < c->timing_used; ++i) {
        float ms = 0.f;
        if (cudaEventSynchronize(c->ev1[i]) != cudaSuccess ||
            cudaEventElapsedTime(&ms, c->ev0[i], c->ev1[i]) != cudaSuccess) {
            cudaGetLastError();
            c->timing_used = 0;
            return SLIMSPEC_ERR_CUDA;
        }
        c->timing_ms += ms;
        c->timing_launches += 1;
    }
    c->timing_used = 0;
    return SLIMSPEC_OK;
}

extern "C" int slimspec_kernel_timing(slimspec_ctx* c, int enable)
{
    if (!c) return SLIMSPEC_ERR_NULL;
    if (enable && !c->ev0) {
        c->ev0 = new (std::nothrow) cudaEvent_t[kTimingEvents];
        c->ev1 = new (std::nothrow) cudaEvent_t[kTimingEvents];
        if (!c->ev0 || !c->ev1) return SLIMSPEC_ERR_NOMEM;
        for (int i = 0; i < kTimingEvents; ++i) {
            if (cudaEventCreate(&c->ev0[i]) != cudaSuccess || cudaEventCreate(&c->ev1[i]) != cudaSuccess)
                return SLIMSPEC_ERR_CUDA;
        }
    }
    if (enable) {
        int rc = timing_drain(c);
        if (rc != SLIMSPEC_OK) return rc;
        c->timing_ms = 0.0;
        c->timing_launches = 0;
    }
    c->timing_on = enable ? 1 : 0;
    return SLIMSPEC_OK;
}

extern "C" int slimspec_kernel_timing_read(slimspec_ctx* c, double* total_ms, long long* launches)
{
    if (!c || !total_ms || !launches) return SLIMSPEC_ERR_NULL;
    int rc = timing_drain(c);
    if (rc != SLIMSPEC_OK) return rc;
    *total_ms = c->timing_ms;
    *launches = c->timing_launches;
    return SLIMSPEC_OK;
}

static bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }

// Grow-only fp32 M x V buffer for the generic top-k path (allocation synchronises).
static int ensure_logits(slimspec_ctx* c, size_t elems)
{
    if (c->s.logits_elems >= elems) return SLIMSPEC_OK;
    if (c->s.logits) { cudaDeviceSynchronize(); cudaFree(c->s.logits); c->s.logits = nullptr; c->s.logits_elems = 0; }
    if (cudaMalloc(&c->s.logits, elems * sizeof(float)) != cudaSuccess) { cudaGetLastError(); return SLIMSPEC_ERR_NOMEM; }
    c->s.logits_elems = elems;
    return SLIMSPEC_OK;
}

#define CK(expr) do { if ((expr) != cudaSuccess) { cudaGetLastError(); return SLIMSPEC_ERR_CUDA; } } while (0)

// Shared body.  K is the contraction length of the streamed matrix Bm (K x V): r for the
// low-rank head (A != null), d for the full-rank head (A == null, z = widened h).
// mode 0: top-k into ids/logprobs; mode 1: raw logits.
static int run_head(slimspec_ctx* c, const bf16* h, const bf16* A, const bf16* Bm, int M, int d, int r, int V,
                    int k, int mode, int32_t* ids, float* logprobs, float* logits, cudaStream_t st)
{
    if (!c || !h || !Bm) return SLIMSPEC_ERR_NULL;
    if (mode == 0 && (!ids || !logprobs)) return SLIMSPEC_ERR_NULL;
    if (mode == 1 && !logits) return SLIMSPEC_ERR_NULL;
    const bool lowrank = (A != nullptr);
    if (M <= 0 || d <= 0 || V <= 0 || (lowrank && r <= 0)) return SLIMSPEC_ERR_DIM;
    if (M > c->max_M || d > c->max_d || V > c->max_V || (lowrank && r > c->max_d)) return SLIMSPEC_ERR_DIM;
    if (mode == 0 && (k <= 0 || k > V || k > SLIMSPEC_MAX_K || k > c->max_k)) return SLIMSPEC_ERR_DIM;
    const int K = lowrank ? r : d;

    int path = c->forced_path;
    const bool ptr_ok = aligned16(h) && aligned16(Bm) && (!lowrank || aligned16(A)) &&
                        (mode == 0 || aligned16(logits));
    StreamPlan sp = stream_plan(M, K, V, mode == 0 ? k : 1, c->sm_count);
    const bool stream_ok = sp.ok && ptr_ok && d % 2 == 0 && (!lowrank || r % 16 == 0);
    const bool tensor_fits = tensor_ok(M, K, V, k, mode) && ptr_ok && (!lowrank || (d % 64 == 0 && r >= 64));
    if (path == SLIMSPEC_PATH_AUTO) {
        // FP32 FMAs keep up with HBM only for a few rows; beyond that the tensor cores take over
        if (M > kStreamMaxRows && tensor_fits) path = SLIMSPEC_PATH_TENSOR;
        else path = stream_ok ? SLIMSPEC_PATH_STREAM : (tensor_fits ? SLIMSPEC_PATH_TENSOR : SLIMSPEC_PATH_GENERIC);
    }
    if (path == SLIMSPEC_PATH_TENSOR && !tensor_fits) return SLIMSPEC_ERR_ALIGN;
    if (path == SLIMSPEC_PATH_STREAM && !stream_ok) return SLIMSPEC_ERR_ALIGN;
    c->last_path = path;

    if (path == SLIMSPEC_PATH_GENERIC) {
        float* lg = logits;
        if (mode == 0) {
            int rc = ensure_logits(c, (size_t)M * V);
            if (rc != SLIMSPEC_OK) return rc;
            lg = c->s.logits;
        }
        if (lowrank) CK(generic_downproj(h, A, M, d, r, c->s.z, st));
        else CK(generic_widen(h, M * d, c->s.z, st));
        CK(generic_upproj(c->s.z, Bm, M, K, V, lg, st));
        c->launches += 2;
        if (mode == 0) { CK(generic_softmax_topk(lg, M, V, k, ids, logprobs, st)); c->launches += 1; }
        return SLIMSPEC_OK;
    }

    if (path == SLIMSPEC_PATH_TENSOR) {
        int n = 0;
        const bf16* X = h;
        const bf16* Xlo = nullptr;
        if (lowrank) {
            // While the call is HBM-bound the tensor cores have time to spare: keep the bf16 rounding
            // remainder of z and feed it through a second MMA, so z is effectively fp32-exact.
            const bool low_part = M <= kSplitCodeRows;
            cudaError_t e0;
            if (M <= kCodeByStreamRows && d % 2 == 0 && r % 16 == 0) {
                // few rows: the streaming path's down-projection (one launch of small CTAs) beats a K-split
                // tcgen05 product plus its reduction
                e0 = stream_code_rows(h, A, M, d, r, c->s.zb, low_part ? c->s.zb_lo : (bf16*)nullptr, c->sm_count, st);
                n = 1;
            } else {
                e0 = tensor_downproj(h, A, M, d, r, low_part, c->s, c->sm_count, &n, st);
            }
            c->launches += n;
            n = 0;
            if (e0 != cudaSuccess) { cudaGetLastError(); return SLIMSPEC_ERR_CUDA; }
            X = c->s.zb;
            if (low_part) Xlo = c->s.zb_lo;
        }
        if (mode == 0 && !tensor_records_fit(M, V, k, c->s, c->sm_count)) return SLIMSPEC_ERR_DIM;
        int slot = -1;
        if (c->timing_on) {
            if (c->timing_used == kTimingEvents) { int rc = timing_drain(c); if (rc != SLIMSPEC_OK) return rc; }
            slot = c->timing_used++;
        }
        cudaError_t e = tensor_head(X, Xlo, Bm, M, K, V, k, mode, ids, logprobs, logits, c->s, c->sm_count, &n,
                                    slot >= 0 ? c->ev0[slot] : (cudaEvent_t) nullptr, slot >= 0 ? c->ev1[slot] : (cudaEvent_t) nullptr, st);
        c->launches += n;
        if (e != cudaSuccess) { cudaGetLastError(); return SLIMSPEC_ERR_CUDA; }
        return SLIMSPEC_OK;
    }

    // streaming path: row tiles of up to 16 rows, each streams the K x V matrix once
    for (int m0 = 0; m0 < M; m0 += kStreamTile) {
        const int mrows = (M - m0 < kStreamTile) ? (M - m0) : kStreamTile;
        const bf16* hm = h + (size_t)m0 * d;
        const int kk = mode == 0 ? k : 1;
        int nl = 0;
        // one or two rows: the FMA kernel, one launch; three to sixteen: the tensor-core streaming kernels
        const FmaPlan fp = fma_plan(mrows, d, lowrank ? r : 0, V, kk, c->sm_count);
        const bool fma = fp.ok && fp.ncta <= c->s.max_parts;
        if (!fma) {
            if (lowrank) CK(stream_code(hm, A, mrows, d, r, V, kk, c->s.zfrag, c->sm_count, st));
            else CK(stream_widen(hm, mrows, d, V, kk, c->s.zfrag, c->sm_count, st));
            nl = 1;
        }
        int slot = -1;
        if (c->timing_on) {
            if (c->timing_used == kTimingEvents) { int rc = timing_drain(c); if (rc != SLIMSPEC_OK) return rc; }
            slot = c->timing_used++;
            CK(cudaEventRecord(c->ev0[slot], st));
        }
        // an event between two kernels serialises them: the timed kernel then runs alone
        int32_t* ids_t = mode == 0 ? ids + (size_t)m0 * k : nullptr;
        float* lp_t = mode == 0 ? logprobs + (size_t)m0 * k : nullptr;
        float* lg_t = mode == 1 ? logits + (size_t)m0 * V : nullptr;
        if (fma) {
            if (++c->epoch == 0) {      // the call numbers have gone round: forget the old ones
                CK(cudaMemsetAsync(c->s.zq, 0, fma_code_words(c->max_d) * sizeof(uint2), st));
                c->epoch = 1;
            }
            CK(fma_head(hm, A, Bm, mrows, fp.mt, d, r, V, kk, mode, ids_t, lp_t, lg_t, c->s, c->epoch, c->sm_count, st));
            nl += 1;
        } else {
            int nh = 0;
            CK(stream_head(c->s.zfrag, lowrank, Bm, mrows, K, V, kk, mode, ids_t, lp_t, lg_t, c->s, c->sm_count, slot < 0, &nh, st));
            nl += nh;
        }
        if (slot >= 0) CK(cudaEventRecord(c->ev1[slot], st));
        c->launches += nl;
    }
    return SLIMSPEC_OK;
}

extern "C" int slimspec_head_topk(slimspec_ctx* c, const void* h, const void* A, const void* B, int M, int d,
                                  int r, int V, int k, int32_t* out_ids, float* out_logprobs, void* stream)
{
    if (!A) return SLIMSPEC_ERR_NULL;
    return run_head(c, (const bf16*)h, (const bf16*)A, (const bf16*)B, M, d, r, V, k, 0, out_ids, out_logprobs,
                    nullptr, (cudaStream_t)stream);
}

extern "C" int slimspec_head_logits(slimspec_ctx* c, const void* h, const void* A, const void* B, int M, int d,
                                    int r, int V, float* out_logits, void* stream)
{
    if (!A) return SLIMSPEC_ERR_NULL;
    return run_head(c, (const bf16*)h, (const bf16*)A, (const bf16*)B, M, d, r, V, 1, 1, nullptr, nullptr,
                    out_logits, (cudaStream_t)stream);
}

extern "C" int fullhead_topk(slimspec_ctx* c, const void* h, const void* W, int M, int d, int V, int k,
                             int32_t* out_ids, float* out_logprobs, void* stream)
{
    return run_head(c, (const bf16*)h, nullptr, (const bf16*)W, M, d, 0, V, k, 0, out_ids, out_logprobs, nullptr,
                    (cudaStream_t)stream);
}

extern "C" int slimspec_head_topk_host(slimspec_ctx* c, const void* h_host, const void* A, const void* B, int M,
                                       int d, int r, int V, int k, int32_t* out_ids_host,
                                       float* out_logprobs_host, void* stream)
{
    if (!c || !h_host || !A || !B || !out_ids_host || !out_logprobs_host) return SLIMSPEC_ERR_NULL;
    if (M <= 0 || d <= 0 || M > c->max_M || d > c->max_d || k <= 0 || k > c->max_k) return SLIMSPEC_ERR_DIM;
    cudaStream_t st = (cudaStream_t)stream;
    CK(cudaMemcpyAsync(c->h_stage, h_host, (size_t)M * d * sizeof(bf16), cudaMemcpyHostToDevice, st));
    int rc = slimspec_head_topk(c, c->h_stage, A, B, M, d, r, V, k, c->ids_stage, c->lp_stage, stream);
    if (rc != SLIMSPEC_OK) return rc;
    CK(cudaStreamSynchronize(st));      // the kernels wrote the results into the mapped host buffer
    memcpy(out_ids_host, c->res_host, (size_t)M * k * sizeof(int32_t));
    memcpy(out_logprobs_host, reinterpret_cast<unsigned char*>(c->res_host) + c->res_half, (size_t)M * k * sizeof(float));
    return SLIMSPEC_OK;
}
