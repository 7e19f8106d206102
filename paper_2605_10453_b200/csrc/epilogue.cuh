// Epilogue shared by the streaming head kernels: from a slab's logits in shared memory to the
// slab's record (maximum, sum of exp, the k best (key, id) pairs), and the merge of all records by
// the last CTA to arrive (softmax of Section 3.2 in online form, and the candidate selection).
#pragma once
#include "ptx.cuh"
#include "select.cuh"
#include <float.h>

namespace slimspec {

static constexpr int kCand = 256;                     // candidates one row may park in a CTA's epilogue
// shared memory the epilogue keeps at the start of the CTA's dynamic area: ticket, group maxima
// [16][64], bound / maximum / count per row, sums of exp [16][16]
static constexpr int kEpFixedBytes = 64 + (16 * 64 + 16 + 16 + 16 + 16 * 16) * 4;

// Arrival counter with release / acquire semantics at GPU scope: what the CTA wrote before its
// barrier is visible to whoever reads the counter's later values.
__device__ __forceinline__ unsigned int ticket_take(unsigned int* ticket)
{
    unsigned int old;
    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(old) : "l"(ticket) : "memory");
    return old;
}
__device__ __forceinline__ unsigned int ld_acquire_gpu_u32(const unsigned int* p)
{
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
static constexpr long long kArrivalPolls = 1ll << 22;      // reads of the counter before a merging CTA gives up (seconds)

// ------------------------------------------------------------------------------------------
// Step (4) of the epilogue and what follows it: a warp per row orders the parked candidates by counting
// and writes the slab's record; then the arrival ticket, and the last CTAs to arrive merge the records.
template <int MT, class Params>
__device__ __forceinline__ void slab_records(const Params& p, unsigned char* smem, unsigned char* scratch, unsigned char* merge_area,
    const float* lg, int ngroups, int gstride, int lpitch, int ncols, int col_base)
{
    unsigned int* s_ticket = reinterpret_cast<unsigned int*>(smem);
    float* gmax_s = reinterpret_cast<float*>(smem + 64);      // [16 rows][64]: maxima of thread groups
    float* tau_s = gmax_s + 16 * 64;                          // [16] candidates must reach this
    float* cmax_s = tau_s + 16;                               // [16] the slab's maximum
    int* cnt_s = reinterpret_cast<int*>(cmax_s + 16);         // [16] candidates parked
    float* wsum_s = reinterpret_cast<float*>(cnt_s + 16);     // [16 rows][16 warps] sums of exp
    uint32_t* ck = reinterpret_cast<uint32_t*>(scratch);      // [MT][kCand]
    int* ci = reinterpret_cast<int*>(ck + MT * kCand);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, nt = blockDim.x, nw = nt >> 5;
    const int cta = blockIdx.x, k = p.k;
    const int mrows = min(p.M, MT);
    auto logit = [&](int row, int c) {
        float x = lg[row * lpitch + c];
        for (int gi = 1; gi < ngroups; ++gi) x += lg[gi * gstride + row * lpitch + c];
        return x + 0.f;             // -0 becomes +0: keys and float compares then agree
    };

    // ---- (4)
    const int P = p.ncta;
    const int RW = p.rec_words;
    for (int row = warp; row < mrows; row += nw) {
        float* rec = p.part + ((size_t)row * P + cta) * RW;
        {
            const float s = warp_sum(lane < nw ? wsum_s[row * 16 + lane] : 0.f);      // fixed order: reproducible
            if (lane == 0) *reinterpret_cast<float2*>(rec) = make_float2(cmax_s[row], s);
        }
        const int n = cnt_s[row];
        if (n <= kCand) {
            // the (key, id) pairs go straight into the record: rank j to words 2 + 2 j, 3 + 2 j
            const uint32_t* rk = ck + row * kCand;
            const int* ri = ci + row * kCand;
            for (int base = 0; base < n; base += 32) {
                const int i = base + lane;
                const uint32_t mk = i < n ? rk[i] : 0u;
                const int mi = i < n ? ri[i] : kNoId;
                int rank = 0;
                for (int j = 0; j < n; ++j) rank += better(rk[j], ri[j], mk, mi) ? 1 : 0;
                if (i < n && rank < k) *reinterpret_cast<float2*>(rec + 2 + 2 * rank) = make_float2(__uint_as_float(mk), __int_as_float(mi));
            }
            for (int j = n + lane; j < k; j += 32) *reinterpret_cast<float2*>(rec + 2 + 2 * j) = make_float2(__uint_as_float(0u), __int_as_float(kNoId));
        } else {
            // Slow path (masses of equal logits, or logits in long ordered runs): k rounds over the
            // row, each taking the best logit that comes after the previous winner in the order;
            // nothing is kept between rounds but that winner.
            uint32_t lk = 0xffffffffu;
            int li = -1;
            for (int j = 0; j < k; ++j) {
                uint32_t bk = 0u;
                int bi = kNoId;
                for (int c = lane; c < ncols; c += 32) {
                    const uint32_t ke = f2key(logit(row, c));
                    const int ie = col_base + c;
                    if (after(ke, ie, lk, li) && better(ke, ie, bk, bi)) { bk = ke; bi = ie; }
                }
                const uint32_t wk = warp_max_u32(bk);
                const uint32_t wi = warp_min_u32(bk == wk ? (uint32_t)bi : 0xffffffffu);
                lk = wk;
                li = (int)wi;
                if (lane == 0) *reinterpret_cast<float2*>(rec + 2 + 2 * j) = make_float2(__uint_as_float(wk), __int_as_float(wk != 0u ? (int)wi : kNoId));
                if (wk == 0u) { lk = 0u; li = kNoId; }      // nothing left: later rounds stay empty
            }
        }
    }

    // ---- arrival.  The CTAs take tickets from a counter that only counts up (the call's first ticket is
    // p.ticket_base).  The last R of them to arrive merge: each takes every R-th row, waits until the counter
    // shows that all P have arrived (they are already running: it is a wait of a microsecond, bounded all
    // the same), and runs two tasks per row, a warp each: the row's log-sum-exp, and its k best entries.
    if (!p.merge_inside) return;
    __syncthreads();
    if (tid == 0) *s_ticket = ticket_take(p.ticket) - p.ticket_base;
    __syncthreads();
    const int rows_at_once = max(1, nw >> 1);
    const int R = min(P, (p.M + rows_at_once - 1) / rows_at_once);
    const int me = (int)*s_ticket - (P - R);             // which of the R mergers this CTA is
    if (me < 0) return;
    if (me != R - 1) {
        if (tid == 0) {
            long long it = 0;
            while (ld_acquire_gpu_u32(p.ticket) - p.ticket_base < (unsigned)P && ++it < kArrivalPolls) {}
            if (it >= kArrivalPolls) atomicCAS(p.err, 0, ERR_WAIT_RECORD);
        }
        __syncthreads();
    }
    float* lse_s = reinterpret_cast<float*>(merge_area);                 // [16] by the CTA's own count of rows
    uint32_t* ok_all = reinterpret_cast<uint32_t*>(lse_s + 16);          // [16 rows][32] ordered keys
    int* oi_all = reinterpret_cast<int*>(ok_all + 16 * 32);              // [16 rows][32] their ids
    uint32_t* mk = reinterpret_cast<uint32_t*>(oi_all + 16 * 32) + warp * 2 * kMergeCand;     // this warp's candidates
    int* mi = reinterpret_cast<int*>(mk + kMergeCand);
    const int mine = (p.M - me + R - 1) / R;             // rows me, me + R, ...
    for (int task = warp; task < 2 * mine; task += nw) {
        const int lr = task >> 1, row = me + lr * R;
        if (P <= 5 * 32) merge_task<5>(p.part, P, RW, k, row, task & 1, lane, lse_s + lr, ok_all + lr * 32, oi_all + lr * 32, mk, mi, &cnt_s[warp]);
        else merge_task<kMergeLists>(p.part, P, RW, k, row, task & 1, lane, lse_s + lr, ok_all + lr * 32, oi_all + lr * 32, mk, mi, &cnt_s[warp]);
    }
    __syncthreads();
    for (int e = tid; e < mine * k; e += nt) {
        const int lr = e / k, j = e - lr * k, row = me + lr * R;
        p.ids[(size_t)row * k + j] = oi_all[lr * 32 + j];
        p.logprobs[(size_t)row * k + j] = key2f(ok_all[lr * 32 + j]) - lse_s[lr];
    }
}

// Epilogue of the head kernel.  The slab's logits lie in shared memory: logit (row, column c) is
// the sum over g < ngroups of lg[g * gstride + row * lpitch + c] (a kernel that leaves one partial sum
// per row group passes ngroups > 1).  The steps, which the two variants below share out differently:
//   (1) maxima of groups of logits (eight threads' logits, or a lane's); (2) the k-th largest of
//   these maxima bounds the slab's k-th largest logit from below; (3) sum of exp against the slab's
//   maximum, logits that reach the bound are parked; (4) a warp per row orders the parked candidates
//   by counting and writes the slab's record; then the arrival ticket, and the last CTAs to arrive
//   merge the records of every row the same way.
// Nothing here depends on the order in which threads or CTAs arrive: results are reproducible.
//
// Three to sixteen rows: a warp per row and no barrier.  The warp walks its row twice in shared memory (lane l
// looks after columns l, l + 32, ...).  First pass: the lanes' maxima; the k-th largest of these 32
// bounds the row's k-th largest logit from below (k <= 32), the largest is the slab's maximum.
// Second pass: sum of exp, and the logits that reach the bound go to the row's list in column order
// (ballot and count: no atomics).  Step (4) then finds its inputs where the other variants leave them.
// Several rows per warp run one after the other: 3 rounds for 16 rows on 7 warps, against block-wide
// steps whose cost grows with every row (measured at 8 rows: steps (1)-(3) 6.4 us).
template <int MT, class Params>
__device__ __forceinline__ void slab_epilogue_rows(const Params& p, unsigned char* smem, unsigned char* scratch, unsigned char* merge_area,
    const float* lg, int lpitch, int ncols, int col_base)
{
    float* gmax_s = reinterpret_cast<float*>(smem + 64);
    float* cmax_s = gmax_s + 16 * 64 + 16;                    // [16] the slab's maximum
    int* cnt_s = reinterpret_cast<int*>(cmax_s + 16);         // [16] candidates parked
    float* wsum_s = reinterpret_cast<float*>(cnt_s + 16);     // [16 rows][16 warps] sums of exp: here all of a row's sum in slot 0
    uint32_t* ck = reinterpret_cast<uint32_t*>(scratch);      // [MT][kCand]
    int* ci = reinterpret_cast<int*>(ck + MT * kCand);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, nt = blockDim.x, nw = nt >> 5;
    const int k = p.k;
    const int mrows = min(p.M, MT);

    if (p.mode == 1) {
        for (int row = 0; row < mrows; ++row)
            for (int c = tid; c < ncols; c += nt) p.logits[(size_t)row * p.V + col_base + c] = lg[row * lpitch + c] + 0.f;
        return;
    }
    for (int row = warp; row < mrows; row += nw) {
        const float* lr = lg + (size_t)row * lpitch;
        float lm = -FLT_MAX;
        for (int c = lane; c < ncols; c += 32) lm = fmaxf(lm, lr[c] + 0.f);       // -0 becomes +0: keys and float compares then agree
        const uint32_t lk = f2key(lm);
        const uint32_t kth = warp_kth_largest(lk, min(k, 32), lane);       // a lone warp waits on latencies: 32 independent shuffles beat k dependent rounds
        const float cm = key2f(warp_max_u32(lk));
        float s = 0.f;
        int n = 0;
        for (int c0 = 0; c0 < ncols; c0 += 32) {
            const int c = c0 + lane;
            const float x = c < ncols ? lr[c] + 0.f : -FLT_MAX;
            const uint32_t key = f2key(x);
            const bool in = c < ncols && key >= kth;
            if (c < ncols) s += __expf(x - cm);
            const unsigned b = __ballot_sync(0xffffffffu, in);
            if (in) {
                const int pos = n + __popc(b & ((1u << lane) - 1u));
                if (pos < kCand) { ck[row * kCand + pos] = key; ci[row * kCand + pos] = col_base + c; }
            }
            n += __popc(b);
        }
        s = warp_sum(s);
        if (lane < 16) wsum_s[row * 16 + lane] = lane == 0 ? s : 0.f;
        if (lane == 0) { cmax_s[row] = cm; cnt_s[row] = n; }
    }
    __syncwarp();       // step (4) of a row is run by the warp that wrote the above
    slab_records<MT>(p, smem, scratch, merge_area, lg, 1, 0, lpitch, ncols, col_base);
}

// One to four rows and at most four columns per thread (ncols <= 4 * blockDim), all warps on every row: a thread
// adds up its logits once and keeps them in registers, group maxima come from one reduction
// instruction per group of eight lanes, and every warp works out the bound and the slab's maximum for
// itself, which saves the second barrier.
template <int MT, class Params>
__device__ __forceinline__ void slab_epilogue_few(const Params& p, unsigned char* smem, unsigned char* scratch, unsigned char* merge_area,
    const float* lg, int ngroups, int gstride, int lpitch, int ncols, int col_base)
{
    unsigned int* s_ticket = reinterpret_cast<unsigned int*>(smem);
    float* gmax_s = reinterpret_cast<float*>(smem + 64);      // [16 rows][64]: maxima of thread groups
    float* tau_s = gmax_s + 16 * 64;                          // [16] candidates must reach this
    float* cmax_s = tau_s + 16;                               // [16] the slab's maximum
    int* cnt_s = reinterpret_cast<int*>(cmax_s + 16);         // [16] candidates parked
    float* wsum_s = reinterpret_cast<float*>(cnt_s + 16);     // [16 rows][16 warps] sums of exp
    uint32_t* ck = reinterpret_cast<uint32_t*>(scratch);      // [MT][kCand]
    int* ci = reinterpret_cast<int*>(ck + MT * kCand);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, nt = blockDim.x, nw = nt >> 5;
    const int cta = blockIdx.x, k = p.k;
    const int mrows = min(p.M, MT);
    auto logit = [&](int row, int c) {
        float x = lg[row * lpitch + c];
        for (int gi = 1; gi < ngroups; ++gi) x += lg[gi * gstride + row * lpitch + c];
        return x + 0.f;             // -0 becomes +0: keys and float compares then agree
    };

    if (p.mode == 1) {
        for (int row = 0; row < mrows; ++row)
            for (int c = tid; c < ncols; c += nt) p.logits[(size_t)row * p.V + col_base + c] = logit(row, c);
        return;
    }
    static_assert(MT <= 4, "rows held in registers");
    float x[MT][4];
#pragma unroll
    for (int m = 0; m < MT; ++m)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int c = tid + j * nt;
            x[m][j] = (m < mrows && c < ncols) ? logit(m, c) : -FLT_MAX;
        }
    // ---- (1) maxima of groups of eight threads
    if (tid < 16) cnt_s[tid] = 0;
#pragma unroll
    for (int m = 0; m < MT; ++m) {
        const float t = fmaxf(fmaxf(x[m][0], x[m][1]), fmaxf(x[m][2], x[m][3]));
        const uint32_t gk = __reduce_max_sync(0xffu << (lane & 24), f2key(t));
        if ((lane & 7) == 0 && m < mrows) gmax_s[m * 64 + warp * 4 + (lane >> 3)] = key2f(gk);
    }
    __syncthreads();
    // ---- (2) + (3): the bound and the maximum (every warp for itself), sum of exp, candidates parked
#pragma unroll
    for (int m = 0; m < MT; ++m) {
        if (m >= mrows) break;
        const uint32_t ka = f2key(gmax_s[m * 64 + lane]), kb2 = f2key(gmax_s[m * 64 + 32 + lane]);
        const uint32_t kth = (k <= 16) ? warp_kth_largest_any(max(ka, kb2), k, lane) : warp_kth_largest64(ka, kb2, min(k, 64), lane);
        const float cm = key2f(warp_max_u32(max(ka, kb2)));
        if (tid == 0) cmax_s[m] = cm;
        float s = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int c = tid + j * nt;
            if (c < ncols) {
                s += __expf(x[m][j] - cm);
                const uint32_t key = f2key(x[m][j]);
                if (key >= kth) {
                    const int pos = atomicAdd(&cnt_s[m], 1);
                    if (pos < kCand) { ck[m * kCand + pos] = key; ci[m * kCand + pos] = col_base + c; }
                }
            }
        }
        s = warp_sum(s);
        if (lane == 0) wsum_s[m * 16 + warp] = s;
    }
    __syncthreads();
    slab_records<MT>(p, smem, scratch, merge_area, lg, ngroups, gstride, lpitch, ncols, col_base);
}


}  // namespace slimspec
