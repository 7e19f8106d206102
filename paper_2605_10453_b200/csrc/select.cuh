// Selection of the k best (logit, id) pairs, shared by the streaming and the tensor-core path:
// warp-level bounds, ordering by counting, and the merge of split-V records.
// Records: per (row, slab) rec_words floats: maximum, sum of exp(logit - maximum), then k
// (key, id) pairs in order, padded to a multiple of four words.
#pragma once
#include "ptx.cuh"
#include <float.h>

namespace slimspec {

static constexpr int kMergeCand = 128;                // candidates one row may park in the final merge
static constexpr int kMergeLists = 10;                // slab records a lane owns in the final merge
static constexpr int kMaxRecords = 32 * kMergeLists;  // records per row the merge can take
static constexpr int kNoId = 0x7fffffff;

// ------------------------------------------------------------------------------------------
// Selection.  Candidates are (key, id) with key = f2key(logit) and key 0 = none; the order is
// (key descending, id ascending).

// The k-th largest (k = 1..32) of the warp's 32 lane values, by counting: a lane's rank is the
// number of lanes ahead of it (larger key, or equal key and lower lane).
__device__ __forceinline__ uint32_t warp_kth_largest(uint32_t key, int k, int lane)
{
    int rank = 0;
#pragma unroll 4
    for (int s = 0; s < 32; ++s) {
        const uint32_t o = __shfl_sync(0xffffffffu, key, s);
        rank += (o > key || (o == key && s < lane)) ? 1 : 0;
    }
    const unsigned hit = __ballot_sync(0xffffffffu, rank == k - 1);
    return __shfl_sync(0xffffffffu, key, __ffs(hit) - 1);
}

// The same for small k by k rounds of "take the maximum out": cheaper than counting up to about a dozen.
__device__ __forceinline__ uint32_t warp_kth_largest_rounds(uint32_t key, int k, int lane)
{
    uint32_t kth = 0u;
    for (int j = 0; j < k; ++j) {
        kth = warp_max_u32(key);
        const unsigned eq = __ballot_sync(0xffffffffu, key == kth);
        if (lane == __ffs(eq) - 1) key = 0u;
    }
    return kth;
}
__device__ __forceinline__ uint32_t warp_kth_largest_any(uint32_t key, int k, int lane)
{
    return k <= 12 ? warp_kth_largest_rounds(key, k, lane) : warp_kth_largest(key, k, lane);
}

// The same over 64 values, two per lane (value a has index lane, value b index lane + 32).
__device__ __forceinline__ uint32_t warp_kth_largest64(uint32_t a, uint32_t b, int k, int lane)
{
    int ra = 0, rb = 0;
#pragma unroll 4
    for (int s = 0; s < 32; ++s) {
        const uint32_t oa = __shfl_sync(0xffffffffu, a, s);
        const uint32_t ob = __shfl_sync(0xffffffffu, b, s);
        ra += (oa > a || (oa == a && s < lane)) ? 1 : 0;
        ra += (ob > a) ? 1 : 0;
        rb += (oa >= b) ? 1 : 0;
        rb += (ob > b || (ob == b && s < lane)) ? 1 : 0;
    }
    const unsigned hit_a = __ballot_sync(0xffffffffu, ra == k - 1);
    const unsigned hit_b = __ballot_sync(0xffffffffu, rb == k - 1);
    const uint32_t va = __shfl_sync(0xffffffffu, a, hit_a ? __ffs(hit_a) - 1 : 0);
    const uint32_t vb = __shfl_sync(0xffffffffu, b, hit_b ? __ffs(hit_b) - 1 : 0);
    return hit_a ? va : vb;
}

// n candidates in shared memory, in any order, distinct ids.  The warp writes the min(n, k)
// best in order to (ok, oi) and pads up to k with empty entries.  By counting: a candidate's
// place is the number of candidates ahead of it.
__device__ __forceinline__ void warp_rank_select(const uint32_t* ck, const int* ci, int n, int k, uint32_t* ok,
                                                 int* oi, int lane)
{
    for (int base = 0; base < n; base += 32) {
        const int i = base + lane;
        const uint32_t mk = i < n ? ck[i] : 0u;
        const int mi = i < n ? ci[i] : kNoId;
        int rank = 0;
        for (int j = 0; j < n; ++j) {
            const uint32_t kj = ck[j];
            const int ij = ci[j];
            rank += (kj > mk || (kj == mk && ij < mi)) ? 1 : 0;
        }
        if (i < n && rank < k) { ok[rank] = mk; oi[rank] = mi; }
    }
    for (int j = n + lane; j < k; j += 32) { ok[j] = 0u; oi[j] = kNoId; }
}

// is (ka, ia) strictly after (kb, ib) in the order, i.e. a worse candidate?
__device__ __forceinline__ bool after(uint32_t ka, int ia, uint32_t kb, int ib)
{
    return ka < kb || (ka == kb && ia > ib);
}
// is (ka, ia) a better candidate than (kb, ib)?
__device__ __forceinline__ bool better(uint32_t ka, int ia, uint32_t kb, int ib)
{
    return ka > kb || (ka == kb && ia < ib);
}

// ------------------------------------------------------------------------------------------
// ------------------------------------------------------------------------------------------
// One task of the merge, run by one warp: kind 0 = the row's log-sum-exp from the records'
// (maximum, sum-exp) pairs, written to *lse_out; kind 1 = its k best entries.  A lane owns the records lane,
// lane + 32, ... (NL of them at most) and keeps what it loads in registers: one round trip to the L2.
template <int NL>
__device__ __forceinline__ void merge_task(const float* part, int P, int RW, int k, int row, int kind, int lane, float* lse_out,
                                           uint32_t* ok, int* oi, uint32_t* mk, int* mi, int* cnt)
{
    const float* rows = part + (size_t)row * P * RW;
    if (kind == 0) {
        float2 ms[NL];
#pragma unroll
        for (int q = 0; q < NL; ++q) {
            const int s = lane + 32 * q;
            ms[q] = s < P ? __ldcg(reinterpret_cast<const float2*>(rows + (size_t)s * RW)) : make_float2(-FLT_MAX, 0.f);
        }
        float gm = -FLT_MAX;
#pragma unroll
        for (int q = 0; q < NL; ++q) gm = fmaxf(gm, ms[q].x);
        gm = warp_max(gm);
        float gs = 0.f;
#pragma unroll
        for (int q = 0; q < NL; ++q) gs += ms[q].y * __expf(ms[q].x - gm);
        gs = warp_sum(gs);
        if (lane == 0) *lse_out = gm + __logf(gs);
        return;
    }
    // the first three entries of every record (words 2..7), then the bound: at least k entries
    // reach the k-th largest of the lanes' best first entries
    float2 e0[NL];
    float4 e12[NL];
#pragma unroll
    for (int q = 0; q < NL; ++q) {
        const int s = lane + 32 * q;
        e0[q] = make_float2(0.f, __int_as_float(kNoId));
        e12[q] = make_float4(0.f, __int_as_float(kNoId), 0.f, __int_as_float(kNoId));
        if (s < P) {
            e0[q] = __ldcg(reinterpret_cast<const float2*>(rows + (size_t)s * RW + 2));
            if (k >= 2) e12[q] = __ldcg(reinterpret_cast<const float4*>(rows + (size_t)s * RW + 4));
        }
    }
    uint32_t hk = 0u;
#pragma unroll
    for (int q = 0; q < NL; ++q) hk = max(hk, __float_as_uint(e0[q].x));
    const uint32_t kth = warp_kth_largest_any(hk, min(k, 32), lane);
    if (lane == 0) *cnt = 0;
    __syncwarp();
#pragma unroll
    for (int q = 0; q < NL; ++q) {
        const uint32_t k0 = __float_as_uint(e0[q].x);
        if (k0 != 0u && k0 >= kth) {
            int pos = atomicAdd(cnt, 1);
            if (pos < kMergeCand) { mk[pos] = k0; mi[pos] = __float_as_int(e0[q].y); }
            const uint32_t k1 = __float_as_uint(e12[q].x);
            if (k >= 2 && k1 != 0u && k1 >= kth) {          // the record's list is in order: rarely more than one entry
                pos = atomicAdd(cnt, 1);
                if (pos < kMergeCand) { mk[pos] = k1; mi[pos] = __float_as_int(e12[q].y); }
                const uint32_t k2 = __float_as_uint(e12[q].z);
                if (k >= 3 && k2 != 0u && k2 >= kth) {
                    pos = atomicAdd(cnt, 1);
                    if (pos < kMergeCand) { mk[pos] = k2; mi[pos] = __float_as_int(e12[q].w); }
                    const float* rec = rows + (size_t)(lane + 32 * q) * RW;
                    for (int j = 3; j < k; ++j) {
                        const float2 en = __ldcg(reinterpret_cast<const float2*>(rec + 2 + 2 * j));
                        const uint32_t kj = __float_as_uint(en.x);
                        if (kj == 0u || kj < kth) break;
                        pos = atomicAdd(cnt, 1);
                        if (pos < kMergeCand) { mk[pos] = kj; mi[pos] = __float_as_int(en.y); }
                    }
                }
            }
        }
    }
    __syncwarp();
    const int n = *cnt;
    if (n <= kMergeCand) {
        warp_rank_select(mk, mi, n, k, ok, oi, lane);
    } else {
        // slow path: k rounds over every entry of the row's records, each round taking the best
        // entry after the previous winner
        uint32_t lk = 0xffffffffu;
        int li = -1;
        for (int j = 0; j < k; ++j) {
            uint32_t bk = 0u;
            int bi = kNoId;
            for (int s = lane; s < P; s += 32) {
                const float* rec = rows + (size_t)s * RW;
                for (int e = 0; e < k; ++e) {
                    const float2 en = __ldcg(reinterpret_cast<const float2*>(rec + 2 + 2 * e));
                    const uint32_t ke = __float_as_uint(en.x);
                    const int ie = __float_as_int(en.y);
                    if (ke != 0u && after(ke, ie, lk, li) && better(ke, ie, bk, bi)) { bk = ke; bi = ie; }
                }
            }
            const uint32_t wk = warp_max_u32(bk);
            const uint32_t wi = warp_min_u32(bk == wk ? (uint32_t)bi : 0xffffffffu);
            lk = wk;
            li = (int)wi;
            if (lane == 0) { ok[j] = wk; oi[j] = wk != 0u ? (int)wi : kNoId; }
            if (wk == 0u) { lk = 0u; li = kNoId; }
        }
    }
}

}  // namespace slimspec
