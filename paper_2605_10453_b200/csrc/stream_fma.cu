// Streaming path for one or two rows, ONE launch per call: the K x V weight matrix is read from HBM
// exactly once, in split-V slabs (one CTA per SM), with coalesced 128-bit loads held in flight in
// registers and consumed by packed FP32 FMAs against the fp32 code.
//
// The down-projection z = h A runs inside the same kernel.  Every CTA first sends for the top of
// its slab (weights may be read ahead of the activations), waits for the kernel before it in the
// stream, computes one job of the down-projection (8 columns of A over a range of its rows),
// publishes the partial sums, each in one 8-byte word with the number of the call, and polls the
// words of all jobs; a CTA that has polled for a long time computes whatever is still missing
// itself, so the wait ends whether or not the other CTAs are running.  With the code in shared memory it streams its slab.  The logits never
// leave the SM: each CTA writes max / sum-exp / top-k of its slab as a record and the last CTA to
// arrive merges the records (Section 4.1: both projections; the softmax of Section 3.2 in online
// form; the candidate selection).
// (Three to sixteen rows take the tensor-core streaming kernel of stream.cu.)
#include "kernels.h"
#include "ptx.cuh"
#include "select.cuh"
#include "epilogue.cuh"
#include <float.h>
#include <type_traits>

namespace slimspec {

static constexpr int kFmaMaxColThreads = 256;   // threads across a slab's columns, 8 columns each
static constexpr int kFmaMaxCtas = 256;         // most slabs
static constexpr int kFmaZChunkBytes = 64 * 1024;   // shared memory for the code, as (z, z) pairs
static constexpr int kFmaEpFixed = (kEpFixedBytes + 127) / 128 * 128;      // the epilogue's fixed area
static constexpr int kFmaMergeBytes = (16 + 2 * 16 * 32 + 8 * 2 * kMergeCand) * 4 + 64;   // the last CTA's merge: up to eight tasks
#ifndef SLIMSPEC_FMA4_MIN_A
#define SLIMSPEC_FMA4_MIN_A (4u << 20)
#endif
static constexpr size_t kFmaFourRowsMinA = SLIMSPEC_FMA4_MIN_A;      // elements of A from which three and four rows take this kernel
static constexpr int kFmaHelpAfter = 256;       // polls of the published code before a CTA computes the missing jobs itself

// Bytes of the weight matrix (all CTAs together) the kernel asks into the L2 while it waits
// for the code: about what HBM delivers in that wait (measured; more only evicts what is needed).
#ifndef SLIMSPEC_PF_MB
#define SLIMSPEC_PF_MB 8
#endif
static constexpr size_t kFmaPrefetchBytes = (size_t)SLIMSPEC_PF_MB << 20;

struct FmaParams {
    const bf16* h;        // [M][d]
    const bf16* A;        // [d][K]; null: the full-rank head, whose code is h itself (K = d)
    const bf16* B;        // [K][V]
    int M, d, K, V, k, mode;
    int ncta;             // slabs
    int units_base, units_rem;   // V/8 column units: slab c has units_base + (c < units_rem)
    int ct, rg;           // column threads (multiple of 32) and row groups: blockDim = ct * rg
    int kc;               // rows of the code per shared-memory chunk (K, or a multiple of rg * U)
    int rec_words;        // words per split-V record: max, sum-exp, k (key, id) pairs, padded to 4
    int merge_inside;     // 1: the last CTA to arrive merges the records
    // the down-projection, shared out among the CTAs as jobs: job j = (split j / code_units, unit j % code_units)
    int njobs;
    int code_units;       // K / 8: 16-byte column units of A
    int nsplit;           // row splits of A
    int job_rows;         // rows of A per split (a multiple of 4)
    uint2* zpart;         // [nsplit][K][MT] partial sums of the code, each an 8-byte word (value, epoch)
    unsigned int epoch;   // differs from call to call, never 0: marks the words this call has published
    int32_t* ids;
    float* logprobs;
    float* logits;
    float* part;          // split-V records [M][ncta][rec_words]
    unsigned int* ticket;
    unsigned int ticket_base;   // what the counter read when the call began
    int* err;
    int pf_rows;          // rows of the slab asked into the L2 while waiting
    int red_bytes;        // shared memory for the row groups' partial sums (at least what the merge needs)
};

__device__ __forceinline__ uint4 fma_ldg(const void* p)
{
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}

// 8-byte words that one CTA publishes and the others poll: single accesses, so a reader sees a
// word whole, old or new
__device__ __forceinline__ void st_relaxed_gpu_u64(uint2* p, uint2 v)
{
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"((unsigned long long)v.x | ((unsigned long long)v.y << 32)) : "memory");
}
__device__ __forceinline__ uint2 ld_relaxed_gpu_u64(const uint2* p)
{
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return make_uint2((uint32_t)v, (uint32_t)(v >> 32));
}

// ------------------------------------------------------------------------------------------
// One job of the down-projection, by the whole CTA: 8 columns of A (unit u) times the rows
// [s * job_rows, (s + 1) * job_rows) of A, for the MT rows of h.  A thread takes runs of four
// consecutive rows; the warp folds its lanes' sums by exchange (halving the columns a lane
// keeps), the warps meet in shared memory.  Sums run in a fixed order, so whoever computes a job
// -- its owner or a helper -- publishes the same bits.
template <int MT>
__device__ __forceinline__ void fma_code_job(const FmaParams& p, int j, float* wpart, const uint4 (&apre)[4], bool have_pre)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nt = blockDim.x, nw = nt >> 5;
    const int s = j / p.code_units, u = j - s * p.code_units;
    const int rbeg = s * p.job_rows, rend = min(p.d, rbeg + p.job_rows);
    const bf16* Ac = p.A + (size_t)u * 8;
    float acc[MT][8];
#pragma unroll
    for (int m = 0; m < MT; ++m)
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[m][c] = 0.f;

    for (int i0 = rbeg + tid * 4; i0 < rend; i0 += nt * 4) {
        uint4 a[4];
        uint2 hv[MT];
        // the first four rows of the CTA's own job were sent for before the wait (weights may be)
        const bool pre = have_pre && i0 == rbeg + tid * 4;
#pragma unroll
        for (int jj = 0; jj < 4; ++jj)
            a[jj] = pre ? apre[jj] : (i0 + jj < rend) ? fma_ldg(Ac + (size_t)(i0 + jj) * p.K) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int m = 0; m < MT; ++m)     // d is a multiple of 4; with one and two rows MT = M
            hv[m] = (MT <= 2 || m < p.M) ? __ldcg(reinterpret_cast<const uint2*>(p.h + (size_t)m * p.d + i0)) : make_uint2(0u, 0u);
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
            const uint32_t w[4] = {a[jj].x, a[jj].y, a[jj].z, a[jj].w};
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                const uint32_t hw = (jj < 2) ? hv[m].x : hv[m].y;
                const float hf = __uint_as_float((jj & 1) ? (hw & 0xffff0000u) : (hw << 16));
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    acc[m][2 * e] = fmaf(hf, __uint_as_float(w[e] << 16), acc[m][2 * e]);
                    acc[m][2 * e + 1] = fmaf(hf, __uint_as_float(w[e] & 0xffff0000u), acc[m][2 * e + 1]);
                }
            }
        }
    }
    // fold the lanes: each exchange halves the columns a lane keeps; lane l ends with column
    // 4 (l >> 4 & 1) + 2 (l >> 3 & 1) + (l >> 2 & 1), summed over the warp
#pragma unroll
    for (int m = 0; m < MT; ++m) {
        float v4[4], v2[2], v1;
        const bool u16 = lane & 16, u8 = lane & 8, u4 = lane & 4;
#pragma unroll
        for (int i = 0; i < 4; ++i)
            v4[i] = (u16 ? acc[m][4 + i] : acc[m][i]) + __shfl_xor_sync(0xffffffffu, u16 ? acc[m][i] : acc[m][4 + i], 16);
#pragma unroll
        for (int i = 0; i < 2; ++i) v2[i] = (u8 ? v4[2 + i] : v4[i]) + __shfl_xor_sync(0xffffffffu, u8 ? v4[i] : v4[2 + i], 8);
        v1 = (u4 ? v2[1] : v2[0]) + __shfl_xor_sync(0xffffffffu, u4 ? v2[0] : v2[1], 4);
        v1 += __shfl_xor_sync(0xffffffffu, v1, 2);
        v1 += __shfl_xor_sync(0xffffffffu, v1, 1);
        if ((lane & 3) == 0) wpart[(warp * MT + m) * 8 + (u16 ? 4 : 0) + (u8 ? 2 : 0) + (u4 ? 1 : 0)] = v1;
    }
    __syncthreads();
    if (tid < MT * 8) {
        const int m = tid >> 3, c = tid & 7;
        float v = 0.f;
        for (int w = 0; w < nw; ++w) v += wpart[(w * MT + m) * 8 + c];
        // value and call number travel in one 8-byte store: whoever reads the number of this call
        // reads this call's value with it, so no fence and no separate flag are needed
        st_relaxed_gpu_u64(p.zpart + ((size_t)s * p.K + u * 8 + c) * MT + m, make_uint2(__float_as_uint(v), p.epoch));
    }
    __syncthreads();      // wpart is free again
}

// ------------------------------------------------------------------------------------------
// The kernel.  One CTA per V slab; thread = (column unit of 8 columns, row group).  Every thread
// keeps U 128-bit loads of its column unit in flight (rows g, g+RG, g+2RG, ...), multiplies each
// arriving row by the code held in shared memory (packed FP32 FMAs) and refills.  The row
// groups' partial sums meet in shared memory, where the epilogue picks them up.
template <int MT, int U>
__global__ void __launch_bounds__(512, 1) k_fma_head(const FmaParams p)
{
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* cand = smem + kFmaEpFixed;                            // the epilogue's parked candidates
    float* red = reinterpret_cast<float*>(cand + MT * kCand * 8);       // [RG][MT][ct*8]; before that, the code jobs' warp sums
    unsigned char* merge_area = reinterpret_cast<unsigned char*>(red);   // the last CTA's merge, when the sums are no longer needed
    const int CT = p.ct, RG = p.rg;
    const int slab_cols = CT * 8;
    float2* zs = reinterpret_cast<float2*>(reinterpret_cast<unsigned char*>(red) + p.red_bytes);   // [kc][MT] (z, z) pairs

    const int tid = threadIdx.x;
    const int g = tid / CT, c = tid - g * CT;        // row group, column unit
    const int cta = blockIdx.x;
    const int K = p.K, V = p.V;
    const int stepU = RG * U;
    const bool lowrank = p.A != nullptr;

    // ---- hints first: this CTA's share of A (it is needed first, and the loads below queue up behind it)
    if (lowrank) {
        for (int j = cta; j < p.njobs; j += p.ncta) {
            const int s = j / p.code_units, u = j - s * p.code_units;
            const int rbeg = s * p.job_rows, rend = min(p.d, rbeg + p.job_rows);
            for (int i = rbeg + tid; i < rend; i += blockDim.x) prefetch_l2(p.A + (size_t)i * K + u * 8);
        }
    }

    // ---- this CTA's slab
    const int my_units = p.units_base + (cta < p.units_rem ? 1 : 0);
    const int unit0 = cta * p.units_base + min(cta, p.units_rem);
    const bool active = c < my_units;
    const bf16* base = p.B + (size_t)(unit0 + c) * 8;

    // the CTA's own job of the down-projection: its first four rows of A per thread go out now,
    // ahead of everything else, so that after the wait only h is missing
    uint4 apre[4];
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) apre[jj] = make_uint4(0u, 0u, 0u, 0u);
    const bool have_pre = lowrank && cta < p.njobs;
    if (have_pre) {
        const int s = cta / p.code_units, u = cta - s * p.code_units;
        const int rbeg = s * p.job_rows, rend = min(p.d, rbeg + p.job_rows);
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
            const int i = rbeg + tid * 4 + jj;
            if (i < rend) apre[jj] = fma_ldg(p.A + (size_t)i * K + u * 8);
        }
    }

    // Two sets of UH loads each: one set is consumed while the other is in flight, so a wait
    // for the older set never waits for loads issued after it.
    constexpr int UH = U / 2;
    uint4 q[2][UH];
#pragma unroll
    for (int hh = 0; hh < 2; ++hh)
#pragma unroll
        for (int j = 0; j < UH; ++j) {
            const int row = g + (hh * UH + j) * RG;
            q[hh][j] = (active && row < K) ? fma_ldg(base + (size_t)row * V) : make_uint4(0u, 0u, 0u, 0u);
        }
    // the weights are on their way; let the next kernel in the stream come up behind this one
    pdl_launch_dependents();
    for (int i = tid; i < MT * 64; i += blockDim.x) reinterpret_cast<float*>(smem + 64)[i] = -FLT_MAX;
    // Until the kernel before this one is complete this CTA can only wait, and while it waits HBM
    // idles: ask the L2 for the rows of the slab that come next (a hint; the loads of the main
    // loop then hit the L2).  Launched early behind a kernel that still runs, the wait is several
    // microseconds.
    if (p.pf_rows > 0) {
        const int lines = (my_units * 16 + 127) / 128 + 1;       // the slab's row segment need not start on a line
        const int r0 = min(K, stepU), r1 = min(K, stepU + p.pf_rows);
        const char* seg = reinterpret_cast<const char*>(p.B + (size_t)unit0 * 8);
        const size_t row_bytes = (size_t)V * sizeof(bf16);
        const int last = my_units * 16 - 1;                      // last byte of the row segment
        for (int i = tid; i < (r1 - r0) * lines; i += blockDim.x) {
            const int r = r0 + i / lines, l = i - (i / lines) * lines;
            prefetch_l2(seg + (size_t)r * row_bytes + min(l * 128, last));
        }
    }
    // the activations, the scratch and the outputs belong to the kernels before this one until here
    pdl_wait();

    // ---- this CTA's jobs of the down-projection
    if (lowrank)
        for (int j = cta; j < p.njobs; j += p.ncta) fma_code_job<MT>(p, j, red, apre, have_pre && j == cta);

    float2 acc[MT][4];
#pragma unroll
    for (int m = 0; m < MT; ++m)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[m][e] = make_float2(0.f, 0.f);

    // rows row, row + RG, ... (U of them): multiply what has arrived, then refill
    auto block = [&](int row, int kc0, int kend, auto checked) {
        constexpr bool kChecked = decltype(checked)::value;
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
#pragma unroll
            for (int j = 0; j < UH; ++j) {
                const int rj = row + (hh * UH + j) * RG;
                if (!kChecked || rj < kend) {
                    const uint32_t w[4] = {q[hh][j].x, q[hh][j].y, q[hh][j].z, q[hh][j].w};
                    float2 b2[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        b2[e] = make_float2(__uint_as_float(w[e] << 16), __uint_as_float(w[e] & 0xffff0000u));
                    const float2* zr = zs + (size_t)(rj - kc0) * MT;
#pragma unroll
                    for (int m = 0; m < MT; ++m) {
                        const float2 z2 = zr[m];
#pragma unroll
                        for (int e = 0; e < 4; ++e) acc[m][e] = __ffma2_rn(b2[e], z2, acc[m][e]);
                    }
                }
            }
            // the set is used up: refill all of it at once
#pragma unroll
            for (int j = 0; j < UH; ++j) {
                const int nr = row + (hh * UH + j) * RG + stepU;
                if (!kChecked || nr < K) q[hh][j] = fma_ldg(base + (size_t)nr * V);
            }
        }
    };

    for (int kc0 = 0; kc0 < K; kc0 += p.kc) {
        const int kend = min(K, kc0 + p.kc);
        // bring this chunk of the code into shared memory as (z, z) pairs
        if (kc0 > 0) __syncthreads();
        if (lowrank) {
            // poll the published words of this chunk until all carry this call's number; a CTA that has
            // polled for long computes the missing jobs itself (the other CTAs may not be running at all,
            // on a GPU shared with other work), so the wait ends either way
            for (int it = 0;; ++it) {
                bool ok = true;
                for (int e = tid; e < (kend - kc0) * MT; e += blockDim.x) {
                    const uint2* src = p.zpart + (size_t)kc0 * MT + e;
                    float zv = 0.f;
                    for (int s = 0; s < p.nsplit; ++s) {
                        const uint2 w = ld_relaxed_gpu_u64(src + (size_t)s * K * MT);
                        ok = ok && w.y == p.epoch;
                        zv += __uint_as_float(w.x);
                    }
                    zs[e] = make_float2(zv, zv);
                }
                if (__syncthreads_and(ok)) break;
                if (it >= kFmaHelpAfter) {
                    for (int j = 0; j < p.njobs; ++j) {
                        const int s = j / p.code_units, u = j - s * p.code_units;
                        const bool missing = ld_relaxed_gpu_u64(p.zpart + ((size_t)s * K + u * 8) * MT).y != p.epoch;
                        if (__syncthreads_or(missing)) fma_code_job<MT>(p, j, red, apre, false);
                    }
                }
            }
        } else {
            for (int e = tid; e < (kend - kc0) * MT; e += blockDim.x) {
                const int i = e / MT, m = e - i * MT;
                const float zv = (MT <= 2 || m < p.M) ? __bfloat162float(p.h[(size_t)m * p.d + kc0 + i]) : 0.f;
                zs[e] = make_float2(zv, zv);
            }
        }
        __syncthreads();
        if (active) {
            for (int row = kc0 + g; row < kend; row += stepU) {
                // unchecked while this block and the next one lie wholly inside K
                if (row - g + 2 * stepU <= K) block(row, kc0, kend, std::false_type());
                else block(row, kc0, kend, std::true_type());
            }
        }
    }
    // ---- the row groups' partial sums meet in shared memory; the epilogue adds them up
    if (active) {
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            float* dst = red + ((size_t)g * MT + m) * slab_cols + c * 8;
            *reinterpret_cast<float4*>(dst) = make_float4(acc[m][0].x, acc[m][0].y, acc[m][1].x, acc[m][1].y);
            *reinterpret_cast<float4*>(dst + 4) = make_float4(acc[m][2].x, acc[m][2].y, acc[m][3].x, acc[m][3].y);
        }
    }
    __syncthreads();
    slab_epilogue_few<MT>(p, smem, cand, merge_area, red, RG, MT * slab_cols, slab_cols, my_units * 8, unit0 * 8);
}

// ------------------------------------------------------------------------------------------
static int fma_pick_mt(int M) { return M <= 2 ? M : 4; }

struct FmaGeometry {
    int ncta, units_base, units_rem, max_units, ct, rg, u, kc, rec_words, threads;
    int njobs, code_units, nsplit, job_rows, red_bytes;
    size_t smem;
};

// One CTA per SM, the slab's column units across ct threads, the rows of the matrix dealt to rg row
// groups.  Shapes whose slabs are wider than kFmaMaxColThreads units are not taken (the tensor-core
// streaming kernel takes them).  r = 0: the full-rank head (K = d, no down-projection).
static bool fma_geometry(int mt, int d, int r, int V, int k, int sm_count, FmaGeometry* g)
{
    const int K = r > 0 ? r : d;
    if (V % 8 != 0 || K < 1 || k > 32 || k < 1) return false;
    const int units = V / 8;
    int ncta = sm_count < kFmaMaxCtas ? sm_count : kFmaMaxCtas;
    if (ncta > units) ncta = units;
    g->ncta = ncta;
    g->units_base = units / ncta;
    g->units_rem = units % ncta;
    g->max_units = g->units_base + (g->units_rem ? 1 : 0);
    if (g->max_units > kFmaMaxColThreads) return false;
    g->ct = (g->max_units + 31) / 32 * 32;
    g->rg = 512 / g->ct;
    if (g->rg > K) g->rg = K;
    if (g->rg < 2) return false;      // the epilogue keeps at most four columns per thread
    g->threads = g->ct * g->rg;
    g->u = mt == 4 ? 8 : 16;      // loads a thread keeps in flight: the registers of four rows leave room for eight
    // rows of the code per shared-memory chunk: all of K if it fits, else a multiple of rg*u
    const int kc_max = kFmaZChunkBytes / (mt * 8);
    if (K <= kc_max) g->kc = K;
    else {
        g->kc = kc_max / (g->rg * g->u) * (g->rg * g->u);
        if (g->kc < 1) return false;
    }
    g->rec_words = (2 + 2 * k + 3) / 4 * 4;
    g->red_bytes = g->threads * mt * 32 > kFmaMergeBytes ? g->threads * mt * 32 : kFmaMergeBytes;
    g->smem = (size_t)kFmaEpFixed + (size_t)mt * kCand * 8 + g->red_bytes + (size_t)g->kc * mt * 8;
    if (g->smem > 200 * 1024) return false;
    // the down-projection's jobs: one 16-byte unit of A's columns each; the rows of A are split while
    // that leaves every CTA a job and a job at least a row per thread
    g->njobs = 0; g->code_units = 0; g->nsplit = 1; g->job_rows = d;
    if (r > 0) {
        if (r % 8 != 0 || d % 4 != 0) return false;
        g->code_units = r / 8;
        int ns = ncta / g->code_units;
        if (ns > 8 / mt) ns = 8 / mt;
        if (ns > d / 512) ns = d / 512;
        if (ns < 1) ns = 1;
        g->job_rows = ((d + ns - 1) / ns + 3) / 4 * 4;
        g->nsplit = (d + g->job_rows - 1) / g->job_rows;
        g->njobs = g->code_units * g->nsplit;
    }
    return true;
}

FmaPlan fma_plan(int M, int d, int r, int V, int k, int sm_count)
{
    FmaPlan sp = {0, 0, 0, 0};
    // three and four rows only where A is large: there the down-projection inside this kernel, on all SMs,
    // beats the other path's separate kernel (d = 8192: 8 to 32 MB of A); on the smaller heads the two are equal
    if (M < 1 || M > 4 || (M > 2 && (r <= 0 || (size_t)d * r < kFmaFourRowsMinA))) return sp;
    const int mt = fma_pick_mt(M);
    FmaGeometry g;
    if (!fma_geometry(mt, d, r, V, k, sm_count, &g)) return sp;
    sp.ok = 1;
    sp.mt = mt;
    sp.ncta = g.ncta;
    sp.launches = 1;
    return sp;
}

// Once per device: load the kernels and allow them their dynamic shared memory.
cudaError_t fma_prepare()
{
    cudaError_t e;
    if ((e = cudaFuncSetAttribute(k_fma_head<1, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(k_fma_head<2, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(k_fma_head<4, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024)) != cudaSuccess) return e;
    return cudaSuccess;
}

// Launched with programmatic stream serialization: the kernel may begin once every CTA of the kernel
// before it in the stream has signalled launch_dependents or left; it orders itself after that
// kernel with griddepcontrol.wait.  Across calls this hides the launch gap and lets a call read the
// top of its slabs under the tail of the call before.
cudaError_t fma_head(const bf16* h, const bf16* A, const bf16* B, int M, int mt, int d, int r, int V, int k, int mode,
                     int32_t* ids, float* logprobs, float* logits, const Scratch& s, unsigned int epoch, int sm_count,
                     cudaStream_t st)
{
    FmaGeometry g;
    if (!fma_geometry(mt, d, A ? r : 0, V, k, sm_count, &g)) return cudaErrorInvalidValue;
    if (g.ncta > s.max_parts || epoch == 0) return cudaErrorInvalidValue;
    const int K = A ? r : d;
    FmaParams hp;
    hp.h = h; hp.A = A; hp.B = B; hp.M = M; hp.d = d; hp.K = K; hp.V = V; hp.k = k; hp.mode = mode;
    hp.ncta = g.ncta; hp.units_base = g.units_base; hp.units_rem = g.units_rem;
    hp.ct = g.ct; hp.rg = g.rg; hp.kc = g.kc; hp.rec_words = g.rec_words; hp.merge_inside = 1;
    hp.njobs = g.njobs; hp.code_units = g.code_units; hp.nsplit = g.nsplit; hp.job_rows = g.job_rows;
    hp.zpart = s.zq; hp.epoch = epoch; hp.red_bytes = g.red_bytes;
    hp.ids = ids; hp.logprobs = logprobs; hp.logits = logits;
    hp.part = s.part; hp.ticket = s.tickets; hp.err = s.err;
    hp.ticket_base = 0;
    if (mode == 0) hp.ticket_base = *s.ticket_base_host;
    {
        const size_t row_bytes = (size_t)g.max_units * 16 * g.ncta;      // one row of every slab
        const size_t rows = row_bytes ? kFmaPrefetchBytes / row_bytes : 0;
        hp.pf_rows = (int)(rows < (size_t)K ? rows : (size_t)K);
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(hp.ncta);
    cfg.blockDim = dim3(g.threads);
    cfg.dynamicSmemBytes = g.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = mt == 1 ? cudaLaunchKernelEx(&cfg, k_fma_head<1, 16>, hp)
                        : mt == 2 ? cudaLaunchKernelEx(&cfg, k_fma_head<2, 16>, hp) : cudaLaunchKernelEx(&cfg, k_fma_head<4, 8>, hp);
    if (e == cudaSuccess && mode == 0) *s.ticket_base_host += (unsigned int)hp.ncta;      // the tickets this launch will take
    return e;
}

}  // namespace slimspec
