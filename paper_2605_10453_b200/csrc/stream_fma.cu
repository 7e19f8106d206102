// Streaming path for one or two rows: the K x V weight matrix is read from HBM exactly once, in
// split-V slabs (one CTA per SM), with coalesced 128-bit loads held in flight in registers and
// consumed by packed FP32 FMAs against the fp32 code.  Two launches per call, chained by
// programmatic dependent launch: a down-projection with one CTA per 16 columns of A, and the head.
// The logits never leave the SM: each CTA keeps a running max / sum-exp / top-k per row and
// the last CTA to finish merges the per-slab records (Section 4.1 up-projection, the
// softmax of Section 3.2 in online form, and the candidate selection).
// (Three to sixteen rows take the tensor-core streaming kernel of stream.cu.  At one row this
// kernel pair is the faster one on every shape measured: the down-projection runs at the HBM rate
// on a large A, and its few, large CTAs leave most SMs to the head CTAs that start early.)
#include "kernels.h"
#include "ptx.cuh"
#include <float.h>
#include <type_traits>

namespace slimspec {

static constexpr int kFmaMaxColThreads = 256;   // threads across one pass's columns, 8 columns each
static constexpr int kFmaMaxColWarps = kFmaMaxColThreads / 32;
static constexpr int kFmaMaxCtas = 256;         // slabs per row the merge can take
static constexpr int kFmaZChunkBytes = 64 * 1024;   // shared memory for the code, as (z, z) pairs
static constexpr int kFmaNoId = 0x7fffffff;

// Bytes of the weight matrix (all CTAs together) the head kernel asks into the L2 while it waits
// for the code: about what HBM delivers in that wait (measured; more only evicts what is needed).
#ifndef SLIMSPEC_PF_MB
#define SLIMSPEC_PF_MB 24
#endif
static constexpr size_t kFmaPrefetchBytes = (size_t)SLIMSPEC_PF_MB << 20;

struct FmaParams {
    const float* zT;      // [K][MT] fp32 code, transposed and zero-padded to MT rows
    const bf16* B;        // [K][V]
    int M, K, V, k, mode;
    int ncta;             // slabs
    int units_base, units_rem;   // V/8 column units: slab c has units_base + (c < units_rem)
    int pass_units;       // most units one pass covers (<= ct)
    int ct, rg;           // column threads (multiple of 32) and row groups: blockDim = ct * rg
    int kc;               // rows of the code per shared-memory chunk (K, or a multiple of rg * U)
    int rec_words;        // words per split-V record: max, sum-exp, k keys, k ids, padded to 4
    int merge_rows;       // rows the last CTA merges per round
    int32_t* ids;
    float* logprobs;
    float* logits;
    float* part;          // split-V records [M][ncta][rec_words]
    unsigned int* ticket;
    int* err;
    int wait_prev;        // 1: zT is written by the kernel launched just before (PDL)
    int pf_rows;          // rows of the slab asked into the L2 while waiting for that kernel
};

// ------------------------------------------------------------------------------------------
// Selection.  Candidates are (key, id) with key = f2key(logit) and key 0 = none; the order is
// (key descending, id ascending).  Every lane offers the head of a list that is already in that
// order; each round takes the best head of the warp and advances that lane's list.  Lane j < k
// ends up with the j-th best.

// One round: does this lane's head win?  The winner has the largest key, and among equal keys
// the lowest id (the second reduction runs only when keys tie).  With no candidate left the
// "winner" is an empty entry (key 0, id kFmaNoId).
__device__ __forceinline__ bool round_winner(uint32_t hk, int hi)
{
    const uint32_t wk = warp_max_u32(hk);
    bool win = hk == wk;
    const unsigned tied = __ballot_sync(0xffffffffu, win);
    if (tied & (tied - 1)) {
        const uint32_t wi = warp_min_u32(win ? (uint32_t)hi : 0xffffffffu);
        win = win && (uint32_t)hi == wi;
    }
    return win;
}

// The winner of round j drops its head into out_k[j], out_i[j] (shared memory, one pair of
// 32-entry arrays per warp), so nothing but the pop of the winner's list sits between two
// rounds, and that pop is a select, not a branch.

// Lists held in registers, NL entries per lane (unused entries: key 0, id kFmaNoId).
template <int NL>
__device__ __forceinline__ void warp_topk_regs(uint32_t (&ck)[NL], int (&ci)[NL], int k, uint32_t* out_k, int* out_i)
{
    for (int j = 0; j < k; ++j) {
        const bool win = round_winner(ck[0], ci[0]);
        if (win) { out_k[j] = ck[0]; out_i[j] = ci[0]; }
#pragma unroll
        for (int s = 0; s + 1 < NL; ++s) { ck[s] = win ? ck[s + 1] : ck[s]; ci[s] = win ? ci[s + 1] : ci[s]; }
        ck[NL - 1] = win ? 0u : ck[NL - 1];
        ci[NL - 1] = win ? kFmaNoId : ci[NL - 1];
    }
}

// Lists held in shared memory: this lane's list is keys[0..len), ids[0..len).  The entry after
// the head is fetched ahead, so a pop never waits for shared memory.
__device__ __forceinline__ void warp_topk_smem(const uint32_t* keys, const int* ids, int len, int k, uint32_t* out_k,
                                               int* out_i)
{
    int pos = 0;
    uint32_t hk = len > 0 ? keys[0] : 0u;
    int hi = len > 0 ? ids[0] : kFmaNoId;
    uint32_t nk = len > 1 ? keys[1] : 0u;
    int ni = len > 1 ? ids[1] : kFmaNoId;
    for (int j = 0; j < k; ++j) {
        const bool win = round_winner(hk, hi);
        if (win) { out_k[j] = hk; out_i[j] = hi; }
        pos += win ? 1 : 0;
        hk = win ? nk : hk;
        hi = win ? ni : hi;
        const bool more = pos + 1 < len;
        const int nx = more ? pos + 1 : 0;
        const uint32_t tk = keys[len > 0 ? nx : 0];
        const int ti = ids[len > 0 ? nx : 0];
        nk = more ? tk : 0u;
        ni = more ? ti : kFmaNoId;
    }
}

// compare-exchange so that (ka, ia) comes before (kb, ib)
__device__ __forceinline__ void order2(uint32_t& ka, int& ia, uint32_t& kb, int& ib)
{
    const bool swap = (ka < kb) || (ka == kb && ia > ib);
    const uint32_t tk = swap ? kb : ka;
    const int ti = swap ? ib : ia;
    kb = swap ? ka : kb;
    ib = swap ? ia : ib;
    ka = tk;
    ia = ti;
}

// sort the first 8 candidates of a 9-entry list (19 compare-exchanges)
__device__ __forceinline__ void sort8(uint32_t (&k)[9], int (&i)[9])
{
#define SLIMSPEC_CE(a, b) order2(k[a], i[a], k[b], i[b])
    SLIMSPEC_CE(0, 1); SLIMSPEC_CE(2, 3); SLIMSPEC_CE(4, 5); SLIMSPEC_CE(6, 7);
    SLIMSPEC_CE(0, 2); SLIMSPEC_CE(1, 3); SLIMSPEC_CE(4, 6); SLIMSPEC_CE(5, 7);
    SLIMSPEC_CE(1, 2); SLIMSPEC_CE(5, 6); SLIMSPEC_CE(0, 4); SLIMSPEC_CE(3, 7);
    SLIMSPEC_CE(1, 5); SLIMSPEC_CE(2, 6);
    SLIMSPEC_CE(1, 4); SLIMSPEC_CE(3, 6);
    SLIMSPEC_CE(2, 4); SLIMSPEC_CE(3, 5);
    SLIMSPEC_CE(3, 4);
#undef SLIMSPEC_CE
}

// ------------------------------------------------------------------------------------------
// z^T = (h A)^T for M <= MT rows.  A CTA owns 16 columns of A (two 16-byte units) over all d
// rows, so no partial sums cross CTAs; a thread owns one unit and every (NT/2)-th row, with
// RB row loads in flight at a time.  Rows M..MT-1 of z^T are written as zeros.
template <int MT, int NT, int RB>
__global__ void __launch_bounds__(NT) k_fma_downproj(const bf16* __restrict__ h, const bf16* __restrict__ A, int M,
                                                         int d, int r, float* __restrict__ zT)
{
    pdl_launch_dependents();
    __shared__ float red[NT / 32][MT][16];
    const int t = threadIdx.x, u = t & 1, rl = t >> 1, lane = t & 31, warp = t >> 5;
    const int c0 = blockIdx.x * 16 + u * 8;
    constexpr int RSTEP = NT / 2;
    // Launched early (programmatic dependent launch), this kernel may start while the kernel before
    // it in the stream is still finishing: until that one is complete it only asks the L2 for its
    // slice of A (a hint; no value is read), then it waits.  h and z^T are touched after the wait.
    if (u == 0) {
        for (int i = rl; i < d; i += RSTEP) prefetch_l2(A + (size_t)i * r + c0);
    }
    pdl_wait();

    float acc[MT][8];
#pragma unroll
    for (int m = 0; m < MT; ++m)
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[m][c] = 0.f;

    for (int i0 = rl; i0 < d; i0 += RSTEP * RB) {
        uint4 a[RB];
        float hv[MT][RB];
#pragma unroll
        for (int j = 0; j < RB; ++j) {
            const int i = i0 + j * RSTEP;
            a[j] = (i < d) ? __ldg(reinterpret_cast<const uint4*>(A + (size_t)i * r + c0)) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
            for (int m = 0; m < MT; ++m) hv[m][j] = (i < d && m < M) ? __bfloat162float(h[(size_t)m * d + i]) : 0.f;
        }
#pragma unroll
        for (int j = 0; j < RB; ++j) {
            const uint32_t w[4] = {a[j].x, a[j].y, a[j].z, a[j].w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float lo = __uint_as_float(w[e] << 16), hi = __uint_as_float(w[e] & 0xffff0000u);
#pragma unroll
                for (int m = 0; m < MT; ++m) {
                    acc[m][2 * e] = fmaf(hv[m][j], lo, acc[m][2 * e]);
                    acc[m][2 * e + 1] = fmaf(hv[m][j], hi, acc[m][2 * e + 1]);
                }
            }
        }
    }
    // the 16 row lanes of a warp share a unit: fold them, then the warps through shared memory
#pragma unroll
    for (int m = 0; m < MT; ++m)
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            float v = acc[m][c];
            v += __shfl_xor_sync(0xffffffffu, v, 2);
            v += __shfl_xor_sync(0xffffffffu, v, 4);
            v += __shfl_xor_sync(0xffffffffu, v, 8);
            v += __shfl_xor_sync(0xffffffffu, v, 16);
            acc[m][c] = v;
        }
    if (lane < 2) {
#pragma unroll
        for (int m = 0; m < MT; ++m)
#pragma unroll
            for (int c = 0; c < 8; ++c) red[warp][m][lane * 8 + c] = acc[m][c];
    }
    __syncthreads();
    if (t < MT * 16) {
        const int m = t >> 4, c = t & 15;
        float v = 0.f;
#pragma unroll
        for (int w = 0; w < NT / 32; ++w) v += red[w][m][c];
        zT[(size_t)(blockIdx.x * 16 + c) * MT + m] = v;
    }
}

// z^T = widened h^T for the full-rank head (no down-projection).
__global__ void k_fma_widen_t(const bf16* __restrict__ h, int M, int MT, int d, float* __restrict__ zT)
{
    pdl_launch_dependents();
    pdl_wait();          // launched early: the kernel before it may still read z^T
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= d * MT) return;
    const int i = e / MT, m = e % MT;
    zT[e] = (m < M) ? __bfloat162float(h[(size_t)m * d + i]) : 0.f;
}

// ------------------------------------------------------------------------------------------
// The streaming head.  One CTA per V slab; thread = (column unit of 8 columns, row group).
// Every thread keeps U 128-bit loads of its column unit in flight (rows g, g+RG, g+2RG, ...),
// multiplies each arriving row by the code held in shared memory (packed FP32 FMAs) and
// refills.  The row groups' partial sums meet in shared memory; the warps of the slab then
// keep the running max / sum-exp / top-k per row (or store the logits).  The last CTA to
// finish merges the per-slab records.
__device__ __forceinline__ uint4 fma_ldg(const void* p)
{
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}

template <int MT, int U>
__global__ void __launch_bounds__(MT <= 4 ? 512 : 256, 1) k_fma_head(const FmaParams p)
{
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned int* s_ticket = reinterpret_cast<unsigned int*>(smem);
    uint32_t* sel_s = reinterpret_cast<uint32_t*>(smem + 128);           // [16 warps][32 keys, 32 ids]
    float* ep_s = reinterpret_cast<float*>(smem + 128 + 16 * 64 * 4);    // [MT][kFmaMaxColWarps][66]
    float* red = ep_s + MT * kFmaMaxColWarps * 66;                          // [RG][MT][ct*8]
    const int CT = p.ct, RG = p.rg;
    const int pass_cols = CT * 8;
    float2* zs = reinterpret_cast<float2*>(red + (size_t)RG * MT * pass_cols);   // [kc][MT] (z, z) pairs

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint32_t* sel_k = sel_s + warp * 64;             // this warp's selection output
    int* sel_i = reinterpret_cast<int*>(sel_k + 32);
    const int g = tid / CT, c = tid - g * CT;        // row group, column unit inside the pass
    const int NW = CT >> 5;                          // warps across a pass
    const int cw = warp - g * NW;                    // this warp's position across the pass
    const int cta = blockIdx.x;
    const int K = p.K, V = p.V, k = p.k;
    const int stepU = RG * U;

    // ---- this CTA's slab and its passes
    const int my_units = p.units_base + (cta < p.units_rem ? 1 : 0);
    const int unit0 = cta * p.units_base + min(cta, p.units_rem);
    const int npass = (my_units + p.pass_units - 1) / p.pass_units;
    const int units_per_pass = npass ? (my_units + npass - 1) / npass : 0;

    // Two sets of UH loads each: one set is consumed while the other is in flight, so a wait
    // for the older set never waits for loads issued after it.
    constexpr int UH = U / 2;
    uint4 q[2][UH];
    auto prologue = [&](int pass) {
        const int pu0 = pass * units_per_pass;
        const int pun = min(units_per_pass, my_units - pu0);
        const bf16* base = p.B + (size_t)(unit0 + pu0 + c) * 8;
#pragma unroll
        for (int hh = 0; hh < 2; ++hh)
#pragma unroll
            for (int j = 0; j < UH; ++j) {
                const int row = g + (hh * UH + j) * RG;
                q[hh][j] = (c < pun && row < K) ? fma_ldg(base + (size_t)row * V) : make_uint4(0u, 0u, 0u, 0u);
            }
    };
    if (npass > 0) prologue(0);
    // the weights are on their way; let the next kernel in the stream come up behind this one,
    // then wait for the kernel that writes the code
    pdl_launch_dependents();
    if (p.wait_prev) {
        // Until the code is there this CTA can only wait, and while it waits HBM idles: ask the L2
        // for the rows of the slab that come next (a hint; the loads of the main loop then hit the
        // L2).  Launched early behind a kernel that still runs, the wait is several microseconds.
        if (p.pf_rows > 0 && npass > 0) {
            const int pun0 = min(units_per_pass, my_units);
            const int lines = (pun0 * 16 + 127) / 128 + 1;          // the slab's row segment need not start on a line
            const int r0 = min(K, stepU), r1 = min(K, stepU + p.pf_rows);
            const char* seg = reinterpret_cast<const char*>(p.B + (size_t)unit0 * 8);
            const size_t row_bytes = (size_t)V * sizeof(bf16);
            const int last = pun0 * 16 - 1;                          // last byte of the row segment
            for (int i = tid; i < (r1 - r0) * lines; i += blockDim.x) {
                const int r = r0 + i / lines, l = i - (i / lines) * lines;
                prefetch_l2(seg + (size_t)r * row_bytes + min(l * 128, last));
            }
        }
        pdl_wait();
    }

    float run_max[MT], run_sum[MT];
    uint32_t lst_k[MT];                              // lane j < k: key of the j-th best so far
    int lst_i[MT];
    bool mine[MT];                                   // rows whose softmax / top-k this warp keeps
#pragma unroll
    for (int m = 0; m < MT; ++m) {
        run_max[m] = -FLT_MAX; run_sum[m] = 0.f; lst_k[m] = 0; lst_i[m] = kFmaNoId;
        mine[m] = (m % RG) == g;
    }

    for (int pass = 0; pass < npass; ++pass) {
        const int pu0 = pass * units_per_pass;
        const int pun = min(units_per_pass, my_units - pu0);
        const bool active = c < pun;
        const bf16* base = p.B + (size_t)(unit0 + pu0 + c) * 8;
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
            if (pass == 0 || p.kc < K) {
                // bring this chunk of the code into shared memory as (z, z) pairs
                if (kc0 > 0 || pass > 0) __syncthreads();
                const float* src = p.zT + (size_t)kc0 * MT;
                for (int e = tid; e < (kend - kc0) * MT; e += blockDim.x) {
                    const float zv = __ldcg(src + e);
                    zs[e] = make_float2(zv, zv);
                }
                __syncthreads();
            }
            if (active) {
                for (int row = kc0 + g; row < kend; row += stepU) {
                    // unchecked while this block and the next one lie wholly inside K
                    if (row - g + 2 * stepU <= K) block(row, kc0, kend, std::false_type());
                    else block(row, kc0, kend, std::true_type());
                }
            }
        }
        // ---- the row groups' partial sums meet in shared memory
        if (active) {
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                float* dst = red + ((size_t)g * MT + m) * pass_cols + c * 8;
                *reinterpret_cast<float4*>(dst) = make_float4(acc[m][0].x, acc[m][0].y, acc[m][1].x, acc[m][1].y);
                *reinterpret_cast<float4*>(dst + 4) = make_float4(acc[m][2].x, acc[m][2].y, acc[m][3].x, acc[m][3].y);
            }
        }
        // next pass's first loads fly while this pass's logits are reduced
        if (pass + 1 < npass) prologue(pass + 1);
        __syncthreads();

        const int col = (unit0 + pu0 + c) * 8;       // first vocabulary id of this thread
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            if (!mine[m] || m >= p.M) continue;
            float l[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) l[e] = 0.f;
            if (active) {
                for (int gg = 0; gg < RG; ++gg) {
                    const float* src = red + ((size_t)gg * MT + m) * pass_cols + c * 8;
                    const float4 a = *reinterpret_cast<const float4*>(src);
                    const float4 b = *reinterpret_cast<const float4*>(src + 4);
                    l[0] += a.x; l[1] += a.y; l[2] += a.z; l[3] += a.w;
                    l[4] += b.x; l[5] += b.y; l[6] += b.z; l[7] += b.w;
                }
            }
            if (p.mode == 1) {
                if (active) {
                    float* dst = p.logits + (size_t)m * V + col;
                    *reinterpret_cast<float4*>(dst) = make_float4(l[0], l[1], l[2], l[3]);
                    *reinterpret_cast<float4*>(dst + 4) = make_float4(l[4], l[5], l[6], l[7]);
                }
                continue;
            }
            // online softmax + running top-k of this warp's columns
            float tmax = -FLT_MAX;
            if (active) {
#pragma unroll
                for (int e = 0; e < 8; ++e) tmax = fmaxf(tmax, l[e]);
            }
            const float wmax = warp_max(tmax);
            const float nm = fmaxf(run_max[m], wmax);
            float ts = 0.f;
            if (active) {
#pragma unroll
                for (int e = 0; e < 8; ++e) ts += __expf(l[e] - nm);
            }
            run_sum[m] = run_sum[m] * __expf(run_max[m] - nm) + warp_sum(ts);
            run_max[m] = nm;
            // skip the selection when nothing here beats the current k-th best
            const uint32_t kth = __shfl_sync(0xffffffffu, lst_k[m], k - 1);
            if (f2key(wmax) < kth) continue;
            // this lane's list: its eight new logits in order, then its entry of the running list
            uint32_t ck[9];
            int ci[9];
#pragma unroll
            for (int e = 0; e < 8; ++e) { ck[e] = active ? f2key(l[e]) : 0u; ci[e] = active ? col + e : kFmaNoId; }
            sort8(ck, ci);
            ck[8] = lst_k[m];
            ci[8] = lst_i[m];
#pragma unroll
            for (int e = 7; e >= 0; --e) order2(ck[e], ci[e], ck[e + 1], ci[e + 1]);
            sel_k[lane] = 0u;
            sel_i[lane] = kFmaNoId;
            __syncwarp();
            warp_topk_regs<9>(ck, ci, k, sel_k, sel_i);
            __syncwarp();
            lst_k[m] = sel_k[lane];
            lst_i[m] = sel_i[lane];
            __syncwarp();
        }
        if (pass + 1 < npass) __syncthreads();       // the partial sums may be overwritten now
    }
    if (p.mode == 1) return;

    // ---- fold the warps across the slab into one record per (row, slab)
    // ep_s: per (row, warp) 66 words: max, sum-exp, 32 keys, 32 ids
#pragma unroll
    for (int m = 0; m < MT; ++m) {
        if (!mine[m] || m >= p.M) continue;
        float* rec = ep_s + ((size_t)m * kFmaMaxColWarps + cw) * 66;
        if (lane == 0) { rec[0] = run_max[m]; rec[1] = run_sum[m]; }
        rec[2 + lane] = __uint_as_float(lst_k[m]);
        rec[34 + lane] = __int_as_float(lst_i[m]);
    }
    __syncthreads();
    const int P = p.ncta;
    const int RW = p.rec_words;
    if (cw == 0) {
        // the lanes share out the NW sorted lists: 32 / NW lanes per list, a run of each list per lane
        const int lpl = 32 / NW;
        const int seg = (k + lpl - 1) / lpl;
        const int lw = lane / lpl, ls = lane - lw * lpl;
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            if (!mine[m] || m >= p.M) continue;
            const float* rows = ep_s + (size_t)m * kFmaMaxColWarps * 66;
            float cm = -FLT_MAX, cs = 0.f;
            if (MT > 1 || NW > 4) {
                // lane w takes warp w's (max, sum-exp); measured better than the loop except for one row
                // with up to four warps
                const float wm = lane < NW ? rows[lane * 66] : -FLT_MAX;
                cm = warp_max(wm);
                cs = warp_sum(lane < NW ? rows[lane * 66 + 1] * __expf(wm - cm) : 0.f);
            } else {
                for (int w = 0; w < NW; ++w) cm = fmaxf(cm, rows[w * 66]);
                for (int w = 0; w < NW; ++w) cs += rows[w * 66 + 1] * __expf(rows[w * 66] - cm);
            }
            const int first = ls * seg;
            const int len = (lw < NW && first < k) ? min(seg, k - first) : 0;
            const int lwc = lw < NW ? lw : 0;
            const uint32_t* lk = reinterpret_cast<const uint32_t*>(rows + lwc * 66 + 2 + first);
            const int* li = reinterpret_cast<const int*>(rows + lwc * 66 + 34 + first);
            sel_k[lane] = 0u;
            sel_i[lane] = kFmaNoId;
            __syncwarp();
            warp_topk_smem(lk, li, len, k, sel_k, sel_i);
            __syncwarp();
            const uint32_t ok = sel_k[lane];
            const int oi = sel_i[lane];
            __syncwarp();
            float* gp = p.part + ((size_t)m * P + cta) * RW;
            if (lane == 0) { gp[0] = cm; gp[1] = cs; }
            if (lane < k) {
                gp[2 + lane] = __uint_as_float(ok);
                gp[2 + k + lane] = __int_as_float(oi);
            }
        }
        __threadfence();
    }
    __syncthreads();
    if (tid == 0) *s_ticket = atomicAdd(p.ticket, 1u);
    __syncthreads();
    if (*s_ticket != (unsigned)(P - 1)) return;

    // ---- last CTA: merge the P slab records of every row, a few rows per round
    __threadfence();
    float* mrg = red;                                // the reduction and code areas are idle now
    __shared__ float lse_s[32];                      // a row's log-sum-exp, by the row's place in the round
    uint32_t* stage_k = reinterpret_cast<uint32_t*>(ep_s);            // [rows][groups][32] keys, then ids
    const int row_words = P * RW;
    const int ngroups = (P + 31) >> 5;               // groups of 32 slabs, one warp each
    const int nwarps = blockDim.x >> 5;
    for (int m0 = 0; m0 < p.M; m0 += p.merge_rows) {
        const int nrows = min(p.merge_rows, p.M - m0);
        const int n4 = nrows * row_words / 4;
        const float4* src = reinterpret_cast<const float4*>(p.part + (size_t)m0 * row_words);
        float4* dst = reinterpret_cast<float4*>(mrg);
        // batches of independent loads: the records sit in L2, one round trip per batch
        for (int i0 = tid; i0 < n4; i0 += blockDim.x * 8) {
            float4 t[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int i = i0 + j * blockDim.x;
                t[j] = (i < n4) ? __ldcg(src + i) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int i = i0 + j * blockDim.x;
                if (i < n4) dst[i] = t[j];
            }
        }
        __syncthreads();
        // first level: a warp takes 32 slabs of one row, a lane per slab list
        int* stage_i = reinterpret_cast<int*>(stage_k + (size_t)nrows * ngroups * 32);
        for (int job = warp; job < nrows * ngroups; job += nwarps) {
            const int rrow = job / ngroups, grp = job - rrow * ngroups;
            const int s = grp * 32 + lane;
            const float* rec = mrg + (size_t)rrow * row_words + (size_t)(s < P ? s : 0) * RW;
            stage_k[(size_t)job * 32 + lane] = 0u;
            stage_i[(size_t)job * 32 + lane] = kFmaNoId;
            __syncwarp();
            warp_topk_smem(reinterpret_cast<const uint32_t*>(rec + 2), reinterpret_cast<const int*>(rec + 2 + k),
                           s < P ? k : 0, k, stage_k + (size_t)job * 32, stage_i + (size_t)job * 32);
        }
        // meanwhile the warps at the other end take the rows' log-sum-exp (it needs no list)
        if (warp >= nwarps - nrows) {
            const int rrow = nwarps - 1 - warp;
            const float* rows = mrg + (size_t)rrow * row_words;
            float gm = -FLT_MAX;
            for (int s = lane; s < P; s += 32) gm = fmaxf(gm, rows[(size_t)s * RW]);
            gm = warp_max(gm);
            float gs = 0.f;
            for (int s = lane; s < P; s += 32) gs += rows[(size_t)s * RW + 1] * __expf(rows[(size_t)s * RW] - gm);
            gs = warp_sum(gs);
            if (lane == 0) lse_s[rrow] = gm + __logf(gs);
        }
        __syncthreads();
        // second level: a warp per row folds the groups' lists and finishes the log-softmax
        if (warp < nrows) {
            const int m = m0 + warp;
            const float lse = lse_s[warp];
            const int lpl = 32 / ngroups;
            const int seg = (k + lpl - 1) / lpl;
            const int lw = lane / lpl, ls = lane - lw * lpl;
            const int first = ls * seg;
            const int len = (lw < ngroups && first < k) ? min(seg, k - first) : 0;
            const size_t off = ((size_t)warp * ngroups + (lw < ngroups ? lw : 0)) * 32 + first;
            sel_k[lane] = 0u;
            sel_i[lane] = kFmaNoId;
            __syncwarp();
            warp_topk_smem(stage_k + off, stage_i + off, len, k, sel_k, sel_i);
            __syncwarp();
            const uint32_t ok = sel_k[lane];
            const int oi = sel_i[lane];
            if (lane < k) {
                p.ids[(size_t)m * k + lane] = oi;
                p.logprobs[(size_t)m * k + lane] = key2f(ok) - lse;
            }
        }
        __syncthreads();
    }
    if (tid == 0) *p.ticket = 0;
}

// ------------------------------------------------------------------------------------------
static int fma_pick_mt(int M) { return M <= 1 ? 1 : 2; }

struct FmaGeometry {
    int ncta, units_base, units_rem, pass_units, ct, rg, u, kc, rec_words, merge_rows, threads;
    size_t smem;
};

static bool fma_geometry(int mt, int K, int V, int k, int sm_count, FmaGeometry* g)
{
    if (V % 8 != 0 || K < 1 || k > 32 || k < 1) return false;
    const int units = V / 8;
    int ncta = sm_count < kFmaMaxCtas ? sm_count : kFmaMaxCtas;
    if (ncta > units) ncta = units;
    g->ncta = ncta;
    g->units_base = units / ncta;
    g->units_rem = units % ncta;
    const int max_units = g->units_base + (g->units_rem ? 1 : 0);
    const int npass = (max_units + kFmaMaxColThreads - 1) / kFmaMaxColThreads;
    g->pass_units = (max_units + npass - 1) / npass;
    g->ct = (g->pass_units + 31) / 32 * 32;
    const int nt_max = mt <= 4 ? 512 : 256;
    g->rg = nt_max / g->ct;
    if (g->rg < 1) g->rg = 1;
    if (g->rg > K) g->rg = K;
    g->threads = g->ct * g->rg;
    g->u = (mt == 4) ? 8 : 16;
    // rows of the code per shared-memory chunk: all of K if it fits, else a multiple of rg*u
    const int kc_max = kFmaZChunkBytes / (mt * 8);
    if (K <= kc_max) g->kc = K;
    else {
        g->kc = kc_max / (g->rg * g->u) * (g->rg * g->u);
        if (g->kc < 1) return false;
    }
    g->rec_words = (2 + 2 * k + 3) / 4 * 4;
    const size_t fixed = 128 + 16 * 64 * 4 + (size_t)mt * kFmaMaxColWarps * 66 * 4;
    const size_t work = (size_t)g->threads * mt * 32 + (size_t)g->kc * mt * 8;
    const size_t one_row = (size_t)ncta * g->rec_words * 4;
    const size_t area = work > one_row ? work : one_row;
    g->merge_rows = (int)(area / one_row);
    if (g->merge_rows > g->threads / 32) g->merge_rows = g->threads / 32;
    // the first merge level parks rows * groups lists of 32 (key, id) pairs where the warps' records were
    const int groups = (ncta + 31) / 32;
    const int park = (int)((size_t)mt * kFmaMaxColWarps * 66 * 4 / ((size_t)groups * 32 * 8));
    if (park < 1) return false;
    if (g->merge_rows > park) g->merge_rows = park;
    g->smem = fixed + area;
    return g->smem <= 200 * 1024;
}

FmaPlan fma_plan(int M, int d, int K, int V, int k, int sm_count)
{
    FmaPlan sp = {0, 0, 0, 0};
    (void)d;
    if (M < 1 || M > 2) return sp;
    const int mt = fma_pick_mt(M);
    FmaGeometry g;
    if (!fma_geometry(mt, K, V, k, sm_count, &g)) return sp;
    sp.ok = 1;
    sp.mt = mt;
    sp.ncta = g.ncta;
    sp.launches = 2;
    return sp;
}

// Launch with programmatic stream serialization: the kernel may begin once every CTA of the kernel
// before it in the stream has signalled launch_dependents or left; it orders itself after that
// kernel with griddepcontrol.wait.  Across calls this hides the launch gap and lets the first
// kernel of a call warm up under the tail of the last kernel of the call before.
template <typename... KArgs, typename... Args>
static cudaError_t fma_launch_early(void (*kern)(KArgs...), int grid, int block, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

cudaError_t fma_downproj(const bf16* h, const bf16* A, int M, int mt, int d, int r, const Scratch& s,
                            cudaStream_t st)
{
    const int grid = r / 16;
    switch (mt) {
    case 1: return fma_launch_early(k_fma_downproj<1, 1024, 8>, grid, 1024, st, h, A, M, d, r, s.z);
    default: return fma_launch_early(k_fma_downproj<2, 1024, 4>, grid, 1024, st, h, A, M, d, r, s.z);
    }
}

cudaError_t fma_widen_t(const bf16* h, int M, int mt, int d, float* zT, cudaStream_t st)
{
    const int n = d * mt;
    return fma_launch_early(k_fma_widen_t, (n + 255) / 256, 256, st, h, M, mt, d, zT);
}

// Once per device: load the kernels and allow the head kernels their dynamic shared memory.
cudaError_t fma_prepare()
{
    cudaError_t e;
    cudaFuncAttributes fa;
    if ((e = cudaFuncGetAttributes(&fa, k_fma_downproj<1, 1024, 8>)) != cudaSuccess) return e;
    if ((e = cudaFuncGetAttributes(&fa, k_fma_downproj<2, 1024, 4>)) != cudaSuccess) return e;
    if ((e = cudaFuncGetAttributes(&fa, k_fma_widen_t)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(k_fma_head<1, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(k_fma_head<2, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024)) != cudaSuccess) return e;
    return cudaSuccess;
}

template <int MT, int U>
static cudaError_t fma_launch_head(const FmaParams& hp, const FmaGeometry& g, bool pdl, cudaStream_t st)
{
    auto kern = k_fma_head<MT, U>;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(hp.ncta);
    cfg.blockDim = dim3(g.threads);
    cfg.dynamicSmemBytes = g.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, hp);
}

cudaError_t fma_head(const float* zT, const bf16* B, int M, int mt, int K, int V, int k, int mode,
                        int32_t* ids, float* logprobs, float* logits, const Scratch& s, int sm_count,
                        bool after_producer_kernel, cudaStream_t st)
{
    FmaGeometry g;
    if (!fma_geometry(mt, K, V, k, sm_count, &g)) return cudaErrorInvalidValue;
    if (g.ncta > s.max_parts) return cudaErrorInvalidValue;
    FmaParams hp;
    hp.zT = zT; hp.B = B; hp.M = M; hp.K = K; hp.V = V; hp.k = k; hp.mode = mode;
    hp.ncta = g.ncta; hp.units_base = g.units_base; hp.units_rem = g.units_rem; hp.pass_units = g.pass_units;
    hp.ct = g.ct; hp.rg = g.rg; hp.kc = g.kc; hp.rec_words = g.rec_words; hp.merge_rows = g.merge_rows;
    hp.ids = ids; hp.logprobs = logprobs; hp.logits = logits;
    hp.part = s.part; hp.ticket = s.tickets; hp.err = s.err;
    hp.wait_prev = after_producer_kernel ? 1 : 0;
    {
        const size_t row_bytes = (size_t)g.pass_units * 16 * g.ncta;      // one row of every slab's first pass
        const size_t rows = row_bytes ? kFmaPrefetchBytes / row_bytes : 0;
        hp.pf_rows = after_producer_kernel ? (int)(rows < (size_t)K ? rows : (size_t)K) : 0;
    }
    switch (mt) {
    case 1: return fma_launch_head<1, 16>(hp, g, after_producer_kernel, st);
    default: return fma_launch_head<2, 16>(hp, g, after_producer_kernel, st);
    }
}

}  // namespace slimspec
