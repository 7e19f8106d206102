// Streaming path for small M (<= 8 rows per launch): the K x V weight matrix is read from HBM
// exactly once, in split-V slabs (one CTA per SM), staged through shared memory by bulk
// asynchronous copies (TMA) and consumed with 128-bit shared loads and FP32 FMAs.
// The logits never leave the SM: each CTA keeps a running max / sum-exp / top-k per row and
// the last CTA to finish merges the per-slab records (Section 4.1 up-projection, the
// softmax of Section 3.2 in online form, and the candidate selection).
#include "kernels.h"
#include "ptx.cuh"
#include <float.h>

namespace slimspec {

static constexpr int kRowsPerStage = 16;     // rows of the K x V matrix per pipeline stage
static constexpr int kColThreads = 128;      // threads across one pass's columns, 8 columns each
static constexpr int kEpiWarps = 4;
static constexpr int kMaxStages = 12;
static constexpr int kMaxCtas = 256;         // slabs per row the merge can take (8 lists per lane)
static constexpr int kListPerLane = kMaxCtas / 32;
// Leave ~28 KB of the SM's shared memory to the kernel that produces z, so that it can share
// the SM with this kernel's prologue under programmatic dependent launch.
static constexpr int kSmemBudget = 200 * 1024;

struct HeadParams {
    const float* zT;      // [K][MT] fp32 code, transposed and zero-padded to MT rows
    const bf16* B;        // [K][V]
    int M, K, V, k, mode;
    int ncta;             // slabs
    int units_base, units_rem;   // V/8 column units: slab c has units_base + (c < units_rem)
    int pass_units;       // most units one pass covers (<= 128)
    int nstages;
    int pitch;            // bytes between staged rows = pass_units * 16
    int32_t* ids;
    float* logprobs;
    float* logits;
    float* part;          // split-V records
    unsigned int* ticket;
    int* err;
    int wait_prev;        // 1: zT is written by the kernel launched just before (PDL)
};

// ------------------------------------------------------------------------------------------
// warp-level selection: every lane holds NC candidates (key = f2key(value), 0 = empty; id).
// Afterwards lane j < k holds the j-th best in (value desc, id asc) order.
template <int NC>
__device__ __forceinline__ void warp_select(uint32_t (&ck)[NC], int (&ci)[NC], int k, int lane, uint32_t& outk,
                                            int& outi)
{
    outk = 0;
    outi = 0x7fffffff;
    for (int j = 0; j < k; ++j) {
        uint32_t bk = ck[0];
        int bi = ci[0];
        int bs = 0;
#pragma unroll
        for (int s = 1; s < NC; ++s) {
            bool better = ck[s] > bk || (ck[s] == bk && ci[s] < bi);
            bk = better ? ck[s] : bk;
            bi = better ? ci[s] : bi;
            bs = better ? s : bs;
        }
        const uint32_t wk = warp_max_u32(bk);
        const uint32_t wi = warp_min_u32(bk == wk ? (uint32_t)bi : 0xffffffffu);
        const bool win = (bk == wk) && ((uint32_t)bi == wi);
#pragma unroll
        for (int s = 0; s < NC; ++s)
            if (win && s == bs) ck[s] = 0;
        if (lane == j) { outk = wk; outi = (int)wi; }
    }
}

// ------------------------------------------------------------------------------------------
// z^T = (h A)^T for M <= 8 rows.  Grid (r/64, S): a CTA sums a slab of d for 64 columns of A,
// the last CTA of a column block adds the S partial sums in slab order (deterministic).
template <int MT>
__global__ void __launch_bounds__(256) k_stream_downproj(const bf16* __restrict__ h, const bf16* __restrict__ A,
                                                          int M, int d, int r, int slab, float* __restrict__ zpart,
                                                          float* __restrict__ zT, unsigned int* __restrict__ tickets)
{
    pdl_launch_dependents();
    __shared__ float red[8][MT][64];
    __shared__ unsigned int s_ticket;
    const int t = threadIdx.x, cg = t & 7, rl = t >> 3, lane = t & 31, warp = t >> 5;
    const int c0 = blockIdx.x * 64;
    const int i0 = blockIdx.y * slab;
    const int i1 = min(i0 + slab, d);
    const int S = gridDim.y;

    float acc[MT][8];
#pragma unroll
    for (int m = 0; m < MT; ++m)
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[m][c] = 0.f;

    for (int i = i0 + rl; i < i1; i += 32) {
        const uint4 q = *reinterpret_cast<const uint4*>(A + (size_t)i * r + c0 + cg * 8);
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
        float a[8];
#pragma unroll
        for (int p = 0; p < 4; ++p) {
            a[2 * p] = __uint_as_float(w[p] << 16);
            a[2 * p + 1] = __uint_as_float(w[p] & 0xffff0000u);
        }
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            if (m < M) {
                const float hv = __bfloat162float(h[(size_t)m * d + i]);
#pragma unroll
                for (int c = 0; c < 8; ++c) acc[m][c] = fmaf(hv, a[c], acc[m][c]);
            }
        }
    }
    // the four row lanes of a warp share a column group: fold them, then the eight warps
#pragma unroll
    for (int m = 0; m < MT; ++m)
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            float v = acc[m][c];
            v += __shfl_xor_sync(0xffffffffu, v, 8);
            v += __shfl_xor_sync(0xffffffffu, v, 16);
            acc[m][c] = v;
        }
    if (lane < 8) {
#pragma unroll
        for (int m = 0; m < MT; ++m)
#pragma unroll
            for (int c = 0; c < 8; ++c) red[warp][m][lane * 8 + c] = acc[m][c];
    }
    __syncthreads();
    for (int e = t; e < MT * 64; e += 256) {
        const int m = e / 64, c = e % 64;
        float v = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) v += red[w][m][c];
        if (S == 1) zT[(size_t)(c0 + c) * MT + m] = v;
        else zpart[((size_t)blockIdx.y * r + c0 + c) * MT + m] = v;
    }
    if (S == 1) return;
    __threadfence();
    __syncthreads();
    if (t == 0) s_ticket = atomicAdd(&tickets[blockIdx.x], 1u);
    __syncthreads();
    if (s_ticket != (unsigned)(S - 1)) return;
    __threadfence();
    for (int e = t; e < MT * 64; e += 256) {
        const int m = e % MT, c = e / MT;
        float v = 0.f;
        for (int s = 0; s < S; ++s) v += __ldcg(&zpart[((size_t)s * r + c0 + c) * MT + m]);
        zT[(size_t)(c0 + c) * MT + m] = v;
    }
    if (t == 0) tickets[blockIdx.x] = 0;
}

// z^T = widened h^T for the full-rank head (no down-projection).
__global__ void k_stream_widen_t(const bf16* __restrict__ h, int M, int MT, int d, float* __restrict__ zT)
{
    pdl_launch_dependents();
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= d * MT) return;
    const int i = e / MT, m = e % MT;
    zT[e] = (m < M) ? __bfloat162float(h[(size_t)m * d + i]) : 0.f;
}

// ------------------------------------------------------------------------------------------
// The streaming head.  Warp roles: warp 0 producer (bulk copies), 4*KG consumer warps
// (thread = 8 columns x one of KG row groups of a stage), 4 epilogue warps (sum the row
// groups' partial sums; running softmax / top-k, or logit store; final merge).
template <int MT, int KG>
__global__ void __launch_bounds__(32 + 128 * KG + 32 * kEpiWarps, 1) k_stream_head(const HeadParams p)
{
    constexpr int RPG = kRowsPerStage / KG;          // rows per group per stage
    constexpr int NCONS = 4 * KG;                    // consumer warps
    extern __shared__ __align__(128) unsigned char smem[];

    // ---- shared memory carve-up
    uint64_t* full = reinterpret_cast<uint64_t*>(smem);            // [kMaxStages]
    uint64_t* empty = full + kMaxStages;                           // [kMaxStages]
    uint64_t* acc_ready = empty + kMaxStages;
    uint64_t* acc_free = acc_ready + 1;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(acc_free + 1);
    unsigned int* s_ticket = reinterpret_cast<unsigned int*>(const_cast<int*>(abort_flag) + 1);
    float* ep_s = reinterpret_cast<float*>(smem + 256);            // [kEpiWarps][MT][66]
    const int pass_cols = p.pass_units * 8;
    float* part_s = ep_s + kEpiWarps * MT * 66;                    // [KG][MT][pass_cols]
    unsigned char* stage0 = reinterpret_cast<unsigned char*>(part_s + (size_t)KG * MT * pass_cols);
    stage0 = reinterpret_cast<unsigned char*>(((uintptr_t)stage0 + 127) & ~(uintptr_t)127);
    const int ztile_bytes = kRowsPerStage * MT * 4;
    const int stage_bytes = kRowsPerStage * p.pitch + ((ztile_bytes + 127) & ~127);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x;

    // ---- this CTA's slab and its passes
    const int my_units = p.units_base + (cta < p.units_rem ? 1 : 0);
    const int unit0 = cta * p.units_base + min(cta, p.units_rem);
    const int npass = (my_units + p.pass_units - 1) / p.pass_units;
    const int units_per_pass = npass ? (my_units + npass - 1) / npass : 0;
    const int kchunks = p.K / kRowsPerStage;
    const int total = npass * kchunks;

    if (tid == 0) {
        for (int s = 0; s < p.nstages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], NCONS); }
        mbar_init(acc_ready, NCONS);
        mbar_init(acc_free, kEpiWarps);
        *abort_flag = 0;
        mbar_fence_init();
    }
    __syncthreads();

    if (warp == 0) {
        // ================= producer =================
        const int prefetch = min(p.nstages, total);
        for (int it = 0; it < total; ++it) {
            const int slot = it % p.nstages, use = it / p.nstages;
            const int pass = it / kchunks, kc = it - pass * kchunks;
            const int pu0 = pass * units_per_pass;
            const int pun = min(units_per_pass, my_units - pu0);
            const uint32_t row_bytes = (uint32_t)pun * 16u;
            unsigned char* st = stage0 + (size_t)slot * stage_bytes;
            if (use > 0 && !mbar_wait(&empty[slot], (use - 1) & 1, abort_flag, p.err, ERR_WAIT_EMPTY)) break;
            if (lane == 0) mbar_arrive_expect_tx(&full[slot], row_bytes * kRowsPerStage + ztile_bytes);
            __syncwarp();
            if (lane < kRowsPerStage) {
                const bf16* src = p.B + (size_t)(kc * kRowsPerStage + lane) * p.V + (size_t)(unit0 + pu0) * 8;
                bulk_g2s(st + (size_t)lane * p.pitch, src, row_bytes, &full[slot]);
            }
            const bool z_now = !(p.wait_prev && it < prefetch);
            if (z_now && lane == kRowsPerStage)
                bulk_g2s(st + kRowsPerStage * p.pitch, p.zT + (size_t)kc * kRowsPerStage * MT, ztile_bytes, &full[slot]);
            if (p.wait_prev && it == prefetch - 1) {
                // weights of the first stages are in flight; now wait for the kernel that writes z
                pdl_wait();
                if (lane == kRowsPerStage) {
                    for (int j = 0; j < prefetch; ++j) {
                        const int kcj = j % kchunks;
                        unsigned char* sj = stage0 + (size_t)(j % p.nstages) * stage_bytes;
                        bulk_g2s(sj + kRowsPerStage * p.pitch, p.zT + (size_t)kcj * kRowsPerStage * MT, ztile_bytes,
                                 &full[j % p.nstages]);
                    }
                }
            }
        }
    } else if (warp <= NCONS) {
        // ================= consumers =================
        const int cw = warp - 1;
        const int g = cw >> 2;                          // row group
        const int ct = ((cw & 3) << 5) | lane;          // column unit inside the pass
        float acc[MT][8];
        int it = 0;
        bool alive = true;
        for (int pass = 0; pass < npass && alive; ++pass) {
            const int pu0 = pass * units_per_pass;
            const int pun = min(units_per_pass, my_units - pu0);
            const bool active = ct < pun;
#pragma unroll
            for (int m = 0; m < MT; ++m)
#pragma unroll
                for (int c = 0; c < 8; ++c) acc[m][c] = 0.f;
            for (int kc = 0; kc < kchunks; ++kc, ++it) {
                const int slot = it % p.nstages, use = it / p.nstages;
                if (!mbar_wait(&full[slot], use & 1, abort_flag, p.err, ERR_WAIT_FULL)) { alive = false; break; }
                const unsigned char* st = stage0 + (size_t)slot * stage_bytes;
                const float* zt = reinterpret_cast<const float*>(st + kRowsPerStage * p.pitch) + g * RPG * MT;
                if (active) {
                    const unsigned char* bp = st + (size_t)(g * RPG) * p.pitch + ct * 16;
#pragma unroll
                    for (int rr = 0; rr < RPG; ++rr) {
                        const uint4 q = *reinterpret_cast<const uint4*>(bp + (size_t)rr * p.pitch);
                        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
                        float zv[MT];
                        if constexpr (MT == 1) {
                            zv[0] = zt[rr];
                        } else if constexpr (MT == 2) {
                            const float2 t2 = *reinterpret_cast<const float2*>(zt + rr * 2);
                            zv[0] = t2.x; zv[1] = t2.y;
                        } else {
#pragma unroll
                            for (int m4 = 0; m4 < MT / 4; ++m4) {
                                const float4 t4 = *reinterpret_cast<const float4*>(zt + rr * MT + m4 * 4);
                                zv[m4 * 4 + 0] = t4.x; zv[m4 * 4 + 1] = t4.y; zv[m4 * 4 + 2] = t4.z; zv[m4 * 4 + 3] = t4.w;
                            }
                        }
#pragma unroll
                        for (int pq = 0; pq < 4; ++pq) {
                            const float lo = __uint_as_float(w[pq] << 16);
                            const float hi = __uint_as_float(w[pq] & 0xffff0000u);
                            if constexpr (MT >= 4) {
#pragma unroll
                                for (int m = 0; m < MT; ++m) {
                                    float2 r2 = __ffma2_rn(make_float2(lo, hi), make_float2(zv[m], zv[m]),
                                                           make_float2(acc[m][2 * pq], acc[m][2 * pq + 1]));
                                    acc[m][2 * pq] = r2.x;
                                    acc[m][2 * pq + 1] = r2.y;
                                }
                            } else {
#pragma unroll
                                for (int m = 0; m < MT; ++m) {
                                    acc[m][2 * pq] = fmaf(lo, zv[m], acc[m][2 * pq]);
                                    acc[m][2 * pq + 1] = fmaf(hi, zv[m], acc[m][2 * pq + 1]);
                                }
                            }
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty[slot]);
            }
            if (!alive) break;
            // hand this pass's partial sums to the epilogue warps
            if (pass > 0 && !mbar_wait(acc_free, (pass - 1) & 1, abort_flag, p.err, ERR_WAIT_FREE)) { alive = false; break; }
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                if (!active) break;        // columns past the pass would land in the next group's row
                float* dst = part_s + ((size_t)g * MT + m) * pass_cols + ct * 8;
                *reinterpret_cast<float4*>(dst) = make_float4(acc[m][0], acc[m][1], acc[m][2], acc[m][3]);
                *reinterpret_cast<float4*>(dst + 4) = make_float4(acc[m][4], acc[m][5], acc[m][6], acc[m][7]);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_ready);
        }
    } else {
        // ================= epilogue =================
        const int ew = warp - 1 - NCONS;
        const int et = (ew << 5) | lane;                 // column unit inside the pass
        const int k = p.k;
        float run_max[MT], run_sum[MT];
        uint32_t lst_k[MT];                              // lane j < k: key of the j-th best so far
        int lst_i[MT];
#pragma unroll
        for (int m = 0; m < MT; ++m) { run_max[m] = -FLT_MAX; run_sum[m] = 0.f; lst_k[m] = 0; lst_i[m] = 0x7fffffff; }
        bool alive = true;
        for (int pass = 0; pass < npass; ++pass) {
            const int pu0 = pass * units_per_pass;
            const int pun = min(units_per_pass, my_units - pu0);
            const bool active = et < pun;
            const int col = (unit0 + pu0 + et) * 8;      // first vocabulary id of this thread
            if (!mbar_wait(acc_ready, pass & 1, abort_flag, p.err, ERR_WAIT_ACC)) { alive = false; break; }
            float l[MT][8];
#pragma unroll
            for (int m = 0; m < MT; ++m) {
#pragma unroll
                for (int c = 0; c < 8; ++c) l[m][c] = 0.f;
                if (active) {
#pragma unroll
                    for (int g = 0; g < KG; ++g) {
                        const float* src = part_s + ((size_t)g * MT + m) * pass_cols + et * 8;
                        const float4 a = *reinterpret_cast<const float4*>(src);
                        const float4 b = *reinterpret_cast<const float4*>(src + 4);
                        l[m][0] += a.x; l[m][1] += a.y; l[m][2] += a.z; l[m][3] += a.w;
                        l[m][4] += b.x; l[m][5] += b.y; l[m][6] += b.z; l[m][7] += b.w;
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_free);
            if (p.mode == 1) {
                if (active) {
#pragma unroll
                    for (int m = 0; m < MT; ++m) {
                        if (m < p.M) {
                            float* dst = p.logits + (size_t)m * p.V + col;
                            *reinterpret_cast<float4*>(dst) = make_float4(l[m][0], l[m][1], l[m][2], l[m][3]);
                            *reinterpret_cast<float4*>(dst + 4) = make_float4(l[m][4], l[m][5], l[m][6], l[m][7]);
                        }
                    }
                }
                continue;
            }
            // online softmax + running top-k of this warp's columns
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                float tmax = -FLT_MAX;
                if (active) {
#pragma unroll
                    for (int c = 0; c < 8; ++c) tmax = fmaxf(tmax, l[m][c]);
                }
                const float wmax = warp_max(tmax);
                const float nm = fmaxf(run_max[m], wmax);
                float ts = 0.f;
                if (active) {
#pragma unroll
                    for (int c = 0; c < 8; ++c) ts += __expf(l[m][c] - nm);
                }
                run_sum[m] = run_sum[m] * __expf(run_max[m] - nm) + warp_sum(ts);
                run_max[m] = nm;
                // skip the selection when nothing here beats the current k-th best
                const uint32_t kth = __shfl_sync(0xffffffffu, lst_k[m], k - 1);
                if (f2key(wmax) < kth) continue;
                uint32_t ck[9];
                int ci[9];
#pragma unroll
                for (int c = 0; c < 8; ++c) { ck[c] = active ? f2key(l[m][c]) : 0u; ci[c] = active ? col + c : 0x7fffffff; }
                ck[8] = lst_k[m];
                ci[8] = lst_i[m];
                warp_select<9>(ck, ci, k, lane, lst_k[m], lst_i[m]);
            }
        }
        if (p.mode == 1 || !alive) return;

        // ---- fold the four epilogue warps into one record per (row, slab)
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            float* rec = ep_s + ((size_t)ew * MT + m) * 66;
            if (lane == 0) { rec[0] = run_max[m]; rec[1] = run_sum[m]; }
            rec[2 + lane] = __uint_as_float(lst_k[m]);
            rec[34 + lane] = __int_as_float(lst_i[m]);
        }
        named_bar_sync(1, 32 * kEpiWarps);
        const int P = p.ncta;
        const size_t rec_stride = (size_t)P * (2 + 2 * k);
        for (int m = ew; m < p.M; m += kEpiWarps) {
            float cm = -FLT_MAX;
#pragma unroll
            for (int w = 0; w < kEpiWarps; ++w) cm = fmaxf(cm, ep_s[((size_t)w * MT + m) * 66]);
            float cs = 0.f;
            uint32_t ck[kEpiWarps];
            int ci[kEpiWarps];
#pragma unroll
            for (int w = 0; w < kEpiWarps; ++w) {
                const float* rec = ep_s + ((size_t)w * MT + m) * 66;
                cs += rec[1] * __expf(rec[0] - cm);
                ck[w] = __float_as_uint(rec[2 + lane]);
                ci[w] = __float_as_int(rec[34 + lane]);
            }
            uint32_t ok;
            int oi;
            warp_select<kEpiWarps>(ck, ci, k, lane, ok, oi);
            float* gp = p.part + (size_t)m * rec_stride;
            if (lane == 0) { gp[cta] = cm; gp[P + cta] = cs; }
            if (lane < k) {
                gp[2 * P + (size_t)cta * k + lane] = __uint_as_float(ok);
                gp[2 * P + (size_t)P * k + (size_t)cta * k + lane] = __int_as_float(oi);
            }
        }
        __threadfence();
        named_bar_sync(1, 32 * kEpiWarps);
        if (ew == 0 && lane == 0) *s_ticket = atomicAdd(p.ticket, 1u);
        named_bar_sync(1, 32 * kEpiWarps);
        if (*s_ticket != (unsigned)(P - 1)) return;

        // ---- last CTA: merge the P slab records of every row
        __threadfence();
        // the pipeline stages are idle now; reuse them to hold one row's candidate lists per warp
        uint32_t* cand = reinterpret_cast<uint32_t*>(stage0) + (size_t)ew * 2 * P * k;
        for (int m = ew; m < p.M; m += kEpiWarps) {
            const float* gp = p.part + (size_t)m * rec_stride;
            float gm = -FLT_MAX;
            for (int c = lane; c < P; c += 32) gm = fmaxf(gm, __ldcg(gp + c));
            gm = warp_max(gm);
            float gs = 0.f;
            for (int c = lane; c < P; c += 32) gs += __ldcg(gp + P + c) * __expf(__ldcg(gp + c) - gm);
            gs = warp_sum(gs);
            const float lse = gm + __logf(gs);
            for (int e = lane; e < 2 * P * k; e += 32) cand[e] = __float_as_uint(__ldcg(gp + 2 * P + e));
            __syncwarp();
            // lane owns slabs lane, lane+32, ...; each slab list is sorted, so only heads compete
            uint32_t hk[kListPerLane];
            int hi[kListPerLane];
            int hp[kListPerLane];
#pragma unroll
            for (int q = 0; q < kListPerLane; ++q) {
                const int c = lane + 32 * q;
                hp[q] = 0;
                hk[q] = (c < P) ? cand[(size_t)c * k] : 0u;
                hi[q] = (c < P) ? (int)cand[(size_t)P * k + (size_t)c * k] : 0x7fffffff;
            }
            uint32_t ok = 0;
            int oi = 0x7fffffff;
            for (int j = 0; j < k; ++j) {
                uint32_t bk = hk[0];
                int bi = hi[0], bs = 0;
#pragma unroll
                for (int q = 1; q < kListPerLane; ++q) {
                    const bool better = hk[q] > bk || (hk[q] == bk && hi[q] < bi);
                    bk = better ? hk[q] : bk;
                    bi = better ? hi[q] : bi;
                    bs = better ? q : bs;
                }
                const uint32_t wk = warp_max_u32(bk);
                const uint32_t wi = warp_min_u32(bk == wk ? (uint32_t)bi : 0xffffffffu);
                const bool win = (bk == wk) && ((uint32_t)bi == wi);
                if (win && wk != 0u) {
#pragma unroll
                    for (int q = 0; q < kListPerLane; ++q) {
                        if (q == bs) {
                            const int c = lane + 32 * q;
                            const int np = hp[q] + 1;
                            hp[q] = np;
                            hk[q] = (np < k) ? cand[(size_t)c * k + np] : 0u;
                            hi[q] = (np < k) ? (int)cand[(size_t)P * k + (size_t)c * k + np] : 0x7fffffff;
                        }
                    }
                }
                if (lane == j) { ok = wk; oi = (int)wi; }
            }
            if (lane < k) {
                p.ids[(size_t)m * k + lane] = oi;
                p.logprobs[(size_t)m * k + lane] = key2f(ok) - lse;
            }
            __syncwarp();
        }
        if (ew == 0 && lane == 0) *p.ticket = 0;
    }
}

// ------------------------------------------------------------------------------------------
static int pick_mt(int M) { return M <= 1 ? 1 : M <= 2 ? 2 : M <= 4 ? 4 : 8; }

struct Geometry {
    int ncta, units_base, units_rem, pass_units, nstages, pitch, kg;
    size_t smem;
};

static bool geometry(int mt, int K, int V, int k, int sm_count, Geometry* g)
{
    if (V % 8 != 0 || K % kRowsPerStage != 0 || k > 32 || k < 1) return false;
    const int units = V / 8;
    int ncta = sm_count < kMaxCtas ? sm_count : kMaxCtas;
    if (ncta > units) ncta = units;
    g->ncta = ncta;
    g->units_base = units / ncta;
    g->units_rem = units % ncta;
    const int max_units = g->units_base + (g->units_rem ? 1 : 0);
    const int npass = (max_units + kColThreads - 1) / kColThreads;
    g->pass_units = (max_units + npass - 1) / npass;
    g->pitch = g->pass_units * 16;
    g->kg = (mt == 8) ? 2 : 4;
    const size_t fixed = 256 + (size_t)kEpiWarps * mt * 66 * 4 + (size_t)g->kg * mt * g->pass_units * 8 * 4 + 128;
    const size_t stage = (size_t)kRowsPerStage * g->pitch + (((size_t)kRowsPerStage * mt * 4 + 127) & ~(size_t)127);
    if (fixed + 2 * stage > (size_t)kSmemBudget) return false;
    int ns = (int)(((size_t)kSmemBudget - fixed) / stage);
    if (ns > kMaxStages) ns = kMaxStages;
    g->nstages = ns;
    // the last CTA's merge keeps 2*P*k words per epilogue warp in the (then idle) stage area
    const size_t merge = (size_t)kEpiWarps * 2 * ncta * k * 4;
    if (fixed + merge > (size_t)kSmemBudget) return false;
    const size_t area = (size_t)ns * stage > merge ? (size_t)ns * stage : merge;
    g->smem = fixed + area;
    return true;
}

StreamPlan stream_plan(int M, int d, int K, int V, int k, int sm_count)
{
    StreamPlan sp = {0, 0, 0, 0};
    (void)d;
    if (M < 1) return sp;
    const int mt = pick_mt(M > 8 ? 8 : M);
    Geometry g;
    if (!geometry(mt, K, V, k, sm_count, &g)) return sp;
    sp.ok = 1;
    sp.mt = mt;
    sp.ncta = g.ncta;
    sp.launches = 2;
    return sp;
}

cudaError_t stream_downproj(const bf16* h, const bf16* A, int M, int mt, int d, int r, const Scratch& s,
                            cudaStream_t st)
{
    const int cblocks = r / 64;
    int S = (2 * 148 + cblocks - 1) / cblocks;
    if (S > 64) S = 64;
    int slab = ((d + S - 1) / S + 31) / 32 * 32;
    S = (d + slab - 1) / slab;
    dim3 grid(cblocks, S);
    switch (mt) {
    case 1: k_stream_downproj<1><<<grid, 256, 0, st>>>(h, A, M, d, r, slab, s.zpart, s.z, s.tickets + 1); break;
    case 2: k_stream_downproj<2><<<grid, 256, 0, st>>>(h, A, M, d, r, slab, s.zpart, s.z, s.tickets + 1); break;
    case 4: k_stream_downproj<4><<<grid, 256, 0, st>>>(h, A, M, d, r, slab, s.zpart, s.z, s.tickets + 1); break;
    default: k_stream_downproj<8><<<grid, 256, 0, st>>>(h, A, M, d, r, slab, s.zpart, s.z, s.tickets + 1); break;
    }
    return cudaGetLastError();
}

cudaError_t stream_widen_t(const bf16* h, int M, int mt, int d, float* zT, cudaStream_t st)
{
    const int n = d * mt;
    k_stream_widen_t<<<(n + 255) / 256, 256, 0, st>>>(h, M, mt, d, zT);
    return cudaGetLastError();
}

template <int MT, int KG>
static cudaError_t launch_head(const HeadParams& hp, size_t smem, bool pdl, cudaStream_t st)
{
    auto kern = k_stream_head<MT, KG>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(hp.ncta);
    cfg.blockDim = dim3(32 + 128 * KG + 32 * kEpiWarps);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, hp);
}

cudaError_t stream_head(const float* zT, const bf16* B, int M, int mt, int K, int V, int k, int mode,
                        int32_t* ids, float* logprobs, float* logits, const Scratch& s, int sm_count,
                        bool after_producer_kernel, cudaStream_t st)
{
    Geometry g;
    if (!geometry(mt, K, V, k, sm_count, &g)) return cudaErrorInvalidValue;
    if (g.ncta > s.max_parts) return cudaErrorInvalidValue;
    HeadParams hp;
    hp.zT = zT; hp.B = B; hp.M = M; hp.K = K; hp.V = V; hp.k = k; hp.mode = mode;
    hp.ncta = g.ncta; hp.units_base = g.units_base; hp.units_rem = g.units_rem; hp.pass_units = g.pass_units;
    hp.nstages = g.nstages; hp.pitch = g.pitch;
    hp.ids = ids; hp.logprobs = logprobs; hp.logits = logits;
    hp.part = s.part; hp.ticket = s.tickets; hp.err = s.err;
    hp.wait_prev = after_producer_kernel ? 1 : 0;
    switch (mt) {
    case 1: return launch_head<1, 4>(hp, g.smem, after_producer_kernel, st);
    case 2: return launch_head<2, 4>(hp, g.smem, after_producer_kernel, st);
    case 4: return launch_head<4, 4>(hp, g.smem, after_producer_kernel, st);
    default: return launch_head<8, 2>(hp, g.smem, after_producer_kernel, st);
    }
}

}  // namespace slimspec
