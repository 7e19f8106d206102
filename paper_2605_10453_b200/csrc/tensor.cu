// Tensor-core path for larger M: out = X W with X[M][K] (rows on the MMA's M side, K-major) and
// W[K][N] (N-major), bf16 inputs, fp32 accumulation in tensor memory (tcgen05).
//   down-projection  z = h A      X = h, W = A, split over K, fp32 partial tiles -> k_tc_reduce_z
//   up-projection    logits = z B X = z (bf16), W = B, fused online log-softmax / top-k epilogue
//   full-rank head   logits = h W X = h, W = W, same epilogue
// (Section 4.1; the softmax of Section 3.2 and the candidate selection.)
//
// One CTA per SM: one warp feeds a ring of shared-memory stages by TMA, one thread of another
// warp issues the MMAs (128 rows x NV columns x 16 per instruction) into one of two
// accumulator buffers in tensor memory, eight epilogue warps read the finished buffer (a thread per
// row and column half) and keep that row's running max / sum-exp / top-k while the next tile's MMAs run.
#include "kernels.h"
#include "ptx.cuh"
#include "select.cuh"
#include <cuda.h>
#include <float.h>
#include <string.h>

namespace slimspec {

static constexpr int kTcRows = 128;          // rows per tile = MMA M
static constexpr int kTcKChunk = 64;         // K per stage: 64 bf16 = one 128-byte swizzle row
// Twelve warps.  A warp reads only the lane quarter (warp id mod 4) of tensor memory and warps are
// dealt to the SM's four schedulers by the same rule, so the rows of quarter q are worked on by the
// scheduler q.  The thread that issues the MMAs loses its issue slots to busy epilogue warps of its
// scheduler, so it (and the TMA thread) sit with the quarters that fill last: warp 2 loads, warp 3
// issues, epilogue warps {0,4} {1,5} {6,10} {7,11} take quarters 0..3, warps 8 and 9 idle.  With up
// to 64 rows in a tile neither special warp shares a scheduler with a busy warp.
static constexpr int kTcThreads = 384;
static constexpr int kTcLoadWarp = 2, kTcMmaWarp = 3;
static constexpr int kTcMaxK = 32;           // largest k
static constexpr int kTcList = 48;           // candidates a row parks before the list is compacted
static constexpr int kTcListPitch = 49;      // words between two rows' lists in shared memory: odd, so lanes hit distinct banks
static constexpr int kTcEpiThreads = 256;    // epilogue threads per CTA
// shared memory the final sort of the lists needs (values and ids of every epilogue thread)
static constexpr size_t kTcSortBytes = (size_t)2 * kTcEpiThreads * kTcListPitch * 4;
static constexpr int kTcNoId = 0x7fffffff;
static constexpr float kLog2e = 1.4426950408889634f;

struct alignas(64) TcParams {
    CUtensorMap mapX;       // X[M][K]: box 64 (K) x 128 rows, 128-byte swizzle
    CUtensorMap mapW;       // W[K][N]: box 64 (N) x 64 (K), 128-byte swizzle
    CUtensorMap mapX2;      // split mode: the low part of X, same shape and box as mapX
    int M, K, N;
    int nrb, nct, nks;      // row blocks, column tiles, K splits
    int chunks_per_split;   // K chunks of 64 per split
    int gct;                // CTAs that share one (row block, split); column tiles go round-robin
    int mode;               // 0: top-k records, 1: fp32 out[M][N], 2: fp32 partial out[nks][nrb*128][N],
                            // 3: per-row maximum of each tile, as a key, to smax[tile][nrb*128]
    uint32_t* smax;         // mode 3 output
    const uint32_t* thr0;   // mode 0: per-row lower bound (key - 1) of the k-th largest logit, or null
    int k;
    int rec_words;
    int ns;                 // stages of the W ring
    int nsx;                // stages of the X ring (unused when X is resident)
    int xbox_bytes;         // bytes of one X box: (rows of the box, 8..128) x 128; rows past the box are garbage in,
                            // garbage out, and belong to no live row
    int split;              // 1: X = X_hi + X_lo (two bf16 matrices): two MMAs per step into one accumulator
    int xres;               // 1: the row block's whole X (K <= 512) is loaded once and stays in shared memory
    float* out;
    float* part;            // records [M][2 * gct][rec_words]: two column halves per CTA
    int* err;
};

// A row's candidate list: up to kTcList (value, id) pairs above the row's threshold, appended in
// the order the columns arrive (ascending id).  topk_compact sorts the list (values descending,
// equal values keep their order, i.e. lower id first), cuts it to the k best and returns the
// new threshold: the k-th value if the list holds k entries, else the old bound.
__device__ __noinline__ float topk_compact(float* cv, int* ci, int& cnt, int k, float thr0)
{
    for (int i = 1; i < cnt; ++i) {
        const float v = cv[i];
        const int id = ci[i];
        int pos = i;
        while (pos > 0 && cv[pos - 1] < v) {
            cv[pos] = cv[pos - 1];
            ci[pos] = ci[pos - 1];
            --pos;
        }
        cv[pos] = v;
        ci[pos] = id;
    }
    if (cnt > k) cnt = k;
    return cnt == k ? cv[k - 1] : thr0;
}

__device__ __forceinline__ float ex2_fast(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float max3(float a, float b, float c)
{
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// What one epilogue thread carries for its row across the tiles of its CTA.
struct EpiRow {
    float run_max, run_sum;     // online softmax: maximum so far, sum of exp(logit - maximum)
    float thr;                  // candidates must beat this
    float tile_max;             // mode 3: maximum of the current tile
    int cnt;                    // candidates parked in the list
};

// One chunk of 32 consecutive columns of one row, as read from tensor memory.
__device__ __forceinline__ void epi_chunk(const TcParams& p, const uint32_t (&v)[32], int col0, int m, int ks, bool live,
                                          EpiRow& st, float* cv, int* ci)
{
    const int nvalid = min(32, p.N - col0);      // same for every thread
    if (nvalid <= 0 || !live) return;
    if (p.mode == 3) {
#pragma unroll
        for (int e = 0; e < 32; ++e) st.tile_max = fmaxf(st.tile_max, e < nvalid ? __uint_as_float(v[e]) : -FLT_MAX);
        return;
    }
    if (p.mode != 0) {
        const size_t orow = (p.mode == 2) ? ((size_t)ks * p.nrb * kTcRows + m) : (size_t)m;
        float* dst = p.out + orow * p.N + col0;
#pragma unroll
        for (int e = 0; e < 32; e += 4) {
            if (e < nvalid)      // N is a multiple of 8, so a group of four is all in or all out
                *reinterpret_cast<float4*>(dst + e) =
                    make_float4(__uint_as_float(v[e]), __uint_as_float(v[e + 1]), __uint_as_float(v[e + 2]),
                                __uint_as_float(v[e + 3]));
        }
        return;
    }
    // ---- online softmax and candidate filter.  Columns past N (last tile only) count as -FLT_MAX.
    float x[32];
#pragma unroll
    for (int e = 0; e < 32; ++e) x[e] = __uint_as_float(v[e]);
    if (nvalid < 32) {
#pragma unroll
        for (int e = 0; e < 32; ++e) x[e] = e < nvalid ? x[e] : -FLT_MAX;
    }
    float m8[4];       // maxima of the four groups of eight columns (three-input max: four steps a group)
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        float g = max3(x[q * 8], x[q * 8 + 1], x[q * 8 + 2]);
        g = max3(g, x[q * 8 + 3], x[q * 8 + 4]);
        g = max3(g, x[q * 8 + 5], x[q * 8 + 6]);
        m8[q] = fmaxf(g, x[q * 8 + 7]);
    }
    const float cmax = fmaxf(max3(m8[0], m8[1], m8[2]), m8[3]);
    if (cmax > st.run_max) {
        st.run_sum *= ex2_fast((st.run_max - cmax) * kLog2e);
        st.run_max = cmax;
    }
    // sum of 2^(x log2(e) - max log2(e)): the scaling and the adds go two columns an instruction
    const float nmb = -st.run_max * kLog2e;
    const float2 sc = make_float2(kLog2e, kLog2e), of = make_float2(nmb, nmb);
    float2 sacc[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
    for (int e = 0; e < 32; e += 2) {
        const float2 t = __ffma2_rn(make_float2(x[e], x[e + 1]), sc, of);
        sacc[(e >> 1) & 1] = __fadd2_rn(sacc[(e >> 1) & 1], make_float2(ex2_fast(t.x), ex2_fast(t.y)));
    }
    st.run_sum += (sacc[0].x + sacc[0].y) + (sacc[1].x + sacc[1].y);
    // top-k: ids arrive in ascending order, so a candidate must beat the threshold strictly.  Some
    // row of the warp has a candidate in most chunks, but a given row rarely has one: a lane with
    // one looks only into the groups of eight whose maximum beats its threshold.  (No warp-wide
    // vote here: lanes of rows past M have returned.)
    if (cmax > st.thr) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            if (m8[q] > st.thr) {
                uint32_t gt = 0u;       // the group's columns above the threshold, built without branches
#pragma unroll
                for (int e = 0; e < 8; ++e) gt |= (x[q * 8 + e] > st.thr) ? (1u << e) : 0u;
                if ((gt & (gt - 1u)) == 0u) {
                    // one column: it is the group's maximum
                    if (st.cnt == kTcList) {
                        int c = st.cnt;      // a copy: the state stays in registers
                        st.thr = topk_compact(cv, ci, c, p.k, st.thr);
                        st.cnt = c;
                    }
                    if (m8[q] > st.thr) {
                        cv[st.cnt] = m8[q];
                        ci[st.cnt] = col0 + q * 8 + __ffs(gt) - 1;
                        ++st.cnt;
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const float xv = x[q * 8 + e];
                        if (xv > st.thr) {
                            if (st.cnt == kTcList) {
                                int c = st.cnt;
                                st.thr = topk_compact(cv, ci, c, p.k, st.thr);
                                st.cnt = c;
                            }
                            if (xv > st.thr) {
                                cv[st.cnt] = xv;
                                ci[st.cnt] = col0 + q * 8 + e;
                                ++st.cnt;
                            }
                        }
                    }
                }
            }
        }
    }
}

// ------------------------------------------------------------------------------------------
template <int NV>
__global__ void __launch_bounds__(kTcThreads, 1) k_tc_gemm(const __grid_constant__ TcParams p)
{
    constexpr int NSMAX = 8;                                // most ring stages
    constexpr int WBOX_BYTES = kTcKChunk * 64 * 2;          // 8 KB: 64 k x 64 columns
    constexpr int W_BYTES = WBOX_BYTES * (NV / 64);
    const int NS = p.ns;
    const bool xres = p.xres != 0, split = p.split != 0;
    const int XH = p.xbox_bytes;                            // one X box (high or low part) of a K chunk
    const int XB = split ? 2 * XH : XH;                     // X bytes per K chunk: high part, then low part
    // Two rings: W chunks (the HBM stream: as many stages as shared memory allows) and, unless X
    // is resident, X chunks (L2 hits: a few stages do).
    const int NSX = p.nsx;
    // instruction descriptor: D fp32, A and B bf16, A K-major, B MN-major, N = NV, M = 128
    constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) |
                               ((uint32_t)(NV >> 3) << 17) | ((uint32_t)(kTcRows >> 4) << 24);

    extern __shared__ unsigned char smem_raw[];
    __shared__ uint64_t full[NSMAX], empty[NSMAX], xfull[4], xempty[4], acc_full[2], acc_empty[2], x_full;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    unsigned char* xarea = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    unsigned char* stages = xarea + (xres ? (size_t)p.chunks_per_split * XB : (size_t)NSX * XB);   // W ring
    volatile int* abort_flag = &abort_s;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x;
    const int rb = cta % p.nrb;
    const int rest = cta / p.nrb;
    const int ks = rest % p.nks;
    const int cg = rest / p.nks;                 // position among the CTAs of this (row block, split)
    const int cps = p.chunks_per_split;
    const int ntiles = cg < p.nct ? (p.nct - cg + p.gct - 1) / p.gct : 0;

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int s = 0; s < 4; ++s) { mbar_init(&xfull[s], 1); mbar_init(&xempty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 256); }
        mbar_init(&x_full, 1);
        abort_s = 0;
        mbar_fence_init();
        prefetch_tensor_map(&p.mapX);
        prefetch_tensor_map(&p.mapW);
        if (p.split) prefetch_tensor_map(&p.mapX2);
    }
    if (warp == kTcMmaWarp) tmem_alloc(&tmem_base_s, 2 * NV);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_base_s;
    // Everything above touched no global data: under programmatic dependent launch it overlaps the
    // kernel before; from here on that kernel's results are needed.
    pdl_launch_dependents();
    pdl_wait();

    if (warp == kTcLoadWarp) {
        // ================= producer: one thread issues the TMA loads =================
        if (lane == 0) {
            // ring positions are kept as (slot, phase) pairs: no division on this thread's path
            int s = 0, ph = 0, sx = 0, phx = 0;
            bool first = true, firstx = true;       // first lap: the slots start out empty
            bool alive = true;
            if (xres && ntiles > 0) {
                mbar_arrive_expect_tx(&x_full, (uint32_t)cps * XB);
                for (int c = 0; c < cps; ++c) {
                    tma_load_2d(xarea + (size_t)c * XB, &p.mapX, c * kTcKChunk, rb * kTcRows, &x_full);
                    if (split) tma_load_2d(xarea + (size_t)c * XB + XH, &p.mapX2, c * kTcKChunk, rb * kTcRows, &x_full);
                }
            }
            for (int t = 0; t < ntiles && alive; ++t) {
                const int ct = cg + t * p.gct;
                for (int c = 0; c < cps; ++c) {
                    const int kx = (ks * cps + c) * kTcKChunk;
                    if (!xres) {
                        if (!firstx && !mbar_wait(&xempty[sx], phx ^ 1, abort_flag, p.err, ERR_WAIT_EMPTY)) { alive = false; break; }
                        unsigned char* xs = xarea + (size_t)sx * XB;
                        mbar_arrive_expect_tx(&xfull[sx], (uint32_t)XB);
                        tma_load_2d(xs, &p.mapX, kx, rb * kTcRows, &xfull[sx]);
                        if (split) tma_load_2d(xs + XH, &p.mapX2, kx, rb * kTcRows, &xfull[sx]);
                        if (++sx == NSX) { sx = 0; phx ^= 1; firstx = false; }
                    }
                    if (!first && !mbar_wait(&empty[s], ph ^ 1, abort_flag, p.err, ERR_WAIT_EMPTY)) { alive = false; break; }
                    unsigned char* st = stages + (size_t)s * W_BYTES;
                    mbar_arrive_expect_tx(&full[s], (uint32_t)W_BYTES);
#pragma unroll
                    for (int i = 0; i < NV / 64; ++i)
                        tma_load_2d(st + i * WBOX_BYTES, &p.mapW, ct * NV + i * 64, kx, &full[s]);
                    if (++s == NS) { s = 0; ph ^= 1; first = false; }
                }
            }
        }
    } else if (warp == kTcMmaWarp) {
        // ================= MMA issuer =================
        // One thread feeds the tensor pipe, so its instruction count per K chunk is what bounds the
        // main loop once the data is there: descriptors are kept as a running low word (start
        // address and leading offset; the high word is the same for every operand) and ring
        // positions as (slot, phase) pairs.
        if (lane == 0) {
            constexpr uint32_t DESC_HI = (1024u >> 4) | (1u << 14) | (2u << 29);     // SBO 1024, version 1, 128-byte swizzle
            const uint32_t a_base = ((smem_u32(xarea) >> 4) & 0x3fffu) | (1u << 16);                       // LBO 16
            const uint32_t b_base = ((smem_u32(stages) >> 4) & 0x3fffu) | ((uint32_t)(WBOX_BYTES >> 4) << 16);
            const uint32_t a_step = (uint32_t)XB >> 4, a_lowpart = (uint32_t)XH >> 4;
            constexpr uint32_t B_STEP = (uint32_t)W_BYTES >> 4;
            const int nsa = xres ? cps : NSX;           // X slots: the resident chunks, or the ring
            int s = 0, ph = 0, sx = 0, phx = 0;
            uint32_t a_lo = a_base, b_lo = b_base;
            bool alive = true;
            if (xres && ntiles > 0 && !mbar_wait(&x_full, 0, abort_flag, p.err, ERR_WAIT_FULL)) alive = false;
            for (int t = 0; t < ntiles && alive; ++t) {
                const int buf = t & 1;
                if (t >= 2 && !mbar_wait(&acc_empty[buf], ((t >> 1) - 1) & 1, abort_flag, p.err, ERR_WAIT_FREE)) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * NV);
                for (int c = 0; c < cps; ++c) {
                    if (!xres && !mbar_try_wait(&xfull[sx], phx) && !mbar_wait(&xfull[sx], phx, abort_flag, p.err, ERR_WAIT_FULL)) { alive = false; break; }
                    if (!mbar_try_wait(&full[s], ph) && !mbar_wait(&full[s], ph, abort_flag, p.err, ERR_WAIT_FULL)) { alive = false; break; }
                    // 16 of K per instruction: 32 bytes along a K-major row of X, two 8-row groups of the N-major W tile
                    tc_mma_bf16_words(d_tmem, a_lo, b_lo, DESC_HI, IDESC, c > 0 ? 1u : 0u);
                    if (split) tc_mma_bf16_words(d_tmem, a_lo + a_lowpart, b_lo, DESC_HI, IDESC, 1u);
#pragma unroll
                    for (int j = 1; j < kTcKChunk / 16; ++j) {
                        tc_mma_bf16_words(d_tmem, a_lo + (uint32_t)(j * 2), b_lo + (uint32_t)(j * 128), DESC_HI, IDESC, 1u);
                        if (split) tc_mma_bf16_words(d_tmem, a_lo + a_lowpart + (uint32_t)(j * 2), b_lo + (uint32_t)(j * 128), DESC_HI, IDESC, 1u);
                    }
                    tc_commit(&empty[s]);
                    b_lo += B_STEP;
                    if (++s == NS) { s = 0; ph ^= 1; b_lo = b_base; }
                    if (!xres) tc_commit(&xempty[sx]);
                    a_lo += a_step;
                    if (++sx == nsa) { sx = 0; phx ^= 1; a_lo = a_base; }
                }
                if (alive) tc_commit(&acc_full[buf]);
            }
        }
    } else if (warp != 8 && warp != 9) {
        // ================= epilogue: thread = row =================
        const int quarter = warp & 3;                        // the lane quarter this warp may read
        const int half = (warp == 4 || warp == 5 || warp >= 10) ? 1 : 0;     // two warps share a quarter: each takes half the columns
        const int slot = (quarter * 2 + half) * 32 + lane;  // 0..255 among the epilogue threads
        const int row = quarter * 32 + lane;
        const int m = rb * kTcRows + row;
        const bool live = m < p.M;
        const int k = p.k;
        EpiRow st;
        st.run_max = -FLT_MAX;
        st.run_sum = 0.f;
        st.cnt = 0;
        float cv[kTcList];
        int ci[kTcList];
        // Candidates must beat thr: the k-th best value once the list is full, before that a bound
        // known to lie below the row's k-th largest logit (from a sample of the vocabulary).
        const uint32_t thr0_key = (p.mode == 0 && p.thr0 != nullptr && live) ? __ldg(p.thr0 + m) : 0u;
        st.thr = thr0_key != 0u ? key2f(thr0_key) : -FLT_MAX;      // key 0: no bound
        bool alive = true;
        constexpr int NCH = NV / 2 / 32;          // chunks of 32 columns per warp and tile: 2 or 4
        for (int t = 0; t < ntiles && alive; ++t) {
            const int buf = t & 1;
            const int ct = cg + t * p.gct;
            if (!mbar_wait_warp(&acc_full[buf], (t >> 1) & 1, abort_flag, p.err, ERR_WAIT_ACC)) { alive = false; break; }
            tc_fence_after_sync();
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * NV + half * (NV / 2));
            const int colbase = ct * NV + half * (NV / 2);
            st.tile_max = -FLT_MAX;
#pragma unroll 1
            for (int i = 0; i < NCH; ++i) {
                uint32_t va[32];
                tmem_ld_32x32(taddr + (uint32_t)(i * 32), va);
                tmem_ld_wait();
                epi_chunk(p, va, colbase + i * 32, m, ks, live, st, cv, ci);
            }
            if (p.mode == 3 && live) p.smax[((size_t)ct * 2 + half) * p.nrb * kTcRows + m] = f2key(st.tile_max);
            tc_fence_before_sync();
            mbar_arrive(&acc_empty[buf]);
        }
        const float run_max = st.run_max, run_sum = st.run_sum, thr = st.thr;
        int cnt = st.cnt;
        if (alive && live && p.mode == 0) {
            // The lists live in local memory, which this kernel's small L1 hardly caches: a sort
            // there pays an L2 round trip per step.  Every MMA has completed by now (the last
            // accumulator was handed over), so the operand rings are dead: sort in that memory.
            float* sv = reinterpret_cast<float*>(xarea) + (size_t)slot * kTcListPitch;
            int* si = reinterpret_cast<int*>(xarea + (size_t)kTcEpiThreads * kTcListPitch * 4) + (size_t)slot * kTcListPitch;
            for (int j = 0; j < cnt; ++j) {
                sv[j] = cv[j];
                si[j] = ci[j];
            }
            topk_compact(sv, si, cnt, k, thr);
            float* rec = p.part + ((size_t)m * (2 * p.gct) + 2 * cg + half) * p.rec_words;
            rec[0] = run_max;
            rec[1] = run_sum;
            for (int j = 0; j < k; ++j)      // (key, id) pairs; -0 and +0 rank alike
                *reinterpret_cast<float2*>(rec + 2 + 2 * j) =
                    make_float2(__uint_as_float(j < cnt ? f2key(sv[j] + 0.f) : 0u), __int_as_float(j < cnt ? si[j] : kTcNoId));
        }
    }
    // ---- teardown: every role is past its last use of tensor memory
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == kTcMmaWarp) tmem_dealloc(tmem_base, 2 * NV);
}

// ------------------------------------------------------------------------------------------
// z = sum of the K-split partial tiles, rounded once to bf16; with zlo set, the rounding error is
// kept as a second bf16 matrix (z = z + zlo to about 2^-17 relative).
__global__ void k_tc_reduce_z(const float* __restrict__ part, int nks, int mpad, int M, int r, bf16* __restrict__ z,
                              bf16* __restrict__ zlo)
{
    pdl_launch_dependents();
    pdl_wait();
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= M * r) return;
    const int m = e / r, j = e - m * r;
    float acc = 0.f;
    for (int s0 = 0; s0 < nks; s0 += 8) {
        float t[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) t[q] = (s0 + q < nks) ? __ldcg(part + ((size_t)(s0 + q) * mpad + m) * r + j) : 0.f;
#pragma unroll
        for (int q = 0; q < 8; ++q) acc += t[q];
    }
    const bf16 hi = __float2bfloat16_rn(acc);
    z[e] = hi;
    if (zlo != nullptr) zlo[e] = __float2bfloat16_rn(acc - __bfloat162float(hi));
}

// ------------------------------------------------------------------------------------------
// thr0[m] = (k-th largest of the row's nst sample-tile maxima) - 1, as a key: at least k logits
// of the row are >= that maximum, so the row's k-th largest logit is too.  One warp per row,
// nst <= 64.  Equal maxima are counted once, which only lowers the bound.  0 if nst < k.
__global__ void __launch_bounds__(256) k_tc_thr0(const uint32_t* __restrict__ smax, int nst, int mpad, int M, int k,
                                                 uint32_t* __restrict__ thr0)
{
    pdl_launch_dependents();
    pdl_wait();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m = blockIdx.x * (blockDim.x >> 5) + warp;
    if (m >= M) return;
    uint32_t a = lane < nst ? __ldcg(smax + (size_t)lane * mpad + m) : 0u;
    uint32_t b = lane + 32 < nst ? __ldcg(smax + (size_t)(lane + 32) * mpad + m) : 0u;
    if (b > a) { const uint32_t t = a; a = b; b = t; }
    uint32_t kth = 0u;
    for (int j = 0; j < k; ++j) {
        kth = warp_max_u32(a);
        if (a == kth) { a = b; b = 0u; }
    }
    if (lane == 0) thr0[m] = (nst >= k && kth > 0u) ? kth - 1u : 0u;
}

// ------------------------------------------------------------------------------------------
// Merge the P per-slab records of each row.  Two rows per CTA, two warps per row: one takes the
// row's log-sum-exp, the other its k best entries (bound from the records' first entries, the few
// entries above it ordered by counting).
__global__ void __launch_bounds__(128) k_tc_merge(const float* __restrict__ part, int M, int P, int RW, int k,
                                                  int32_t* __restrict__ ids, float* __restrict__ logprobs)
{
    __shared__ float lse_s[2];
    __shared__ uint32_t ok_s[2][32];
    __shared__ int oi_s[2][32];
    __shared__ uint32_t mk_s[4][kMergeCand];
    __shared__ int mi_s[4][kMergeCand];
    __shared__ int cnt_s[4];
    pdl_launch_dependents();     // the first kernel of the next call may come up behind this one
    pdl_wait();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r2 = warp >> 1, row = blockIdx.x * 2 + r2;
    if (row < M) {
        if (P <= 5 * 32) merge_task<5>(part, P, RW, k, row, warp & 1, lane, &lse_s[r2], ok_s[r2], oi_s[r2], mk_s[warp], mi_s[warp], &cnt_s[warp]);
        else merge_task<kMergeLists>(part, P, RW, k, row, warp & 1, lane, &lse_s[r2], ok_s[r2], oi_s[r2], mk_s[warp], mi_s[warp], &cnt_s[warp]);
    }
    __syncthreads();
    if ((warp & 1) == 0 && row < M && lane < k) {
        ids[(size_t)row * k + lane] = oi_s[r2][lane];
        logprobs[(size_t)row * k + lane] = key2f(ok_s[r2][lane]) - lse_s[r2];
    }
}

// ------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)ptr;
    }
    return fn;
}

// bf16 matrix [rows][cols] (cols contiguous), box = box_cols x box_rows, 128-byte swizzle, zero fill
static bool make_map(CUtensorMap* map, const void* base, int rows, int cols, int box_cols, int box_rows)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    cuuint32_t es[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, es,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool tensor_ok(int M, int K, int N, int k, int mode)
{
    if (M < 1 || K < kTcKChunk || K % kTcKChunk != 0 || N % 8 != 0 || N < 64) return false;
    if (mode == 0 && (k < 1 || k > kTcMaxK)) return false;
    return true;
}

static constexpr size_t kTcSmemMax = 227 * 1024 - 512;   // dynamic shared memory per CTA (a little static on top)

// Launch with (or without) the programmatic-dependent-launch attribute: the kernel may start while
// the one before it in the stream is still running and meets it at griddepcontrol.wait.
template <typename... KArgs, typename... Args>
static cudaError_t launch_chain(void (*kern)(KArgs...), int grid, int block, size_t smem, bool pdl, cudaStream_t st,
                                Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, args...);
}

// Merge kernel: P split-V records per row -> ids / log-probs; launched early behind the kernel that writes them.
cudaError_t merge_records(const float* part, int M, int P, int RW, int k, int32_t* ids, float* logprobs, cudaStream_t st)
{
    return launch_chain(k_tc_merge, (M + 1) / 2, 128, 0, true, st, part, M, P, RW, k, ids, logprobs);
}

// Chooses the ring depth (and whether X can stay resident) and launches.
template <int NV>
static cudaError_t launch_gemm(TcParams p, int grid, bool pdl, cudaStream_t st)
{
    const size_t x_bytes = (size_t)p.xbox_bytes * (p.split ? 2 : 1), w_bytes = (size_t)kTcKChunk * NV * 2;
    const size_t x_all = (size_t)p.chunks_per_split * x_bytes;
    p.xres = (p.nks == 1 && x_all + 3 * w_bytes + 1024 <= kTcSmemMax) ? 1 : 0;
    p.nsx = 4;
    const size_t fixed = 1024 + (p.xres ? x_all : (size_t)p.nsx * x_bytes);
    const size_t stage = w_bytes;
    int ns = (int)((kTcSmemMax - fixed) / stage);
    if (ns > 8) ns = 8;
    if (ns < 2) return cudaErrorInvalidValue;
    p.ns = ns;
    size_t smem = fixed + (size_t)ns * stage;
    if (p.mode == 0 && smem < 1024 + kTcSortBytes) smem = 1024 + kTcSortBytes;      // room for the final sort of the lists
    auto kern = k_tc_gemm<NV>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    return launch_chain(kern, grid, kTcThreads, smem, pdl, st, p);
}

// Does the context's scratch hold the split-V records of this call?  (Same arithmetic as tensor_head.)
bool tensor_records_fit(int M, int N, int k, const Scratch& s, int sm_count)
{
    const int nrb = (M + kTcRows - 1) / kTcRows;
    const int nv = (nrb == 1) ? 128 : 256;
    const int nct = (N + nv - 1) / nv;
    int gct = sm_count / nrb;
    if (gct < 1) gct = 1;
    if (gct > nct) gct = nct;
    if (gct > kMaxRecords / 2) gct = kMaxRecords / 2;
    return (size_t)M * 2 * gct * ((2 + 2 * k + 3) / 4 * 4) <= s.part_elems;
}

// out = X W through the tensor cores.  mode 0: top-k records then merge into ids / logprobs;
// mode 1: fp32 logits.  X is bf16 [M][K], W bf16 [K][N].
cudaError_t tensor_head(const bf16* X, const bf16* Xlo, const bf16* W, int M, int K, int N, int k, int mode, int32_t* ids,
                        float* logprobs, float* logits, const Scratch& s, int sm_count, int* launches,
                        cudaEvent_t ev0, cudaEvent_t ev1, cudaStream_t st)
{
    // Every kernel here orders itself after its predecessor with griddepcontrol.wait before it touches
    // global memory, so each one, the first included, is launched early.
    const bool after_kernel = true;
    TcParams p;
    memset(&p, 0, sizeof(p));
    // a single row block loads only as many rows of X as there are (in whole groups of eight)
    const int xrows = M >= kTcRows ? kTcRows : (M + 7) / 8 * 8;
    if (!make_map(&p.mapX, X, M, K, kTcKChunk, xrows) || !make_map(&p.mapW, W, K, N, 64, kTcKChunk))
        return cudaErrorInvalidValue;
    if (Xlo != nullptr) {
        if (!make_map(&p.mapX2, Xlo, M, K, kTcKChunk, xrows)) return cudaErrorInvalidValue;
        p.split = 1;
    }
    p.xbox_bytes = xrows * kTcKChunk * 2;
    p.M = M; p.K = K; p.N = N;
    p.nrb = (M + kTcRows - 1) / kTcRows;
    const int nv = (p.nrb == 1) ? 128 : 256;
    p.nct = (N + nv - 1) / nv;
    p.nks = 1;
    p.chunks_per_split = K / kTcKChunk;
    p.gct = sm_count / p.nrb;
    if (p.gct < 1) p.gct = 1;
    if (p.gct > p.nct) p.gct = p.nct;
    if (p.gct > kMaxRecords / 2) p.gct = kMaxRecords / 2;       // the merge takes up to 320 lists per row
    p.mode = mode;
    p.k = k;
    p.rec_words = (2 + 2 * k + 3) / 4 * 4;
    p.out = logits;
    p.part = s.part;
    p.err = s.err;
    if (mode == 0 && (size_t)M * 2 * p.gct * p.rec_words > s.part_elems) return cudaErrorInvalidValue;
    cudaError_t e;
    if (mode == 0) {
        // A bound below each row's k-th largest logit, from the first sample tiles of the vocabulary:
        // it keeps the per-row candidate lists of the main pass almost idle.
        // (each sample tile yields two maxima per row, one per column half; k_tc_thr0 takes up to 64)
        // as many sample tiles as one wave of CTAs takes (the launch costs the same) and k_tc_thr0 reads
        int nst = 32;
        if (nst * p.nrb > sm_count) nst = sm_count / p.nrb;
        if (nst < 1) nst = 1;
        if (nst > p.nct) nst = p.nct;
        if (2 * nst >= k && (size_t)2 * nst * p.nrb * kTcRows <= s.smax_elems) {
            TcParams q = p;
            q.mode = 3;
            q.nct = nst;
            q.gct = nst;
            q.smax = s.smax;
            e = (nv == 128) ? launch_gemm<128>(q, nst * p.nrb, after_kernel, st) : launch_gemm<256>(q, nst * p.nrb, after_kernel, st);
            if (e != cudaSuccess) return e;
            e = launch_chain(k_tc_thr0, (M + 7) / 8, 256, 0, true, st, (const uint32_t*)s.smax, 2 * nst, p.nrb * kTcRows, M, k,
                             s.thr0);
            if (e != cudaSuccess) return e;
            *launches += 2;
            p.thr0 = s.thr0;
        }
    }
    const int grid = p.gct * p.nrb;
    // optional events directly around the kernel that streams the weights (they also keep it from
    // overlapping its neighbours)
    if (ev0 && (e = cudaEventRecord(ev0, st)) != cudaSuccess) return e;
    e = (nv == 128) ? launch_gemm<128>(p, grid, after_kernel && !ev0, st) : launch_gemm<256>(p, grid, after_kernel && !ev0, st);
    if (e != cudaSuccess) return e;
    if (ev1 && (e = cudaEventRecord(ev1, st)) != cudaSuccess) return e;
    *launches += 1;
    if (mode == 0) {
        e = merge_records(s.part, M, 2 * p.gct, p.rec_words, k, ids, logprobs, st);
        *launches += 1;
    }
    return e;
}

// z (bf16, [M][r]) = h A through the tensor cores: K-split partial tiles, then one reduction.
cudaError_t tensor_downproj(const bf16* h, const bf16* A, int M, int d, int r, bool with_low_part, const Scratch& s,
                            int sm_count, int* launches, cudaStream_t st)
{
    TcParams p;
    memset(&p, 0, sizeof(p));
    const int xrows = M >= kTcRows ? kTcRows : (M + 7) / 8 * 8;
    if (!make_map(&p.mapX, h, M, d, kTcKChunk, xrows) || !make_map(&p.mapW, A, d, r, 64, kTcKChunk))
        return cudaErrorInvalidValue;
    p.xbox_bytes = xrows * kTcKChunk * 2;
    p.M = M; p.K = d; p.N = r;
    p.nrb = (M + kTcRows - 1) / kTcRows;
    p.nct = (r + 127) / 128;
    const int chunks = d / kTcKChunk;
    // as many K splits as fill the SMs once, each a whole number of chunks
    int nks = sm_count / (p.nrb * p.nct);
    if (nks < 1) nks = 1;
    if (nks > chunks) nks = chunks;
    while (chunks % nks != 0) --nks;
    p.nks = nks;
    p.chunks_per_split = chunks / nks;
    p.gct = p.nct;
    p.mode = 2;
    p.out = s.zpart;
    p.err = s.err;
    const size_t need = (size_t)nks * p.nrb * kTcRows * r;
    if (need > s.zpart_elems) return cudaErrorInvalidValue;
    // Launched early even as the first kernel of a call: it touches global memory only after its
    // griddepcontrol.wait, so it may come up under the tail of whatever kernel precedes it.
    cudaError_t e = launch_gemm<128>(p, p.nrb * p.nct * nks, true, st);
    if (e != cudaSuccess) return e;
    const int n = M * r;
    e = launch_chain(k_tc_reduce_z, (n + 255) / 256, 256, 0, true, st, (const float*)s.zpart, nks, p.nrb * kTcRows, M, r,
                     s.zb, with_low_part ? s.zb_lo : (bf16*)nullptr);
    *launches += 2;
    return e;
}

}  // namespace slimspec
