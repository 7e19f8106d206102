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
#include "select.cuh"
#include "epilogue.cuh"
#include <float.h>
#include <type_traits>

namespace slimspec {

static constexpr int kFmaMaxColThreads = 256;   // threads across one pass's columns, 8 columns each
static constexpr int kFmaMaxCtas = 256;         // most slabs
static constexpr int kFmaZChunkBytes = 64 * 1024;   // shared memory for the code, as (z, z) pairs
static constexpr int kFmaEpFixed = (kEpFixedBytes + 127) / 128 * 128;      // the epilogue's fixed area
static constexpr int kFmaMergeBytes = (16 + 2 * 16 * 32 + 4 * 2 * kMergeCand) * 4 + 64;   // the last CTA's merge: up to four tasks

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
    int ct, rg;           // column threads (multiple of 32) and row groups: blockDim = ct * rg
    int kc;               // rows of the code per shared-memory chunk (K, or a multiple of rg * U)
    int rec_words;        // words per split-V record: max, sum-exp, k (key, id) pairs, padded to 4
    int merge_inside;     // 1: the last CTA to arrive merges the records
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
__global__ void __launch_bounds__(512, 1) k_fma_head(const FmaParams p)
{
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* cand = smem + kFmaEpFixed;                            // the epilogue's parked candidates
    unsigned char* merge_area = cand + MT * kCand * 8;                   // the last CTA's merge
    float* red = reinterpret_cast<float*>(merge_area + kFmaMergeBytes);  // [RG][MT][ct*8]
    const int CT = p.ct, RG = p.rg;
    const int slab_cols = CT * 8;
    float2* zs = reinterpret_cast<float2*>(red + (size_t)RG * MT * slab_cols);   // [kc][MT] (z, z) pairs

    const int tid = threadIdx.x;
    const int g = tid / CT, c = tid - g * CT;        // row group, column unit
    const int cta = blockIdx.x;
    const int K = p.K, V = p.V;
    const int stepU = RG * U;

    // ---- this CTA's slab
    const int my_units = p.units_base + (cta < p.units_rem ? 1 : 0);
    const int unit0 = cta * p.units_base + min(cta, p.units_rem);
    const bool active = c < my_units;
    const bf16* base = p.B + (size_t)(unit0 + c) * 8;

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
    // the weights are on their way; let the next kernel in the stream come up behind this one,
    // then wait for the kernel that writes the code
    pdl_launch_dependents();
    for (int i = tid; i < MT * 64; i += blockDim.x) reinterpret_cast<float*>(smem + 64)[i] = -FLT_MAX;
    if (p.wait_prev) {
        // Until the code is there this CTA can only wait, and while it waits HBM idles: ask the L2
        // for the rows of the slab that come next (a hint; the loads of the main loop then hit the
        // L2).  Launched early behind a kernel that still runs, the wait is several microseconds.
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
        pdl_wait();
    }

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
        const float* src = p.zT + (size_t)kc0 * MT;
        for (int e = tid; e < (kend - kc0) * MT; e += blockDim.x) {
            const float zv = __ldcg(src + e);
            zs[e] = make_float2(zv, zv);
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
    slab_epilogue<MT>(p, smem, cand, merge_area, red, RG, MT * slab_cols, slab_cols, my_units * 8, unit0 * 8);
}

// ------------------------------------------------------------------------------------------
static int fma_pick_mt(int M) { return M <= 1 ? 1 : 2; }

struct FmaGeometry {
    int ncta, units_base, units_rem, max_units, ct, rg, u, kc, rec_words, threads;
    size_t smem;
};

// One CTA per SM, the slab's column units across ct threads, the rows of the matrix dealt to rg row
// groups.  Shapes whose slabs are wider than kFmaMaxColThreads units are not taken (the tensor-core
// streaming kernel takes them).
static bool fma_geometry(int mt, int K, int V, int k, int sm_count, FmaGeometry* g)
{
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
    g->threads = g->ct * g->rg;
    g->u = 16;
    // rows of the code per shared-memory chunk: all of K if it fits, else a multiple of rg*u
    const int kc_max = kFmaZChunkBytes / (mt * 8);
    if (K <= kc_max) g->kc = K;
    else {
        g->kc = kc_max / (g->rg * g->u) * (g->rg * g->u);
        if (g->kc < 1) return false;
    }
    g->rec_words = (2 + 2 * k + 3) / 4 * 4;
    g->smem = (size_t)kFmaEpFixed + (size_t)mt * kCand * 8 + kFmaMergeBytes + (size_t)g->threads * mt * 32 + (size_t)g->kc * mt * 8;
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
    hp.ncta = g.ncta; hp.units_base = g.units_base; hp.units_rem = g.units_rem;
    hp.ct = g.ct; hp.rg = g.rg; hp.kc = g.kc; hp.rec_words = g.rec_words; hp.merge_inside = 1;
    hp.ids = ids; hp.logprobs = logprobs; hp.logits = logits;
    hp.part = s.part; hp.ticket = s.tickets; hp.err = s.err;
    hp.wait_prev = after_producer_kernel ? 1 : 0;
    {
        const size_t row_bytes = (size_t)g.max_units * 16 * g.ncta;      // one row of every slab
        const size_t rows = row_bytes ? kFmaPrefetchBytes / row_bytes : 0;
        hp.pf_rows = after_producer_kernel ? (int)(rows < (size_t)K ? rows : (size_t)K) : 0;
    }
    switch (mt) {
    case 1: return fma_launch_head<1, 16>(hp, g, after_producer_kernel, st);
    default: return fma_launch_head<2, 16>(hp, g, after_producer_kernel, st);
    }
}

}  // namespace slimspec
