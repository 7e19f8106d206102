// Streaming path for three to sixteen rows per launch (one and two rows: stream_fma.cu): the K x V
// weight matrix is read from HBM exactly once, in split-V slabs, every warp instruction fetching
// 512 contiguous bytes of one row.  The logits never leave the SM: every CTA keeps max / sum-exp /
// top-k per row for its slab, and the slab records are merged at the end (Section 4.1
// up-projection, the softmax of Section 3.2 in online form, and the candidate selection).
//
//   k_stream_code      the down-projection: h A with the rows of the batch on the 16-row side of
//                      warp-level tensor-core instructions, split over K across the CTAs of a
//                      cluster and folded through distributed shared memory; leaves the code as
//                      bf16 value + bf16 remainder in the form the head kernel reads.
//   k_stream_head_mma  a cp.async ring in shared memory, ldmatrix and mma.sync m16n8k16 (bf16 in,
//                      fp32 accumulate).  On this GPU one such instruction holds the SM's legacy
//                      tensor pipe for 8 cycles: 8 of them per 2 KB of weights keep up with HBM,
//                      16 do not -- hence the packed fragments below.
#include "kernels.h"
#include "ptx.cuh"
#include "select.cuh"
#include "epilogue.cuh"
#include <float.h>
#include <string.h>

namespace slimspec {

static constexpr int kMmaWarps = 7;                   // warps of a CTA of the tensor-core kernel (two CTAs per SM): 64 columns each;
                                                      // eight where that saves the epilogue a round of rows (see mma_warps)
// The epilogue gives each row to one warp: 8 rows on 7 warps take two rounds, 16 rows three.  An eighth
// warp (idle in the stream when the slab has no columns for it) saves a round there: M = 8: 41.1 -> 39.6 us,
// M = 16: 48.1 -> 46.4 us; with other row counts it only adds a party to the barriers (+0.4 to 0.7 us).
static int mma_warps(int M) { return (M == 8 || M >= 15) ? 8 : kMmaWarps; }
static constexpr size_t kMmaSmem = 76 * 1024;         // its shared memory: two such CTAs and the down-projection's CTA of the next call share an SM
static constexpr int kMaxStages = 8;                  // most stages of the shared-memory ring
enum : int { kCodePacked = 1, kCodeSplit = 2, kCodePlain = 3, kCodeRows = 4 };
static constexpr size_t kZOneChunkBytes = 16 * 1024;  // code fragments up to this size stay whole in shared memory
static constexpr size_t kZChunkBytes = 8 * 1024;      // else they pass through two buffers of this size

struct HeadParams {
    const uint32_t* zfrag;    // code fragments [nkb][ZP][32 lanes][4 words]
    const bf16* B;            // [K][V]
    int M, K, V, k, mode;
    int ncta;                 // slabs
    int units_base, units_rem;    // V/8 column units: slab c has units_base + (c < units_rem)
    int pitch_units;          // 16-byte units between two rows of a stage (odd, >= the widest slab)
    int ns;                   // stages of the ring
    int nkb;                  // 16-row blocks of the matrix: ceil(K / 16)
    int kb_chunk, nchunks;    // blocks of code fragments per shared-memory chunk, chunks
    unsigned int zarea_bytes; // shared memory the code takes
    int rec_words;            // words per record: max, sum-exp, k (key, id) pairs, padded to 4
    int32_t* ids;
    float* logprobs;
    float* logits;
    float* part;              // records [M][ncta * npass][rec_words]
    unsigned int* ticket;
    unsigned int ticket_base; // what the counter read when the call began
    int* err;
    int wait_prev;            // 1: the code is written by the kernel launched just before (PDL)
    int merge_inside;         // 1: the last CTAs to arrive merge the records; 0: raw logits, nothing to merge
};

// ------------------------------------------------------------------------------------------
// Small PTX helpers of this file.

// D (16 x 8, fp32) += A (16 x 16, bf16, row-major fragment) * B (16 x 8, bf16, column fragment)
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint4& a, uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void cp_async16(void* dst_smem, const void* src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst_smem)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
// wait until at most n of this thread's committed groups are still in flight
__device__ __forceinline__ void cp_async_wait_pending(int n)
{
    switch (n) {
    case 0: asm volatile("cp.async.wait_group 0;" ::: "memory"); break;
    case 1: asm volatile("cp.async.wait_group 1;" ::: "memory"); break;
    case 2: asm volatile("cp.async.wait_group 2;" ::: "memory"); break;
    case 3: asm volatile("cp.async.wait_group 3;" ::: "memory"); break;
    case 4: asm volatile("cp.async.wait_group 4;" ::: "memory"); break;
    case 5: asm volatile("cp.async.wait_group 5;" ::: "memory"); break;
    default: asm volatile("cp.async.wait_group 6;" ::: "memory"); break;
    }
}

// four 8 x 8 bf16 matrices from shared memory, transposed on the way: lane l supplies the address
// of row (l & 7) of matrix (l >> 3); register i of lane (g, t) receives rows 2t, 2t+1 of column g
// of matrix i
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}

// The code z (or, for the full-rank head, h itself) leaves this file's kernels in one of four forms:
//   kCodePacked  fragments, one part: rows 0-7 hold the value rounded to bf16 and rows 8-15 the
//                rounding remainders of those same rows, so ONE instruction multiplies both
//                (M <= 8; the two halves of its result are summed at the end)
//   kCodeSplit   fragments, two parts: value and remainder of up to 16 rows (two instructions)
//   kCodePlain   fragments, one part: up to 16 rows that are exact in bf16 (the full-rank head)
//   kCodeRows    plain row-major bf16 matrices [M][r], value and remainder: the operand the tcgen05
//                kernels load by TMA (any M: grid.z walks tiles of 16 rows)
// Fragments: word (kb, part, lane, reg) holds, for the 16-row block kb of the streamed matrix
// (contraction indices 16 kb .. 16 kb + 15), the two bf16 values
//     row  = (lane >> 2) + 8 (reg & 1),   index = 16 kb + 2 (lane & 3) + 8 (reg >> 1), + 1
// (the lower index in the lower half): the "A" operand of mma.m16n8k16 as lane `lane` wants it.
__host__ __device__ __forceinline__ size_t zfrag_word(int kb, int zparts, int part, int row, int idx16)
{
    const int lane = (row & 7) * 4 + ((idx16 & 7) >> 1);
    const int reg = ((idx16 >> 3) << 1) | (row >> 3);
    return (((size_t)kb * zparts + part) * 32 + lane) * 4 + reg;
}

// z = h A for up to 16 rows.  Grid (S, column tiles of 32), cluster (S, 1, 1): the CTAs of a
// cluster split the d rows of A, each of their four warps takes a contiguous run of 16-row
// blocks, and the partial tiles meet in the shared memory of the cluster's first CTA, which
// rounds and writes the fragments.  Sums run in a fixed order: results do not depend on timing.
struct CodeParams {
    const bf16* h;
    const bf16* A;
    int M, d, r;
    int S;            // K splits = CTAs per cluster
    int nkb;          // 16-row blocks of A: ceil(d / 16)
    int chunk_kbs;    // 16-row blocks of A per shared-memory buffer
    int nbuf;         // buffers
    int fmt;          // kCodePacked, kCodeSplit or kCodeRows
    uint32_t* zfrag;  // the code in that form
    bf16* zrows;      // kCodeRows: value [M][r]
    bf16* zrows_lo;   // kCodeRows: remainder [M][r], or null
};

static constexpr int kCodePitch = 80;            // bytes between two rows of the A slice in shared memory: 5 units (odd)
static constexpr int kCodeSliceRows = 640;       // rows of A a CTA holds at once when its whole share fits (50 KB: it then
                                                 // shares the SM with a head CTA) ...
static constexpr int kCodeChunkRows = 320;       // ... else it works through its share in chunks of this many rows,
static constexpr int kCodeRing = 4;              // through a ring of this many buffers, two CTAs per SM
static constexpr size_t kCodeSmemMax = (size_t)kCodeRing * kCodeChunkRows * kCodePitch + 128;   // most dynamic shared memory of that kernel

__global__ void __launch_bounds__(128, 8) k_stream_code(const CodeParams p)
{
    __shared__ __align__(16) float wt[4][16 * 32];      // the warps' partial tiles
    __shared__ __align__(16) float ct[8][16 * 32];      // the cluster's partial tiles (used in its first CTA)
    extern __shared__ __align__(128) unsigned char aslice[];     // [buffers][rows][kCodePitch]: 32 columns of A
    pdl_launch_dependents();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int rank = blockIdx.x;
    const int j0 = blockIdx.y * 32;
    const int d = p.d, r = p.r;
    const int m0 = blockIdx.z * 16;                      // first row of this CTA's tile of the batch
    const int mrows = min(16, p.M - m0);
    const bf16* hrows = p.h + (size_t)m0 * d;
    // this CTA's run of 16-row blocks, whole or in chunks through two buffers
    const int cta_kb0 = (int)((long long)p.nkb * rank / p.S), cta_kb1 = (int)((long long)p.nkb * (rank + 1) / p.S);
    const int chunk_kbs = p.chunk_kbs;
    const int nchunks = (cta_kb1 - cta_kb0 + chunk_kbs - 1) / chunk_kbs;
    const uint32_t buf_bytes = (uint32_t)chunk_kbs * 16u * kCodePitch;
    const int nbuf = p.nbuf, depth = max(1, nbuf - 1);         // chunks in flight
    auto fetch = [&](int c) {
        // weights may be read before the kernel ahead in the stream has finished: they are final before
        // the call is made (the contract of the library); only h comes from that kernel
        if (c < nchunks) {
            const int kb0 = cta_kb0 + c * chunk_kbs, kb1 = min(cta_kb1, kb0 + chunk_kbs);
            unsigned char* dst = aslice + (size_t)(c % nbuf) * buf_bytes;
            const int rows = 16 * (kb1 - kb0);
            for (int idx = tid; idx < rows * 4; idx += 128) {
                const int row = idx >> 2, u = idx & 3;
                const int grow = min(16 * kb0 + row, d - 1);             // rows past d re-read the last row (their h is zero)
                const int col = min(j0 + 8 * u, r - 8);                  // a ragged last tile re-reads the last columns
                cp_async16(dst + (size_t)row * kCodePitch + u * 16, p.A + (size_t)grow * r + col);
            }
        }
        cp_async_commit();
    };
    for (int c = 0; c < depth; ++c) fetch(c);
    pdl_wait();

    float acc[4][4];
#pragma unroll
    for (int e = 0; e < 4; ++e)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[e][c] = 0.f;
    const uint32_t lane_off = (uint32_t)((lane & 7) + ((lane >> 3) & 1) * 8) * kCodePitch + (uint32_t)(lane >> 4) * 16u;
    const uint32_t as_s = smem_u32(aslice);

    for (int c = 0; c < nchunks; ++c) {
        const int c0 = cta_kb0 + c * chunk_kbs, c1 = min(cta_kb1, c0 + chunk_kbs);
        // the warp's blocks of this chunk; their h fragments are the only loads that wait for the kernel ahead
        const int n = c1 - c0;
        const int wb0 = c0 + n * warp / 4, wb1 = c0 + n * (warp + 1) / 4;
        cp_async_wait_pending(depth - 1);          // chunk c is in (later ones may still be on their way)
        __syncthreads();                           // ... for everyone, and everyone is done with chunk c - 1
        fetch(c + depth);                          // into the buffer chunk c - 1 has left
        const uint32_t cbase = as_s + (uint32_t)(c % nbuf) * buf_bytes;
        for (int kb = wb0; kb < wb1; kb += 4) {
            uint4 hf[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int k0 = 16 * (kb + i) + 2 * t;
                const bool on = kb + i < wb1;
                const bool lo_ok = on && k0 < d, hi_ok = on && k0 + 8 < d;
                const uint32_t* h0 = reinterpret_cast<const uint32_t*>(hrows + (size_t)g * d + k0);
                const uint32_t* h1 = reinterpret_cast<const uint32_t*>(hrows + (size_t)(g + 8) * d + k0);
                hf[i].x = (g < mrows && lo_ok) ? __ldcg(h0) : 0u;
                hf[i].y = (g + 8 < mrows && lo_ok) ? __ldcg(h1) : 0u;
                hf[i].z = (g < mrows && hi_ok) ? __ldcg(h0 + 4) : 0u;
                hf[i].w = (g + 8 < mrows && hi_ok) ? __ldcg(h1 + 4) : 0u;
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if (kb + i < wb1) {
                    const uint32_t a = cbase + (uint32_t)(kb + i - c0) * 16u * kCodePitch + lane_off;
                    uint32_t b0, b1, b2, b3;
                    ldmatrix_x4_trans(b0, b1, b2, b3, a);
                    mma_bf16(acc[0], hf[i], b0, b1);
                    mma_bf16(acc[1], hf[i], b2, b3);
                    ldmatrix_x4_trans(b0, b1, b2, b3, a + 32u);
                    mma_bf16(acc[2], hf[i], b0, b1);
                    mma_bf16(acc[3], hf[i], b2, b3);
                }
            }
        }
    }
    // tile e of the instruction holds columns 8 e .. 8 e + 7 of the 32: lane (g, t) has columns
    // 8 e + 2 t, + 1 for rows g (values 0, 1) and g + 8 (values 2, 3)
    {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            *reinterpret_cast<float2*>(&wt[warp][g * 32 + 8 * e + 2 * t]) = make_float2(acc[e][0], acc[e][1]);
            *reinterpret_cast<float2*>(&wt[warp][(g + 8) * 32 + 8 * e + 2 * t]) = make_float2(acc[e][2], acc[e][3]);
        }
    }
    __syncthreads();
    float4 v = *reinterpret_cast<const float4*>(&wt[0][tid * 4]);
#pragma unroll
    for (int w = 1; w < 4; ++w) {
        const float4 o = *reinterpret_cast<const float4*>(&wt[w][tid * 4]);
        v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w;
    }
    if (p.S > 1) {
        // every CTA of the cluster drops its tile into slot `rank` of the first CTA's shared memory
        uint32_t remote;
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_u32(&ct[rank][tid * 4])), "r"(0));
        asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(remote), "f"(v.x), "f"(v.y), "f"(v.z),
                     "f"(v.w)
                     : "memory");
        asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
        if (rank != 0) return;
        v = *reinterpret_cast<const float4*>(&ct[0][tid * 4]);
        for (int s = 1; s < p.S; ++s) {
            const float4 o = *reinterpret_cast<const float4*>(&ct[s][tid * 4]);
            v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w;
        }
    }
    // four consecutive columns of one row
    const int row = tid >> 3, j = j0 + (tid & 7) * 4;
    if (j >= r) return;
    const float z[4] = {v.x, v.y, v.z, v.w};
    uint32_t hi[4], lo[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const bf16 hb = __float2bfloat16_rn(z[e]);
        const bf16 lb = __float2bfloat16_rn(z[e] - __bfloat162float(hb));
        hi[e] = (uint32_t)__bfloat16_as_ushort(hb);
        lo[e] = (uint32_t)__bfloat16_as_ushort(lb);
    }
    if (p.fmt == kCodeRows) {
        if (row < mrows) {
            const size_t o = (size_t)(m0 + row) * r + j;          // four bf16: 8 bytes, aligned (j is a multiple of 4)
            *reinterpret_cast<uint2*>(p.zrows + o) = make_uint2(hi[0] | (hi[1] << 16), hi[2] | (hi[3] << 16));
            if (p.zrows_lo) *reinterpret_cast<uint2*>(p.zrows_lo + o) = make_uint2(lo[0] | (lo[1] << 16), lo[2] | (lo[3] << 16));
        }
        return;
    }
#pragma unroll
    for (int pr = 0; pr < 2; ++pr) {
        const int jj = j + 2 * pr;
        const uint32_t hw = hi[2 * pr] | (hi[2 * pr + 1] << 16), lw = lo[2 * pr] | (lo[2 * pr + 1] << 16);
        if (p.fmt == kCodePacked) {
            if (row < 8) {
                p.zfrag[zfrag_word(jj >> 4, 1, 0, row, jj & 15)] = hw;
                p.zfrag[zfrag_word(jj >> 4, 1, 0, row + 8, jj & 15)] = lw;
            }
        } else {
            p.zfrag[zfrag_word(jj >> 4, 2, 0, row, jj & 15)] = hw;
            p.zfrag[zfrag_word(jj >> 4, 2, 1, row, jj & 15)] = lw;
        }
    }
}

// The full-rank head has no down-projection: its "code" is h itself, exact in bf16
// (kCodePlain).
__global__ void k_stream_widen(const bf16* __restrict__ h, int M, int d, int nkb, uint32_t* __restrict__ zfrag)
{
    pdl_launch_dependents();
    pdl_wait();          // launched early: the kernel before it may still read the code
    const int w = blockIdx.x * blockDim.x + threadIdx.x;
    if (w >= nkb * 128) return;
    const int kb = w >> 7, lane = (w >> 2) & 31, reg = w & 3;
    const int row = (lane >> 2) + 8 * (reg & 1);
    const int idx = 16 * kb + 2 * (lane & 3) + 8 * (reg >> 1);
    uint32_t word = 0u;
    if (row < M && idx < d) word = *reinterpret_cast<const uint32_t*>(h + (size_t)row * d + idx);
    zfrag[w] = word;
}


// ------------------------------------------------------------------------------------------
// Three to sixteen rows.  One CTA per V slab, seven warps, two CTAs per SM: all warps of a CTA meet
// at a barrier once per stage and then issue their tensor-core instructions together, so a second,
// independent CTA on the SM keeps the tensor pipe and the memory system busy meanwhile (one CTA of
// 14 warps spent as long at the barrier as in the instructions).  The slab's rows arrive through a ring
// of shared-memory stages (16 rows of the matrix each), filled by cp.async.  A warp owns 64 columns
// of the slab (two such chunks when the slab is wider than 7 x 64 columns) and all K rows: per
// stage it reads the "B" fragments of eight m16n8k16 instructions per chunk with ldmatrix.trans
// (the row pitch is an odd number of 16-byte units, so the eight rows of a matrix fall into
// distinct banks) and the code fragment from its own area of shared memory.  Lane (g, t) ends up
// with the logits of rows g and g + 8 at columns 8 e + 2 t, 8 e + 2 t + 1 of every 8-column unit e
// of its chunks.  MT = 8: rows 8-15 of the code fragment are the remainders of rows 0-7 (or zero),
// and the two halves of the result are summed.
template <int MT, int ZP, int NCH>
__global__ void __launch_bounds__(256, 2) k_stream_head_mma(const HeadParams p)      // at most 128 registers: a small CTA fits beside two of these
{
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* zarea = smem + ((kEpFixedBytes + 127) / 128) * 128;
    unsigned char* ring = zarea + p.zarea_bytes;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int nw = blockDim.x >> 5;
    const int cta = blockIdx.x;
    const int K = p.K;
    const size_t Vb = (size_t)p.V * sizeof(bf16);

    const int my_units = p.units_base + (cta < p.units_rem ? 1 : 0);
    const int unit0 = cta * p.units_base + min(cta, p.units_rem);
    const char* slab = reinterpret_cast<const char*>(p.B + (size_t)unit0 * 8);

    pdl_launch_dependents();
    for (int i = tid; i < 16 * 64; i += blockDim.x) reinterpret_cast<float*>(smem + 64)[i] = -FLT_MAX;

    // ---- this thread's share of a stage: 16-byte pieces (row, unit), the same for every stage
    constexpr int kMaxCopies = 8;
    uint32_t src_off[kMaxCopies], dst_off[kMaxCopies];
    const int pitch = p.pitch_units;                    // units between two rows of a stage (odd)
    const uint32_t stage_bytes = 16u * (uint32_t)pitch * 16u;
#pragma unroll
    for (int i = 0; i < kMaxCopies; ++i) {
        const int idx = tid + i * (int)blockDim.x;
        const int row = my_units > 0 ? idx / my_units : 16;
        const int c = idx - row * my_units;
        src_off[i] = row < 16 ? (uint32_t)((size_t)row * Vb) + (uint32_t)c * 16u : 0xffffffffu;
        dst_off[i] = ((uint32_t)row * (uint32_t)pitch + (uint32_t)c) * 16u;
    }
    const int nkb = p.nkb, NS = p.ns;
    auto issue_stage = [&](int kb, int slot) {
        if (kb < nkb) {
            unsigned char* dst = ring + (size_t)slot * stage_bytes;
            if (16 * kb + 16 <= K) {
                const char* src = slab + (size_t)(16 * kb) * Vb;
#pragma unroll
                for (int i = 0; i < kMaxCopies; ++i)
                    if (src_off[i] != 0xffffffffu) cp_async16(dst + dst_off[i], src + src_off[i]);
            } else {
                // the last block of a K that is no multiple of 16: rows past the end re-read the last
                // row (their code entries are zero)
                for (int idx = tid; idx < 16 * my_units; idx += blockDim.x) {
                    const int row = idx / my_units, c = idx - row * my_units;
                    cp_async16(dst + ((size_t)row * pitch + c) * 16, slab + (size_t)min(16 * kb + row, K - 1) * Vb + (size_t)c * 16);
                }
            }
        }
    };
    // code fragments: whole in shared memory, or chunk by chunk through two buffers
    const size_t kb_bytes = (size_t)ZP * 512;
    const size_t zchunk_bytes = (size_t)p.kb_chunk * kb_bytes;
    auto copy_zchunk = [&](int c) {
        const int kb0 = c * p.kb_chunk;
        if (kb0 >= nkb) return;
        unsigned char* dst = zarea + (p.nchunks > 1 ? (size_t)(c & 1) * zchunk_bytes : 0);
        const int n16 = (int)((size_t)(min(nkb, kb0 + p.kb_chunk) - kb0) * kb_bytes / 16);
        const uint4* src = reinterpret_cast<const uint4*>(p.zfrag) + (size_t)kb0 * kb_bytes / 16;
        for (int i = tid; i < n16; i += blockDim.x) cp_async16(dst + (size_t)i * 16, src + i);
    };

    // ---- the warp's chunks of 64 columns and its ldmatrix lane address inside a stage
    bool chunk_on[NCH];
    int cb[NCH];                                        // first unit of the chunk
#pragma unroll
    for (int ch = 0; ch < NCH; ++ch) { cb[ch] = 8 * (warp + nw * ch); chunk_on[ch] = cb[ch] < my_units; }
    // lane l gives the address of row (l & 7) of matrix (l >> 3): matrices 0, 1 are rows 0-7 and
    // 8-15 of a unit, matrices 2, 3 the same rows of the next unit
    const uint32_t lane_off = ((uint32_t)((lane & 7) + ((lane >> 3) & 1) * 8) * (uint32_t)pitch + (uint32_t)(lane >> 4)) * 16u;
    const uint32_t ring_s = smem_u32(ring);

    float acc[NCH][8][4];
#pragma unroll
    for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
        for (int e = 0; e < 8; ++e)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[ch][e][c] = 0.f;

    // ---- the pipeline: NS - 1 stages in flight.  The first stages go out before the kernel ahead in
    // the stream is waited for (weights are final before the call is made: the contract of the
    // library); the code, which that kernel writes, after it -- it travels with stage NS - 2.
    for (int s = 0; s < NS - 2; ++s) { issue_stage(s, s); cp_async_commit(); }
    if (p.wait_prev) pdl_wait();
    copy_zchunk(0);
    issue_stage(NS - 2, NS - 2);
    cp_async_commit();
    int slot = 0, fill_slot = NS - 1;
    int zc = 0, zkb0 = 0, zkb1 = min(nkb, p.kb_chunk);      // current chunk of the code
    for (int kb = 0; kb < nkb; ++kb) {
        cp_async_wait_pending(kb == 0 ? 0 : NS - 2);        // the first time round the code, which went out last, must be in too
        __syncthreads();            // stage kb has landed for everyone; everyone is done with stage kb - 1
        if (kb == zkb1) { ++zc; zkb0 = zkb1; zkb1 = min(nkb, zkb0 + p.kb_chunk); }
        if (kb == zkb0 && p.nchunks > 1) copy_zchunk(zc + 1);
        issue_stage(kb + NS - 1, fill_slot);
        cp_async_commit();
        if (++fill_slot == NS) fill_slot = 0;

        const unsigned char* zbuf = zarea + (p.nchunks > 1 ? (size_t)(zc & 1) * zchunk_bytes : 0);
        const uint4* zp = reinterpret_cast<const uint4*>(zbuf) + (size_t)(kb - zkb0) * (ZP * 32) + lane;
        const uint4 zh = zp[0];
        uint4 zl = make_uint4(0u, 0u, 0u, 0u);
        if (ZP == 2) zl = zp[32];
        const uint32_t st = ring_s + (uint32_t)slot * stage_bytes + lane_off;
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch) {
            if (chunk_on[ch]) {
                const uint32_t a = st + (uint32_t)cb[ch] * 16u;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    uint32_t b0, b1, b2, b3;
                    ldmatrix_x4_trans(b0, b1, b2, b3, a + (uint32_t)j * 32u);
                    mma_bf16(acc[ch][2 * j], zh, b0, b1);
                    mma_bf16(acc[ch][2 * j + 1], zh, b2, b3);
                    if (ZP == 2) {
                        mma_bf16(acc[ch][2 * j], zl, b0, b1);
                        mma_bf16(acc[ch][2 * j + 1], zl, b2, b3);
                    }
                }
            }
        }
        if (++slot == NS) slot = 0;
    }
    cp_async_wait_pending(0);
    __syncthreads();                // the ring is idle from here on: it takes the logits and the epilogue's lists

    // ---- the slab's logits to shared memory, [MT][lpitch].  Unit e of chunk ch exists if
    // cb[ch] + e < my_units; its columns 2 t, 2 t + 1 are values (0, 1) of the tile for row g and
    // (2, 3) for row g + 8.
    const int lpitch = pitch * 8 + 8;
    float* lg = reinterpret_cast<float*>(ring);
#pragma unroll
    for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            if (chunk_on[ch] && cb[ch] + e < my_units) {
                float* dst = lg + (size_t)g * lpitch + (cb[ch] + e) * 8 + 2 * t;
                if (MT == 8) {
                    *reinterpret_cast<float2*>(dst) = make_float2(acc[ch][e][0] + acc[ch][e][2], acc[ch][e][1] + acc[ch][e][3]);
                } else {
                    *reinterpret_cast<float2*>(dst) = make_float2(acc[ch][e][0], acc[ch][e][1]);
                    *reinterpret_cast<float2*>(dst + (size_t)8 * lpitch) = make_float2(acc[ch][e][2], acc[ch][e][3]);
                }
            }
        }
    __syncthreads();
    unsigned char* lists = reinterpret_cast<unsigned char*>(lg + (size_t)MT * lpitch);
    slab_epilogue_rows<MT>(p, smem, lists, zarea, lg, lpitch, my_units * 8, unit0 * 8);
}

// ------------------------------------------------------------------------------------------
struct Geometry {
    int ncta, units_base, units_rem, rec_words;
    int nch, pitch_units, ns, nkb, kb_chunk, nchunks, warps;
    size_t zarea_bytes, smem;
};

static constexpr size_t kHeadSmemMax = 226 * 1024;

static size_t merge_bytes(int) { return (size_t)(16 + 2 * 16 * 32 + 16 * 2 * kMergeCand) * 4; }

// zparts: 1 or 2 parts of code fragments (tensor-core kernel)
static bool geometry(int M, int zparts, int K, int V, int k, int sm_count, Geometry* g)
{
    if (V % 8 != 0 || K < 1 || k > 32 || k < 1 || M < 1 || M > 16) return false;
    const int units = V / 8;
    g->rec_words = (2 + 2 * k + 3) / 4 * 4;
    const size_t fixed0 = ((kEpFixedBytes + 127) / 128) * 128;
    const int mt = M <= 8 ? 8 : 16;
    // two CTAs per SM
    int ncta = 2 * sm_count;
    if (ncta > units) ncta = units;
    if (ncta > kMaxRecords) ncta = kMaxRecords;
    g->ncta = ncta;
    g->units_base = units / ncta;
    g->units_rem = units % ncta;
    const int mma_units = g->units_base + (g->units_rem ? 1 : 0);
    g->warps = mma_warps(M);
    g->nch = (mma_units + 8 * g->warps - 1) / (8 * g->warps);
    if (g->nch > 2) return false;
    g->pitch_units = mma_units | 1;
    g->nkb = (K + 15) / 16;
    const size_t kb_bytes = (size_t)zparts * 512;
    const size_t zbytes = (size_t)g->nkb * kb_bytes;
    if (zbytes <= kZOneChunkBytes) {
        g->kb_chunk = g->nkb;
        g->nchunks = 1;
        g->zarea_bytes = zbytes;
    } else {
        g->kb_chunk = (int)(kZChunkBytes / kb_bytes);
        g->nchunks = (g->nkb + g->kb_chunk - 1) / g->kb_chunk;
        g->zarea_bytes = 2 * (size_t)g->kb_chunk * kb_bytes;
    }
    // the ring takes what is left; the logits, the epilogue's lists and the last CTA's merge reuse it
    const size_t fixed = fixed0 + g->zarea_bytes + 256;
    const size_t stage = (size_t)16 * g->pitch_units * 16;
    const size_t ep = (size_t)mt * (g->pitch_units * 8 + 8) * 4 + (size_t)mt * kCand * 8;
    if (fixed + 3 * stage > kMmaSmem) return false;
    int ns = (int)((kMmaSmem - fixed) / stage);
    if (ns > kMaxStages) ns = kMaxStages;
    g->ns = ns;
    size_t ringb = (size_t)ns * stage;
    if (ringb < ep) ringb = ep;
    if (g->zarea_bytes + ringb < merge_bytes(ncta)) ringb = merge_bytes(ncta) - g->zarea_bytes;     // the merge works in both areas
    g->smem = fixed + ringb;
    return g->smem <= kHeadSmemMax;
}

// The form of the code the head kernel for (M, low-rank or not) reads.
static int code_format(const Geometry& g, int M, bool lowrank)
{
    (void)g;
    if (!lowrank) return kCodePlain;
    return M <= 8 ? kCodePacked : kCodeSplit;
}

StreamPlan stream_plan(int M, int K, int V, int k, int sm_count)
{
    StreamPlan sp = {0, 0, 0, 0, 0};
    if (M < 1) return sp;
    Geometry g;
    if (!geometry(M > 16 ? 16 : M, 2, K, V, k, sm_count, &g)) return sp;
    sp.ok = 1;
    sp.mt = M <= 8 ? 8 : 16;
    sp.ncta = g.ncta;
    sp.parts = g.ncta;
    sp.launches = 2;
    return sp;
}

size_t stream_code_bytes(int K) { return (size_t)((K + 15) / 16) * 2 * 512 + 1024; }

static bool plan_code(int M, bool lowrank, int K, int V, int k, int sm_count, Geometry* g, int* fmt)
{
    const int zparts = (lowrank && M > 8) ? 2 : 1;
    if (!geometry(M, zparts, K, V, k, sm_count, g)) return false;
    *fmt = code_format(*g, M, lowrank);
    return true;
}

// Launch with programmatic stream serialization: the kernel may begin once every CTA of the kernel
// before it in the stream has signalled launch_dependents or left; it orders itself after that
// kernel with griddepcontrol.wait.  Across calls this hides the launch gap and lets the first
// kernel of a call warm up under the tail of the last kernel of the call before.
static cudaError_t launch_code(CodeParams cp, int sm_count, size_t head_smem, cudaStream_t st)
{
    cp.nkb = (cp.d + 15) / 16;
    const int nct = (cp.r + 31) / 32;
    const int ntiles = (cp.M + 15) / 16;
    // One CTA per SM at most while a CTA's whole share of A fits beside a head CTA; a larger A goes
    // through a ring of buffers with two CTAs per SM (what counts then is the bandwidth of this kernel).
    int S = 8;
    while (S > 1 && (S * nct * ntiles > sm_count || S * 4 > cp.nkb)) S >>= 1;
    if (((cp.nkb + S - 1) / S) * 16 > kCodeSliceRows) {
        S = 8;
        while (S > 1 && (S * nct * ntiles > 2 * sm_count || S * 4 > cp.nkb)) S >>= 1;
    }
    cp.S = S;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(S, nct, ntiles);
    cfg.blockDim = dim3(128);
    {
        const int kbs = (cp.nkb + S - 1) / S;
        if (kbs * 16 <= kCodeSliceRows) {
            cp.chunk_kbs = kbs; cp.nbuf = 1; cfg.dynamicSmemBytes = (size_t)kbs * 16 * kCodePitch + 128;
            // The block scheduler fills an SM with as many of these CTAs as fit (two or three on 60 of the
            // SMs, measured), and a head CTA of the same call that finds its place taken starts only when
            // they have left, without the rows it would have fetched meanwhile.  Asking for enough shared
            // memory that two of these CTAs do not fit beside one head CTA, while one still fits beside
            // two, spreads them over the SMs (one each on 92, two on 18).  It does not cure the late starts
            // (a head CTA still comes up late on most SMs that hold one of these), but it is never slower
            // and up to 2.3 us per call faster (small head, 8 rows: 30.5 -> 28.2 us).
            if (head_smem > 0) {
                const size_t sm_bytes = 228 * 1024, per_cta = 1024, fixed = 24 * 1024 + per_cta;      // static arrays, reserve
                const size_t head_cost = head_smem + per_cta;
                const size_t lower = (sm_bytes - head_cost) / 2 + 1024;       // head + 2 x this: too much
                const size_t upper = sm_bytes - 2 * head_cost;                // 2 heads + this: fits
                if (lower <= upper && lower > fixed + cfg.dynamicSmemBytes && lower - fixed <= kCodeSmemMax) cfg.dynamicSmemBytes = lower - fixed;
            }
        }
        else { cp.chunk_kbs = kCodeChunkRows / 16; cp.nbuf = kCodeRing; cfg.dynamicSmemBytes = (size_t)kCodeRing * kCodeChunkRows * kCodePitch + 128; }
    }
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = S;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, k_stream_code, cp);
}

cudaError_t stream_code(const bf16* h, const bf16* A, int M, int d, int r, int V, int k, uint32_t* zfrag, int sm_count,
                        cudaStream_t st)
{
    Geometry g;
    CodeParams cp;
    memset(&cp, 0, sizeof(cp));
    if (!plan_code(M, true, r, V, k, sm_count, &g, &cp.fmt)) return cudaErrorInvalidValue;
    cp.h = h; cp.A = A; cp.M = M; cp.d = d; cp.r = r; cp.zfrag = zfrag;
    return launch_code(cp, sm_count, g.smem, st);
}

cudaError_t stream_code_rows(const bf16* h, const bf16* A, int M, int d, int r, bf16* z, bf16* z_lo, int sm_count, cudaStream_t st)
{
    if (d % 2 != 0 || r % 16 != 0 || M < 1) return cudaErrorInvalidValue;
    CodeParams cp;
    memset(&cp, 0, sizeof(cp));
    cp.fmt = kCodeRows;
    cp.h = h; cp.A = A; cp.M = M; cp.d = d; cp.r = r; cp.zrows = z; cp.zrows_lo = z_lo;
    return launch_code(cp, sm_count, 0, st);
}

cudaError_t stream_widen(const bf16* h, int M, int d, int V, int k, uint32_t* zfrag, int sm_count, cudaStream_t st)
{
    Geometry g;
    int fmt;
    if (!plan_code(M, false, d, V, k, sm_count, &g, &fmt)) return cudaErrorInvalidValue;
    const int nkb = (d + 15) / 16;
    const int n = nkb * 128;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((n + 255) / 256);
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, k_stream_widen, h, M, d, nkb, zfrag);
}

// Once per device: load the kernels of this file and allow the head kernels their dynamic shared
// memory, so that no call on the hot path has to (module loading allocates and may synchronise).
template <typename Kern>
static cudaError_t allow_smem(Kern kern)
{
    return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kHeadSmemMax);
}

cudaError_t stream_prepare()
{
    cudaError_t e;
    cudaFuncAttributes fa;
    if ((e = cudaFuncGetAttributes(&fa, k_stream_code)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(k_stream_code, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kCodeSmemMax)) != cudaSuccess) return e;
    if ((e = cudaFuncGetAttributes(&fa, k_stream_widen)) != cudaSuccess) return e;
    if ((e = allow_smem(k_stream_head_mma<8, 1, 1>)) != cudaSuccess) return e;
    if ((e = allow_smem(k_stream_head_mma<8, 1, 2>)) != cudaSuccess) return e;
    if ((e = allow_smem(k_stream_head_mma<16, 1, 1>)) != cudaSuccess) return e;
    if ((e = allow_smem(k_stream_head_mma<16, 1, 2>)) != cudaSuccess) return e;
    if ((e = allow_smem(k_stream_head_mma<16, 2, 1>)) != cudaSuccess) return e;
    if ((e = allow_smem(k_stream_head_mma<16, 2, 2>)) != cudaSuccess) return e;
    return cudaSuccess;
}

template <typename Kern>
static cudaError_t launch_head(Kern kern, const HeadParams& hp, const Geometry& g, bool pdl, cudaStream_t st)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(hp.ncta);
    cfg.blockDim = dim3(g.warps * 32);
    cfg.dynamicSmemBytes = g.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, hp);
}

cudaError_t stream_head(const uint32_t* zfrag, bool lowrank, const bf16* B, int M, int K, int V, int k, int mode,
                        int32_t* ids, float* logprobs, float* logits, const Scratch& s, int sm_count,
                        bool after_producer_kernel, int* launches, cudaStream_t st)
{
    Geometry g;
    int fmt;
    if (!plan_code(M, lowrank, K, V, k, sm_count, &g, &fmt)) return cudaErrorInvalidValue;
    if (g.ncta > s.max_parts) return cudaErrorInvalidValue;
    HeadParams hp;
    memset(&hp, 0, sizeof(hp));
    hp.zfrag = zfrag; hp.B = B; hp.M = M; hp.K = K; hp.V = V; hp.k = k; hp.mode = mode;
    hp.ncta = g.ncta; hp.units_base = g.units_base; hp.units_rem = g.units_rem;
    hp.rec_words = g.rec_words;
    hp.zarea_bytes = (unsigned int)g.zarea_bytes;
    hp.ids = ids; hp.logprobs = logprobs; hp.logits = logits;
    hp.part = s.part; hp.ticket = s.tickets; hp.err = s.err;
    hp.wait_prev = after_producer_kernel ? 1 : 0;
    hp.merge_inside = 1;
    hp.ticket_base = 0;
    if (mode == 0) hp.ticket_base = *s.ticket_base_host;
    const bool pdl = after_producer_kernel;
    cudaError_t e;
    {
        hp.pitch_units = g.pitch_units; hp.ns = g.ns;
        hp.nkb = g.nkb; hp.kb_chunk = g.kb_chunk; hp.nchunks = g.nchunks;
        if (fmt == kCodeSplit)
            e = g.nch == 1 ? launch_head(k_stream_head_mma<16, 2, 1>, hp, g, pdl, st) : launch_head(k_stream_head_mma<16, 2, 2>, hp, g, pdl, st);
        else if (M <= 8)
            e = g.nch == 1 ? launch_head(k_stream_head_mma<8, 1, 1>, hp, g, pdl, st) : launch_head(k_stream_head_mma<8, 1, 2>, hp, g, pdl, st);
        else
            e = g.nch == 1 ? launch_head(k_stream_head_mma<16, 1, 1>, hp, g, pdl, st) : launch_head(k_stream_head_mma<16, 1, 2>, hp, g, pdl, st);
    }
    if (launches) *launches += 1;
    if (e == cudaSuccess && mode == 0) *s.ticket_base_host += (unsigned int)hp.ncta;      // the tickets this launch will take
    return e;
}

}  // namespace slimspec
