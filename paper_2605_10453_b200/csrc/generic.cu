// Generic path: correct for every shape and alignment, one thread per output element.
// It is the fallback for shapes the fast kernels do not take (odd V, tiny r, ...) and a
// second, independent GPU implementation the fast paths are compared with.
#include "kernels.h"
#include <float.h>

namespace slimspec {

// z[m][j] = sum_i h[m][i] A[i][j]    (Section 4.1: W_down h)
__global__ void k_generic_downproj(const bf16* __restrict__ h, const bf16* __restrict__ A, int d, int r,
                                   float* __restrict__ z)
{
    int j = blockIdx.x * blockDim.x + threadIdx.x;
    int m = blockIdx.y;
    if (j >= r) return;
    float acc = 0.f;
    for (int i = 0; i < d; ++i)
        acc = fmaf(__bfloat162float(h[(size_t)m * d + i]), __bfloat162float(A[(size_t)i * r + j]), acc);
    z[(size_t)m * r + j] = acc;
}

__global__ void k_generic_widen(const bf16* __restrict__ h, int n, float* __restrict__ z)
{
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) z[i] = __bfloat162float(h[i]);
}

// logits[m][v] = sum_j z[m][j] B[j][v]    (Section 4.1: W_up applied to the code)
__global__ void k_generic_upproj(const float* __restrict__ z, const bf16* __restrict__ B, int r, int V,
                                 float* __restrict__ logits)
{
    int v = blockIdx.x * blockDim.x + threadIdx.x;
    int m = blockIdx.y;
    if (v >= V) return;
    float acc = 0.f;
    for (int j = 0; j < r; ++j)
        acc = fmaf(z[(size_t)m * r + j], __bfloat162float(B[(size_t)j * V + v]), acc);
    logits[(size_t)m * V + v] = acc;
}

// (value desc, id asc) order: is (a, ia) strictly before (b, ib)?
__device__ __forceinline__ bool before(float a, int ia, float b, int ib)
{
    return a > b || (a == b && ia < ib);
}

// One block per row: max, sum of exp, then k rounds of "best element after the previous winner".
__global__ void k_generic_softmax_topk(const float* __restrict__ logits, int V, int k,
                                       int32_t* __restrict__ ids, float* __restrict__ logprobs)
{
    __shared__ float s_val[256];
    __shared__ int s_idx[256];
    const int t = threadIdx.x, nt = blockDim.x;
    const float* row = logits + (size_t)blockIdx.x * V;

    float mx = -FLT_MAX;
    for (int v = t; v < V; v += nt) mx = fmaxf(mx, row[v]);
    s_val[t] = mx;
    __syncthreads();
    for (int s = nt / 2; s > 0; s >>= 1) {
        if (t < s) s_val[t] = fmaxf(s_val[t], s_val[t + s]);
        __syncthreads();
    }
    mx = s_val[0];
    __syncthreads();

    float sum = 0.f;
    for (int v = t; v < V; v += nt) sum += expf(row[v] - mx);
    s_val[t] = sum;
    __syncthreads();
    for (int s = nt / 2; s > 0; s >>= 1) {
        if (t < s) s_val[t] += s_val[t + s];
        __syncthreads();
    }
    const float lse = mx + logf(s_val[0]);
    __syncthreads();

    float pv = FLT_MAX;   // previous winner; everything must come strictly after it
    int pi = -1;
    for (int j = 0; j < k; ++j) {
        float bv = -FLT_MAX;
        int bi = 0x7fffffff;
        for (int v = t; v < V; v += nt) {
            float x = row[v];
            if (before(pv, pi, x, v) && before(x, v, bv, bi)) { bv = x; bi = v; }
        }
        s_val[t] = bv;
        s_idx[t] = bi;
        __syncthreads();
        for (int s = nt / 2; s > 0; s >>= 1) {
            if (t < s && before(s_val[t + s], s_idx[t + s], s_val[t], s_idx[t])) {
                s_val[t] = s_val[t + s];
                s_idx[t] = s_idx[t + s];
            }
            __syncthreads();
        }
        pv = s_val[0];
        pi = s_idx[0];
        if (t == 0) {
            ids[(size_t)blockIdx.x * k + j] = pi;
            logprobs[(size_t)blockIdx.x * k + j] = pv - lse;
        }
        __syncthreads();
    }
}

cudaError_t generic_downproj(const bf16* h, const bf16* A, int M, int d, int r, float* z, cudaStream_t st)
{
    dim3 g((r + 127) / 128, M);
    k_generic_downproj<<<g, 128, 0, st>>>(h, A, d, r, z);
    return cudaGetLastError();
}

cudaError_t generic_widen(const bf16* h, int n, float* z, cudaStream_t st)
{
    k_generic_widen<<<(n + 255) / 256, 256, 0, st>>>(h, n, z);
    return cudaGetLastError();
}

cudaError_t generic_upproj(const float* z, const bf16* B, int M, int r, int V, float* logits, cudaStream_t st)
{
    dim3 g((V + 255) / 256, M);
    k_generic_upproj<<<g, 256, 0, st>>>(z, B, r, V, logits);
    return cudaGetLastError();
}

cudaError_t generic_softmax_topk(const float* logits, int M, int V, int k, int32_t* ids, float* logprobs,
                                 cudaStream_t st)
{
    k_generic_softmax_topk<<<M, 256, 0, st>>>(logits, V, k, ids, logprobs);
    return cudaGetLastError();
}

}  // namespace slimspec
