// slimspec_head_topk_static: the streaming low-rank head for callers that cannot allocate.
//
// The ordinary entry points take a context whose scratch comes from cudaMalloc.  Some callers
// must not allocate once they are running: a serving loop whose memory pool already owns every
// byte of the device, a plugin invoked by a runtime that forbids driver allocations on its worker
// threads, a latency-critical section where the implicit device synchronisation of cudaMalloc /
// cudaFree is unacceptable.  For them the scratch of the streaming kernels (the fp32 code z, the
// per-slab softmax / top-k records, the arrival ticket and the error word) lives in one file-scope
// device array of fixed size that is part of the library image: every GPU that loads the library
// holds these bytes until the process exits.
#include "../../include/slimspec.h"
#include "kernels.h"
#include <mutex>

using namespace slimspec;

namespace {

// Layout of the static scratch, in bytes.  Limits: M <= 8 rows, r <= SLIMSPEC_STATIC_MAX_R,
// k <= 32, at most 320 split-V records per row.
constexpr size_t kZBytes = (size_t)(SLIMSPEC_STATIC_MAX_R / 16) * 2 * 512 + 1024;   // the code, in its largest form
constexpr size_t kRecWords = 68;                                                     // 2 + 2*32, padded to 4
constexpr int kStaticParts = 320;
constexpr size_t kPartBytes = (size_t)8 * kStaticParts * kRecWords * sizeof(float);  // [8 rows][320 records]
constexpr size_t kCtlBytes = 256;                                                    // ticket, error word
constexpr size_t kZqBytes = (size_t)4 * SLIMSPEC_STATIC_MAX_R * 8;                   // one- and two-row calls: the code as published (value, call number) words
constexpr size_t kScratchBytes = kZBytes + kPartBytes + kCtlBytes + kZqBytes;

static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

struct DeviceSetup {
    bool ready;
    unsigned char* base;     // device address of g_static_scratch on this device
    int sm_count;
    unsigned int epoch;      // number of the last one- or two-row call on this device
};
constexpr int kMaxDevices = 64;
DeviceSetup g_setup[kMaxDevices];
std::mutex g_setup_mutex;

// Once per device, with that device current: ask the runtime where the array lives on this
// device.  The name g_static_scratch is only a handle in host code, never a device pointer.
int setup_current_device(DeviceSetup** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return SLIMSPEC_ERR_CUDA; }
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    DeviceSetup& s = g_setup[dev];
    if (!s.ready) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) { cudaGetLastError(); return SLIMSPEC_ERR_CUDA; }
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) { cudaGetLastError(); return SLIMSPEC_ERR_CUDA; }
        // load the kernels now, so that no later call has to (loading a module allocates)
        if (stream_prepare() != cudaSuccess || fma_prepare() != cudaSuccess) { cudaGetLastError(); return SLIMSPEC_ERR_CUDA; }
        s.base = static_cast<unsigned char*>(ptr);
        s.sm_count = sms;
        s.ready = true;
    }
    *out = &s;
    return SLIMSPEC_OK;
}

bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }

}  // namespace

extern "C" int slimspec_head_topk_static(const void* h, const void* A, const void* B, int M, int d, int r, int V, int k,
                                         int32_t* out_ids, float* out_logprobs, void* stream)
{
    if (!h || !A || !B || !out_ids || !out_logprobs) return SLIMSPEC_ERR_NULL;
    if (M <= 0 || d <= 0 || r <= 0 || V <= 0 || k <= 0 || k > V) return SLIMSPEC_ERR_DIM;
    // beyond the fixed scratch: say so instead of overrunning it
    if (M > SLIMSPEC_STATIC_MAX_M || r > SLIMSPEC_STATIC_MAX_R || k > SLIMSPEC_STATIC_MAX_K) return SLIMSPEC_ERR_STATIC_LIMIT;
    DeviceSetup* dev = nullptr;
    int rc = setup_current_device(&dev);
    if (rc != SLIMSPEC_OK) return rc;
    StreamPlan plan = stream_plan(M, r, V, k, dev->sm_count);
    if (!plan.ok || r % 16 != 0 || d % 2 != 0 || !aligned16(h) || !aligned16(A) || !aligned16(B)) return SLIMSPEC_ERR_ALIGN;
    if (plan.parts > kStaticParts) return SLIMSPEC_ERR_STATIC_LIMIT;

    Scratch s = {};
    s.zfrag = reinterpret_cast<uint32_t*>(dev->base);
    s.part = reinterpret_cast<float*>(dev->base + kZBytes);
    s.tickets = reinterpret_cast<unsigned int*>(dev->base + kZBytes + kPartBytes);
    s.err = reinterpret_cast<int*>(dev->base + kZBytes + kPartBytes + 128);
    s.zq = reinterpret_cast<uint2*>(dev->base + kZBytes + kPartBytes + kCtlBytes);
    s.max_parts = kStaticParts;
    unsigned int ticket_base = 0;           // the counter is cleared below, before every call
    s.ticket_base_host = &ticket_base;
    cudaStream_t st = (cudaStream_t)stream;
    // The array keeps whatever the last call left; the ticket and the error word must start at 0.
    if (cudaMemsetAsync(dev->base + kZBytes + kPartBytes, 0, kCtlBytes, st) != cudaSuccess) { cudaGetLastError(); return SLIMSPEC_ERR_CUDA; }
    // the same choice of kernels as the context-based entry point: one or two rows, the FMA kernel
    const FmaPlan fp = fma_plan(M, d, r, V, k, dev->sm_count);
    cudaError_t e;
    if (fp.ok && fp.ncta <= kStaticParts) {
        // the words of that area start as zeros (static storage) and only these calls write them; each call
        // takes the next number, under the lock that also guards the set-up
        unsigned int epoch;
        {
            std::lock_guard<std::mutex> lock(g_setup_mutex);
            epoch = ++dev->epoch;
            if (epoch == 0) {
                if (cudaMemsetAsync(s.zq, 0, kZqBytes, st) != cudaSuccess) { cudaGetLastError(); return SLIMSPEC_ERR_CUDA; }
                epoch = dev->epoch = 1;
            }
        }
        e = fma_head((const bf16*)h, (const bf16*)A, (const bf16*)B, M, fp.mt, d, r, V, k, 0, out_ids, out_logprobs, nullptr, s, epoch, dev->sm_count, st);
    } else {
        e = stream_code((const bf16*)h, (const bf16*)A, M, d, r, V, k, s.zfrag, dev->sm_count, st);
        if (e == cudaSuccess) e = stream_head(s.zfrag, true, (const bf16*)B, M, r, V, k, 0, out_ids, out_logprobs, nullptr, s, dev->sm_count, true, nullptr, st);
    }
    if (e != cudaSuccess) { cudaGetLastError(); return SLIMSPEC_ERR_CUDA; }
    return SLIMSPEC_OK;
}
