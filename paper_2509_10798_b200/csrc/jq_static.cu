// jq_score_static: the tensor-core scoring of jq_score for callers that cannot allocate device memory.
//
// The scratch that jq_score takes from the caller's workspace (the status block with the grid counters,
// the merged row normalisers and the per-CTA partial row statistics of pass 1) lives here in one
// file-scope device array instead.  Every GPU that loads the library holds the array until the process
// exits.  In host code the array's name is only a handle: the device address is asked for once per
// device with cudaGetSymbolAddress, with that device current, and that address is what the kernel gets.
#include "jq_internal.cuh"
#include <mutex>

namespace jq {
namespace {

constexpr int kStaticRows = 2048;   // largest Hkv * group * w (query rows over all KV heads) the array serves
constexpr size_t kStaticStatusBytes = 256;
constexpr size_t kStaticMrowBytes = (size_t)kStaticRows * sizeof(float);
constexpr size_t kStaticPartBytes = (size_t)kStaticRows * kSlots * sizeof(float2);
constexpr size_t kStaticBytes = kStaticStatusBytes + kStaticMrowBytes + kStaticPartBytes;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

// Device address of the array on the current device; nullptr if the runtime refuses.
unsigned char *static_scratch_address()
{
    static unsigned char *addr[64] = {};
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return nullptr;
        }
        addr[dev] = (unsigned char *)p;
    }
    return addr[dev];
}

}  // namespace
}  // namespace jq

using namespace jq;

extern "C" jq_status jq_score_static(const void *K, const void *Qwin, const jq_shape *s, float *scores,
                                     jq_stream_t stream)
{
    jq_status rc = jq_check_shape(s);
    if (rc != JQ_OK) return rc;
    if (!K || !Qwin || !scores || ((uintptr_t)K & 15u) || ((uintptr_t)Qwin & 15u) || ((uintptr_t)scores & 15u))
        return JQ_ERR_INVALID_ARG;
    const long long rows = (long long)s->Hkv * s->group * s->w;
    if (rows > kStaticRows) return JQ_ERR_UNSUPPORTED;   // beyond what the built-in scratch array serves
    unsigned char *base = static_scratch_address();
    if (!base) return JQ_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    // The array keeps what the last call left.  Only the status block (status word, grid counters) must
    // start at zero; the normalisers and partials are written before they are read.
    if (cudaMemsetAsync(base, 0, kStaticStatusBytes, st) != cudaSuccess) return JQ_ERR_CUDA;
    Workspace w = {};
    w.status = (int *)base;
    w.Mrow = (float *)(base + kStaticStatusBytes);
    w.part = (float2 *)(base + kStaticStatusBytes + kStaticMrowBytes);
    w.bytes = kStaticBytes;
    return launch_score_tc(K, Qwin, *s, scores, w, st);
}
