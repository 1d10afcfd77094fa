// The record of the bounds-checked build (see jq_debug.cuh).  Empty in the ordinary build.
#include "jq_internal.cuh"
#include "jq_debug.cuh"
#ifdef JQ_DEBUG
#include <mutex>

namespace jq {
namespace {
static __device__ DebugRecord g_record;
}

DebugRecord *debug_record()
{
    static DebugRecord *addr[64] = {};
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_record) != cudaSuccess) { cudaGetLastError(); return nullptr; }
        addr[dev] = (DebugRecord *)p;
    }
    return addr[dev];
}
}  // namespace jq

// out: violations, kernel, site, index, extent of the first violation.  Synchronises the device.  0 on success.
extern "C" int jq_debug_read(long long out[5])
{
    jq::DebugRecord *p = jq::debug_record(), r;
    if (!p || cudaDeviceSynchronize() != cudaSuccess || cudaMemcpy(&r, p, sizeof r, cudaMemcpyDeviceToHost) != cudaSuccess) return 1;
    out[0] = (long long)r.violations; out[1] = r.kernel; out[2] = r.site; out[3] = r.index; out[4] = r.extent;
    return 0;
}

extern "C" int jq_debug_reset(void)
{
    jq::DebugRecord *p = jq::debug_record();
    return (!p || cudaDeviceSynchronize() != cudaSuccess || cudaMemset(p, 0, sizeof(jq::DebugRecord)) != cudaSuccess) ? 1 : 0;
}
#endif
