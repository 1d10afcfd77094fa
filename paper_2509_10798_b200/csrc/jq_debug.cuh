// Bounds-checked build of the kernels (-DJQ_DEBUG; build.build(debug=True) makes libjq_debug.so from the same
// sources).  It stands in for a memory checker: every index that score_fused, select_cluster, gather_rows and
// decode_step compute into global, shared or tensor memory goes through JQ_IN(index, extent, kernel, site) before
// the access.  An index outside [0, extent) is counted in a record in device memory, the first one is kept
// (which kernel, which site, the index and the extent), and the access is skipped: the kernel never traps and
// always runs to its end.  The host reads the record with jq_debug_read (exported by the debug library only).
// In the ordinary build JQ_IN is the constant true and the extra kernel parameter does not exist.
#pragma once

namespace jq {

struct DebugRecord {
    unsigned long long violations;   // accesses that were skipped
    int kernel, site;                // of the first one
    long long index, extent;
};
enum { kDbgScore = 1, kDbgSelect = 2, kDbgGather = 3, kDbgDecode = 4 };

#ifdef JQ_DEBUG
DebugRecord *debug_record();   // host: device address of the record on the current device (nullptr on error)
__device__ __forceinline__ bool dbg_in(DebugRecord *r, long long i, long long n, int kernel, int site)
{
    if (i >= 0 && i < n) return true;
    if (atomicAdd(&r->violations, 1ull) == 0ull) { r->kernel = kernel; r->site = site; r->index = i; r->extent = n; }
    return false;
}
#define JQ_DBG_PARAM , ::jq::DebugRecord *dbg
#define JQ_DBG_ARG , ::jq::debug_record()
#define JQ_DBG_ARG_DEV , dbg
#define JQ_IN(i, n, kernel, site) ::jq::dbg_in(dbg, (long long)(i), (long long)(n), kernel, site)
#else
#define JQ_DBG_PARAM
#define JQ_DBG_ARG
#define JQ_DBG_ARG_DEV
#define JQ_IN(i, n, kernel, site) true
#endif

}  // namespace jq
