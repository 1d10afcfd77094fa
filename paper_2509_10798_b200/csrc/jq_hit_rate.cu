// Eq. 6, the critical key-value hit rate |I_cur ^ I_ref| / |I_ref| of two kept-index sets, per KV head.
// Both rows are strictly ascending (what jq_select_topk writes): a thread takes an element of the reference
// row and looks it up in the other row by binary search; one block per KV head counts the hits.
#include "jq_internal.cuh"

namespace jq {
namespace {

__global__ void __launch_bounds__(256)
hit_rate_rows(const int32_t *__restrict__ cur, const int32_t *__restrict__ ref, int ncur, int nref, float *__restrict__ rate)
{
    const int32_t *a = cur + (size_t)blockIdx.x * ncur, *b = ref + (size_t)blockIdx.x * nref;
    __shared__ int hits;
    if (threadIdx.x == 0) hits = 0;
    __syncthreads();
    int mine = 0;
    for (int i = threadIdx.x; i < nref; i += blockDim.x) {
        const int32_t x = b[i];
        int lo = 0, hi = ncur;                 // first position of a with a[pos] >= x
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (a[mid] < x) lo = mid + 1; else hi = mid;
        }
        mine += (lo < ncur && a[lo] == x);
    }
    for (int o = 16; o >= 1; o >>= 1) mine += __shfl_xor_sync(0xffffffffu, mine, o);
    if ((threadIdx.x & 31) == 0 && mine) atomicAdd(&hits, mine);
    __syncthreads();
    if (threadIdx.x == 0) rate[blockIdx.x] = (float)hits / (float)nref;
}

}  // namespace
}  // namespace jq

extern "C" jq_status jq_hit_rate(const int32_t *cur, const int32_t *ref, int Hkv, int ncur, int nref, float *rate,
                                 jq_stream_t stream)
{
    if (!cur || !ref || !rate || Hkv < 1 || ncur < 1 || nref < 1 || Hkv > 65535 * 32767) return JQ_ERR_INVALID_ARG;
    jq::hit_rate_rows<<<(unsigned)Hkv, 256, 0, (cudaStream_t)stream>>>(cur, ref, ncur, nref, rate);
    jq::count_launch(1);
    return jq::check_launch();
}
