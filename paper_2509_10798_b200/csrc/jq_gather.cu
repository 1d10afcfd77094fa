// Compaction of the pruned cache: row gather of K and V by the kept indices, 16-byte vectors.
// One half-warp copies one 256-byte row; rows of K and V of all heads share one grid.
#include "jq_internal.cuh"
#include "jq_debug.cuh"

namespace jq {
namespace {

constexpr int kVecPerRow = kD * 2 / 16;  // 16 uint4 per bf16 row of 128

__global__ void __launch_bounds__(256)
gather_rows(const uint4 *__restrict__ K, const uint4 *__restrict__ V, const int32_t *__restrict__ idx,
            int L, int nkeep, long long nrows, uint4 *__restrict__ Kout, uint4 *__restrict__ Vout, int Hkv JQ_DBG_PARAM)
{
    const int lane16 = threadIdx.x & 15;
    long long row = (long long)blockIdx.x * (blockDim.x / 16) + (threadIdx.x >> 4);
    const long long stride = (long long)gridDim.x * (blockDim.x / 16);
    for (; row < 2 * nrows; row += stride) {
        const bool isv = row >= nrows;
        const long long r = isv ? row - nrows : row;   // r = kv * nkeep + t
        const int kv = (int)(r / nkeep);
        int j = idx[r];
        j = min(max(j, 0), L - 1);
        const uint4 *src = (isv ? V : K) + ((size_t)kv * L + j) * kVecPerRow;
        uint4 *dst = (isv ? Vout : Kout) + (size_t)r * kVecPerRow;
        if (JQ_IN((long long)kv * L + j, (long long)Hkv * L, kDbgGather, 1) && JQ_IN(r, nrows, kDbgGather, 2))
            dst[lane16] = src[lane16];
    }
}

}  // namespace

jq_status launch_gather(const void *K, const void *V, const int32_t *idx, const jq_shape &s,
                        void *Kout, void *Vout, cudaStream_t st)
{
    const int nkeep = s.budget < s.L ? s.budget : s.L;
    const long long nrows = (long long)s.Hkv * nkeep;
    long long blocks = (2 * nrows + 15) / 16;
    if (blocks > 148 * 16) blocks = 148 * 16;
    gather_rows<<<(unsigned)blocks, 256, 0, st>>>((const uint4 *)K, (const uint4 *)V, idx, s.L, nkeep, nrows,
                                                  (uint4 *)Kout, (uint4 *)Vout, s.Hkv JQ_DBG_ARG);
    count_launch(1);
    return check_launch();
}

}  // namespace jq
