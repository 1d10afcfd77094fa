// Max-pool + exact top-k selection per KV head.
//
//   1. pool_keys: pooled[j] = max of the centred window (edges clipped); stored as an
//      order-preserving 32-bit integer key (float order == unsigned order).
//   2. radix_select: 4 rounds of 8 bits, most significant first, over integer histograms, find the
//      key tau of the nkeep-th largest element and how many elements equal to tau are kept.
//      Max-pooling copies every peak into up to `pool` neighbours, so ties at tau are the normal
//      case: all keys > tau are kept, then the lowest-index keys == tau.
//   3. ordered compaction: kept positions are written in ascending order.
// Everything is integer arithmetic on bit patterns, hence deterministic and exact.
#include "jq_internal.cuh"

namespace jq {
namespace {

constexpr int kSelThreads = 1024;

__device__ __forceinline__ uint32_t order_key(float x)
{
    uint32_t b = __float_as_uint(x + 0.0f);  // -0 -> +0
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// grid (ceil(L/256), Hkv), block 256.
__global__ void __launch_bounds__(256)
pool_keys(const float *__restrict__ scores, int L, int radius, uint32_t *__restrict__ keys,
          float *__restrict__ pooled)
{
    const int kv = blockIdx.y;
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= L) return;
    const float *s = scores + (size_t)kv * L;
    const int lo = max(j - radius, 0), hi = min(j + radius, L - 1);
    float best = s[j];
    for (int u = lo; u <= hi; ++u) best = fmaxf(best, s[u]);
    keys[(size_t)kv * L + j] = order_key(best);
    if (pooled) pooled[(size_t)kv * L + j] = best;
}

// Block-wide exclusive scan of one int per thread (1024 threads); returns the exclusive prefix and
// the block total through `total`.
__device__ __forceinline__ int block_excl_scan(int v, int *warp_sums, int &total)
{
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
    }
    if (lane == 31) warp_sums[wid] = inc;
    __syncthreads();
    if (wid == 0) {
        int ws = warp_sums[lane];
        int winc = ws;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int n = __shfl_up_sync(0xffffffffu, winc, o);
            if (lane >= o) winc += n;
        }
        warp_sums[lane] = winc - ws;       // exclusive warp offsets
        if (lane == 31) warp_sums[32] = winc;
    }
    __syncthreads();
    const int excl = warp_sums[wid] + inc - v;
    total = warp_sums[32];
    __syncthreads();
    return excl;
}

// grid (Hkv), block 1024.
__global__ void __launch_bounds__(kSelThreads)
radix_select_compact(const uint32_t *__restrict__ keys, int L, int nkeep, int32_t *__restrict__ idx)
{
    __shared__ int hist[256];
    __shared__ int warp_sums[33];
    __shared__ uint32_t s_prefix;
    __shared__ int s_krem;
    const int kv = blockIdx.x;
    const uint32_t *key = keys + (size_t)kv * L;
    int32_t *out = idx + (size_t)kv * nkeep;

    if (nkeep >= L) {  // everything is kept
        for (int j = threadIdx.x; j < L; j += blockDim.x) out[j] = j;
        return;
    }
    if (threadIdx.x == 0) { s_prefix = 0; s_krem = nkeep; }
    for (int round = 0; round < 4; ++round) {
        const int shift = 24 - 8 * round;
        if (threadIdx.x < 256) hist[threadIdx.x] = 0;
        __syncthreads();
        const uint32_t prefix = s_prefix;
        // uniform trip count so that the warp-level match sees whole warps
        for (int base = 0; base < L; base += blockDim.x) {
            const int j = base + threadIdx.x;
            bool live = false;
            uint32_t digit = 0;
            if (j < L) {
                const uint32_t k = key[j];
                live = (round == 0) || ((k >> (shift + 8)) == prefix);
                digit = (k >> shift) & 255u;
            }
            const uint32_t tag = live ? digit : 256u;
            const uint32_t peers = __match_any_sync(0xffffffffu, tag);
            if (live && (__ffs(peers) - 1) == (threadIdx.x & 31)) atomicAdd(&hist[digit], __popc(peers));
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            int krem = s_krem, above = 0, dsel = 0;
            for (int dg = 255; dg >= 0; --dg) {
                const int h = hist[dg];
                if (above + h >= krem) { dsel = dg; break; }
                above += h;
            }
            s_krem = krem - above;
            s_prefix = (prefix << 8) | (uint32_t)dsel;
        }
        __syncthreads();
    }
    const uint32_t tau = s_prefix;
    const int need_eq = s_krem;  // how many of the keys == tau are kept (lowest indices first)

    // ordered compaction: thread t owns the contiguous positions [t*seg, (t+1)*seg)
    const int seg = (L + blockDim.x - 1) / blockDim.x;
    const int j0 = min(threadIdx.x * seg, L), j1 = min(j0 + seg, L);
    int gt = 0, eq = 0;
    for (int j = j0; j < j1; ++j) {
        const uint32_t k = key[j];
        gt += (k > tau);
        eq += (k == tau);
    }
    int tot_gt, tot_eq;
    int gt_before = block_excl_scan(gt, warp_sums, tot_gt);
    int eq_before = block_excl_scan(eq, warp_sums, tot_eq);
    for (int j = j0; j < j1; ++j) {
        const uint32_t k = key[j];
        if (k > tau) {
            out[gt_before + min(eq_before, need_eq)] = j;
            ++gt_before;
        } else if (k == tau) {
            if (eq_before < need_eq) out[gt_before + eq_before] = j;
            ++eq_before;
        }
    }
}

}  // namespace

jq_status launch_select(const float *scores, const jq_shape &s, int32_t *idx, float *pooled,
                        const Workspace &w, cudaStream_t st)
{
    const int nkeep = s.budget < s.L ? s.budget : s.L;
    pool_keys<<<dim3((s.L + 255) / 256, s.Hkv), 256, 0, st>>>(scores, s.L, (s.pool - 1) / 2, w.keys, pooled);
    radix_select_compact<<<s.Hkv, kSelThreads, 0, st>>>(w.keys, s.L, nkeep, idx);
    count_launch(2);
    return check_launch();
}

}  // namespace jq
