// Max-pool + exact top-k selection per KV head.  Two kernels share the arithmetic: select_cluster, one
// thread-block cluster per head (8 CTAs when the call has few heads, 4 or 2 when it has more heads than
// clusters fit on the GPU at a time, see choose_plan), and, for calls over 128 heads or more, select_stream
// further down, one CTA per head.  The cluster kernel:
//
//   1. pool: pooled[j] = max of the centred window (edges clipped), turned into an order-preserving
//      32-bit integer key (float order == unsigned order).  Each CTA owns a contiguous share of
//      the positions and keeps its keys in shared memory (in the workspace for very long prefixes).
//   2. radix select, 3 rounds of 11/11/10 bits, most significant first: local integer histograms
//      are summed into the leading CTA through distributed shared memory, which finds the digit
//      holding the nkeep-th largest key and broadcasts it.  After the first round the keys that
//      share that digit are normally few: they are then copied into the leading CTA, which runs
//      the two remaining rounds on them alone (no further pass over all keys, no further
//      histogram traffic).  Result: the key tau of the nkeep-th largest element and how many
//      elements equal to tau are kept.  Max-pooling copies every peak
//      into up to `pool` neighbours, so ties at tau are the normal case: all keys > tau are kept,
//      then the lowest-index keys == tau.
//   3. ordered compaction: kept positions are written in ascending order (CTA rank, warp,
//      iteration and lane order all follow the position order).
//   4. (fused layer path only) the cluster copies the kept K and V rows of its head.
// Everything is integer arithmetic on bit patterns, hence deterministic and exact.
#include "jq_internal.cuh"
#include "jq_debug.cuh"
#include <cooperative_groups.h>

namespace cg = cooperative_groups;

namespace jq {
namespace {

constexpr int kClMax = 8;          // most CTAs per cluster (= per KV head); the kernel also exists for 4 and 2
constexpr int kSelThreads = 1024;
constexpr int kBins = 2048;
constexpr int kRawTile = 20480;    // most scores staged per pooling step (a CTA's whole share unless the prefix is very long)
constexpr int kHalo = 32;          // >= pool radius
constexpr int kKeysSmemMax = 24576; // keys a CTA can keep in shared memory
constexpr int kCandMax = 8192;     // candidates the leading CTA finishes alone (they live in its staging buffer)
static_assert(kCandMax <= kRawTile, "candidates are kept in the staging buffer");

// Extents of what the kernel indexes (read by the bounds-checked build only).
struct SelExtents {
    long long scores;     // floats in the scores array (and keys in the global key array)
    long long out_rows;   // rows of the stacked outputs (kept indices, compacted K and V)
    long long src_heads;  // heads in one source buffer of K / V
};

struct SelCtl {
    uint32_t prefix;
    int krem;
    int found_prefix_digit, found_krem, found_count;
    int cand_total;      // keys sharing the first-round digit (broadcast by the leading CTA)
    int cand_count;      // leading CTA only: candidates appended so far
    int counts_gt[kClMax], counts_eq[kClMax];
    int warp_gt[32], warp_eq[32];
    int tot_gt, tot_eq;
    int scan[33];
};

__device__ __forceinline__ uint32_t order_key(float x)
{
    uint32_t b = __float_as_uint(x + 0.0f);  // -0 -> +0
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

__device__ __forceinline__ float max3f(float a, float b, float c)
{
    float y;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(y) : "f"(a), "f"(b), "f"(c));
    return y;
}

// Block-wide exclusive scan of one int per thread (1024 threads).
__device__ __forceinline__ int block_excl_scan(int v, int *warp_sums)
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
    }
    __syncthreads();
    const int excl = warp_sums[wid] + inc - v;
    __syncthreads();
    return excl;
}

// All 1024 threads of a CTA: in a histogram of kBins bins find, walking the bins from the top, the bin
// that holds the krem-th element; leaves the bin, the rank within it and its population in ctl.
__device__ __forceinline__ void find_digit(const uint32_t *g, int krem, SelCtl &ctl)
{
    // bins in descending order: thread t looks at bins 2047-2t and 2046-2t
    const int hi = kBins - 1 - 2 * (int)threadIdx.x, lo = hi - 1;
    const int h_hi = (int)g[hi], h_lo = (int)g[lo];
    const int above = block_excl_scan(h_hi + h_lo, ctl.scan);
    if (above < krem && krem <= above + h_hi) {
        ctl.found_prefix_digit = hi; ctl.found_krem = krem - above; ctl.found_count = h_hi;
    } else if (above + h_hi < krem && krem <= above + h_hi + h_lo) {
        ctl.found_prefix_digit = lo; ctl.found_krem = krem - above - h_hi; ctl.found_count = h_lo;
    }
    __syncthreads();
}

// The cluster copies the kept K and V rows of its head (256 bytes each: 16 lanes x 16 bytes), CTA r the
// r-th share of them, once every index of the head has been written.
// kv_in: the head's index within the buffer the rows come from; orow: the head's first row in the outputs.
template <int CL>
__device__ __forceinline__ void copy_kept_rows(cg::cluster_group &cluster, const int32_t *out, int kv_in, long long orow, int L, int nkeep,
                                               const uint4 *Kin, const uint4 *Vin, uint4 *Kout, uint4 *Vout, int src_rows,
                                               const SelExtents &ext JQ_DBG_PARAM)
{
    __threadfence();
    cluster.sync();
    const int rank = (int)cluster.block_rank();
    const int r0 = (int)((long long)rank * nkeep / CL), r1 = (int)((long long)(rank + 1) * nkeep / CL);
    const int lane16 = threadIdx.x & 15;
    for (int t = r0 + (int)(threadIdx.x >> 4); t < r1; t += kSelThreads / 16) {
        const int j = min(max(__ldcg(out + t), 0), L - 1);
        const size_t src = ((size_t)kv_in * src_rows + j) * 16 + lane16, dst = (size_t)(orow + t) * 16 + lane16;
        if (JQ_IN((long long)kv_in * src_rows + j, ext.src_heads * src_rows, kDbgSelect, 1) && JQ_IN(orow + t, ext.out_rows, kDbgSelect, 2)) {
            Kout[dst] = Kin[src];
            Vout[dst] = Vin[src];
        }
    }
}

// grid (Hkv * CL), cluster CL, block 1024.  With htab (ragged calls) every head has a length, a budget, offsets
// into the scores, the keys and the outputs, and a source buffer of its own; L, nkeep, chunk, keys_in_smem are
// then those of the longest head and only size the shared memory.
template <int CL>
__global__ void __cluster_dims__(CL, 1, 1) __launch_bounds__(kSelThreads, 2)
select_cluster(const float *__restrict__ scores, int L, int nkeep, int radius, int32_t *__restrict__ idx,
               float *__restrict__ pooled, uint32_t *__restrict__ gkeys, int chunk, int keys_in_smem, int raw_tile,
               const uint4 *__restrict__ Kin, const uint4 *__restrict__ Vin, uint4 *__restrict__ Kout,
               uint4 *__restrict__ Vout, const HeadRec *__restrict__ htab, const uint4 *const *__restrict__ Ktab,
               const uint4 *const *__restrict__ Vtab, int src_rows, int out_rows, const SelExtents ext JQ_DBG_PARAM)
{
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();
    const int kv = blockIdx.x / CL;
    int kv_in = kv;                                  // the head's index within the buffer its rows come from
    long long soff = (long long)kv * L, orow = (long long)kv * nkeep;   // offsets of the head's scores and of its kept indices
    long long krow = (long long)kv * out_rows;                          // first row of the head in the compacted outputs
    extern __shared__ __align__(16) uint8_t sm[];
    uint32_t *ghist = (uint32_t *)sm;                       // [kBins]; the leading CTA's copy accumulates the cluster's histogram of a round
    uint32_t *hist = ghist + kBins;                         // [kBins]
    float *raw = (float *)(hist + kBins);                   // [raw_tile + 2*kHalo]; later the candidate keys
    uint32_t *keys_s = (uint32_t *)(raw + raw_tile + 2 * kHalo);
    __shared__ SelCtl ctl;

    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int raw_cap = raw_tile + 2 * kHalo, keys_cap = keys_in_smem ? chunk : 0;   // shared-memory extents (those of the launch)
    (void)raw_cap; (void)keys_cap;
    cudaGridDependencySynchronize();   // everything above ran while the previous kernel of the stream was finishing
    if (htab) {
        const HeadRec r = htab[kv];
        L = r.L; nkeep = r.nkeep; kv_in = r.kv_in; soff = r.soff; orow = r.ooff; krow = r.ooff; src_rows = L;
        chunk = ((L + CL - 1) / CL + 31) / 32 * 32;   // (keys_in_smem stays the launch's: the longest head decides whether the region exists)
        if (Ktab) { Kin = Ktab[r.unit]; Vin = Vtab[r.unit]; }
    }
    const int j0 = min(rank * chunk, L), j1 = min(j0 + chunk, L), n = j1 - j0;
    const float *s = scores + soff;
    uint32_t *mykeys = keys_in_smem ? keys_s : gkeys + soff + j0;
    int32_t *out = idx + orow;
    if (pooled) pooled += soff;

    // ---- 1. max-pool -> keys
    // With the keys in shared memory and a window of at most 9, a thread pools four neighbouring
    // positions from three 16-byte reads and the first-round histogram is built on the way.
    const bool fast_pool = keys_in_smem && radius <= 4;
    for (int i = tid; i < kBins; i += kSelThreads) hist[i] = 0;
    for (int t0 = 0; t0 < n; t0 += raw_tile) {
        const int tile = min(raw_tile, n - t0);
        __syncthreads();
        // eight loads in flight per thread: the scores come from L2, one round trip each
        for (int i0 = tid; i0 < tile + 2 * radius; i0 += 8 * kSelThreads) {
            float vals[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                const int j = j0 + t0 - radius + i0 + q * kSelThreads;
                vals[q] = (i0 + q * kSelThreads < tile + 2 * radius && j >= 0 && j < L && JQ_IN(soff + j, ext.scores, kDbgSelect, 3)) ? __ldcg(s + j) : -INFINITY;
            }
#pragma unroll
            for (int q = 0; q < 8; ++q)
                if (i0 + q * kSelThreads < tile + 2 * radius && JQ_IN(i0 + q * kSelThreads, raw_cap, kDbgSelect, 4)) raw[i0 + q * kSelThreads] = vals[q];
        }
        if (fast_pool) for (int i = tid; i < 8; i += kSelThreads) if (JQ_IN(tile + 2 * radius + i, raw_cap, kDbgSelect, 5)) raw[tile + 2 * radius + i] = -INFINITY;   // its 16-byte reads run a little past the window
        __syncthreads();
        if (fast_pool) {
            const int nquads = (tile + 3) / 4;
            const float4 *raw4 = (const float4 *)raw;
            for (int base = 0; base < nquads; base += kSelThreads) {      // uniform trip count: whole warps reach the votes
                const int g4 = base + tid;
                const bool act = g4 < nquads;
                float x[12];
                {
                    const bool rd = act && JQ_IN(4 * (g4 + 2) + 3, raw_cap, kDbgSelect, 6);
                    const float4 a = rd ? raw4[g4] : make_float4(0.f, 0.f, 0.f, 0.f);
                    const float4 b = rd ? raw4[g4 + 1] : a, c = rd ? raw4[g4 + 2] : a;
                    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
                    x[8] = c.x; x[9] = c.y; x[10] = c.z; x[11] = c.w;
                }
                uint32_t key[4];
                float best[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float m = x[i];
#pragma unroll
                    for (int u = 1; u <= 8; ++u) if (u <= 2 * radius) m = fmaxf(m, x[i + u]);
                    best[i] = m;
                    key[i] = order_key(m);
                }
                const int nval = act ? min(4, tile - 4 * g4) : 0;          // positions of this quad inside the tile
                if (act && JQ_IN(t0 + 4 * g4 + nval - 1, keys_cap, kDbgSelect, 7) && (!pooled || JQ_IN(soff + j0 + t0 + 4 * g4 + nval - 1, ext.scores, kDbgSelect, 8))) {
                    if (nval == 4) *(uint4 *)(mykeys + t0 + 4 * g4) = make_uint4(key[0], key[1], key[2], key[3]);
                    else for (int i = 0; i < nval; ++i) mykeys[t0 + 4 * g4 + i] = key[i];
                    if (pooled) for (int i = 0; i < nval; ++i) pooled[j0 + t0 + 4 * g4 + i] = best[i];
                }
                // first-round histogram: one addition per warp when all its positions share the digit (the usual
                // case: 128 neighbouring positions of similar size), else runs of equal digits per thread
                const uint32_t d0 = key[0] >> 21;
                bool same = true;
                for (int i = 1; i < 4; ++i) if (i < nval && (key[i] >> 21) != d0) same = false;
                const uint32_t lead = __shfl_sync(0xffffffffu, d0, 0);
                if (__all_sync(0xffffffffu, nval == 0 || (same && d0 == lead))) {
                    const int tot = __reduce_add_sync(0xffffffffu, nval);
                    if (lane == 0 && tot && JQ_IN(lead, kBins, kDbgSelect, 9)) atomicAdd(&hist[lead], (uint32_t)tot);
                } else {
                    uint32_t cur = 0, cnt = 0;
                    for (int i = 0; i < nval; ++i) {
                        const uint32_t d = key[i] >> 21;
                        if (cnt && d != cur) { atomicAdd(&hist[cur], cnt); cnt = 0; }
                        cur = d; ++cnt;
                    }
                    if (cnt) atomicAdd(&hist[cur], cnt);
                }
            }
            continue;
        }
#pragma unroll 4
        for (int e = tid; e < tile; e += kSelThreads) {
            if (!JQ_IN(e + 2 * radius, raw_cap, kDbgSelect, 10)) continue;
            float best = raw[e];
            for (int u = 1; u <= 2 * radius; ++u) best = fmaxf(best, raw[e + u]);
            if (JQ_IN(keys_in_smem ? t0 + e : soff + j0 + t0 + e, keys_in_smem ? keys_cap : ext.scores, kDbgSelect, 11)) mykeys[t0 + e] = order_key(best);
            if (pooled && JQ_IN(soff + j0 + t0 + e, ext.scores, kDbgSelect, 12)) pooled[j0 + t0 + e] = best;
        }
    }
    if (nkeep >= L) {   // everything is kept (uniform over the cluster; no cluster traffic yet)
        for (int e = tid; e < n; e += kSelThreads) if (JQ_IN(orow + j0 + e, ext.out_rows, kDbgSelect, 13)) out[j0 + e] = j0 + e;
        if (Kin) copy_kept_rows<CL>(cluster, out, kv_in, krow, L, nkeep, Kin, Vin, Kout, Vout, src_rows, ext JQ_DBG_ARG_DEV);
        return;
    }
    for (int i = tid; i < kBins; i += kSelThreads) ghist[i] = 0;
    if (tid == 0) { ctl.prefix = 0; ctl.krem = nkeep; ctl.cand_count = 0; ctl.cand_total = 0; }
    cluster.sync();

    // ---- 2. radix select
    const int n_up = (n + kSelThreads - 1) / kSelThreads * kSelThreads;
    for (int round = 0; round < 3; ++round) {
        const int shift = (round == 0) ? 21 : (round == 1 ? 10 : 0);
        const int width = (round == 2) ? 10 : 11;
        const uint32_t mask = (1u << width) - 1u;
        const bool have_hist = round == 0 && fast_pool;          // built while pooling
        if (!have_hist) for (int i = tid; i < kBins; i += kSelThreads) hist[i] = 0;
        __syncthreads();
        const uint32_t prefix = ctl.prefix;
        // A thread takes a run of consecutive keys and adds equal neighbouring digits as one count: the
        // max-pool leaves plateaus, so a few additions per thread replace one per key.
        if (!have_hist) {
            const int per = (n + kSelThreads - 1) / kSelThreads;
            const int e0 = min(tid * per, n), e1 = min(e0 + per, n);
            uint32_t cur = 0xffffffffu, cnt = 0;
            int pos = per ? tid % per : 0;                      // rotated start: neighbouring threads hit different banks
            for (int i = 0; i < per; ++i) {
                const int e = e0 + pos;
                if (++pos == per) pos = 0;
                if (e >= e1) continue;
                if (!JQ_IN(keys_in_smem ? e : soff + j0 + e, keys_in_smem ? keys_cap : ext.scores, kDbgSelect, 14)) continue;
                const uint32_t k = mykeys[e];
                const bool live = (round == 0) || ((k >> (shift + width)) == prefix);
                const uint32_t digit = live ? ((k >> shift) & mask) : 0xffffffffu;
                if (digit != cur) {
                    if (cnt && cur != 0xffffffffu) atomicAdd(&hist[cur], cnt);
                    cur = digit; cnt = 0;
                }
                ++cnt;
            }
            if (cnt && cur != 0xffffffffu) atomicAdd(&hist[cur], cnt);
        }
        __syncthreads();
        uint32_t *g0 = cluster.map_shared_rank(ghist, 0);
        for (int i = tid; i < kBins; i += kSelThreads) {
            const uint32_t v = hist[i];
            if (v) atomicAdd(&g0[i], v);
        }
        cluster.sync();
        if (rank == 0) {
            find_digit(ghist, ctl.krem, ctl);
            if (tid < CL) {
                SelCtl *rc = cluster.map_shared_rank(&ctl, tid);
                rc->prefix = (prefix << width) | (uint32_t)ctl.found_prefix_digit;
                rc->krem = ctl.found_krem;
                rc->cand_total = ctl.found_count;
            }
            for (int i = tid; i < kBins; i += kSelThreads) ghist[i] = 0;   // for the next round, before anybody adds to it
        }
        cluster.sync();
        if (round == 0 && ctl.cand_total <= kCandMax) {
            // The keys with the winning first digit go to the leading CTA (order does not matter: only
            // their values decide the threshold), which finishes the selection on them alone.
            const uint32_t d0 = ctl.prefix;
            uint32_t *cand = (uint32_t *)cluster.map_shared_rank(raw, 0);
            int *cand_count = &cluster.map_shared_rank(&ctl, 0)->cand_count;
            for (int base = 0; base < n_up; base += kSelThreads) {
                const int e = base + tid;
                const uint32_t k = (e < n && JQ_IN(keys_in_smem ? e : soff + j0 + e, keys_in_smem ? keys_cap : ext.scores, kDbgSelect, 19)) ? mykeys[e] : 0u;
                const bool hit = e < n && (k >> 21) == d0;
                const uint32_t votes = __ballot_sync(0xffffffffu, hit);
                if (votes) {
                    int at = 0;
                    if (lane == 0) at = atomicAdd(cand_count, __popc(votes));
                    at = __shfl_sync(0xffffffffu, at, 0);
                    if (hit && JQ_IN(at + __popc(votes & ((1u << lane) - 1u)), raw_cap, kDbgSelect, 15)) cand[at + __popc(votes & ((1u << lane) - 1u))] = k;
                }
            }
            cluster.sync();
            if (rank == 0) {
                const int nc = ctl.cand_total;
                const uint32_t *mine = (const uint32_t *)raw;
                uint32_t pre = d0;
                for (int r2 = 1; r2 < 3; ++r2) {
                    const int sh = (r2 == 1) ? 10 : 0, wd = (r2 == 2) ? 10 : 11;
                    for (int i = tid; i < kBins; i += kSelThreads) hist[i] = 0;
                    __syncthreads();
                    for (int e = tid; e < nc; e += kSelThreads) {
                        const uint32_t k = mine[e];
                        if ((k >> (sh + wd)) == pre && JQ_IN((k >> sh) & ((1u << wd) - 1u), kBins, kDbgSelect, 16)) atomicAdd(&hist[(k >> sh) & ((1u << wd) - 1u)], 1u);
                    }
                    __syncthreads();
                    find_digit(hist, ctl.krem, ctl);
                    pre = (pre << wd) | (uint32_t)ctl.found_prefix_digit;
                    if (tid == 0) ctl.krem = ctl.found_krem;
                    __syncthreads();
                }
                if (tid < CL) {
                    SelCtl *rc = cluster.map_shared_rank(&ctl, tid);
                    rc->prefix = pre;
                    rc->krem = ctl.found_krem;
                }
            }
            cluster.sync();
            break;
        }
    }
    const uint32_t tau = ctl.prefix;
    const int need_eq = ctl.krem;   // how many of the keys == tau are kept (lowest positions first)

    // ---- 3. ordered compaction; warp w owns the contiguous elements [w*seg, (w+1)*seg)
    const int seg = ((n + 31) / 32 + 31) / 32 * 32;
    const int w0 = min(wid * seg, n), w1 = min(w0 + seg, n);
    int cgt = 0, ceq = 0;
    for (int base = w0; base < w1; base += 32) {
        const int e = base + lane;
        const uint32_t k = (e < w1 && JQ_IN(keys_in_smem ? e : soff + j0 + e, keys_in_smem ? keys_cap : ext.scores, kDbgSelect, 20)) ? mykeys[e] : 0u;
        const bool in = e < w1;
        cgt += __popc(__ballot_sync(0xffffffffu, in && k > tau));
        ceq += __popc(__ballot_sync(0xffffffffu, in && k == tau));
    }
    if (lane == 0) { ctl.warp_gt[wid] = cgt; ctl.warp_eq[wid] = ceq; }
    __syncthreads();
    if (wid == 0) {
        const int g = ctl.warp_gt[lane], q = ctl.warp_eq[lane];
        int gi = g, qi = q;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int a = __shfl_up_sync(0xffffffffu, gi, o), b = __shfl_up_sync(0xffffffffu, qi, o);
            if (lane >= o) { gi += a; qi += b; }
        }
        ctl.warp_gt[lane] = gi - g; ctl.warp_eq[lane] = qi - q;   // exclusive
        if (lane == 31) { ctl.tot_gt = gi; ctl.tot_eq = qi; }
    }
    __syncthreads();
    if (tid < CL) {
        SelCtl *rc = cluster.map_shared_rank(&ctl, tid);
        rc->counts_gt[rank] = ctl.tot_gt;
        rc->counts_eq[rank] = ctl.tot_eq;
    }
    cluster.sync();
    int gt_before = ctl.warp_gt[wid], eq_before = ctl.warp_eq[wid];
    for (int q = 0; q < rank; ++q) { gt_before += ctl.counts_gt[q]; eq_before += ctl.counts_eq[q]; }
    const uint32_t lt_mask = (1u << lane) - 1u;
    for (int base = w0; base < w1; base += 32) {
        const int e = base + lane;
        const bool in = e < w1;
        const uint32_t k = (in && JQ_IN(keys_in_smem ? e : soff + j0 + e, keys_in_smem ? keys_cap : ext.scores, kDbgSelect, 21)) ? mykeys[e] : 0u;
        const uint32_t bg = __ballot_sync(0xffffffffu, in && k > tau);
        const uint32_t be = __ballot_sync(0xffffffffu, in && k == tau);
        const int g_here = gt_before + __popc(bg & lt_mask), e_here = eq_before + __popc(be & lt_mask);
        if (in) {
            if (k > tau) { if (JQ_IN(g_here + min(e_here, need_eq), nkeep, kDbgSelect, 17)) out[g_here + min(e_here, need_eq)] = j0 + e; }
            else if (k == tau && e_here < need_eq) { if (JQ_IN(g_here + e_here, nkeep, kDbgSelect, 18)) out[g_here + e_here] = j0 + e; }
        }
        gt_before += __popc(bg);
        eq_before += __popc(be);
    }
    if (Kin) copy_kept_rows<CL>(cluster, out, kv_in, krow, L, nkeep, Kin, Vin, Kout, Vout, src_rows, ext JQ_DBG_ARG_DEV);
}

// ------------------------------------------------------------------ many heads: one CTA per head, no cluster
//
// A call over many heads (the layers of a cache, a ragged batch) has more heads than clusters fit on the GPU, and the
// cluster kernel's time per head is mostly the latency of its barrier-separated phases.  Here a head is one CTA that
// keeps a histogram, a candidate list and a small staging buffer per warp in shared memory, so that several heads are
// resident per SM, and that walks the head's scores three times, pooling on the fly.  Every warp owns a contiguous
// share of the head and takes it 512 positions at a time: four 16-byte asynchronous copies per lane into one of the
// warp's two staging buffers, with one quad of halo on either side, from where a lane pools four neighbouring
// positions while the copies of the next 512 positions are in flight.
//   pass 1  pooled keys -> histogram of the top 11 bits (and the pooled values, when the caller wants them);
//   pass 2  the keys that share the winning digit -> candidate list (key and position), and per warp the number of
//           keys with a larger digit (passes 2 and 3 pool only the quads whose 12 staged scores reach the threshold); rounds 2 and 3 run on the list, and the list then also gives every warp its
//           number of kept keys.  (When the list would not fit, rounds 2 and 3 and the counts are passes of their own.)
//   pass 3  ordered compaction of the kept positions, then the copy of the kept rows.
// Same integer arithmetic as the cluster kernel: the same threshold key and the same ties, hence the same indices.
constexpr int kStrCand = 2048;      // candidates finished in shared memory
constexpr int kStrMaxWarps = 32;
constexpr int kStepQuads = 128;     // quads a warp takes per step
constexpr int kStageQuads = kStepQuads + 2;
constexpr int kStreamMinHeads = 128;   // calls with at least this many heads take this kernel

struct StrCtl {
    int scan[kStrMaxWarps + 1];
    int digit, krem, count;         // find_digit_cta: the bin of the krem-th key, the rank within it, its population
    int cand_count;
    int warp_gt[kStrMaxWarps], warp_eq[kStrMaxWarps];
};

// Quad q (positions 4q .. 4q+3) of a head of L scores at s; positions outside [0, L) read as -inf.
// vec: s is 16-byte aligned.
__device__ __forceinline__ float4 load_quad(const float *__restrict__ s, int L, int q, bool vec, long long soff,
                                            const SelExtents &ext JQ_DBG_PARAM)
{
    (void)soff; (void)ext;
    const float ninf = -INFINITY;
    if (q < 0 || 4 * q >= L) return make_float4(ninf, ninf, ninf, ninf);
    if (vec && 4 * q + 4 <= L && JQ_IN(soff + 4 * q + 3, ext.scores, kDbgSelect, 22)) return *(const float4 *)(s + 4 * q);
    float v[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] = (4 * q + i < L && JQ_IN(soff + 4 * q + i, ext.scores, kDbgSelect, 23)) ? s[4 * q + i] : ninf;
    return make_float4(v[0], v[1], v[2], v[3]);
}

// The warp requests quads [base - 1, base + 129) of the head into one of its two buffers: 16-byte asynchronous copies
// for the quads that lie inside the head (and are aligned), plain stores of -inf-padded values for the others.
__device__ __forceinline__ void stage_issue(float4 *dst, const float *__restrict__ s, int L, int base, bool vec, long long soff,
                                            const SelExtents &ext JQ_DBG_PARAM)
{
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int u = 0; u < 5; ++u) {
        if (u == 4 && lane >= 2) break;
        const int q = u < 4 ? base + 32 * u + lane : (lane == 0 ? base - 1 : base + kStepQuads);
        float4 *d = dst + (u < 4 ? 1 + 32 * u + lane : (lane == 0 ? 0 : kStageQuads - 1));
        if (vec && q >= 0 && 4 * q + 4 <= L && JQ_IN(soff + 4 * q + 3, ext.scores, kDbgSelect, 22))
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(d)), "l"(s + 4 * q) : "memory");
        else
            *d = load_quad(s, L, q, vec, soff, ext JQ_DBG_ARG_DEV);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
}

// The staged quads of the step at `base` of the warp's walk over [qa, qb), 128 quads per step: waits for the step's
// copies and has the next step's under way (two buffers per warp), so that a step's reads from memory overlap the
// pooling of the step before.  Every lane of the warp calls it once per step, in order.
__device__ __forceinline__ const float4 *stage_step(float4 *bufs, const float *__restrict__ s, int L, int base, int qa, int qb, bool vec,
                                                    long long soff, const SelExtents &ext JQ_DBG_PARAM)
{
    const int step = (base - qa) / kStepQuads;
    float4 *cur = bufs + (step & 1) * kStageQuads, *nxt = bufs + ((step + 1) & 1) * kStageQuads;
    if (step == 0) {
        __syncwarp();                                        // the reads of an earlier pass are done
        stage_issue(cur, s, L, base, vec, soff, ext JQ_DBG_ARG_DEV);
    }
    __syncwarp();                                            // the previous step's reads of the other buffer are done
    if (base + kStepQuads < qb) {
        stage_issue(nxt, s, L, base + kStepQuads, vec, soff, ext JQ_DBG_ARG_DEV);
        asm volatile("cp.async.wait_group 1;" ::: "memory");
    } else {
        asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncwarp();
    return cur;
}

// Pooled order keys (and values) of the four positions of quad `at` (0 .. 127) of the staged step.
__device__ __forceinline__ void pooled_quad(const float4 *buf, int at, int radius, uint32_t (&key)[4], float (&best)[4])
{
    const float4 a = buf[at], b = buf[at + 1], c = buf[at + 2];
    const float x[12] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w, c.x, c.y, c.z, c.w};
    if (radius == 3) {
        // window of 7: the four windows share x4..x7; the rest are running maxima of the three neighbours on either side
        const float core = fmaxf(max3f(x[4], x[5], x[6]), x[7]);
        const float l2 = fmaxf(x[2], x[3]), l1 = fmaxf(x[1], l2);
        const float r9 = fmaxf(x[8], x[9]), r10 = fmaxf(r9, x[10]);
        best[0] = fmaxf(core, l1);
        best[1] = max3f(core, l2, x[8]);
        best[2] = max3f(core, x[3], r9);
        best[3] = fmaxf(core, r10);
    } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float m = x[4 + i];
#pragma unroll
            for (int u = 1; u <= 4; ++u) if (u <= radius) m = fmaxf(m, fmaxf(x[4 + i - u], x[4 + i + u]));
            best[i] = m;
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) key[i] = order_key(best[i]);
}

// Order key of the largest of the 12 staged scores around quad `at`: an upper bound of the quad's four pooled keys
// (every window lies inside those 12), so a quad whose bound is below a threshold holds nothing at or above it and
// the passes that only look for such keys skip its pooling.
__device__ __forceinline__ uint32_t quad_bound_key(const float4 *buf, int at)
{
    const float4 a = buf[at], b = buf[at + 1], c = buf[at + 2];
    const float m = max3f(max3f(a.x, a.y, a.z), max3f(a.w, b.x, b.y), max3f(max3f(b.z, b.w, c.x), max3f(c.y, c.z, c.w), -INFINITY));
    return order_key(m);
}

// Block-wide exclusive scan of one int per thread, any number of whole warps.
__device__ __forceinline__ int cta_excl_scan(int v, int *warp_sums)
{
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
    }
    if (lane == 31) warp_sums[wid] = inc;
    __syncthreads();
    if (wid == 0) {
        const int ws = lane < nw ? warp_sums[lane] : 0;
        int winc = ws;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int n = __shfl_up_sync(0xffffffffu, winc, o);
            if (lane >= o) winc += n;
        }
        if (lane < nw) warp_sums[lane] = winc - ws;
    }
    __syncthreads();
    const int excl = warp_sums[wid] + inc - v;
    __syncthreads();
    return excl;
}

// All threads of a CTA of 512 or 1024: the bin of h[kBins] that holds the krem-th key counted from the top.
__device__ __forceinline__ void find_digit_cta(const uint32_t *h, int krem, StrCtl &ctl)
{
    const int per = kBins / (int)blockDim.x;                  // 4 or 2 bins per thread, descending
    const int hi = kBins - 1 - per * (int)threadIdx.x;
    int tot = 0;
    for (int i = 0; i < per; ++i) tot += (int)h[hi - i];
    int above = cta_excl_scan(tot, ctl.scan);
    for (int i = 0; i < per; ++i) {
        const int c = (int)h[hi - i];
        if (above < krem && krem <= above + c) { ctl.digit = hi - i; ctl.krem = krem - above; ctl.count = c; }
        above += c;
    }
    __syncthreads();
}

// Adds the digits of a thread's (up to) four neighbouring keys to the histogram: runs of equal digits as one count (the
// max-pool leaves plateaus); digit 0xffffffff marks a key that does not take part.
__device__ __forceinline__ void hist_add_runs(uint32_t *hist, const uint32_t (&digit)[4], int nval JQ_DBG_PARAM)
{
    uint32_t cur = 0xffffffffu, cnt = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if (i < nval) {
            if (digit[i] != cur) {
                if (cnt && cur != 0xffffffffu && JQ_IN(cur, kBins, kDbgSelect, 24)) atomicAdd(&hist[cur], cnt);
                cur = digit[i]; cnt = 0;
            }
            ++cnt;
        }
    }
    if (cnt && cur != 0xffffffffu && JQ_IN(cur, kBins, kDbgSelect, 24)) atomicAdd(&hist[cur], cnt);
}

// grid (Hkv), block kThreads = 512 (two CTAs to an SM) or 1024 (one); dynamic shared memory: two staging buffers of
// kStageQuads float4 per warp.  Arguments as for select_cluster.
__host__ __device__ constexpr int stream_ctas_per_sm(int threads) { return threads == 512 ? 2 : 1; }
template <int kThreads>
__global__ void __launch_bounds__(kThreads, stream_ctas_per_sm(kThreads))
select_stream(const float *__restrict__ scores, int L, int nkeep, int radius, int32_t *__restrict__ idx,
              float *__restrict__ pooled, const uint4 *__restrict__ Kin, const uint4 *__restrict__ Vin,
              uint4 *__restrict__ Kout, uint4 *__restrict__ Vout, const HeadRec *__restrict__ htab,
              const uint4 *const *__restrict__ Ktab, const uint4 *const *__restrict__ Vtab, int src_rows, int out_rows,
              const SelExtents ext JQ_DBG_PARAM)
{
    extern __shared__ __align__(16) uint8_t sm[];
    __shared__ uint32_t hist[kBins];
    __shared__ uint32_t cand_key[kStrCand];
    __shared__ int cand_pos[kStrCand];
    __shared__ StrCtl ctl;
    constexpr int T = kThreads, nw = T / 32;
    const int kv = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    float4 *buf = (float4 *)sm + wid * 2 * kStageQuads;   // the warp's two staging buffers
    int kv_in = kv;
    long long soff = (long long)kv * L, orow = (long long)kv * nkeep, krow = (long long)kv * out_rows;
    cudaGridDependencySynchronize();   // everything above ran while the previous kernel of the stream was finishing
    if (htab) {
        const HeadRec r = htab[kv];
        L = r.L; nkeep = r.nkeep; kv_in = r.kv_in; soff = r.soff; orow = r.ooff; krow = r.ooff; src_rows = L;
        if (Ktab) { Kin = Ktab[r.unit]; Vin = Vtab[r.unit]; }
    }
    if (nkeep > L) nkeep = L;
    const float *s = scores + soff;
    int32_t *out = idx + orow;
    if (pooled) pooled += soff;
    const bool vec = (((size_t)s) & 15) == 0;
    const int nq = (L + 3) / 4;
    // warp w owns the contiguous quads [qa, qb); every warp makes the same number of steps
    const int segq = (nq + nw - 1) / nw;
    const int qa = min(wid * segq, nq), qb = min(qa + segq, nq);

    // ---- pass 1: histogram of the top 11 bits of the pooled keys
    for (int i = tid; i < kBins; i += T) hist[i] = 0;
    if (tid == 0) ctl.cand_count = 0;
    __syncthreads();
    for (int base = qa; base < qb; base += kStepQuads) {
        const float4 *bf = stage_step(buf, s, L, base, qa, qb, vec, soff, ext JQ_DBG_ARG_DEV);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int q = base + 32 * u + lane;
            const int nval = q < qb ? min(4, L - 4 * q) : 0;
            uint32_t key[4];
            float best[4];
            pooled_quad(bf, 32 * u + lane, radius, key, best);
            if (pooled && nval && JQ_IN(soff + 4 * q + nval - 1, ext.scores, kDbgSelect, 25))
                for (int i = 0; i < nval; ++i) pooled[4 * q + i] = best[i];
            // one addition per warp when all its positions share the digit (the usual case: 128 neighbouring
            // positions of similar size), else runs of equal digits per thread
            const uint32_t d0 = key[0] >> 21;
            bool same = true;
            for (int i = 1; i < 4; ++i) if (i < nval && (key[i] >> 21) != d0) same = false;
            const uint32_t lead = __shfl_sync(0xffffffffu, d0, 0);
            if (__all_sync(0xffffffffu, nval == 0 || (same && d0 == lead))) {
                const int tot = __reduce_add_sync(0xffffffffu, nval);
                if (lane == 0 && tot && JQ_IN(lead, kBins, kDbgSelect, 24)) atomicAdd(&hist[lead], (uint32_t)tot);
            } else {
                const uint32_t dg[4] = {key[0] >> 21, key[1] >> 21, key[2] >> 21, key[3] >> 21};
                hist_add_runs(hist, dg, nval JQ_DBG_ARG_DEV);
            }
        }
    }
    __syncthreads();
    if (nkeep >= L) {                                          // everything is kept
        for (int e = tid; e < L; e += T) if (JQ_IN(orow + e, ext.out_rows, kDbgSelect, 26)) out[e] = e;
    } else {
        // ---- the threshold key tau and how many keys equal to it are kept
        find_digit_cta(hist, nkeep, ctl);
        uint32_t pre = (uint32_t)ctl.digit;
        int krem = ctl.krem;
        const bool listed = ctl.count <= kStrCand;
        if (lane == 0) { ctl.warp_gt[wid] = 0; ctl.warp_eq[wid] = 0; }
        __syncthreads();
        if (listed) {
            // pass 2: the keys with the winning first digit, with their positions; the warp's keys above that digit
            int hi_cnt = 0;
            for (int base = qa; base < qb; base += kStepQuads) {
                const float4 *bf = stage_step(buf, s, L, base, qa, qb, vec, soff, ext JQ_DBG_ARG_DEV);
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int q = base + 32 * u + lane;
                    const int nval = q < qb ? min(4, L - 4 * q) : 0;
                    if (nval == 0 || (quad_bound_key(bf, 32 * u + lane) >> 21) < pre) continue;
                    uint32_t key[4];
                    float best[4];
                    pooled_quad(bf, 32 * u + lane, radius, key, best);
                    int nhit = 0;
                    for (int i = 0; i < 4; ++i) if (i < nval) { nhit += (key[i] >> 21) == pre; hi_cnt += (key[i] >> 21) > pre; }
                    if (nhit) {
                        int at = atomicAdd(&ctl.cand_count, nhit);
                        for (int i = 0; i < 4; ++i)
                            if (i < nval && (key[i] >> 21) == pre) {
                                if (JQ_IN(at, kStrCand, kDbgSelect, 27)) { cand_key[at] = key[i]; cand_pos[at] = 4 * q + i; }
                                ++at;
                            }
                    }
                }
            }
            hi_cnt = __reduce_add_sync(0xffffffffu, hi_cnt);
            if (lane == 0) ctl.warp_gt[wid] = hi_cnt;
            __syncthreads();
        }
        const int nc = listed ? ctl.cand_count : 0;
        for (int r2 = 1; r2 < 3; ++r2) {
            const int sh = (r2 == 1) ? 10 : 0, wd = (r2 == 2) ? 10 : 11;
            const uint32_t mask = (1u << wd) - 1u;
            for (int i = tid; i < kBins; i += T) hist[i] = 0;
            __syncthreads();
            if (listed) {
                for (int e = tid; e < nc; e += T) {
                    const uint32_t k = cand_key[e];
                    if ((k >> (sh + wd)) == pre && JQ_IN((k >> sh) & mask, kBins, kDbgSelect, 24)) atomicAdd(&hist[(k >> sh) & mask], 1u);
                }
            } else {
                for (int base = qa; base < qb; base += kStepQuads) {
                    const float4 *bf = stage_step(buf, s, L, base, qa, qb, vec, soff, ext JQ_DBG_ARG_DEV);
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int q = base + 32 * u + lane;
                        const int nval = q < qb ? min(4, L - 4 * q) : 0;
                        if (nval == 0 || (quad_bound_key(bf, 32 * u + lane) >> (sh + wd)) < pre) continue;
                        uint32_t key[4], dg[4];
                        float best[4];
                        pooled_quad(bf, 32 * u + lane, radius, key, best);
                        for (int i = 0; i < 4; ++i) dg[i] = (key[i] >> (sh + wd)) == pre ? ((key[i] >> sh) & mask) : 0xffffffffu;
                        hist_add_runs(hist, dg, nval JQ_DBG_ARG_DEV);
                    }
                }
            }
            __syncthreads();
            find_digit_cta(hist, krem, ctl);
            pre = (pre << wd) | (uint32_t)ctl.digit;
            krem = ctl.krem;
            __syncthreads();
        }
        const uint32_t tau = pre;
        const int need_eq = krem;       // how many of the keys == tau are kept (lowest positions first)

        // ---- kept keys per warp: from the list, or by a pass of its own
        if (listed) {
            for (int e = tid; e < nc; e += T) {
                const uint32_t k = cand_key[e];
                const int w = min((cand_pos[e] >> 2) / segq, nw - 1);
                if (k > tau) atomicAdd(&ctl.warp_gt[w], 1);
                else if (k == tau) atomicAdd(&ctl.warp_eq[w], 1);
            }
        } else {
            int cgt = 0, ceq = 0;
            for (int base = qa; base < qb; base += kStepQuads) {
                const float4 *bf = stage_step(buf, s, L, base, qa, qb, vec, soff, ext JQ_DBG_ARG_DEV);
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int q = base + 32 * u + lane;
                    const int nval = q < qb ? min(4, L - 4 * q) : 0;
                    if (nval == 0 || quad_bound_key(bf, 32 * u + lane) < tau) continue;
                    uint32_t key[4];
                    float best[4];
                    pooled_quad(bf, 32 * u + lane, radius, key, best);
                    for (int i = 0; i < 4; ++i) if (i < nval) { cgt += key[i] > tau; ceq += key[i] == tau; }
                }
            }
            cgt = __reduce_add_sync(0xffffffffu, cgt);
            ceq = __reduce_add_sync(0xffffffffu, ceq);
            if (lane == 0) { ctl.warp_gt[wid] = cgt; ctl.warp_eq[wid] = ceq; }
        }
        __syncthreads();
        int gt_before = 0, eq_before = 0;
        for (int w = 0; w < wid; ++w) { gt_before += ctl.warp_gt[w]; eq_before += ctl.warp_eq[w]; }

        // ---- pass 3: ordered compaction (position order = warp, step, quad, position within the quad)
        for (int base = qa; base < qb; base += kStepQuads) {
            const float4 *bf = stage_step(buf, s, L, base, qa, qb, vec, soff, ext JQ_DBG_ARG_DEV);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int q = base + 32 * u + lane;
                const int nval = q < qb ? min(4, L - 4 * q) : 0;
                const bool may = nval != 0 && quad_bound_key(bf, 32 * u + lane) >= tau;
                if (!__any_sync(0xffffffffu, may)) continue;         // nothing of these 128 quads is at or above tau
                uint32_t key[4] = {0u, 0u, 0u, 0u};
                float best[4];
                if (may) pooled_quad(bf, 32 * u + lane, radius, key, best);
                int g = 0, e = 0;
                for (int i = 0; i < 4; ++i) if (may && i < nval) { g += key[i] > tau; e += key[i] == tau; }
                const int mine = g | (e << 16);
                int inc = mine;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int n = __shfl_up_sync(0xffffffffu, inc, o);
                    if (lane >= o) inc += n;
                }
                const int total = __shfl_sync(0xffffffffu, inc, 31);
                int g_here = gt_before + ((inc - mine) & 0xffff), e_here = eq_before + ((inc - mine) >> 16);
                for (int i = 0; i < 4; ++i) {
                    if (!may || i >= nval) continue;
                    if (key[i] > tau) {
                        if (JQ_IN(g_here + min(e_here, need_eq), nkeep, kDbgSelect, 28)) out[g_here + min(e_here, need_eq)] = 4 * q + i;
                        ++g_here;
                    } else if (key[i] == tau) {
                        if (e_here < need_eq && JQ_IN(g_here + e_here, nkeep, kDbgSelect, 29)) out[g_here + e_here] = 4 * q + i;
                        ++e_here;
                    }
                }
                gt_before += total & 0xffff;
                eq_before += total >> 16;
            }
        }
    }
    if (!Kin) return;

    // ---- the kept rows (256 bytes each: 16 lanes x 16 bytes), four rows in flight per 16 lanes
    __syncthreads();
    const int lane16 = tid & 15, grp = tid >> 4, ngrp = T >> 4;
    for (int t0 = 4 * grp; t0 < nkeep; t0 += 4 * ngrp) {
        int j[4];
        uint4 a[4], b[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) j[r] = t0 + r < nkeep ? min(max(__ldcg(out + t0 + r), 0), L - 1) : 0;
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const size_t src = ((size_t)kv_in * src_rows + j[r]) * 16 + lane16;
            const bool in = t0 + r < nkeep && JQ_IN((long long)kv_in * src_rows + j[r], ext.src_heads * src_rows, kDbgSelect, 30);
            a[r] = in ? Kin[src] : make_uint4(0u, 0u, 0u, 0u);
            b[r] = in ? Vin[src] : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const size_t dst = (size_t)(krow + t0 + r) * 16 + lane16;
            if (t0 + r < nkeep && JQ_IN(krow + t0 + r, ext.out_rows, kDbgSelect, 31)) { Kout[dst] = a[r]; Vout[dst] = b[r]; }
        }
    }
}

// Shared memory of a CTA whose cluster has `cl` CTAs, the share of the head it holds, and whether its keys stay on chip.
struct SelPlan { int cl, chunk, in_smem, raw_tile; size_t smem; };

// small_stage: stage the scores in pieces of kCandMax (the least the buffer must hold) instead of a CTA's whole
// share, so that two CTAs fit on an SM; worth it when the call has more heads than clusters fit at a time.
SelPlan plan_for(int L, int cl, bool small_stage)
{
    SelPlan p;
    p.cl = cl;
    p.chunk = ((L + cl - 1) / cl + 31) / 32 * 32;
    p.in_smem = p.chunk <= kKeysSmemMax;
    // the staging buffer holds a CTA's share of the scores (at most kRawTile) and later up to kCandMax candidates
    p.raw_tile = p.chunk < kRawTile ? p.chunk : kRawTile;
    if (small_stage && p.in_smem) p.raw_tile = kCandMax;
    if (p.raw_tile < kCandMax) p.raw_tile = kCandMax;
    p.smem = (size_t)(2 * kBins + p.raw_tile + 2 * kHalo) * 4 + (p.in_smem ? (size_t)p.chunk * 4 : 0);
    return p;
}

// Cluster size for Hkv heads of L keys.  The kernel is a chain of short phases between cluster barriers
// (about 20 k cycles of them) plus work in proportion to a CTA's share (about 1.7 cycles per key); few heads
// want the largest cluster (shortest chain per head), many heads want smaller ones (more heads at a time,
// and the chain is paid once per head either way).  Estimated as rounds of resident clusters times the
// time of one.
SelPlan choose_plan(int Hkv, int L, int sms)
{
    const bool many = Hkv > sms / kClMax;        // more heads than 8-CTA clusters fit at one CTA per SM
    SelPlan best = plan_for(L, kClMax, many);
    double best_cost = 0;
    for (int cl = kClMax; cl >= 2; cl >>= 1) {
        const SelPlan p = plan_for(L, cl, many);
        if (cl != kClMax && !p.in_smem) break;
        const int per_sm = p.smem <= 112 * 1024 + 512 ? 2 : 1;
        const int resident = sms * per_sm / cl > 0 ? sms * per_sm / cl : 1;
        const double cost = (double)((Hkv + resident - 1) / resident) * (20000.0 + 1.7 * p.chunk);
        if (cl == kClMax || cost < best_cost) { best = p; best_cost = cost; }
    }
    return best;
}

template <int CL>
jq_status launch_select_cl(const SelPlan &p, const float *scores, const jq_shape &s, int nkeep, int32_t *idx, float *pooled,
                           const Workspace &w, cudaStream_t st, const void *K, const void *V, void *Kout, void *Vout, int dev,
                           const UnitTables *tables, int src_rows, int out_rows)
{
    static bool attr_done[64] = {};
    if (!attr_done[dev]) {
        const int max_smem = (2 * kBins + kRawTile + 2 * kHalo + kKeysSmemMax) * 4;
        if (cudaFuncSetAttribute(select_cluster<CL>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem) != cudaSuccess)
            return JQ_ERR_CUDA;
        attr_done[dev] = true;
    }
    SelExtents ext;
    ext.scores = tables ? tables->total_keys : (long long)s.Hkv * s.L;
    ext.out_rows = tables ? tables->total_rows : (long long)s.Hkv * out_rows;
    ext.src_heads = tables ? tables->hpu : s.Hkv;
    // Launched with programmatic stream serialisation: the CTAs may be set up while the kernel before it in
    // the stream (the scoring kernel) drains; the kernel waits for that kernel's memory before reading anything.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(s.Hkv * CL));
    cfg.blockDim = dim3(kSelThreads);
    cfg.dynamicSmemBytes = p.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, select_cluster<CL>, scores, s.L, nkeep, (s.pool - 1) / 2, idx, pooled, w.keys, p.chunk,
                           p.in_smem, p.raw_tile, (const uint4 *)K, (const uint4 *)V, (uint4 *)Kout, (uint4 *)Vout,
                           tables ? tables->heads : nullptr, (const uint4 *const *)(tables && Kout ? tables->K : nullptr),
                           (const uint4 *const *)(tables && Kout ? tables->V : nullptr), src_rows, out_rows, ext JQ_DBG_ARG) != cudaSuccess) {
        cudaGetLastError();
        return JQ_ERR_CUDA;
    }
    count_launch(1);
    return check_launch();
}

// The many-head kernel: 512 threads per head (measured best from 8K to 64K keys per head, 256 to 1024 heads), 1024
// when the scores of the heads that 512 would hold in flight (a head is read three times) are far more than the L2.
jq_status launch_select_stream(const float *scores, const jq_shape &s, int nkeep, int Lmax, int32_t *idx, float *pooled,
                               cudaStream_t st, const void *K, const void *V, void *Kout, void *Vout, int sms, int dev,
                               const UnitTables *tables, int src_rows, int out_rows)
{
    const long long resident = (long long)sms * stream_ctas_per_sm(512), inflight = s.Hkv < resident ? s.Hkv : resident;
    const int threads = inflight * Lmax * 4 <= (96ll << 20) ? 512 : 1024;
    const auto kernel = threads == 512 ? select_stream<512> : select_stream<1024>;
    const size_t dyn = (size_t)(threads / 32) * 2 * kStageQuads * sizeof(float4);
    static bool attr_done[64][2] = {};
    const int which = threads == 512 ? 0 : 1;
    if (dev < 0 || dev >= 64) return JQ_ERR_CUDA;
    if (!attr_done[dev][which]) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess) return JQ_ERR_CUDA;
        attr_done[dev][which] = true;
    }
    SelExtents ext;
    ext.scores = tables ? tables->total_keys : (long long)s.Hkv * s.L;
    ext.out_rows = tables ? tables->total_rows : (long long)s.Hkv * out_rows;
    ext.src_heads = tables ? tables->hpu : s.Hkv;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)s.Hkv);
    cfg.blockDim = dim3((unsigned)threads);
    cfg.dynamicSmemBytes = dyn;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // as for the cluster kernel
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kernel, scores, s.L, nkeep, (s.pool - 1) / 2, idx, pooled, (const uint4 *)K,
                           (const uint4 *)V, (uint4 *)Kout, (uint4 *)Vout, tables ? tables->heads : nullptr,
                           (const uint4 *const *)(tables && Kout ? tables->K : nullptr),
                           (const uint4 *const *)(tables && Kout ? tables->V : nullptr), src_rows, out_rows, ext JQ_DBG_ARG) != cudaSuccess) {
        cudaGetLastError();
        return JQ_ERR_CUDA;
    }
    count_launch(1);
    return check_launch();
}

}  // namespace

jq_status launch_select(const float *scores, const jq_shape &s, int32_t *idx, float *pooled,
                        const Workspace &w, cudaStream_t st, const void *K, const void *V, void *Kout, void *Vout,
                        const UnitTables *tables, int src_head_rows, int out_head_rows)
{
    const int src_rows = src_head_rows > s.L ? src_head_rows : s.L;
    // with tables: the plan and the shared memory follow the longest head; every head reads its own record
    const int Lmax = tables ? tables->max_L : s.L;
    const int nkeep = s.budget < Lmax ? s.budget : Lmax;
    static int sms[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return JQ_ERR_CUDA;
    if (!sms[dev] && cudaDeviceGetAttribute(&sms[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return JQ_ERR_CUDA;
    // many heads and a window the quad pooling covers: one CTA per head
    if (s.Hkv >= kStreamMinHeads && (s.pool - 1) / 2 <= 4)
        return launch_select_stream(scores, s, nkeep, Lmax, idx, pooled, st, K, V, Kout, Vout, sms[dev], dev, tables, src_rows,
                                    out_head_rows > nkeep ? out_head_rows : nkeep);
    const SelPlan p = choose_plan(s.Hkv, Lmax, sms[dev]);
    switch (p.cl) {
    case 2: return launch_select_cl<2>(p, scores, s, nkeep, idx, pooled, w, st, K, V, Kout, Vout, dev, tables, src_rows, out_head_rows > nkeep ? out_head_rows : nkeep);
    case 4: return launch_select_cl<4>(p, scores, s, nkeep, idx, pooled, w, st, K, V, Kout, Vout, dev, tables, src_rows, out_head_rows > nkeep ? out_head_rows : nkeep);
    default: return launch_select_cl<8>(p, scores, s, nkeep, idx, pooled, w, st, K, V, Kout, Vout, dev, tables, src_rows, out_head_rows > nkeep ? out_head_rows : nkeep);
    }
}

}  // namespace jq
