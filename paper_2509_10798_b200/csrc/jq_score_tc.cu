// Tensor-core scoring for sm_100a: Eq. 3 in two streaming passes over K, ONE persistent kernel per call.
//
// The grid is one CTA per SM, launched cooperatively (all CTAs are resident, so they may wait on one
// another).  A CTA is warp-specialised:
//   warp 0      TMA producer: K tiles of 128 keys (two 64-column halves, 128-byte swizzle) into a
//               ring of shared-memory stages; the query rows of a KV head into one of two stationary buffers;
//   warp 1      issues tcgen05.mma (bf16 x bf16 -> fp32 in tensor memory) and owns the TMEM allocation;
//   warps 2-9   two epilogue groups of 128 threads that read accumulators with tcgen05.ld;
//   warp 10     merges the per-CTA partial row statistics of pass 1 across the grid.
// The operand roles are swapped between the passes so that no reduction crosses threads:
//   pass 1  S[R x 128] = Q K^T   (A = query rows, M = 128): a thread owns a QUERY ROW and keeps its
//           running max m and sum l = sum_j exp2(c (s_j - m)); per-CTA partial (m, l) go to the workspace;
//   pass 2  S^T[128 x R] = K Q^T (A = key tile, N = R):     a thread owns a KEY and adds
//           exp2(c s - M_r) over the R rows, M_r = c m_r + log2(l_r) merged from the partials.
//
// KV heads are taken in groups whose keys fit in a share of the L2.  The tiles of a group are split
// statically and contiguously over the CTAs, the same split in both passes, and pass 2 walks its range
// backwards, so a CTA re-reads what it read itself, most recent first.  The segments are ordered
//   P1(0) P1(1) P2(0) P1(2) P2(1) ... P2(last)
// so that the grid-wide merge of group g (counter -> merge warp -> counter) happens while every CTA is busy
// with pass 1 of group g+1; only the epilogue warps ever wait for it, and normally find it done.
//
// Grid-wide counters live in the status block at the head of the workspace (zeroed by
// jq_workspace_init): a ring of four per kind, with cumulative targets, reset by the last CTA to
// leave.  Every wait (mbarrier or counter) is bounded: when one runs out, the CTA records
// JQ_ERR_TIMEOUT in the status word, raises a CTA-wide abort flag that every other wait polls, runs
// through its remaining barriers without touching data, and leaves through the common exit (which
// frees the tensor memory).
#include "jq_internal.cuh"
#include "jq_tmem_ld.cuh"
#include <cuda.h>
#include <cstddef>
#include <cstdlib>
#include <mutex>

namespace jq {
namespace {

constexpr int kTile = 128;                       // keys per tile
constexpr int kMaxStages = 5;                    // K ring depth (5 when R <= 128, 3 above)
constexpr int kThreads = 352;                    // 11 warps
constexpr uint32_t kHalfBytes = kTile * 128;     // one 64-column half of a K tile (128-byte rows)
constexpr uint32_t kStageBytes = 2 * kHalfBytes; // 32 KiB
constexpr uint32_t kCtlBytes = 2048;             // barriers, flags, M_r
constexpr uint32_t kTmemCols = 512;
constexpr long long kWaitCycles = 4000000000ll;  // about 2 s of SM clock per wait
constexpr int kRing = 4;                         // grid counters per kind
// words of the workspace status block
constexpr int kWStatus = 0, kWDone = 1, kWCnt1 = 8, kWCnt2 = 12;

struct Ctl {
    uint64_t full[kMaxStages], empty[kMaxStages];
    uint64_t q_full[2], q_empty[2];
    uint64_t t_full[4], t_empty[4];
    uint32_t tmem_base;
    int abort_flag;
    alignas(16) float Ms[kMaxR];   // read as float4
};
static_assert(offsetof(Ctl, Ms) % 16 == 0, "Ms must be 16-byte aligned");
static_assert(sizeof(Ctl) <= kCtlBytes, "control block too large");

struct Params {
    int L, R, Rbox, Rpad;    // Rbox = 128 or 256: query rows staged per KV head (rows >= R are zero)
    int Hkv, tph;            // KV heads; tiles per head
    int hpg, ngroups;        // heads per group, groups
    int stages;              // K ring depth
    int pipelined;           // 1: P1(0) P1(1) P2(0) P1(2) ... ; 0: P1(0) P2(0) P1(1) P2(1) ...
    float c;                 // log2(e) / sqrt(d)
    float2 *part;            // [Hkv][kSlots][R]
    float *Mrow;             // [Hkv][R]   c*m + log2(l) per query row
    float *scores;           // [Hkv][L]
    int *status;             // status block (kStatusWords ints)
};

// ------------------------------------------------------------------ PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  false: the wait ran out (status recorded) or another thread of the CTA aborted.
// The clock is only consulted after a few thousand failed polls, so a normal wait never pays for it.
__device__ __noinline__ bool mbar_wait_slow(uint64_t *bar, uint32_t parity, Ctl *ctl, int *status)
{
    if (*(volatile int *)&ctl->abort_flag) return false;
    for (int i = 0; i < 4096; ++i)
        if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        for (int i = 0; i < 256; ++i)
            if (mbar_try(bar, parity)) return true;
        if (*(volatile int *)&ctl->abort_flag) return false;
        if (clock64() - t0 > kWaitCycles) {
            *(volatile int *)&ctl->abort_flag = 1;
            atomicMax(status + kWStatus, (int)JQ_ERR_TIMEOUT);
            return false;
        }
    }
}
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, Ctl *ctl, int *status)
{
    if (mbar_try(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, ctl, status);
}

// Bounded wait for a grid-wide counter to reach `target` (acquire).
__device__ __noinline__ bool wait_counter(const int *p, int target, Ctl *ctl, int *status)
{
    const long long t0 = clock64();
    for (;;) {
        int v;
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
        if (v >= target) return true;
        if (*(volatile int *)&ctl->abort_flag) return false;
        if (clock64() - t0 > kWaitCycles) {
            *(volatile int *)&ctl->abort_flag = 1;
            atomicMax(status + kWStatus, (int)JQ_ERR_TIMEOUT);
            return false;
        }
        __nanosleep(64);
    }
}

// Barrier among the 256 epilogue threads only.
__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *map, uint64_t *bar, int c0, int c1, int c2)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// D[tmem] (+)= A[smem] * B[smem]^T, both operands K-major bf16, fp32 accumulate.
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

// Shared-memory matrix descriptor: K-major, 128-byte swizzle, rows of 128 bytes, 8-row groups 1024
// bytes apart (stride byte offset), leading byte offset 16 (unused for swizzled K-major), version 1.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr)
{
    return (uint64_t)((addr >> 4) & 0x3fffu) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}

// Instruction descriptor, kind::f16: D fp32, A and B bf16, both K-major, shape M x N.
__host__ __device__ constexpr uint32_t instr_desc(int M, int N)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float max3(float a, float b, float c)
{
    float y;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(y) : "f"(a), "f"(b), "f"(c));
    return y;
}

// acc (two lanes) += exp2(v * c + b) for two accumulator columns, on packed fp32 pairs.
__device__ __forceinline__ void exp_acc2(float2 &acc, uint32_t v0, uint32_t v1, float2 cc, float2 b)
{
    const float2 x = __ffma2_rn(make_float2(__uint_as_float(v0), __uint_as_float(v1)), cc, b);
    acc = __fadd2_rn(acc, make_float2(ex2(x.x), ex2(x.y)));
}

// Largest of the 128 values of a row segment.
__device__ __forceinline__ float max128(const uint32_t (&v)[128])
{
    float c0 = -INFINITY, c1 = -INFINITY, c2 = -INFINITY, c3 = -INFINITY;
#pragma unroll
    for (int t = 0; t < 128; t += 8) {
        c0 = max3(c0, __uint_as_float(v[t + 0]), __uint_as_float(v[t + 1]));
        c1 = max3(c1, __uint_as_float(v[t + 2]), __uint_as_float(v[t + 3]));
        c2 = max3(c2, __uint_as_float(v[t + 4]), __uint_as_float(v[t + 5]));
        c3 = max3(c3, __uint_as_float(v[t + 6]), __uint_as_float(v[t + 7]));
    }
    return fmaxf(fmaxf(c0, c1), fmaxf(c2, c3));
}

// Which CTA owns tile t when T tiles are split contiguously over G CTAs as [b*T/G, (b+1)*T/G).
__device__ __forceinline__ int owner_of_tile(long long t, long long T, long long G)
{
    return (int)(((t + 1) * G - 1) / T);
}

// ------------------------------------------------------------------ schedule

// Segment s of the 2 * ngroups segments every CTA walks: a pass over this CTA's share of one group.
struct Seg {
    int pass, g, h0, t_begin, t_end;
};

__device__ __forceinline__ Seg segment(int s, const Params &P)
{
    Seg sg;
    const int NG = P.ngroups;
    if (!P.pipelined) { sg.g = s >> 1; sg.pass = 1 + (s & 1); }
    else if (s == 0) { sg.pass = 1; sg.g = 0; }
    else if (s == 2 * NG - 1) { sg.pass = 2; sg.g = NG - 1; }
    else if (s & 1) { sg.pass = 1; sg.g = (s + 1) >> 1; }
    else { sg.pass = 2; sg.g = (s >> 1) - 1; }
    sg.h0 = sg.g * P.hpg;
    const int nh = min(P.hpg, P.Hkv - sg.h0);
    const long long T = (long long)nh * P.tph, G = gridDim.x;
    sg.t_begin = (int)((long long)blockIdx.x * T / G);
    sg.t_end = (int)(((long long)blockIdx.x + 1) * T / G);
    return sg;
}

// Merge of two partial (max, sum of exp2(c (s - max))) pairs; an empty partial has l == 0.
__device__ __forceinline__ void merge_ml(float &m, float &l, float m2, float l2, float c)
{
    if (l2 > 0.f) {
        if (l > 0.f) {
            const float mn = fmaxf(m, m2);
            l = l * ex2(c * (m - mn)) + l2 * ex2(c * (m2 - mn));
            m = mn;
        } else {
            m = m2; l = l2;
        }
    }
}

// ------------------------------------------------------------------ the kernel

__global__ void __launch_bounds__(kThreads, 1)
score_fused(const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapQ, const Params P)
{
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;   // 1024-byte aligned data
    uint8_t *data = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t q_bytes = (uint32_t)P.Rbox * kD * 2;
    uint8_t *qbuf = data;                                    // two query buffers
    uint8_t *kbuf = data + 2 * (size_t)q_bytes;              // K ring
    Ctl *ctl = (Ctl *)(kbuf + (size_t)P.stages * kStageBytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = gridDim.x, stages = P.stages;
    const int nslots = (P.Rbox == 256) ? 2 : 4;
    const uint32_t slot_cols = kTmemCols / nslots;
    const int nseg = 2 * P.ngroups;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(&ctl->q_full[s], 1); mbar_init(&ctl->q_empty[s], 1); }
        for (int s = 0; s < 4; ++s) { mbar_init(&ctl->t_full[s], 1); mbar_init(&ctl->t_empty[s], P.Rbox == 256 ? 256 : 128); }
        ctl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *(volatile uint32_t *)&ctl->tmem_base;

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            uint32_t it = 0, qn = 0;
            int prev_kv = -1;
            bool ok = true;
            for (int s = 0; s < nseg && ok; ++s) {
                const Seg sg = segment(s, P);
                const int ntiles = sg.t_end - sg.t_begin;
                for (int n = 0; n < ntiles; ++n, ++it) {
                    const int i = (sg.pass == 1) ? sg.t_begin + n : sg.t_end - 1 - n;
                    const int kv = sg.h0 + i / P.tph, j0 = (i % P.tph) * kTile;
                    if (kv != prev_kv) {
                        const uint32_t qb = qn & 1;
                        if (!mbar_wait(&ctl->q_empty[qb], ((qn >> 1) & 1) ^ 1, ctl, P.status)) { ok = false; break; }
                        mbar_expect_tx(&ctl->q_full[qb], q_bytes);
                        tma_load_3d(qbuf + (size_t)qb * q_bytes, &mapQ, &ctl->q_full[qb], 0, 0, kv);
                        tma_load_3d(qbuf + (size_t)qb * q_bytes + q_bytes / 2, &mapQ, &ctl->q_full[qb], 64, 0, kv);
                        prev_kv = kv; ++qn;
                    }
                    const uint32_t st = it % stages;
                    if (!mbar_wait(&ctl->empty[st], ((it / stages) & 1) ^ 1, ctl, P.status)) { ok = false; break; }
                    mbar_expect_tx(&ctl->full[st], kStageBytes);
                    tma_load_3d(kbuf + (size_t)st * kStageBytes, &mapK, &ctl->full[st], 0, j0, kv);
                    tma_load_3d(kbuf + (size_t)st * kStageBytes + kHalfBytes, &mapK, &ctl->full[st], 64, j0, kv);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            const uint32_t idesc1 = instr_desc(128, kTile), idesc2 = instr_desc(kTile, P.Rpad);
            const int nmb = P.Rbox / 128;                     // pass 1: accumulator blocks of 128 query rows
            uint32_t it = 0, qn = 0;
            int prev_kv = -1;
            bool ok = true;
            for (int s = 0; s < nseg && ok; ++s) {
                const Seg sg = segment(s, P);
                const int ntiles = sg.t_end - sg.t_begin;
                for (int n = 0; n < ntiles; ++n, ++it) {
                    const int i = (sg.pass == 1) ? sg.t_begin + n : sg.t_end - 1 - n;
                    const int kv = sg.h0 + i / P.tph;
                    if (kv != prev_kv) {
                        if (qn > 0) tc_commit(&ctl->q_empty[(qn - 1) & 1]);   // the previous head's queries are free once its MMAs retire
                        if (!mbar_wait(&ctl->q_full[qn & 1], (qn >> 1) & 1, ctl, P.status)) { ok = false; break; }
                        prev_kv = kv; ++qn;
                    }
                    const uint32_t st = it % stages, slot = it % nslots;
                    if (!mbar_wait(&ctl->full[st], (it / stages) & 1, ctl, P.status)) { ok = false; break; }
                    if (!mbar_wait(&ctl->t_empty[slot], ((it / nslots) & 1) ^ 1, ctl, P.status)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t k_addr = smem_u32(kbuf + (size_t)st * kStageBytes);
                    const uint32_t q_addr = smem_u32(qbuf + (size_t)((qn - 1) & 1) * q_bytes);
                    const uint32_t d = tmem + slot * slot_cols;
                    if (sg.pass == 1) {
                        for (int mb = 0; mb < nmb; ++mb) {
#pragma unroll
                            for (int ks = 0; ks < kD / 16; ++ks) {
                                const uint32_t koff = (uint32_t)(ks >> 2) * kHalfBytes + (uint32_t)(ks & 3) * 32u;
                                const uint32_t qoff = (uint32_t)(ks >> 2) * (q_bytes / 2) + (uint32_t)(ks & 3) * 32u;
                                tc_mma(d + (uint32_t)mb * 128u, smem_desc(q_addr + qoff + (uint32_t)mb * kHalfBytes),
                                       smem_desc(k_addr + koff), idesc1, ks > 0);
                            }
                        }
                    } else {
#pragma unroll
                        for (int ks = 0; ks < kD / 16; ++ks) {
                            const uint32_t koff = (uint32_t)(ks >> 2) * kHalfBytes + (uint32_t)(ks & 3) * 32u;
                            const uint32_t qoff = (uint32_t)(ks >> 2) * (q_bytes / 2) + (uint32_t)(ks & 3) * 32u;
                            tc_mma(d, smem_desc(k_addr + koff), smem_desc(q_addr + qoff), idesc2, ks > 0);
                        }
                    }
                    tc_commit(&ctl->t_full[slot]);
                    tc_commit(&ctl->empty[st]);
                }
            }
        }
    } else if (warp < 10) {
        // ---------------------------------------------------------------- epilogue groups
        const int grp = (warp - 2) >> 2, quarter = warp & 3;
        const int et = threadIdx.x - 64;                        // 0..255
        const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16);
        const bool wide = P.Rbox == 256;
        const int my_row = (wide ? grp * 128 : 0) + quarter * 32 + lane;   // pass 1: the query row this thread owns
        const float c = P.c;
        uint32_t it = 0;
        bool ok = true;

        for (int s = 0; s < nseg; ++s) {
            const Seg sg = segment(s, P);
            const int ntiles = sg.t_end - sg.t_begin;
            int prev_kv = -1;
            if (sg.pass == 1) {
                // l = sum_j exp2(c (s_j - m_run)) against a REFERENCE m_run that need not be the row max: it
                // is the max of the first tile seen and is only raised when a later tile would push the sum
                // towards overflow (the tile is then redone from its registers).  Any reference gives the
                // same M_r = c m + log2(l) after the merge.
                float m_run = -INFINITY;
                float2 l01 = make_float2(0.f, 0.f), l23 = make_float2(0.f, 0.f);
                auto flush_partial = [&](int kv) {
                    if (my_row < P.R && ok)
                        P.part[((size_t)kv * kSlots + 2 * blockIdx.x + grp) * P.R + my_row] =
                            make_float2(m_run, (l01.x + l01.y) + (l23.x + l23.y));
                    m_run = -INFINITY;
                    l01 = l23 = make_float2(0.f, 0.f);
                };
                for (int n = 0; n < ntiles; ++n, ++it) {
                    const int i = sg.t_begin + n;
                    const int kv = sg.h0 + i / P.tph, j0 = (i % P.tph) * kTile;
                    if (kv != prev_kv) {
                        if (prev_kv >= 0) flush_partial(prev_kv);
                        prev_kv = kv;
                    }
                    if (!wide && (int)(it & 1) != grp) continue;
                    const uint32_t slot = it % nslots;
                    if (ok) ok = mbar_wait(&ctl->t_full[slot], (it / nslots) & 1, ctl, P.status);
                    if (!ok) continue;
                    tc_fence_after();
                    const uint32_t taddr = lane_addr + slot * slot_cols + (wide ? (uint32_t)grp * 128u : 0u);
                    uint32_t v[128];
                    // the whole 128-key row segment in one tensor-memory read; the slot is free right after
                    JQ_TMEM_LD128(taddr, v);
                    tmem_ld_wait();
                    tc_fence_before();
                    mbar_arrive(&ctl->t_empty[slot], 1);
                    const int valid = min(kTile, P.L - j0);
                    if (valid < kTile) {
#pragma unroll
                        for (int t = 0; t < 128; ++t) if (t >= valid) v[t] = 0xff800000u;   // -inf: not a key
                    }
                    if (m_run == -INFINITY) m_run = max128(v);
                    const float2 keep01 = l01, keep23 = l23;
                    const float2 cc = make_float2(c, c);
                    float2 mb = make_float2(-m_run * c, -m_run * c);
#pragma unroll
                    for (int t = 0; t < 128; t += 4) {
                        exp_acc2(l01, v[t + 0], v[t + 1], cc, mb);
                        exp_acc2(l23, v[t + 2], v[t + 3], cc, mb);
                    }
                    const float lsum = (l01.x + l01.y) + (l23.x + l23.y);
                    if (!(lsum < 1.0e30f)) {
                        // the reference is too far below this tile's values: raise it to the tile max and redo the tile
                        const float cm = fmaxf(max128(v), m_run);
                        const float f = ex2(c * (m_run - cm));
                        l01 = make_float2(keep01.x * f, keep01.y * f);
                        l23 = make_float2(keep23.x * f, keep23.y * f);
                        m_run = cm;
                        mb = make_float2(-m_run * c, -m_run * c);
#pragma unroll
                        for (int t = 0; t < 128; t += 4) {
                            exp_acc2(l01, v[t + 0], v[t + 1], cc, mb);
                            exp_acc2(l23, v[t + 2], v[t + 3], cc, mb);
                        }
                    }
                }
                if (prev_kv >= 0) flush_partial(prev_kv);
                // this CTA's share of pass 1 of the group is published: count it in
                __threadfence();
                epi_sync();
                if (et == 0) atomicAdd(P.status + kWCnt1 + (sg.g & (kRing - 1)), 1);
            } else {
                if (et == 0 && ok)
                    ok = wait_counter(P.status + kWCnt2 + (sg.g & (kRing - 1)), (sg.g / kRing + 1) * G, ctl, P.status);
                for (int n = 0; n < ntiles; ++n, ++it) {
                    const int i = sg.t_end - 1 - n;
                    const int kv = sg.h0 + i / P.tph, j0 = (i % P.tph) * kTile;
                    if (kv != prev_kv) {
                        // stage the row normalisers M_r of the new head (all readers of the old ones are past them)
                        epi_sync();
                        if (et < P.R) ctl->Ms[et] = -__ldcg(&P.Mrow[(size_t)kv * P.R + et]);   // stored negated: x = c s + (-M_r)
                        epi_sync();
                        if (*(volatile int *)&ctl->abort_flag) ok = false;
                        prev_kv = kv;
                    }
                    if ((int)(it & 1) != grp) continue;
                    const uint32_t slot = it % nslots;
                    if (ok) ok = mbar_wait(&ctl->t_full[slot], (it / nslots) & 1, ctl, P.status);
                    if (!ok) continue;
                    tc_fence_after();
                    const uint32_t taddr = lane_addr + slot * slot_cols;
                    const uint32_t arrive_n = wide ? 2u : 1u;
                    const float *Ms = ctl->Ms;
                    const int Rpad = P.Rpad;
                    uint32_t v[128];
                    float2 a01 = make_float2(0.f, 0.f), a23 = make_float2(0.f, 0.f);
                    const float2 cc = make_float2(c, c);
#pragma unroll 1
                    for (int c0 = 0; c0 < Rpad; c0 += 128) {
                        if (Rpad - c0 >= 128) {
                            JQ_TMEM_LD128(taddr + c0, v);
                            tmem_ld_wait();
                            if (c0 + 128 >= Rpad) { tc_fence_before(); mbar_arrive(&ctl->t_empty[slot], arrive_n); }
                            const int nv = P.R - c0;             // columns that are real query rows
                            if (nv >= 128) {
#pragma unroll
                                for (int t = 0; t < 128; t += 4) {
                                    const float4 mm = *(const float4 *)(Ms + c0 + t);
                                    exp_acc2(a01, v[t + 0], v[t + 1], cc, make_float2(mm.x, mm.y));
                                    exp_acc2(a23, v[t + 2], v[t + 3], cc, make_float2(mm.z, mm.w));
                                }
                            } else {
#pragma unroll
                                for (int t = 0; t < 128; ++t) if (t < nv) a01.x += ex2(fmaf(__uint_as_float(v[t]), c, Ms[c0 + t]));
                            }
                        } else {
#pragma unroll 1
                            for (int c1 = c0; c1 < Rpad; c1 += 32) {
                                JQ_TMEM_LD32(taddr + c1, v);
                                tmem_ld_wait();
                                if (c1 + 32 >= Rpad) { tc_fence_before(); mbar_arrive(&ctl->t_empty[slot], arrive_n); }
                                const int nv = P.R - c1;
                                if (nv >= 32) {
#pragma unroll
                                    for (int t = 0; t < 32; t += 4) {
                                        const float4 mm = *(const float4 *)(Ms + c1 + t);
                                        exp_acc2(a01, v[t + 0], v[t + 1], cc, make_float2(mm.x, mm.y));
                                        exp_acc2(a23, v[t + 2], v[t + 3], cc, make_float2(mm.z, mm.w));
                                    }
                                } else {
#pragma unroll
                                    for (int t = 0; t < 32; ++t) if (t < nv) a01.x += ex2(fmaf(__uint_as_float(v[t]), c, Ms[c1 + t]));
                                }
                            }
                        }
                    }
                    const int key = j0 + quarter * 32 + lane;
                    if (key < P.L) P.scores[(size_t)kv * P.L + key] = (a01.x + a01.y) + (a23.x + a23.y);
                }
            }
        }
    } else {
        // ---------------------------------------------------------------- grid-wide merge of the pass-1 partials
        // Group g: once every CTA has published its partials, this CTA combines the rows b, b+G, b+2G, ...
        // of the group (lanes over the contributing slots, then a butterfly: a fixed order, hence
        // deterministic) into M_r = c*m_r + log2(l_r), and counts itself in.
        const float c = P.c;
        for (int g = 0; g < P.ngroups; ++g) {
            int ok = 1;
            if (lane == 0) ok = wait_counter(P.status + kWCnt1 + (g & (kRing - 1)), (g / kRing + 1) * G, ctl, P.status) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            const int h0 = g * P.hpg, nh = min(P.hpg, P.Hkv - h0);
            const long long T = (long long)nh * P.tph;
            const int ng = (P.Rbox == 256) ? 1 : 2;
            for (int item = blockIdx.x; item < nh * P.R; item += G) {
                const int hl = item / P.R, r = item - hl * P.R, kv = h0 + hl;
                const long long first = (long long)hl * P.tph;
                const int b_lo = owner_of_tile(first, T, G), b_hi = owner_of_tile(first + P.tph - 1, T, G);
                const int g0 = (P.Rbox == 256) ? (r >> 7) : 0;
                const int nsl = (b_hi - b_lo + 1) * ng;
                float m = -INFINITY, l = 0.f;
                for (int i = lane; i < nsl; i += 32) {
                    const int b = b_lo + i / ng, gg = g0 + i % ng;
                    if ((long long)b * T / G == ((long long)b + 1) * T / G) continue;   // CTA b had no tile
                    const float2 p = __ldcg(&P.part[((size_t)kv * kSlots + 2 * b + gg) * P.R + r]);
                    merge_ml(m, l, p.x, p.y, c);
                }
#pragma unroll
                for (int o = 16; o >= 1; o >>= 1) {
                    const float m2 = __shfl_xor_sync(0xffffffffu, m, o), l2 = __shfl_xor_sync(0xffffffffu, l, o);
                    merge_ml(m, l, m2, l2, c);
                }
                if (lane == 0) P.Mrow[(size_t)kv * P.R + r] = c * m + log2f(l);
            }
            __syncwarp();
            if (lane == 0) {
                __threadfence();
                atomicAdd(P.status + kWCnt2 + (g & (kRing - 1)), 1);
            }
        }
    }

    // ---------------------------------------------------------------- common exit
    tc_fence_before();
    __syncthreads();
    if (*(volatile int *)&ctl->abort_flag) __nanosleep(200000);   // let copies still in flight land before the CTA goes
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
    if (threadIdx.x == 0) {
        // the last CTA to leave clears the grid counters for the next call on this workspace
        __threadfence();
        if (atomicAdd(P.status + kWDone, 1) == G - 1) {
            for (int i = 0; i < kRing; ++i) { P.status[kWCnt1 + i] = 0; P.status[kWCnt2 + i] = 0; }
            P.status[kWDone] = 0;
        }
    }
}

// ------------------------------------------------------------------ host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    });
    return fn;
}

// bf16 tensor [heads][rows][128] viewed as 3-D (128, rows, heads); box = 64 columns x box_rows rows of
// one head, 128-byte swizzle; rows past `rows` read as zero.
bool make_map(CUtensorMap *map, const void *ptr, int rows, int heads, int box_rows)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {(cuuint64_t)kD, (cuuint64_t)rows, (cuuint64_t)heads};
    cuuint64_t strides[2] = {(cuuint64_t)kD * 2, (cuuint64_t)rows * kD * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr size_t smem_bytes(int Rbox, int stages)
{
    return 1024 + 2 * (size_t)Rbox * kD * 2 + (size_t)stages * kStageBytes + kCtlBytes;
}

struct DeviceInfo {
    int sms = 0;        // CTAs of score_fused that can be resident at once (one per SM)
    long long l2 = 0;
    bool ready = false;
};

bool device_info(DeviceInfo *out)
{
    static DeviceInfo info[64];
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    std::lock_guard<std::mutex> lock(mu);
    DeviceInfo &d = info[dev];
    if (!d.ready) {
        int l2 = 0, sms = 0, coop = 0, per_sm = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return false;
        if (cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, dev) != cudaSuccess) return false;
        if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop) return false;
        const size_t smem = smem_bytes(256, 3) > smem_bytes(128, 5) ? smem_bytes(256, 3) : smem_bytes(128, 5);
        if (cudaFuncSetAttribute(score_fused, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return false;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, score_fused, kThreads, smem) != cudaSuccess || per_sm < 1)
            return false;
        d.sms = sms;
        d.l2 = l2;
        d.ready = true;
    }
    *out = d;
    return true;
}

// Overrides for tuning runs (read once): JQ_SCORE_GROUP_MIB = K bytes per head group, JQ_SCORE_ORDER = 0
// for the unpipelined segment order.
long long env_ll(const char *name, long long dflt)
{
    const char *v = getenv(name);
    return (v && *v) ? atoll(v) : dflt;
}

}  // namespace

jq_status launch_score_tc(const void *K, const void *Q, const jq_shape &s, float *scores, const Workspace &w,
                          cudaStream_t st)
{
    DeviceInfo dev;
    if (!device_info(&dev)) return JQ_ERR_CUDA;
    static const long long group_mib = env_ll("JQ_SCORE_GROUP_MIB", 32);
    static const long long order = env_ll("JQ_SCORE_ORDER", 1);
    const int R = s.group * s.w;
    Params P;
    P.L = s.L; P.R = R; P.Rbox = R <= 128 ? 128 : 256; P.Rpad = (R + 15) & ~15;
    P.Hkv = s.Hkv;
    P.tph = (s.L + kTile - 1) / kTile;
    P.stages = P.Rbox == 128 ? 5 : 3;
    P.pipelined = order != 0;
    P.c = 1.4426950408889634f / sqrtf((float)s.d);
    P.part = w.part; P.Mrow = w.Mrow; P.scores = scores; P.status = w.status;
    CUtensorMap mapK, mapQ;
    if (!make_map(&mapK, K, s.L, s.Hkv, kTile) || !make_map(&mapQ, Q, R, s.Hkv, P.Rbox)) return JQ_ERR_CUDA;

    int sms = dev.sms;
    if (2 * sms > kSlots) sms = kSlots / 2;
    // KV heads are scored in groups whose keys fit in a share of the L2, so that pass 2 finds them there.
    // Among the admissible group sizes, take the one that wastes the fewest CTA-tile slots.
    const long long head_bytes = (long long)s.L * kD * 2;
    long long hmax = (group_mib << 20) / head_bytes;
    if (hmax < 1) hmax = 1;
    if (hmax > s.Hkv) hmax = s.Hkv;
    int best_hpg = 1;
    double best_eff = -1.0;
    for (int hpg = 1; hpg <= (int)hmax; ++hpg) {
        long long work = 0, slots = 0;
        for (int h0 = 0; h0 < s.Hkv; h0 += hpg) {
            const long long T = (long long)(h0 + hpg <= s.Hkv ? hpg : s.Hkv - h0) * P.tph;
            work += T;
            slots += (T + sms - 1) / sms;
        }
        const double eff = (double)work / ((double)slots * sms);
        if (eff >= best_eff - 1e-9) { best_eff = eff > best_eff ? eff : best_eff; best_hpg = hpg; }
        if (hmax > 64 && hpg >= 64) break;   // the scan is only worth it over a small range
    }
    P.hpg = best_hpg;
    P.ngroups = (s.Hkv + P.hpg - 1) / P.hpg;
    long long tmax = (long long)(P.hpg < s.Hkv ? P.hpg : s.Hkv) * P.tph;
    const int grid = (int)(tmax < sms ? tmax : sms);

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem_bytes(P.Rbox, P.stages);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, score_fused, mapK, mapQ, P) != cudaSuccess) {
        cudaGetLastError();
        return JQ_ERR_CUDA;
    }
    count_launch(1);
    return check_launch();
}

}  // namespace jq
