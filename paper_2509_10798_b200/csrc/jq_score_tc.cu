// Tensor-core scoring for sm_100a: Eq. 3 in two streaming passes over K.
//
// Both passes are persistent, warp-specialised kernels (one CTA per SM):
//   warp 0      TMA producer: K tiles of 128 keys (two 64-column halves, 128-byte swizzle) into a
//               ring of shared-memory stages; the query rows of a KV head into a stationary buffer;
//   warp 1      issues tcgen05.mma (bf16 x bf16 -> fp32 in tensor memory) and owns the TMEM allocation;
//   warps 2-9   two epilogue groups of 128 threads that read accumulators with tcgen05.ld.
// The operand roles are swapped between the passes so that no reduction crosses threads:
//   pass 1  S[R x 128] = Q K^T   (A = query rows, M = 128): a thread owns a QUERY ROW and keeps its
//           running max m and sum l = sum_j exp2(c (s_j - m)); per-CTA partial (m, l) go to the workspace;
//   pass 2  S^T[128 x R] = K Q^T (A = key tile, N = R):     a thread owns a KEY and adds
//           exp2(c s - M_r) over the R rows, M_r = c m_r + log2(l_r) merged from the partials.
// Tiles are split statically and contiguously over the CTAs; pass 2 walks its range backwards so the
// tiles pass 1 read last (most likely still in L2) are read first.
//
// Every wait is bounded: when one runs out, the CTA records JQ_ERR_TIMEOUT in the workspace status
// word, raises a CTA-wide abort flag that every other wait polls, and leaves through the common exit
// (which frees the tensor memory).
#include "jq_internal.cuh"
#include "jq_tmem_ld.cuh"
#include <cuda.h>
#include <cstddef>
#include <mutex>

namespace jq {
namespace {

constexpr int kTile = 128;                       // keys per tile
constexpr int kStages = 4;                       // K ring depth
constexpr int kThreads = 320;
constexpr uint32_t kHalfBytes = kTile * 128;     // one 64-column half of a K tile (128-byte rows)
constexpr uint32_t kStageBytes = 2 * kHalfBytes; // 32 KiB
constexpr uint32_t kCtlBytes = 4096;             // barriers, flags, M_r
constexpr uint32_t kTmemCols = 512;
constexpr long long kWaitCycles = 4000000000ll;         // about 2 s of SM clock per wait

struct Ctl {
    uint64_t full[kStages], empty[kStages];
    uint64_t q_full[2], q_empty[2];
    uint64_t t_full[4], t_empty[4];
    uint64_t m_ready[2];
    uint32_t tmem_base;
    int abort_flag;
    alignas(16) float Ms[2][kMaxR];   // read as float4
};
static_assert(offsetof(Ctl, Ms) % 16 == 0, "Ms must be 16-byte aligned");
static_assert(sizeof(Ctl) <= kCtlBytes, "control block too large");

struct Params {
    int L, R, Rbox;          // Rbox = 128 or 256: query rows staged per KV head (rows >= R are zero)
    int h0, nheads, tph;     // KV heads [h0, h0+nheads) ; tiles per head
    float c;                 // log2(e) / sqrt(d)
    float2 *part;            // [Hkv][kSlots][R]
    float *Mrow;             // [Hkv][R]   c*m + log2(l) per query row
    float *scores;           // [Hkv][L]
    int *status;
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
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
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
    for (int i = 0; i < 4096; ++i)
        if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        for (int i = 0; i < 256; ++i)
            if (mbar_try(bar, parity)) return true;
        if (*(volatile int *)&ctl->abort_flag) return false;
        if (clock64() - t0 > kWaitCycles) {
            *(volatile int *)&ctl->abort_flag = 1;
            atomicMax(status, (int)JQ_ERR_TIMEOUT);
            return false;
        }
    }
}
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, Ctl *ctl, int *status)
{
    if (mbar_try(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, ctl, status);
}

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

// Which CTA owns tile t when T tiles are split contiguously over G CTAs as [b*T/G, (b+1)*T/G).
__device__ __forceinline__ int owner_of_tile(long long t, long long T, long long G)
{
    return (int)(((t + 1) * G - 1) / T);
}

// ------------------------------------------------------------------ the kernel

template <int PASS>
__global__ void __launch_bounds__(kThreads, 1)
score_pass(const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapQ, const Params P)
{
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    Ctl *ctl = (Ctl *)smem_raw;
    const uint32_t base = (smem_u32(smem_raw) + kCtlBytes + 1023u) & ~1023u;   // 1024-byte aligned data
    uint8_t *data = smem_raw + (base - smem_u32(smem_raw));
    const int nq = (P.Rbox == 128) ? 2 : 1;                  // query buffers (double-buffered when they fit)
    const uint32_t q_bytes = (uint32_t)P.Rbox * kD * 2;
    uint8_t *qbuf = data;
    uint8_t *kbuf = data + (size_t)nq * q_bytes;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long T = (long long)P.nheads * P.tph, G = gridDim.x;
    const int t_begin = (int)((long long)blockIdx.x * T / G), t_end = (int)(((long long)blockIdx.x + 1) * T / G);
    const int ntiles = t_end - t_begin;
    const int nmb = (PASS == 1) ? P.Rbox / 128 : 1;          // accumulator blocks per tile
    const int Rpad = (P.R + 15) & ~15;
    const int nslots = (PASS == 1) ? 4 : (Rpad <= 128 ? 4 : 2);
    const uint32_t slot_cols = kTmemCols / nslots;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(&ctl->q_full[s], 1); mbar_init(&ctl->q_empty[s], 1); mbar_init(&ctl->m_ready[s], 256); }
        for (int s = 0; s < 4; ++s) { mbar_init(&ctl->t_full[s], 1); mbar_init(&ctl->t_empty[s], 128); }
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
            int seg = -1, prev_kv = -1;
            for (int n = 0; n < ntiles; ++n) {
                const int i = (PASS == 1) ? t_begin + n : t_end - 1 - n;
                const int kv = P.h0 + i / P.tph, j0 = (i % P.tph) * kTile;
                if (kv != prev_kv) {
                    prev_kv = kv; ++seg;
                    const int qb = seg % nq;
                    if (!mbar_wait(&ctl->q_empty[qb], ((seg / nq) & 1) ^ 1, ctl, P.status)) break;
                    mbar_expect_tx(&ctl->q_full[qb], q_bytes);
                    tma_load_3d(qbuf + (size_t)qb * q_bytes, &mapQ, &ctl->q_full[qb], 0, 0, kv);
                    tma_load_3d(qbuf + (size_t)qb * q_bytes + q_bytes / 2, &mapQ, &ctl->q_full[qb], 64, 0, kv);
                }
                const int st = n % kStages;
                if (!mbar_wait(&ctl->empty[st], ((n / kStages) & 1) ^ 1, ctl, P.status)) break;
                mbar_expect_tx(&ctl->full[st], kStageBytes);
                tma_load_3d(kbuf + (size_t)st * kStageBytes, &mapK, &ctl->full[st], 0, j0, kv);
                tma_load_3d(kbuf + (size_t)st * kStageBytes + kHalfBytes, &mapK, &ctl->full[st], 64, j0, kv);
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            const uint32_t idesc = (PASS == 1) ? instr_desc(128, kTile) : instr_desc(kTile, Rpad);
            int seg = -1, prev_kv = -1;
            uint32_t unit = 0;
            bool ok = true;
            for (int n = 0; n < ntiles && ok; ++n) {
                const int i = (PASS == 1) ? t_begin + n : t_end - 1 - n;
                const int kv = P.h0 + i / P.tph;
                if (kv != prev_kv) {
                    if (seg >= 0) tc_commit(&ctl->q_empty[seg % nq]);   // previous head's queries are free once its MMAs retire
                    prev_kv = kv; ++seg;
                    if (!mbar_wait(&ctl->q_full[seg % nq], (seg / nq) & 1, ctl, P.status)) break;
                }
                const int st = n % kStages;
                if (!mbar_wait(&ctl->full[st], (n / kStages) & 1, ctl, P.status)) break;
                tc_fence_after();
                const uint32_t k_addr = smem_u32(kbuf + (size_t)st * kStageBytes);
                const uint32_t q_addr = smem_u32(qbuf + (size_t)(seg % nq) * q_bytes);
                for (int mb = 0; mb < nmb; ++mb, ++unit) {
                    const uint32_t slot = unit % nslots;
                    if (!mbar_wait(&ctl->t_empty[slot], ((unit / nslots) & 1) ^ 1, ctl, P.status)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t d = tmem + slot * slot_cols;
#pragma unroll
                    for (int ks = 0; ks < kD / 16; ++ks) {
                        const uint32_t koff = (uint32_t)(ks >> 2) * kHalfBytes + (uint32_t)(ks & 3) * 32u;
                        const uint32_t qoff = (uint32_t)(ks >> 2) * (q_bytes / 2) + (uint32_t)(ks & 3) * 32u;
                        if (PASS == 1)
                            tc_mma(d, smem_desc(q_addr + qoff + (uint32_t)mb * kHalfBytes), smem_desc(k_addr + koff), idesc, ks > 0);
                        else
                            tc_mma(d, smem_desc(k_addr + koff), smem_desc(q_addr + qoff), idesc, ks > 0);
                    }
                    tc_commit(&ctl->t_full[slot]);
                }
                tc_commit(&ctl->empty[st]);
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue groups
        const int grp = (warp - 2) >> 2, quarter = warp & 3;
        const int et = threadIdx.x - 64;                        // 0..255
        const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16);
        int seg = -1, prev_kv = -1;
        uint32_t unit = 0;
        float m_run = -INFINITY, l0 = 0.f, l1 = 0.f, l2 = 0.f, l3 = 0.f;
        bool ok = true;
        const float c = P.c;

        auto flush_partial = [&](int kv) {                      // pass 1: one (m, l) per row and group
            const int row = ((nmb == 2) ? grp * 128 : 0) + quarter * 32 + lane;
            if (row < P.R)
                P.part[((size_t)kv * kSlots + 2 * blockIdx.x + grp) * P.R + row] = make_float2(m_run, (l0 + l1) + (l2 + l3));
            m_run = -INFINITY; l0 = l1 = l2 = l3 = 0.f;
        };

        for (int n = 0; n < ntiles && ok; ++n) {
            const int i = (PASS == 1) ? t_begin + n : t_end - 1 - n;
            const int kv = P.h0 + i / P.tph, j0 = (i % P.tph) * kTile;
            if (kv != prev_kv) {
                if (PASS == 1) {
                    if (seg >= 0) flush_partial(prev_kv);
                } else {
                    // stage the row normalisers M_r of the new head
                    const int sb = (seg + 1) & 1;
                    if (et < P.R) ctl->Ms[sb][et] = __ldcg(&P.Mrow[(size_t)kv * P.R + et]);
                    mbar_arrive(&ctl->m_ready[sb]);
                    if (!mbar_wait(&ctl->m_ready[sb], ((seg + 1) >> 1) & 1, ctl, P.status)) break;
                }
                prev_kv = kv; ++seg;
            }
            for (int mb = 0; mb < nmb; ++mb, ++unit) {
                if ((int)(unit & 1) != grp) continue;
                const uint32_t slot = unit % nslots;
                if (!mbar_wait(&ctl->t_full[slot], (unit / nslots) & 1, ctl, P.status)) { ok = false; break; }
                tc_fence_after();
                const uint32_t taddr = lane_addr + slot * slot_cols;
                uint32_t v[128];
                if (PASS == 1) {
                    // the whole 128-key row segment in one tensor-memory read; the slot is free right after
                    JQ_TMEM_LD128(taddr, v);
                    tmem_ld_wait();
                    tc_fence_before();
                    mbar_arrive(&ctl->t_empty[slot]);
                    const int valid = min(kTile, P.L - j0);
                    if (valid < kTile) {
#pragma unroll
                        for (int t = 0; t < 128; ++t) if (t >= valid) v[t] = 0xff800000u;   // -inf: not a key
                    }
                    float c0 = -INFINITY, c1 = -INFINITY, c2 = -INFINITY, c3 = -INFINITY;
#pragma unroll
                    for (int t = 0; t < 128; t += 4) {
                        c0 = fmaxf(c0, __uint_as_float(v[t + 0])); c1 = fmaxf(c1, __uint_as_float(v[t + 1]));
                        c2 = fmaxf(c2, __uint_as_float(v[t + 2])); c3 = fmaxf(c3, __uint_as_float(v[t + 3]));
                    }
                    const float cm = fmaxf(fmaxf(c0, c1), fmaxf(c2, c3));
                    if (cm > m_run) {
                        const float f = ex2(c * (m_run - cm));
                        l0 *= f; l1 *= f; l2 *= f; l3 *= f;
                        m_run = cm;
                    }
                    const float mc = m_run * c;
#pragma unroll
                    for (int t = 0; t < 128; t += 4) {
                        l0 += ex2(fmaf(__uint_as_float(v[t + 0]), c, -mc));
                        l1 += ex2(fmaf(__uint_as_float(v[t + 1]), c, -mc));
                        l2 += ex2(fmaf(__uint_as_float(v[t + 2]), c, -mc));
                        l3 += ex2(fmaf(__uint_as_float(v[t + 3]), c, -mc));
                    }
                } else {
                    const float *Ms = ctl->Ms[seg & 1];
                    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll 1
                    for (int c0 = 0; c0 < Rpad; c0 += 128) {
                        if (Rpad - c0 >= 128) {
                            JQ_TMEM_LD128(taddr + c0, v);
                            tmem_ld_wait();
                            if (c0 + 128 >= Rpad) { tc_fence_before(); mbar_arrive(&ctl->t_empty[slot]); }
                            const int nv = P.R - c0;             // columns that are real query rows
                            if (nv >= 128) {
#pragma unroll
                                for (int t = 0; t < 128; t += 4) {
                                    const float4 mm = *(const float4 *)(Ms + c0 + t);
                                    a0 += ex2(fmaf(__uint_as_float(v[t + 0]), c, -mm.x));
                                    a1 += ex2(fmaf(__uint_as_float(v[t + 1]), c, -mm.y));
                                    a2 += ex2(fmaf(__uint_as_float(v[t + 2]), c, -mm.z));
                                    a3 += ex2(fmaf(__uint_as_float(v[t + 3]), c, -mm.w));
                                }
                            } else {
#pragma unroll
                                for (int t = 0; t < 128; ++t) if (t < nv) a0 += ex2(fmaf(__uint_as_float(v[t]), c, -Ms[c0 + t]));
                            }
                        } else {
#pragma unroll 1
                            for (int c1 = c0; c1 < Rpad; c1 += 32) {
                                JQ_TMEM_LD32(taddr + c1, v);
                                tmem_ld_wait();
                                if (c1 + 32 >= Rpad) { tc_fence_before(); mbar_arrive(&ctl->t_empty[slot]); }
                                const int nv = P.R - c1;
                                if (nv >= 32) {
#pragma unroll
                                    for (int t = 0; t < 32; t += 4) {
                                        const float4 mm = *(const float4 *)(Ms + c1 + t);
                                        a0 += ex2(fmaf(__uint_as_float(v[t + 0]), c, -mm.x));
                                        a1 += ex2(fmaf(__uint_as_float(v[t + 1]), c, -mm.y));
                                        a2 += ex2(fmaf(__uint_as_float(v[t + 2]), c, -mm.z));
                                        a3 += ex2(fmaf(__uint_as_float(v[t + 3]), c, -mm.w));
                                    }
                                } else {
#pragma unroll
                                    for (int t = 0; t < 32; ++t) if (t < nv) a0 += ex2(fmaf(__uint_as_float(v[t]), c, -Ms[c1 + t]));
                                }
                            }
                        }
                    }
                    const int key = j0 + quarter * 32 + lane;
                    if (key < P.L) P.scores[(size_t)kv * P.L + key] = (a0 + a1) + (a2 + a3);
                }
            }
        }
        if (PASS == 1 && seg >= 0 && ok) flush_partial(prev_kv);
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
}

// Combines the per-CTA partial (m, l) of pass 1 into M_r = c*m_r + log2(l_r).  One warp per query
// row, lanes over the partial slots, then a butterfly; the order is fixed, hence deterministic.
// grid (ceil(R/8), nheads), block 256.
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

__global__ void __launch_bounds__(256)
merge_partials(const float2 *__restrict__ part, float *__restrict__ Mrow, int R, int Rbox, int h0, int tph,
               int nheads, int G, float c)
{
    const int lane = threadIdx.x & 31, r = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (r >= R) return;
    const int kv = h0 + blockIdx.y;
    const long long T = (long long)nheads * tph, first = (long long)blockIdx.y * tph;
    const int b_lo = owner_of_tile(first, T, G), b_hi = owner_of_tile(first + tph - 1, T, G);
    const int ng = (Rbox == 256) ? 1 : 2, g0 = (Rbox == 256) ? (r >> 7) : 0;
    const int nsl = (b_hi - b_lo + 1) * ng;
    float m = -INFINITY, l = 0.f;
    for (int i = lane; i < nsl; i += 32) {
        const int b = b_lo + i / ng, g = g0 + i % ng;
        if ((long long)b * T / G == ((long long)b + 1) * T / G) continue;   // CTA b had no tile
        const float2 p = __ldcg(&part[((size_t)kv * kSlots + 2 * b + g) * R + r]);
        merge_ml(m, l, p.x, p.y, c);
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, m, o), l2 = __shfl_xor_sync(0xffffffffu, l, o);
        merge_ml(m, l, m2, l2, c);
    }
    if (lane == 0) Mrow[(size_t)kv * R + r] = c * m + log2f(l);
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

struct DeviceInfo {
    int sms = 0;
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
        int l2 = 0;
        if (cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return false;
        if (cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, dev) != cudaSuccess) return false;
        d.l2 = l2;
        const int smem = (int)(kCtlBytes + 1024 + 2 * 128 * kD * 2 + kStages * kStageBytes);
        if (cudaFuncSetAttribute(score_pass<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return false;
        if (cudaFuncSetAttribute(score_pass<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return false;
        d.ready = true;
    }
    *out = d;
    return true;
}

}  // namespace

jq_status launch_score_tc(const void *K, const void *Q, const jq_shape &s, float *scores, const Workspace &w,
                          cudaStream_t st)
{
    DeviceInfo dev;
    if (!device_info(&dev)) return JQ_ERR_CUDA;
    const int R = s.group * s.w;
    Params P;
    P.L = s.L; P.R = R; P.Rbox = R <= 128 ? 128 : 256;
    P.tph = (s.L + kTile - 1) / kTile;
    P.c = 1.4426950408889634f / sqrtf((float)s.d);
    P.part = w.part; P.Mrow = w.Mrow; P.scores = scores; P.status = w.status;
    CUtensorMap mapK, mapQ;
    if (!make_map(&mapK, K, s.L, s.Hkv, kTile) || !make_map(&mapQ, Q, R, s.Hkv, P.Rbox)) return JQ_ERR_CUDA;
    const size_t smem = kCtlBytes + 1024 + (size_t)(P.Rbox == 128 ? 2 : 1) * P.Rbox * kD * 2 + (size_t)kStages * kStageBytes;
    int grid = dev.sms;
    if (2 * grid > kSlots) grid = kSlots / 2;
    // KV heads are scored in groups whose keys fit in a share of the L2, so that pass 2 finds them there.
    const long long head_bytes = (long long)s.L * kD * 2;
    long long per_group = (dev.l2 / 2) / head_bytes;
    if (per_group < 1) per_group = 1;
    const long long ngroups = (s.Hkv + per_group - 1) / per_group;
    per_group = (s.Hkv + ngroups - 1) / ngroups;       // even split
    for (int h0 = 0; h0 < s.Hkv; h0 += (int)per_group) {
        P.h0 = h0;
        P.nheads = (int)(h0 + per_group <= s.Hkv ? per_group : s.Hkv - h0);
        score_pass<1><<<grid, kThreads, smem, st>>>(mapK, mapQ, P);
        merge_partials<<<dim3((R + 7) / 8, P.nheads), 256, 0, st>>>(w.part, w.Mrow, R, P.Rbox, h0, P.tph, P.nheads, grid, P.c);
        score_pass<2><<<grid, kThreads, smem, st>>>(mapK, mapQ, P);
        count_launch(3);
    }
    return check_launch();
}

}  // namespace jq
