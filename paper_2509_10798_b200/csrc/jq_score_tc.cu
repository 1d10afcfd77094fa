// Tensor-core scoring for sm_100a: Eq. 3 in two streaming passes over K, ONE persistent kernel per call.
//
// The grid is one CTA per SM, launched cooperatively (all CTAs are resident, so they may wait on one
// another).  A CTA is warp-specialised; the first four warps run the machinery:
//   warp 0        TMA producer: K tiles of 128 keys (two 64-column halves, 128-byte swizzle) into a ring of
//                 shared-memory stages; the query rows of a KV head into one of two stationary buffers;
//   warp 1        issues tcgen05.mma (bf16 x bf16 -> fp32 in tensor memory; the warp stays converged, one
//                 elected lane issues) and owns the TMEM allocation;
//   warp 2        merges the per-warp partial row statistics of pass 1 across the grid;
//   warp 3        stages the merged row normalisers of the next KV head of pass 2;
//   warps 4..     kGroups epilogue groups of 128 threads.  Accumulator block u (128 TMEM lanes x 128
//                 columns) sits in slot u % 4 and is taken by group u % kGroups.
// The operand roles are swapped between the passes so that no reduction crosses threads:
//   pass 1  S[128 x 128] = Q K^T  (A = a block of 128 query rows): a thread owns a QUERY ROW and keeps
//           the running max m and l = sum_j exp2(c (s_j - m)); per-warp partial (m, l) go to the workspace;
//   pass 2  S^T[128 x N] = K Q^T  (A = key tile, B = a block of up to 128 query rows): a thread owns a KEY
//           and adds exp2(c s - M_r) over the rows, M_r = c m_r + log2(l_r) merged from the partials.
//           With more than 128 query rows a key gets two blocks, added into the scores with red.add
//           (two commutative additions onto zero: the result does not depend on their order).
// A share of the exponentials is evaluated on the FMA pipe (round, degree-4 polynomial on
// [-1/2, 1/2], exponent insertion) because the ex2 unit, at 16 results per clock per SM, is the binding unit.
//
// An epilogue warp is the only source of work for the ex2 unit of its scheduler, and it has two or three
// peers there: whatever it does between two exponentials leaves the unit idle unless a peer happens to be
// inside its own stream.  So an epilogue warp reads its accumulators 16 columns at a time into two
// register arrays that alternate: the read of the next 16 columns - of the same block, or of the warp's
// next block if that one is already complete - is in flight while the current 16 are exponentiated, the
// accumulator slot goes back to the MMA warp as soon as its last columns are in registers, and the
// bookkeeping per block (which tile, which head, where the result goes) is a handful of integer
// operations on a cursor that moves by a fixed stride.
//
// KV heads are taken in groups whose keys fit in a share of the L2.  The tiles of a group are split
// statically and contiguously over the CTAs, the same split in both passes, and pass 2 walks its range
// backwards, so a CTA re-reads what it read itself, most recent first.  The segments are ordered
//   P1(0) P1(1) P2(0) P1(2) P2(1) ... P2(last)
// so that the grid-wide merge of group g (counter -> merge warps -> counter) happens while every CTA is
// busy with pass 1 of group g+1.
//
// Grid-wide counters live in the status block at the head of the workspace (zeroed by
// jq_workspace_init): a ring of four per kind, with cumulative targets, reset by the last CTA to
// leave.  Every wait (mbarrier or counter) is bounded: when one runs out, the CTA records
// JQ_ERR_TIMEOUT in the status word and raises a CTA-wide abort flag that every other wait polls; all
// roles then run out of their loops without touching data and leave through the common exit (which
// frees the tensor memory).
#include "jq_internal.cuh"
#include "jq_tmem_ld.cuh"
#include "jq_debug.cuh"
#include <cuda.h>
#include <cstddef>
#include <cstring>
#include <mutex>

namespace jq {
namespace {

constexpr int kTile = 128;                       // keys per tile
constexpr int kMaxStages = 5;                    // K ring depth (5 when R <= 128, 3 above)
constexpr int kGroupsNarrow = 3, kGroupsWide = 4;   // epilogue groups for R <= 128 / R > 128
constexpr int kTSlots = 4;                       // accumulator slots in tensor memory
constexpr int kSpecialWarps = 4;                 // producer, MMA, merge, stage: one warpgroup
__host__ __device__ constexpr int threads_for(int groups) { return (kSpecialWarps + 4 * groups) * 32; }
constexpr uint32_t kHalfBytes = kTile * 128;     // one 64-column half of a K tile (128-byte rows)
constexpr uint32_t kStageBytes = 2 * kHalfBytes; // 32 KiB
constexpr uint32_t kCtlBytes = 3072;             // barriers, flags, M_r
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kSlotCols = kTmemCols / kTSlots;
constexpr long long kWaitCycles = 4000000000ll;  // about 2 s of SM clock per wait
constexpr int kRing = 4;                         // grid counters per kind
constexpr int kMergeLoads = 16;                  // partial slots a lane of the merge warp has in flight
constexpr uint32_t kSleepLong = 256;             // ns between polls of a waiter that runs ahead (producer, stager)
constexpr uint32_t kSleepShort = 32;             // ns between polls of a waiter on the critical path
constexpr int kPolyOf8 = 2;                      // of every 8 pairs of exponentials, this many go to the FMA pipe
// words of the workspace status block
constexpr int kWStatus = 0, kWDone = 1, kWCnt1 = 8, kWCnt2 = 12;
static_assert(kSlots >= kGroupsWide * 148 && kSlots >= kGroupsNarrow * 148, "one partial slot per epilogue group and CTA");
// A group waits for its block on the slot's barrier by phase parity, which tells two consecutive fillings apart and no
// more: a group may be at most one filling of a slot ahead of the MMA warp, which holds as long as every group has a
// slot of its own to wait on.
static_assert(kGroupsWide <= kTSlots && kGroupsNarrow <= kTSlots, "no more epilogue groups than accumulator slots");

struct Ctl {
    uint64_t full[kMaxStages], empty[kMaxStages];
    uint64_t q_full[2], q_empty[2];
    uint64_t t_full[kTSlots], t_empty[kTSlots];
    uint64_t ms_full[2], ms_empty[2];
    uint64_t p1_done[4];               // all epilogue warps have published their pass-1 partials of a group
    uint32_t tmem_base;
    int abort_flag;
    alignas(16) float Ms[2][kMaxR];   // -M_r of the KV head being scored in pass 2, double-buffered; read as float4
};
static_assert(offsetof(Ctl, Ms) % 16 == 0, "Ms must be 16-byte aligned");
static_assert(sizeof(Ctl) <= kCtlBytes, "control block too large");

struct Params {
    int L, R, Rbox, Rpad;    // Rbox = 128 or 256: query rows staged per KV head (rows >= R are zero); Rpad = R rounded up to 32
    int Hkv, tph;            // KV heads; tiles per head (the window tile included)
    int hpg, ngroups;        // heads per group, groups
    int stages;              // K ring depth
    int depth;               // pass 2 of a group starts after pass 1 of `depth` groups: 1 = P1(0) P2(0) P1(1) ..., 2 = P1(0) P1(1) P2(0) P1(2) ...
    float c;                 // log2(e) / sqrt(d)
    float2 *part;            // [Hkv][kSlots][R]
    float *Mrow;             // [Hkv][R]   c*m + log2(l) per query row
    float *scores;           // [Hkv][L]
    int *status;             // status block (kStatusWords ints)
    int wtile;               // 1 in window-inclusive mode: every head has one more tile, the last, holding the w window keys
    int w;                   // soft-token queries per query head
    // Units in buffers of their own (ragged calls): the head groups, their lengths and score offsets come from
    // gtab [ngroups] (L, tph, hpg above are then unused) and the tiles through maps [units][2] (K, Qwin).
    const GroupRec *gtab;
    const CUtensorMap *maps;
    int hpu;                 // KV heads per unit (a group may run over consecutive units of one length)
    uint32_t grid_magic, tph_magic;   // ceil(2^32 / gridDim.x), ceil(2^32 / tph) (see fast_div)
#ifdef JQ_DEBUG
    DebugRecord *dbg_rec;    // bounds-checked build: the violation record, and the floats in the scores array
    long long n_scores;
#endif
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
// One look at the barrier, no waiting.
__device__ __forceinline__ bool mbar_test(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  false: the wait ran out (status recorded) or another thread of the CTA aborted.
// A waiter that can afford it sleeps `sleep_ns` between polls: a spinning warp takes issue slots and
// queue entries of the shared-memory pipe away from the epilogue warps on its scheduler.  The clock is
// only consulted after many failed polls, so a normal wait never pays for it.
__device__ __noinline__ bool mbar_wait_slow(uint64_t *bar, uint32_t parity, Ctl *ctl, int *status, uint32_t sleep_ns)
{
    if (*(volatile int *)&ctl->abort_flag) return false;
    for (int i = 0; i < 2048; ++i) {
        if (mbar_try(bar, parity)) return true;
        if (sleep_ns) __nanosleep(sleep_ns);
    }
    const long long t0 = clock64();
    for (;;) {
        for (int i = 0; i < 64; ++i) {
            if (mbar_try(bar, parity)) return true;
            if (sleep_ns) __nanosleep(sleep_ns);
        }
        if (*(volatile int *)&ctl->abort_flag) return false;
        if (clock64() - t0 > kWaitCycles) {
            *(volatile int *)&ctl->abort_flag = 1;
            atomicMax(status + kWStatus, (int)JQ_ERR_TIMEOUT);
            return false;
        }
    }
}
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, Ctl *ctl, int *status, uint32_t sleep_ns = 0)
{
    if (mbar_try(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, ctl, status, sleep_ns);
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

__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *map, uint64_t *bar, int c0, int c1, int c2)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2) : "memory");
}

// A tensor map that the host wrote into global memory (with an ordinary copy) must be acquired by the
// tensor-map proxy before a TMA instruction of this CTA reads it.
__device__ __forceinline__ void tensormap_acquire(const CUtensorMap *map)
{
    asm volatile("fence.proxy.tensormap::generic.acquire.sys [%0], 128;" ::"l"(map) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Issued by ONE lane of a converged warp (the whole warp runs the issuing code so that its address
// arithmetic stays warp-uniform; only the tensor-core instructions themselves are predicated).
__device__ __forceinline__ void tc_commit(uint64_t *bar)
{
    __syncwarp();
    asm volatile(
        "{\n\t.reg .pred pe;\n\t"
        "elect.sync _|pe, 0xffffffff;\n\t"
        "@pe tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
        ::"r"(smem_u32(bar)) : "memory");
}

// Instruction descriptor, kind::f16: D fp32, A and B bf16, both K-major, shape M x N.
__host__ __device__ constexpr uint32_t instr_desc(int M, int N)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

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

// Shared-memory matrix descriptor: K-major, 128-byte swizzle, rows of 128 bytes, 8-row groups 1024
// bytes apart (stride byte offset), leading byte offset 16 (unused for swizzled K-major), version 1.
// Only the low word depends on the address (in 16-byte units); the high word is a constant.
constexpr uint32_t kDescHi = (uint32_t)(1024 >> 4) | (1u << 14) | (2u << 29);
__device__ __forceinline__ uint32_t desc_lo(uint32_t addr) { return ((addr >> 4) & 0x3fffu) | (1u << 16); }

// One accumulator block: D[tmem] = A[smem] * B[smem]^T over the whole head dimension (8 steps of 16),
// both operands K-major bf16 in two 64-column halves `a_half` / `b_half` bytes apart, fp32 accumulate.
// A single straight-line sequence run by the whole (converged) warp with one elected lane issuing: the
// warp shares its scheduler with epilogue warps, so every instruction it does not execute is time the
// tensor pipe does not wait.
__device__ __forceinline__ void tc_mma_block(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t a_half,
                                             uint32_t b_half, uint32_t idesc)
{
    const uint32_t a1 = a_lo + (a_half >> 4), b1 = b_lo + (b_half >> 4);
    __syncwarp();
    asm volatile(
        "{\n\t"
        ".reg .pred pz, po, pe;\n\t"
        ".reg .b64 da, db;\n\t"
        ".reg .b32 ta, tb;\n\t"
        "setp.ne.u32 pz, %0, %0;\n\t"
        "setp.eq.u32 po, %0, %0;\n\t"
        "elect.sync _|pe, 0xffffffff;\n\t"
        "mov.b64 da, {%1, %5};\n\t mov.b64 db, {%2, %5};\n\t"
        "@pe tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %6, pz;\n\t"
        "add.u32 ta, %1, 2;\n\t add.u32 tb, %2, 2;\n\t mov.b64 da, {ta, %5};\n\t mov.b64 db, {tb, %5};\n\t"
        "@pe tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %6, po;\n\t"
        "add.u32 ta, %1, 4;\n\t add.u32 tb, %2, 4;\n\t mov.b64 da, {ta, %5};\n\t mov.b64 db, {tb, %5};\n\t"
        "@pe tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %6, po;\n\t"
        "add.u32 ta, %1, 6;\n\t add.u32 tb, %2, 6;\n\t mov.b64 da, {ta, %5};\n\t mov.b64 db, {tb, %5};\n\t"
        "@pe tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %6, po;\n\t"
        "mov.b64 da, {%3, %5};\n\t mov.b64 db, {%4, %5};\n\t"
        "@pe tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %6, po;\n\t"
        "add.u32 ta, %3, 2;\n\t add.u32 tb, %4, 2;\n\t mov.b64 da, {ta, %5};\n\t mov.b64 db, {tb, %5};\n\t"
        "@pe tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %6, po;\n\t"
        "add.u32 ta, %3, 4;\n\t add.u32 tb, %4, 4;\n\t mov.b64 da, {ta, %5};\n\t mov.b64 db, {tb, %5};\n\t"
        "@pe tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %6, po;\n\t"
        "add.u32 ta, %3, 6;\n\t add.u32 tb, %4, 6;\n\t mov.b64 da, {ta, %5};\n\t mov.b64 db, {tb, %5};\n\t"
        "@pe tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %6, po;\n\t"
        "}"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(a1), "r"(b1), "r"(kDescHi), "r"(idesc) : "memory");
}

// Which CTA owns tile t when T tiles are split contiguously over G CTAs as [b*T/G, (b+1)*T/G).
// (T * G stays far below 2^32: a group has at most 2^17 tiles and the grid at most 160 CTAs.)
__device__ __forceinline__ int owner_of_tile(uint32_t t, uint32_t T, uint32_t G)
{
    return (int)(((t + 1) * G - 1) / T);
}

// Whether CTA b gets a tile at all when T < G tiles are split over G CTAs (rare; kept out of line).
__device__ __noinline__ bool cta_has_tile(uint32_t b, uint32_t T, uint32_t G) { return b * T / G != (b + 1) * T / G; }

// ------------------------------------------------------------------ exponentials

// exp2 of a pair on the FMA pipe, for x < 100 (pass 1 asks for at most +64, see p1_half; pass 2 for
// x <= 0: a logit minus the row's log-sum-exp).  x is clamped to >= -126 (so that the exponent
// insertion cannot wrap; 2^-126 stands in for anything smaller), split into n = round(x) and
// r = x - n in [-1/2, 1/2] by the add-a-large-constant trick, 2^r comes from a degree-4 polynomial
// (relative error < 3e-6, a least-maximum fit of 2^r on that interval) and n is added into the
// exponent field.
__device__ __forceinline__ float2 exp2_fma_pair(float2 x)
{
    const float kMagic = 12582912.f;   // 1.5 * 2^23: x + kMagic holds round(x) in its low mantissa bits
    x.x = fmaxf(x.x, -126.f);
    x.y = fmaxf(x.y, -126.f);
    const float2 t = __fadd2_rn(x, make_float2(kMagic, kMagic));
    const float2 nn = __ffma2_rn(t, make_float2(-1.f, -1.f), make_float2(kMagic, kMagic));   // -round(x)
    const float2 r = __fadd2_rn(x, nn);
    float2 p = __ffma2_rn(make_float2(0.009570101276040077f, 0.009570101276040077f), r,
                          make_float2(0.05591785907745361f, 0.05591785907745361f));
    p = __ffma2_rn(p, r, make_float2(0.240247443318367f, 0.240247443318367f));
    p = __ffma2_rn(p, r, make_float2(0.6931217908859253f, 0.6931217908859253f));
    p = __ffma2_rn(p, r, make_float2(0.9999992847442627f, 0.9999992847442627f));
    return make_float2(__int_as_float(__float_as_int(p.x) + (__float_as_int(t.x) << 23)),
                       __int_as_float(__float_as_int(p.y) + (__float_as_int(t.y) << 23)));
}

// acc += exp2(v * c + b) for two values; POLY picks the pipe.
template <bool POLY>
__device__ __forceinline__ void exp_acc2(float2 &acc, uint32_t v0, uint32_t v1, float2 cc, float2 b)
{
    const float2 x = __ffma2_rn(make_float2(__uint_as_float(v0), __uint_as_float(v1)), cc, b);
    acc = __fadd2_rn(acc, POLY ? exp2_fma_pair(x) : make_float2(ex2(x.x), ex2(x.y)));
}

// Pair i of the 8 pairs of a 16-column read goes to the FMA pipe when this says so: kPolyOf8 of them, spread evenly.
__host__ __device__ constexpr bool poly_pair(int i) { return ((i + 1) * kPolyOf8) / 8 != (i * kPolyOf8) / 8; }

// 16 values against 16 biases (pass 2: the negated row normalisers, from shared memory).
__device__ __forceinline__ void exp_acc16(float2 &a0, float2 &a1, const uint32_t (&v)[16], float2 cc, const float4 *bias)
{
    const float4 b0 = bias[0], b1 = bias[1], b2 = bias[2], b3 = bias[3];
    exp_acc2<poly_pair(0)>(a0, v[0], v[1], cc, make_float2(b0.x, b0.y));
    exp_acc2<poly_pair(1)>(a1, v[2], v[3], cc, make_float2(b0.z, b0.w));
    exp_acc2<poly_pair(2)>(a0, v[4], v[5], cc, make_float2(b1.x, b1.y));
    exp_acc2<poly_pair(3)>(a1, v[6], v[7], cc, make_float2(b1.z, b1.w));
    exp_acc2<poly_pair(4)>(a0, v[8], v[9], cc, make_float2(b2.x, b2.y));
    exp_acc2<poly_pair(5)>(a1, v[10], v[11], cc, make_float2(b2.z, b2.w));
    exp_acc2<poly_pair(6)>(a0, v[12], v[13], cc, make_float2(b3.x, b3.y));
    exp_acc2<poly_pair(7)>(a1, v[14], v[15], cc, make_float2(b3.z, b3.w));
}

// 16 values against one bias (pass 1: minus the running maximum of the row).
__device__ __forceinline__ void exp_acc16(float2 &a0, float2 &a1, const uint32_t (&v)[16], float2 cc, float2 b)
{
    exp_acc2<poly_pair(0)>(a0, v[0], v[1], cc, b);
    exp_acc2<poly_pair(1)>(a1, v[2], v[3], cc, b);
    exp_acc2<poly_pair(2)>(a0, v[4], v[5], cc, b);
    exp_acc2<poly_pair(3)>(a1, v[6], v[7], cc, b);
    exp_acc2<poly_pair(4)>(a0, v[8], v[9], cc, b);
    exp_acc2<poly_pair(5)>(a1, v[10], v[11], cc, b);
    exp_acc2<poly_pair(6)>(a0, v[12], v[13], cc, b);
    exp_acc2<poly_pair(7)>(a1, v[14], v[15], cc, b);
}

__device__ __forceinline__ float max_of16(const uint32_t (&v)[16])
{
    float c0 = -INFINITY, c1 = -INFINITY;
#pragma unroll
    for (int t = 0; t < 16; t += 4) {
        c0 = max3(c0, __uint_as_float(v[t + 0]), __uint_as_float(v[t + 1]));
        c1 = max3(c1, __uint_as_float(v[t + 2]), __uint_as_float(v[t + 3]));
    }
    return fmaxf(c0, c1);
}

// Pass 1, 16 keys of a query row: online softmax statistics (m, l = sum_j exp2(c (s_j - m))).  Any
// reference m gives the same row normaliser c m + log2 l as long as nothing overflows, so m is not kept
// equal to the running max: it is raised (and l rescaled) only when the keys bring a value more than
// `lazy` above it, lazy = 64 / c, i.e. when an exponential would pass 2^64.  A warp of 32 rows restarts
// its statistics at every segment and would otherwise take the rescaling branch on most reads; now it
// takes it once per segment.  (exp2 arguments reach +64 at most, l stays below 2^64 times the keys of
// a segment: far inside fp32.)  The max runs on the ALU pipe and, unlike a check of the sum, does not
// wait for the exponentials in flight.  Keys at column >= valid are not keys (-inf).
struct RowState { float m; float2 l01, l23; };
__device__ __forceinline__ void p1_half(uint32_t (&v)[16], int c0, int valid, float c, float lazy, float2 cc, RowState &st)
{
    if (valid < c0 + 16) {
#pragma unroll
        for (int t = 0; t < 16; ++t) if (c0 + t >= valid) v[t] = 0xff800000u;
    }
    const float cm = max_of16(v);
    if (cm > st.m + lazy) {
        const float f = ex2(c * (st.m - cm));   // 0 for the first keys (m = -inf)
        st.l01 = make_float2(st.l01.x * f, st.l01.y * f);
        st.l23 = make_float2(st.l23.x * f, st.l23.y * f);
        st.m = cm;
    }
    const float nb = -st.m * c;
    exp_acc16(st.l01, st.l23, v, cc, make_float2(nb, nb));
}

// ------------------------------------------------------------------ schedule

// x / d for x < 2^25 with magic = ceil(2^32 / d) computed on the host: one multiplication and a correction
// instead of the compiler's division sequence (dozens of instructions and a reciprocal that would queue behind
// the exponentials in the special-function unit; every role runs the schedule arithmetic once per segment).
__device__ __forceinline__ uint32_t fast_div(uint32_t x, uint32_t d, uint32_t magic)
{
    uint32_t q = __umulhi(x, magic);
    if (q * d > x) --q;          // for d > 1 the estimate is never low and at most one high
    if ((q + 1) * d <= x) ++q;   // d == 1 (magic 2^32 - 1): one low
    return q;
}

// Segment s of the 2 * ngroups segments every CTA walks: a pass over this CTA's share of one group.
struct Seg {
    int pass, g, h0, ntiles;
    int kv0, t0;   // KV head and tile within the head of the first tile in walking order
    int tph, L;    // tiles per head and prefix length of the group's heads
    int unit, c20; // the buffer the group's heads live in and the index of head h0 within it
    long long sbase;   // offset (floats) of head h0's scores
};

// Head group g: from the table of a ragged call, else g-th run of hpg heads of the one stacked tensor.
__device__ __forceinline__ GroupRec group_of(int g, const Params &P)
{
#ifdef JQ_DEBUG
    DebugRecord *dbg = P.dbg_rec;
#endif
    if (P.gtab) {
        // read through the read-only path: a 128-byte line holds three records, so most reads of a role hit the L1
        const GroupRec *p = P.gtab + (JQ_IN(g, P.ngroups, kDbgScore, 1) ? g : 0);
        GroupRec r;
        r.h0 = __ldg(&p->h0); r.nh = __ldg(&p->nh); r.tph = __ldg(&p->tph); r.L = __ldg(&p->L);
        r.unit = __ldg(&p->unit); r.c20 = __ldg(&p->c20); r.sbase = __ldg(&p->sbase); r.tph_magic = __ldg(&p->tph_magic);
        return r;
    }
    GroupRec r;
    r.h0 = g * P.hpg; r.nh = min(P.hpg, P.Hkv - r.h0);
    r.tph = P.tph; r.L = P.L; r.unit = 0; r.c20 = r.h0; r.tph_magic = P.tph_magic;
    r.sbase = (long long)r.h0 * P.L;
    return r;
}

// This CTA's share of a group of nh heads of tph tiles: a role keeps the last one it computed, since consecutive
// groups mostly have the same shape and the divisions are then not repeated.
struct Share {
    int nh = -1, tph = -1;
    int ntiles;
    int hd1, t01;      // head (relative to the group's first) and tile within it of the share's first tile
    int hd2, t02;      // and of its last tile, where pass 2 starts
};

// (Inlined into the four roles that call it once per segment: out of line it took 1200-1400 cycles per call, the
// kernel parameters being read through a reference and the result returned through local memory, and while the MMA
// warp sat in it no group got a block.)
__device__ __forceinline__ Seg segment(int s, const Params &P, Share &sh)
{
    Seg sg;
    const int NG = P.ngroups;
    const int D = min(P.depth, NG), t = s - D;
    if (s < D) { sg.pass = 1; sg.g = s; }                                  // lead-in: pass 1 of the first D groups
    else if (t < 2 * (NG - D)) { sg.pass = (t & 1) ? 1 : 2; sg.g = (t & 1) ? D + (t >> 1) : (t >> 1); }
    else { sg.pass = 2; sg.g = s - NG; }                                   // tail: the last D groups' pass 2
    const GroupRec r = group_of(sg.g, P);
    sg.h0 = r.h0; sg.tph = r.tph; sg.L = r.L; sg.unit = r.unit; sg.c20 = r.c20; sg.sbase = r.sbase;
    if (r.nh != sh.nh || r.tph != sh.tph) {
        const uint32_t T = (uint32_t)r.nh * r.tph, G = gridDim.x;
        const uint32_t t_begin = fast_div(blockIdx.x * T, G, P.grid_magic), t_end = fast_div((blockIdx.x + 1) * T, G, P.grid_magic);
        const uint32_t last = t_end > 0 ? t_end - 1 : 0;
        const uint32_t hd1 = fast_div(t_begin, (uint32_t)r.tph, r.tph_magic), hd2 = fast_div(last, (uint32_t)r.tph, r.tph_magic);
        sh.nh = r.nh; sh.tph = r.tph;
        sh.ntiles = (int)(t_end - t_begin);
        sh.hd1 = (int)hd1; sh.t01 = (int)(t_begin - hd1 * (uint32_t)r.tph);
        sh.hd2 = (int)hd2; sh.t02 = (int)(last - hd2 * (uint32_t)r.tph);
    }
    sg.ntiles = sh.ntiles;
    sg.kv0 = sg.h0 + (sg.pass == 1 ? sh.hd1 : sh.hd2);
    sg.t0 = sg.pass == 1 ? sh.t01 : sh.t02;
    return sg;
}

// Next tile in walking order (forwards in pass 1, backwards in pass 2), without a division: the
// reciprocal a division needs would queue behind the exponentials in the special-function unit.
__device__ __forceinline__ void walk(int pass, int tph, int &kv, int &t)
{
    if (pass == 1) { if (++t == tph) { t = 0; ++kv; } }
    else { if (--t < 0) { t = tph - 1; --kv; } }
}

// ------------------------------------------------------------------ the kernel

template <int kGroups>
__global__ void __launch_bounds__(threads_for(kGroups), 1)
score_fused(const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapQ,
            const __grid_constant__ CUtensorMap mapW, const __grid_constant__ Params P)
{
    constexpr int kEpiWarps = 4 * kGroups;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    if (smem_u32(smem_raw) & 1023u) {   // the swizzled tiles need 1024-byte alignment; nothing has been started yet
        if (threadIdx.x == 0) atomicMax(P.status + kWStatus, (int)JQ_ERR_CUDA);
        return;
    }
    const uint32_t q_bytes = (uint32_t)P.Rbox * kD * 2;
    uint8_t *qbuf = smem_raw;                                 // two query buffers
    uint8_t *kbuf = smem_raw + 2 * (size_t)q_bytes;           // K ring
    Ctl *ctl = (Ctl *)(kbuf + (size_t)P.stages * kStageBytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = gridDim.x, stages = P.stages;
    const int R = P.R, Rpad = P.Rpad;                         // register copies: the loops below must not touch memory for them
    int *const status = P.status;
    const int nblk = P.Rbox / 128;                            // accumulator blocks per tile, both passes
    const int nseg = 2 * P.ngroups;
#ifdef JQ_DEBUG
    DebugRecord *const dbg = P.dbg_rec;
    const long long n_part = (long long)P.Hkv * kSlots * R, n_scores = P.n_scores;
#endif

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxStages; ++s) { mbar_init(&ctl->full[s], 1); mbar_init(&ctl->empty[s], 1); }
        for (int s = 0; s < 2; ++s) {
            mbar_init(&ctl->q_full[s], 1); mbar_init(&ctl->q_empty[s], 1);
            mbar_init(&ctl->ms_full[s], 1); mbar_init(&ctl->ms_empty[s], kEpiWarps);
        }
        for (int s = 0; s < kTSlots; ++s) { mbar_init(&ctl->t_full[s], 1); mbar_init(&ctl->t_empty[s], 4); mbar_init(&ctl->p1_done[s], kEpiWarps); }
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
    cudaGridDependencySynchronize();   // no global memory has been touched so far

    if (warp < kSpecialWarps) {
        if (warp == 0) {
            // ---------------------------------------------------------------- TMA producer
            if (lane == 0) {
                uint32_t st = 0, ph = 0, qn = 0;                  // ring stage and its phase; query loads so far
                Share share;
                int prev_kv = -1, prev_unit = -1;
                const CUtensorMap *head_mapK = &mapK, *head_mapQ = &mapQ;   // maps and head coordinate of the current KV head
                int head_c2 = 0;
                bool ok = true;
#pragma unroll 1
                for (int s = 0; s < nseg && ok; ++s) {
                    const Seg sg = segment(s, P, share);
                    const int pass = sg.pass, ntiles = sg.ntiles, tph = sg.tph;
                    int kv = sg.kv0, tt = sg.t0;
#pragma unroll 1
                    for (int n = 0; n < ntiles; ++n, walk(pass, tph, kv, tt)) {
                        if (kv != prev_kv) {
                            head_c2 = sg.c20 + (kv - sg.h0);
                            if (P.maps) {                         // every unit has tensor maps of its own; the group may run over several units
                                const int du = head_c2 / P.hpu, unit = sg.unit + du;
                                head_c2 -= du * P.hpu;
                                if (unit != prev_unit) {
                                    head_mapK = P.maps + 2 * unit; head_mapQ = head_mapK + 1;
                                    tensormap_acquire(head_mapK); tensormap_acquire(head_mapQ);
                                    prev_unit = unit;
                                }
                            }
                            const uint32_t qb = qn & 1;
                            if (!mbar_wait(&ctl->q_empty[qb], ((qn >> 1) & 1) ^ 1, ctl, status, kSleepLong)) { ok = false; break; }
                            mbar_expect_tx(&ctl->q_full[qb], q_bytes);
                            tma_load_3d(qbuf + (size_t)qb * q_bytes, head_mapQ, &ctl->q_full[qb], 0, 0, head_c2);
                            tma_load_3d(qbuf + (size_t)qb * q_bytes + q_bytes / 2, head_mapQ, &ctl->q_full[qb], 64, 0, head_c2);
                            prev_kv = kv; ++qn;
                        }
                        if (!mbar_wait(&ctl->empty[st], ph ^ 1, ctl, status, kSleepLong)) { ok = false; break; }
                        mbar_expect_tx(&ctl->full[st], kStageBytes);
                        // window-inclusive mode: in pass 1 the last tile of a head is its window keys (rows past w read as
                        // zero); in pass 2 that tile lies past the prefix, reads as zero and its scores are never stored
                        const bool wt = P.wtile && pass == 1 && tt == tph - 1;
                        const CUtensorMap *map = wt ? &mapW : head_mapK;
                        const int j0 = wt ? 0 : tt * kTile;
                        if (JQ_IN(st, stages, kDbgScore, 2)) {
                            tma_load_3d(kbuf + (size_t)st * kStageBytes, map, &ctl->full[st], 0, j0, head_c2);
                            tma_load_3d(kbuf + (size_t)st * kStageBytes + kHalfBytes, map, &ctl->full[st], 64, j0, head_c2);
                        }
                        if (++st == (uint32_t)stages) { st = 0; ph ^= 1; }
                    }
                }
            }
        } else if (warp == 1) {
            // ---------------------------------------------------------------- MMA issuer (all 32 lanes walk the loop)
            const uint32_t idesc1 = instr_desc(128, kTile);
            // pass 2: a block's columns are the query rows it covers, rounded up to 32 (the rows past R are zero)
            const uint32_t idesc2a = instr_desc(kTile, min(128, Rpad)), idesc2b = instr_desc(kTile, max(32, Rpad - 128));
            uint32_t st = 0, ph = 0, qn = 0, u = 0;           // ring stage and phase, query loads, accumulator blocks so far
            Share share;
            int prev_kv = -1;
            bool ok = true;
#pragma unroll 1
            for (int s = 0; s < nseg && ok; ++s) {
                const Seg sg = segment(s, P, share);
                const int pass = sg.pass, ntiles = sg.ntiles, tph = sg.tph;
                int kv = sg.kv0, tt = sg.t0;
#pragma unroll 1
                for (int n = 0; n < ntiles && ok; ++n, walk(pass, tph, kv, tt)) {
                    if (kv != prev_kv) {
                        if (qn > 0) tc_commit(&ctl->q_empty[(qn - 1) & 1]);   // the previous head's queries are free once its MMAs retire
                        if (!mbar_wait(&ctl->q_full[qn & 1], (qn >> 1) & 1, ctl, status, kSleepShort)) { ok = false; break; }
                        prev_kv = kv; ++qn;
                    }
                    if (!mbar_wait(&ctl->full[st], ph, ctl, status, kSleepShort)) { ok = false; break; }
                    const uint32_t k_lo = desc_lo(smem_u32(kbuf) + st * kStageBytes);
                    const uint32_t q_lo = desc_lo(smem_u32(qbuf) + ((qn - 1) & 1) * q_bytes);
#pragma unroll 1
                    for (int blk = 0; blk < nblk; ++blk, ++u) {
                        const uint32_t slot = u % kTSlots;
                        if (!mbar_wait(&ctl->t_empty[slot], ((u / kTSlots) & 1) ^ 1, ctl, status, kSleepShort)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t d = tmem + slot * kSlotCols;
                        if (!JQ_IN(slot * kSlotCols + kSlotCols - 1, kTmemCols, kDbgScore, 3) || !JQ_IN(st, stages, kDbgScore, 4)) { ok = false; break; }
                        const uint32_t qb_lo = q_lo + (uint32_t)blk * (kHalfBytes >> 4);   // query rows [128 blk, 128 blk + 128)
                        if (pass == 1) tc_mma_block(d, qb_lo, k_lo, q_bytes / 2, kHalfBytes, idesc1);
                        else tc_mma_block(d, k_lo, qb_lo, kHalfBytes, q_bytes / 2, blk == 0 ? idesc2a : idesc2b);
                        tc_commit(&ctl->t_full[slot]);
                    }
                    if (ok) tc_commit(&ctl->empty[st]);
                    if (++st == (uint32_t)stages) { st = 0; ph ^= 1; }
                }
            }
        } else if (warp == 2) {
            // ---------------------------------------------------------------- grid-wide merge of the pass-1 partials
            // Group g: once every epilogue warp of every CTA has published its partials, this CTA combines its
            // share of the group's rows into M_r = c*m_r + log2(l_r), and counts itself in.
            const float c = P.c;
            const uint32_t Gu = (uint32_t)G;
#pragma unroll 1
            for (int g = 0; g < P.ngroups; ++g) {
                int ok = 1;
                // this CTA's epilogue warps first (their partial stores happen-before the arrival), then the grid
                ok = mbar_wait(&ctl->p1_done[g & 3], (g >> 2) & 1, ctl, P.status, kSleepLong) ? 1 : 0;
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                if (lane == 0) {
                    __threadfence();
                    atomicAdd(P.status + kWCnt1 + (g & (kRing - 1)), 1);
                    ok = wait_counter(P.status + kWCnt1 + (g & (kRing - 1)), (g / kRing + 1) * G, ctl, P.status) ? 1 : 0;
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                const GroupRec gr = group_of(g, P);
                const int h0 = gr.h0, nh = gr.nh, tph = gr.tph;
                const uint32_t T = (uint32_t)nh * tph;
                // This CTA's rows of the group are blockIdx.x + k G.  They are taken `rows_par` at a time, each by a
                // sub-group of 32 / rows_par lanes that splits the row's partial slots, kMergeLoads loads in flight per
                // lane (the merge is a chain of L2 round trips: the fewer, the sooner pass 2 of the group may start);
                // an empty partial (or one of a CTA that had no tile of the head) counts as (-inf, 0).
                const int nitems = nh * P.R;
                const int nrows = (nitems > (int)blockIdx.x) ? (nitems - 1 - (int)blockIdx.x) / G + 1 : 0;
                int rows_par = 1;
                while (rows_par < nrows && rows_par < 32) rows_par <<= 1;
                const int lpr = 32 / rows_par, sub = lane % lpr;
#pragma unroll 1
                for (int base = 0; base < nrows; base += rows_par) {
                    const int my = base + lane / lpr;
                    const bool have = my < nrows;
                    const int item = blockIdx.x + (have ? my : 0) * G;
                    const int hl = item / P.R, r = item - hl * P.R, kv = h0 + hl;
                    const uint32_t first = (uint32_t)hl * tph;
                    const int b_lo = owner_of_tile(first, T, Gu), b_hi = owner_of_tile(first + tph - 1, T, Gu);
                    const int nsl = have ? (b_hi - b_lo + 1) * kGroups : 0;   // every epilogue group of a contributing CTA wrote a partial
                    const float2 *src = P.part + ((size_t)kv * kSlots + kGroups * b_lo) * P.R + r;
                    float m = -INFINITY, l = 0.f;
#pragma unroll 1
                    for (int i0 = sub; i0 < nsl; i0 += lpr * kMergeLoads) {
                        float2 p[kMergeLoads];
#pragma unroll
                        for (int k = 0; k < kMergeLoads; ++k) {
                            const int i = i0 + lpr * k;
                            p[k] = make_float2(-INFINITY, 0.f);
                            // (a CTA between b_lo and b_hi always has a tile of this head unless the group has fewer tiles than CTAs)
                            if (i < nsl && (T >= Gu || cta_has_tile(b_lo + i / kGroups, T, Gu)))
                                if (JQ_IN(((long long)kv * kSlots + kGroups * b_lo + i) * P.R + r, n_part, kDbgScore, 5)) p[k] = __ldcg(src + (size_t)i * P.R);
                        }
                        float mn = m;
#pragma unroll
                        for (int k = 0; k < kMergeLoads; ++k) if (p[k].y > 0.f) mn = fmaxf(mn, p[k].x);
                        if (mn > -INFINITY) {
                            float acc = (l > 0.f) ? l * ex2(c * (m - mn)) : 0.f;
#pragma unroll
                            for (int k = 0; k < kMergeLoads; ++k) if (p[k].y > 0.f) acc += p[k].y * ex2(c * (p[k].x - mn));
                            m = mn; l = acc;
                        }
                    }
                    // butterfly over the sub-group (a fixed order, hence deterministic): first the common
                    // reference, then the sum against it
                    float mw = (l > 0.f) ? m : -INFINITY;
                    for (int o = lpr >> 1; o >= 1; o >>= 1) mw = fmaxf(mw, __shfl_xor_sync(0xffffffffu, mw, o));
                    l = (l > 0.f) ? l * ex2(c * (m - mw)) : 0.f;
                    for (int o = lpr >> 1; o >= 1; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
                    const float M = c * mw + log2f(l);
                    if (have && sub == 0 && JQ_IN((long long)kv * P.R + r, (long long)P.Hkv * P.R, kDbgScore, 6)) P.Mrow[(size_t)kv * P.R + r] = M;
                }
                __syncwarp();
                if (lane == 0) {
                    __threadfence();
                    atomicAdd(P.status + kWCnt2 + (g & (kRing - 1)), 1);
                }
            }
        } else {
            // ---------------------------------------------------------------- pass-2 stager
            // Walks the pass-2 segments in order.  Per segment: with two blocks per key, zeroes the scores of
            // this CTA's keys (the epilogue adds into them); waits until the group's normalisers are merged;
            // then feeds -M_r of each KV head of the segment into the double-buffered shared array.
            uint32_t hs = 0;
            int ok = 1;
            Share share;
#pragma unroll 1
            for (int s = 0; s < nseg && ok; ++s) {
                const Seg sg = segment(s, P, share);
                if (sg.pass != 2 || sg.ntiles == 0) continue;
                const int tph = sg.tph;
                if (nblk == 2) {
                    int kv = sg.kv0, tt = sg.t0;
                    for (int n = 0; n < sg.ntiles; ++n, walk(2, tph, kv, tt)) {
                        float *dst = P.scores + sg.sbase + (size_t)(kv - sg.h0) * sg.L + tt * kTile;
                        for (int t = lane; t < kTile && tt * kTile + t < sg.L; t += 32)
                            if (JQ_IN(sg.sbase + (long long)(kv - sg.h0) * sg.L + tt * kTile + t, n_scores, kDbgScore, 7)) dst[t] = 0.f;
                    }
                    __threadfence();
                }
                if (lane == 0)
                    ok = wait_counter(P.status + kWCnt2 + (sg.g & (kRing - 1)), (sg.g / kRing + 1) * G, ctl, P.status) ? 1 : 0;
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                int prev_kv = -1;
                int kv = sg.kv0, tt = sg.t0;
#pragma unroll 1
                for (int n = 0; n < sg.ntiles && ok; ++n, walk(2, tph, kv, tt)) {
                    if (kv == prev_kv) continue;
                    prev_kv = kv;
                    const uint32_t buf = hs & 1;
                    ok = mbar_wait(&ctl->ms_empty[buf], ((hs >> 1) & 1) ^ 1, ctl, status, kSleepLong) ? 1 : 0;
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    for (int r = lane; r < kMaxR; r += 32)   // stored negated: x = c s + (-M_r); -inf silences a padding column
                        ctl->Ms[buf][r] = (r < P.R && JQ_IN((long long)kv * P.R + r, (long long)P.Hkv * P.R, kDbgScore, 8)) ? -__ldcg(&P.Mrow[(size_t)kv * P.R + r]) : -INFINITY;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&ctl->ms_full[buf], 1);
                    ++hs;
                }
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue groups
        const int grp = (warp - kSpecialWarps) >> 2, quarter = warp & 3;
        const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16);
        const int row0 = quarter * 32 + lane;                   // TMEM lane: query row within its block (pass 1), key within its tile (pass 2)
        const int bs = nblk - 1;                                // blocks per tile is 1 or 2: shift and mask
        const float c = P.c, lazy = 64.f / c;
        const float2 cc = make_float2(c, c);
        float *const scores_out = P.scores;
        float2 *const part_out = P.part + (size_t)(kGroups * blockIdx.x + grp) * R;
        const int win_i0 = row0 % P.w, win_i1 = (row0 + 128) % P.w;   // soft-token index of this thread's row in block 0 / block 1
        const int np0 = min(128, Rpad) >> 5, np1 = (Rpad - 128) >> 5; // pass 2: 32-column pieces of a key's first / second block
        uint32_t u = 0;                                         // accumulator blocks of the CTA before this segment
        int hs = 0;                                             // pass-2 heads of the CTA before this segment
        bool ok = true;
        uint32_t va[16], vb[16];                                // the two alternating 16-column reads
        Share share;

        // Slot and parity of the CTA's accumulator block number uu; the block after this group's block uu is uu + kGroups.
        // Giving a slot back: the warp's reads of it are complete (tcgen05.wait::ld is warp-wide), one lane tells the MMA warp.
        auto release = [&](uint32_t slot) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&ctl->t_empty[slot], 1);
        };
        // One look whether block uu is complete; if so its first 16 columns are requested (into va).  Warp-uniform.
        // (With as many groups as slots a group's next block cannot be complete before the group gives its slot
        // back, so the look is not taken at all: it sits between the hand-over and the last exponentials of a block.)
        constexpr bool kLookAhead = kGroups < kTSlots;
        auto try_begin = [&](uint32_t uu) -> bool {
            const uint32_t slot = uu % kTSlots;
            if (!__all_sync(0xffffffffu, mbar_test(&ctl->t_full[slot], (uu / kTSlots) & 1))) return false;
            tc_fence_after();
            JQ_TMEM_LD16(lane_addr + slot * kSlotCols, va);
            return true;
        };
        auto begin = [&](uint32_t uu) -> bool {
            const uint32_t slot = uu % kTSlots;
            if (!mbar_wait(&ctl->t_full[slot], (uu / kTSlots) & 1, ctl, status, kSleepShort)) return false;
            tc_fence_after();
            JQ_TMEM_LD16(lane_addr + slot * kSlotCols, va);
            return true;
        };

#pragma unroll 1
        for (int s = 0; s < nseg && ok; ++s) {
            const Seg sg = segment(s, P, share);
            const int ntiles = sg.ntiles, nunits = ntiles << bs, tph = sg.tph, L = sg.L;
            int kv = sg.kv0, tt = sg.t0, at = 0;                // tile cursor: head, tile in head, index in the segment
            int k = (grp + kGroups - (int)(u % kGroups)) % kGroups;   // this group's first block of the segment
            bool pre = false;                                   // the first read of block k has already been requested
            if (sg.pass == 1) {
                // Per block of 128 query rows: running max m and l = sum_j exp2(c (s_j - m)).
                RowState st0 = {-INFINITY, make_float2(0.f, 0.f), make_float2(0.f, 0.f)}, st1 = st0;
                int pub = sg.kv0;                               // next head whose partials this warp has to publish
                // Every group publishes a partial for every head of the CTA's range, an empty one if it saw no block of it.
                auto publish_upto = [&](int head_end) {
#pragma unroll 1
                    for (; pub < head_end; ++pub) {
                        float2 *dst = part_out + (size_t)pub * kSlots * R;
                        const bool in_part = JQ_IN(((long long)pub * kSlots + kGroups * blockIdx.x + grp) * R + (R - 1), n_part, kDbgScore, 9);
                        if (row0 < R && in_part) dst[row0] = make_float2(st0.m, (st0.l01.x + st0.l01.y) + (st0.l23.x + st0.l23.y));
                        if (nblk == 2 && row0 + 128 < R && in_part)
                            dst[row0 + 128] = make_float2(st1.m, (st1.l01.x + st1.l01.y) + (st1.l23.x + st1.l23.y));
                        st0.m = st1.m = -INFINITY;
                        st0.l01 = st0.l23 = st1.l01 = st1.l23 = make_float2(0.f, 0.f);
                    }
                };
#pragma unroll 1
                for (; k < nunits; k += kGroups) {
                    const int tl = k >> bs, blk = k & bs;
                    tt += tl - at; at = tl;
                    while (tt >= tph) { tt -= tph; ++kv; }
                    if (kv != pub) publish_upto(kv);
                    const uint32_t uu = u + (uint32_t)k, slot = uu % kTSlots;
                    if (!pre && !begin(uu)) { ok = false; break; }
                    const uint32_t taddr = lane_addr + slot * kSlotCols;
                    if (!JQ_IN(slot * kSlotCols + kTile - 1, kTmemCols, kDbgScore, 10)) { ok = false; break; }
                    // keys of this block that count for this thread's row: the prefix keys of the tile, or, in the window
                    // tile, the window keys up to the row's own position (causal)
                    const int valid = (P.wtile && tt == tph - 1) ? min(P.w, (blk ? win_i1 : win_i0) + 1) : min(kTile, L - tt * kTile);
                    // one copy of the block code: the second row block borrows the first one's registers
                    if (blk == 1) { const RowState t = st0; st0 = st1; st1 = t; }
#pragma unroll 1
                    for (int c0 = 0; c0 < kTile; c0 += 32) {
                        JQ_TMEM_WAIT16(va);
                        JQ_TMEM_LD16(taddr + c0 + 16, vb);
                        p1_half(va, c0, valid, c, lazy, cc, st0);
                        JQ_TMEM_WAIT16(vb);
                        if (c0 + 32 < kTile) JQ_TMEM_LD16(taddr + c0 + 32, va);
                        else {
                            release(slot);
                            if (kLookAhead) pre = (k + kGroups < nunits) && try_begin(uu + kGroups);
                        }
                        p1_half(vb, c0 + 16, valid, c, lazy, cc, st0);
                    }
                    if (blk == 1) { const RowState t = st0; st0 = st1; st1 = t; }
                }
                if (ok && ntiles > 0) {
                    tt += ntiles - 1 - at;
                    while (tt >= tph) { tt -= tph; ++kv; }
                    publish_upto(kv + 1);
                }
                // this warp's share of pass 1 of the group is published: tell the merge warp, which makes the
                // stores visible to the grid and counts the CTA in (an epilogue warp does not wait for that)
                __syncwarp();
                if (lane == 0) mbar_arrive(&ctl->p1_done[sg.g & 3], 1);
            } else {
                // Heads of the segment are numbered hs, hs + 1, ... in walking order (descending KV head); the
                // stage warp fills buffer (number & 1).  `held` is the number of the head whose normalisers
                // this warp currently reads, hs - 1 before the first.
                int held = hs - 1;
                auto hold = [&](int want) {
#pragma unroll 1
                    while (held < want && ok) {
                        if (held >= hs) { __syncwarp(); if (lane == 0) mbar_arrive(&ctl->ms_empty[held & 1], 1); }
                        ++held;
                        ok = mbar_wait(&ctl->ms_full[held & 1], (held >> 1) & 1, ctl, status, kSleepShort);
                    }
                };
#pragma unroll 1
                for (; k < nunits; k += kGroups) {
                    const int tl = k >> bs, blk = k & bs;
                    tt -= tl - at; at = tl;
                    while (tt < 0) { tt += tph; --kv; }
                    hold(hs + (sg.kv0 - kv));
                    if (!ok) break;
                    const uint32_t uu = u + (uint32_t)k, slot = uu % kTSlots;
                    if (!pre && !begin(uu)) { ok = false; break; }
                    const uint32_t taddr = lane_addr + slot * kSlotCols;
                    const int np = blk ? np1 : np0;                     // 32-column pieces of this block
                    const float4 *bias = (const float4 *)(ctl->Ms[held & 1] + blk * 128);  // columns that are not query rows carry a bias of -inf
                    if (!JQ_IN(slot * kSlotCols + 32 * np - 1, kTmemCols, kDbgScore, 11) || !JQ_IN(blk * 128 + 32 * np - 1, kMaxR, kDbgScore, 12)) { ok = false; break; }
                    float2 a01 = make_float2(0.f, 0.f), a23 = make_float2(0.f, 0.f);
#pragma unroll 1
                    for (int p = 0; p < np; ++p) {
                        JQ_TMEM_WAIT16(va);
                        JQ_TMEM_LD16(taddr + 32 * p + 16, vb);
                        exp_acc16(a01, a23, va, cc, bias + 8 * p);
                        JQ_TMEM_WAIT16(vb);
                        if (p + 1 < np) JQ_TMEM_LD16(taddr + 32 * p + 32, va);
                        else {
                            release(slot);
                            if (kLookAhead) pre = (k + kGroups < nunits) && try_begin(uu + kGroups);
                        }
                        exp_acc16(a01, a23, vb, cc, bias + 8 * p + 4);
                    }
                    const int key = tt * kTile + row0;
                    if (key < L && JQ_IN(sg.sbase + (long long)(kv - sg.h0) * L + key, n_scores, kDbgScore, 13)) {
                        float *dst = scores_out + sg.sbase + (size_t)(kv - sg.h0) * L + key;
                        const float sum = (a01.x + a01.y) + (a23.x + a23.y);
                        if (nblk == 1) *dst = sum;
                        else atomicAdd(dst, sum);              // two blocks per key, onto a zero the stage warp wrote
                    }
                }
                // take part in the hand-over of every remaining head of the segment, then give the last one back
                if (ntiles > 0) {
                    tt -= ntiles - 1 - at;
                    while (tt < 0) { tt += tph; --kv; }
                    const int nheads = sg.kv0 - kv + 1;
                    hold(hs + nheads - 1);
                    if (ok) { __syncwarp(); if (lane == 0) mbar_arrive(&ctl->ms_empty[held & 1], 1); }
                    hs += nheads;
                }
            }
            u += (uint32_t)nunits;
        }
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");   // (a read requested ahead on a path that gave up)
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

// bf16 tensor [heads][head_rows][128] of which the first `rows` rows of every head are data, viewed as 3-D
// (128, rows, heads); box = 64 columns x box_rows rows of one head, 128-byte swizzle; rows past `rows` read
// as zero.  A tensor map is a pure function of these
// arguments, so the last few are kept per host thread: a caller that evicts layer after layer (or the same
// cache again) pays for the driver's encoding once per buffer, not on every call.
bool make_map(CUtensorMap *map, const void *ptr, int rows, int heads, int box_rows, int head_rows = 0)
{
    if (head_rows < rows) head_rows = rows;
    struct Entry { const void *ptr; int rows, heads, box_rows, head_rows; bool valid; CUtensorMap map; };
    constexpr int kEntries = 1024;                      // direct-mapped
    static thread_local Entry cache[kEntries] = {};
    const uint64_t h = ((uint64_t)(uintptr_t)ptr >> 8) * 0x9E3779B97F4A7C15ull + (uint64_t)rows * 0xC2B2AE3D27D4EB4Full + (uint64_t)head_rows * 0x165667B19E3779F9ull + (uint64_t)(heads * 4 + box_rows / 128);
    Entry &e = cache[(h >> 40) % kEntries];
    if (e.valid && e.ptr == ptr && e.rows == rows && e.heads == heads && e.box_rows == box_rows && e.head_rows == head_rows) { *map = e.map; return true; }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {(cuuint64_t)kD, (cuuint64_t)rows, (cuuint64_t)heads};
    cuuint64_t strides[2] = {(cuuint64_t)kD * 2, (cuuint64_t)head_rows * kD * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    if (fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(ptr), dims, strides, box, estr,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    e.ptr = ptr; e.rows = rows; e.heads = heads; e.box_rows = box_rows; e.head_rows = head_rows; e.map = *map; e.valid = true;
    return true;
}

constexpr size_t smem_bytes(int Rbox, int stages)
{
    return 2 * (size_t)Rbox * kD * 2 + (size_t)stages * kStageBytes + kCtlBytes;
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
        if (cudaFuncSetAttribute(score_fused<kGroupsNarrow>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return false;
        if (cudaFuncSetAttribute(score_fused<kGroupsWide>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return false;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, score_fused<kGroupsNarrow>, threads_for(kGroupsNarrow), smem) != cudaSuccess || per_sm < 1)
            return false;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, score_fused<kGroupsWide>, threads_for(kGroupsWide), smem) != cudaSuccess || per_sm < 1)
            return false;
        d.sms = sms;
        d.l2 = l2;
        d.ready = true;
    }
    *out = d;
    return true;
}

}  // namespace

bool make_tensor_map(void *map, const void *ptr, int rows, int heads, int box_rows)
{
    static_assert(sizeof(CUtensorMap) == kTensorMapBytes, "tensor map size");
    return make_map((CUtensorMap *)map, ptr, rows, heads, box_rows);
}

int score_sms()
{
    DeviceInfo dev;
    return device_info(&dev) ? dev.sms : 0;
}

// KV heads are scored in groups whose keys fit in a share of the L2 (32 MiB), so that pass 2 finds them there.
// Among the admissible group sizes, the one that wastes the fewest CTA-tile slots.
int heads_per_group(int L, int heads, int tiles_per_head, int sms)
{
    const long long head_bytes = (long long)L * kD * 2;
    long long hmax = (32ll << 20) / head_bytes;
    if (hmax < 1) hmax = 1;
    if (hmax > heads) hmax = heads;
    int best_hpg = 1;
    double best_eff = -1.0;
    for (int hpg = 1; hpg <= (int)hmax; ++hpg) {
        long long work = 0, slots = 0;
        for (int h0 = 0; h0 < heads; h0 += hpg) {
            const long long T = (long long)(h0 + hpg <= heads ? hpg : heads - h0) * tiles_per_head;
            work += T;
            slots += (T + sms - 1) / sms;
        }
        const double eff = (double)work / ((double)slots * sms);
        if (eff >= best_eff - 1e-9) { best_eff = eff > best_eff ? eff : best_eff; best_hpg = hpg; }
        if (hmax > 64 && hpg >= 64) break;   // the scan is only worth it over a small range
    }
    return best_hpg;
}

jq_status launch_score_tc(const void *K, const void *Q, const jq_shape &s, float *scores, const Workspace &w,
                          cudaStream_t st, const void *Kwin, const UnitTables *tables, int k_head_rows)
{
    DeviceInfo dev;
    if (!device_info(&dev)) return JQ_ERR_CUDA;
    const int R = s.group * s.w;
    Params P;
    P.R = R; P.Rbox = R <= 128 ? 128 : 256; P.Rpad = (R + 31) & ~31;
    P.Hkv = s.Hkv;
    P.wtile = Kwin ? 1 : 0;
    P.stages = P.Rbox == 128 ? 5 : 3;
    P.depth = 2;
    P.c = 1.4426950408889634f / sqrtf((float)s.d);
    P.part = w.part; P.Mrow = w.Mrow; P.scores = scores; P.status = w.status;
    P.w = s.w;
    const int groups = R > 128 ? kGroupsWide : kGroupsNarrow;
    int sms = dev.sms;
    if (groups * sms > kSlots) sms = kSlots / groups;
    CUtensorMap mapK, mapQ, mapW;
    long long tmax;
    if (tables) {
        // every unit has tensor maps of its own in device memory; the three parameter maps are not used
        memset(&mapK, 0, sizeof mapK); mapQ = mapK; mapW = mapK;
        P.L = 0; P.tph = 0; P.hpg = 0;
        P.gtab = tables->groups; P.maps = (const CUtensorMap *)tables->maps; P.hpu = tables->hpu;
        P.ngroups = tables->ngroups;
        tmax = tables->max_group_tiles;
    } else {
        P.L = s.L;
        P.tph = (s.L + kTile - 1) / kTile + P.wtile;
        P.gtab = nullptr; P.maps = nullptr; P.hpu = s.Hkv;
        if (!make_map(&mapK, K, s.L, s.Hkv, kTile, k_head_rows) || !make_map(&mapQ, Q, R, s.Hkv, P.Rbox)) return JQ_ERR_CUDA;
        if (Kwin) { if (!make_map(&mapW, Kwin, s.w, s.Hkv, kTile)) return JQ_ERR_CUDA; } else mapW = mapK;
        P.hpg = heads_per_group(s.L, s.Hkv, P.tph, sms);
        P.ngroups = (s.Hkv + P.hpg - 1) / P.hpg;
        tmax = (long long)(P.hpg < s.Hkv ? P.hpg : s.Hkv) * P.tph;
    }
    const int grid = (int)(tmax < sms ? tmax : sms);
    P.grid_magic = div_magic((uint32_t)grid);
    P.tph_magic = tables ? 0u : div_magic((uint32_t)P.tph);
#ifdef JQ_DEBUG
    P.dbg_rec = debug_record();
    P.n_scores = tables ? tables->total_keys : (long long)s.Hkv * s.L;
    if (!P.dbg_rec) return JQ_ERR_CUDA;
#endif

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)threads_for(groups));
    cfg.dynamicSmemBytes = smem_bytes(P.Rbox, P.stages);
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    // the CTAs may be set up (barriers, tensor-memory allocation) while the previous kernel of the stream drains
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    const cudaError_t err = groups == kGroupsWide ? cudaLaunchKernelEx(&cfg, score_fused<kGroupsWide>, mapK, mapQ, mapW, P)
                                                  : cudaLaunchKernelEx(&cfg, score_fused<kGroupsNarrow>, mapK, mapQ, mapW, P);
    if (err != cudaSuccess) {
        cudaGetLastError();
        return JQ_ERR_CUDA;
    }
    count_launch(1);
    return check_launch();
}

}  // namespace jq
