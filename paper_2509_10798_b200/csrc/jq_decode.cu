// One decoding step over the pruned cache (the step after the eviction pass: decoding continues with the
// retained pairs only).  Single-position GQA attention, out[h] = softmax_j(q[h] . Kc[kv,j] / sqrt(d)) Vc[kv],
// split over the keys:
//   one CTA per (chunk of 64 keys, KV head) stages the chunk's K and V rows in shared memory with coalesced
//   16-byte loads, computes the logits of every query head of the group, their chunk-local softmax statistics
//   (m, l) and the unnormalised weighted sum of the V rows, and writes them to the workspace; the CTA that
//   finishes last for a KV head (a ticket counter per head, zeroed by the call) merges the chunks' (m, l, o)
//   of the head's query heads by the usual rescaling, in chunk order, so the result does not depend on which
//   CTA that is.
// The work is a single read of the two compacted arrays (2 * Hkv * n * 256 bytes): bound by HBM/L2 latency at
// these sizes, no tensor cores (a matrix-vector product per head).
#include <cuda_bf16.h>

#include "jq_internal.cuh"
#include "jq_debug.cuh"

namespace jq {
namespace {

constexpr int kDecChunk = 64;       // keys per CTA
constexpr int kDecThreads = 256;
constexpr int kDecMaxGroup = 8;     // query heads per KV head
constexpr int kKRow = kD + 8;       // padded K row in shared memory (bf16 elements): 272 bytes, conflict-free 16-byte reads
constexpr int kPartial = kD + 2;    // floats per (chunk, head): m, l, o[128]

__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

__global__ void __launch_bounds__(kDecThreads)
decode_step(const uint4 *__restrict__ Kc, const uint4 *__restrict__ Vc, const __nv_bfloat16 *__restrict__ q, int n,
            int group, float scale_log2, float *__restrict__ part, unsigned int *__restrict__ tickets, float *__restrict__ out JQ_DBG_PARAM)
{
    __shared__ int is_last;
    __shared__ __align__(16) __nv_bfloat16 Ks[kDecChunk * kKRow];
    __shared__ __align__(16) __nv_bfloat16 Vs[kDecChunk * kD];
    __shared__ float qs[kDecMaxGroup * kD];
    __shared__ float ps[kDecMaxGroup * kDecChunk];
    const int tid = threadIdx.x, split = blockIdx.x, kv = blockIdx.y, nsplit = gridDim.x;
    const int j0 = split * kDecChunk, valid = min(kDecChunk, n - j0);

    const long long n_rows = (long long)gridDim.y * n, n_part = (long long)gridDim.y * nsplit * group * kPartial;   // extents, for the bounds-checked build
    (void)n_rows; (void)n_part;
    for (int i = tid; i < group * kD; i += kDecThreads)
        if (JQ_IN(i, kDecMaxGroup * kD, kDbgDecode, 1)) qs[i] = __bfloat162float(q[(size_t)kv * group * kD + i]);
    for (int i = tid; i < kDecChunk * 16; i += kDecThreads) {       // 16 x 16 bytes per row
        const int r = i >> 4, c = i & 15;
        uint4 k4 = make_uint4(0u, 0u, 0u, 0u), v4 = k4;
        if (r < valid && JQ_IN((long long)kv * n + j0 + r, n_rows, kDbgDecode, 2)) {
            k4 = Kc[((size_t)kv * n + j0 + r) * 16 + c];
            v4 = Vc[((size_t)kv * n + j0 + r) * 16 + c];
        }
        if (JQ_IN(r * kKRow + c * 8 + 7, kDecChunk * kKRow, kDbgDecode, 3)) *(uint4 *)(Ks + r * kKRow + c * 8) = k4;
        if (JQ_IN(r * kD + c * 8 + 7, kDecChunk * kD, kDbgDecode, 4)) *(uint4 *)(Vs + r * kD + c * 8) = v4;
    }
    __syncthreads();

    // logits (times log2 e / sqrt(d)): thread = (key, head slot)
    {
        const int j = tid & (kDecChunk - 1);
        for (int h = tid >> 6; h < group; h += kDecThreads / kDecChunk) {
            const float *qh = qs + h * kD;
            float acc = 0.f;
#pragma unroll
            for (int c = 0; c < 16; ++c) {
                const uint4 k4 = *(const uint4 *)(Ks + j * kKRow + c * 8);
                acc = fmaf(bf16_lo(k4.x), qh[c * 8 + 0], acc); acc = fmaf(bf16_hi(k4.x), qh[c * 8 + 1], acc);
                acc = fmaf(bf16_lo(k4.y), qh[c * 8 + 2], acc); acc = fmaf(bf16_hi(k4.y), qh[c * 8 + 3], acc);
                acc = fmaf(bf16_lo(k4.z), qh[c * 8 + 4], acc); acc = fmaf(bf16_hi(k4.z), qh[c * 8 + 5], acc);
                acc = fmaf(bf16_lo(k4.w), qh[c * 8 + 6], acc); acc = fmaf(bf16_hi(k4.w), qh[c * 8 + 7], acc);
            }
            if (JQ_IN(h * kDecChunk + j, kDecMaxGroup * kDecChunk, kDbgDecode, 5)) ps[h * kDecChunk + j] = (j < valid) ? acc * scale_log2 : -INFINITY;
        }
    }
    __syncthreads();

    // chunk-local softmax statistics: warp h takes head h
    {
        const int h = tid >> 5, lane = tid & 31;
        if (h < group) {
            const float a = ps[h * kDecChunk + lane], b = ps[h * kDecChunk + lane + 32];
            float m = fmaxf(a, b);
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
            const float pa = exp2f(a - m), pb = exp2f(b - m);       // the chunk holds at least one key: m is finite
            float l = pa + pb;
#pragma unroll
            for (int o = 16; o >= 1; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
            ps[h * kDecChunk + lane] = pa;
            ps[h * kDecChunk + lane + 32] = pb;
            if (lane == 0) {
                float *dst = part + ((size_t)(kv * nsplit + split) * group + h) * kPartial;
                if (JQ_IN(((long long)(kv * nsplit + split) * group + h) * kPartial + 1, n_part, kDbgDecode, 6)) { dst[0] = m; dst[1] = l; }
            }
        }
    }
    __syncthreads();

    // unnormalised output: thread = (pair of columns, head slot)
    {
        const int cp = tid & 63;
        for (int h = tid >> 6; h < group; h += kDecThreads / 64) {
            const float *ph = ps + h * kDecChunk;
            float o0 = 0.f, o1 = 0.f;
#pragma unroll 8
            for (int j = 0; j < kDecChunk; ++j) {
                const uint32_t v2 = *(const uint32_t *)(Vs + j * kD + 2 * cp);
                o0 = fmaf(ph[j], bf16_lo(v2), o0);
                o1 = fmaf(ph[j], bf16_hi(v2), o1);
            }
            float *dst = part + ((size_t)(kv * nsplit + split) * group + h) * kPartial + 2;
            if (JQ_IN(((long long)(kv * nsplit + split) * group + h) * kPartial + 2 + 2 * cp + 1, n_part, kDbgDecode, 7))
                *(float2 *)(dst + 2 * cp) = make_float2(o0, o1);
        }
    }

    // the last CTA of the head to get here merges all chunks (release/acquire through the ticket)
    __threadfence();
    __syncthreads();
    if (tid == 0) is_last = (atomicAdd(&tickets[kv], 1u) == (unsigned)nsplit - 1u);
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    for (int item = tid; item < group * kD; item += kDecThreads) {
        const int h = item / kD, c = item - h * kD;
        // the head's maximum first, then plain sums in chunk order: no value depends on the previous load
        const float *base = part + ((size_t)kv * nsplit * group + h) * kPartial;
        const size_t step = (size_t)group * kPartial;
        float M = -INFINITY;
#pragma unroll 8
        for (int sp = 0; sp < nsplit; ++sp) M = fmaxf(M, __ldcg(base + sp * step));
        float Lsum = 0.f, O = 0.f;
#pragma unroll 8
        for (int sp = 0; sp < nsplit; ++sp) {
            const float *src = base + sp * step;
            const float f = exp2f(__ldcg(src) - M);
            Lsum = fmaf(__ldcg(src + 1), f, Lsum);
            O = fmaf(__ldcg(src + 2 + c), f, O);
        }
        if (JQ_IN(((long long)kv * group + h) * kD + c, (long long)gridDim.y * group * kD, kDbgDecode, 8) &&
            JQ_IN(((long long)kv * nsplit * group + h) * kPartial + (long long)(nsplit - 1) * step + 2 + c, n_part, kDbgDecode, 9))
            out[((size_t)kv * group + h) * kD + c] = O / Lsum;
    }
}

}  // namespace
}  // namespace jq

extern "C" size_t jq_decode_workspace_bytes(int Hkv, int Hq, int n)
{
    if (Hkv < 1 || Hq < 1 || Hq % Hkv || Hq / Hkv > jq::kDecMaxGroup || n < 1) return 0;
    const size_t nsplit = ((size_t)n + jq::kDecChunk - 1) / jq::kDecChunk;
    return jq::align_up((size_t)Hq * nsplit * jq::kPartial * sizeof(float), 256) + jq::align_up((size_t)Hkv * sizeof(unsigned int), 256);
}

extern "C" jq_status jq_decode_attention(const void *Kc, const void *Vc, const void *q, int Hkv, int Hq, int n, float *out,
                                         void *workspace, size_t workspace_bytes, jq_stream_t stream)
{
    if (!Kc || !Vc || !q || !out || Hkv < 1 || Hq < 1 || n < 1 || Hq % Hkv) return JQ_ERR_INVALID_ARG;
    if (((uintptr_t)Kc | (uintptr_t)Vc | (uintptr_t)out | (uintptr_t)workspace) & 15u) return JQ_ERR_INVALID_ARG;
    if (((uintptr_t)q) & 1u) return JQ_ERR_INVALID_ARG;
    const int group = Hq / Hkv;
    if (group > jq::kDecMaxGroup || Hkv > 65535) return JQ_ERR_UNSUPPORTED;
    const size_t need = jq_decode_workspace_bytes(Hkv, Hq, n);
    if (!workspace || workspace_bytes < need) return JQ_ERR_WORKSPACE;
    const int nsplit = (n + jq::kDecChunk - 1) / jq::kDecChunk;
    cudaStream_t st = (cudaStream_t)stream;
    const float scale_log2 = 1.4426950408889634f / sqrtf((float)jq::kD);
    unsigned int *tickets = (unsigned int *)((char *)workspace + jq::align_up((size_t)Hq * nsplit * jq::kPartial * sizeof(float), 256));
    if (cudaMemsetAsync(tickets, 0, (size_t)Hkv * sizeof(unsigned int), st) != cudaSuccess) return JQ_ERR_CUDA;
    jq::decode_step<<<dim3((unsigned)nsplit, (unsigned)Hkv), jq::kDecThreads, 0, st>>>(
        (const uint4 *)Kc, (const uint4 *)Vc, (const __nv_bfloat16 *)q, n, group, scale_log2, (float *)workspace, tickets, out JQ_DBG_ARG);
    jq::count_launch(1);
    return jq::check_launch();
}
