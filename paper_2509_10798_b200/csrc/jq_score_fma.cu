// CUDA-core (fp32 FMA) scoring: the comparator the tensor-core path is profiled against.
//
// Eq. 3 in two streaming passes over K:
//   pass 1  one thread per query row; K tiles staged in shared memory and read as broadcasts;
//           each thread keeps the running max m and sum l = sum_j exp2(c*(s_j - m)) of its row;
//   merge   partial (m, l) of the key chunks combined in chunk order -> M_r = c*m + log2(l);
//   pass 2  one thread per key; the R query rows staged in shared memory and read as broadcasts;
//           score_j = sum_r exp2(c*s_rj - M_r),  c = log2(e)/sqrt(d).
#include "jq_internal.cuh"
#include <cuda_bf16.h>

namespace jq {
namespace {

constexpr int kTileKeys = 32;

__device__ __forceinline__ float bf16lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// grid (nslot, Hkv); block = R rounded up to a warp multiple.
__global__ void __launch_bounds__(256)
score_fma_pass1(const uint16_t *__restrict__ K, const uint16_t *__restrict__ Q, int L, int R,
                int nslot, float c, float2 *__restrict__ part)
{
    __shared__ uint4 ktile[kTileKeys * (kD / 8)];
    const int kv = blockIdx.y, slot = blockIdx.x, r = threadIdx.x;
    const int ntile = (L + kTileKeys - 1) / kTileKeys;
    const int t0 = (int)((long long)slot * ntile / nslot), t1 = (int)((long long)(slot + 1) * ntile / nslot);

    float q[kD];
    if (r < R) {
        const uint4 *qrow = (const uint4 *)(Q + ((size_t)kv * R + r) * kD);
#pragma unroll
        for (int v = 0; v < kD / 8; ++v) {
            uint4 u = qrow[v];
            q[8 * v + 0] = bf16lo(u.x); q[8 * v + 1] = bf16hi(u.x);
            q[8 * v + 2] = bf16lo(u.y); q[8 * v + 3] = bf16hi(u.y);
            q[8 * v + 4] = bf16lo(u.z); q[8 * v + 5] = bf16hi(u.z);
            q[8 * v + 6] = bf16lo(u.w); q[8 * v + 7] = bf16hi(u.w);
        }
    }
    float m = -INFINITY, l = 0.f;
    const uint4 *Kh = (const uint4 *)(K + (size_t)kv * L * kD);
    for (int t = t0; t < t1; ++t) {
        const int j0 = t * kTileKeys;
        const int nk = min(kTileKeys, L - j0);
        __syncthreads();
        for (int v = threadIdx.x; v < nk * (kD / 8); v += blockDim.x) ktile[v] = Kh[(size_t)j0 * (kD / 8) + v];
        __syncthreads();
        if (r < R) {
            for (int j = 0; j < nk; ++j) {
                float s = 0.f;
#pragma unroll
                for (int v = 0; v < kD / 8; ++v) {
                    uint4 u = ktile[j * (kD / 8) + v];
                    s = fmaf(q[8 * v + 0], bf16lo(u.x), s); s = fmaf(q[8 * v + 1], bf16hi(u.x), s);
                    s = fmaf(q[8 * v + 2], bf16lo(u.y), s); s = fmaf(q[8 * v + 3], bf16hi(u.y), s);
                    s = fmaf(q[8 * v + 4], bf16lo(u.z), s); s = fmaf(q[8 * v + 5], bf16hi(u.z), s);
                    s = fmaf(q[8 * v + 6], bf16lo(u.w), s); s = fmaf(q[8 * v + 7], bf16hi(u.w), s);
                }
                if (s > m) {
                    l *= exp2f(c * (m - s));
                    m = s;
                }
                l += exp2f(c * (s - m));
            }
        }
    }
    if (r < R) part[((size_t)kv * kSlots + slot) * R + r] = make_float2(m, l);
}

// grid (ceil(L/128), Hkv); block 128; dynamic shared memory R*256 + R*4 bytes.
__global__ void __launch_bounds__(128)
score_fma_pass2(const uint16_t *__restrict__ K, const uint16_t *__restrict__ Q, int L, int R,
                float c, const float *__restrict__ Mrow, float *__restrict__ scores)
{
    extern __shared__ uint4 smem[];
    uint4 *qs = smem;                                  // [R][16]
    float *Ms = (float *)(smem + (size_t)R * (kD / 8)); // [R]
    const int kv = blockIdx.y;
    const uint4 *Qh = (const uint4 *)(Q + (size_t)kv * R * kD);
    for (int v = threadIdx.x; v < R * (kD / 8); v += blockDim.x) qs[v] = Qh[v];
    for (int v = threadIdx.x; v < R; v += blockDim.x) Ms[v] = Mrow[(size_t)kv * R + v];
    __syncthreads();
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= L) return;
    float k[kD];
    const uint4 *krow = (const uint4 *)(K + ((size_t)kv * L + j) * kD);
#pragma unroll
    for (int v = 0; v < kD / 8; ++v) {
        uint4 u = krow[v];
        k[8 * v + 0] = bf16lo(u.x); k[8 * v + 1] = bf16hi(u.x);
        k[8 * v + 2] = bf16lo(u.y); k[8 * v + 3] = bf16hi(u.y);
        k[8 * v + 4] = bf16lo(u.z); k[8 * v + 5] = bf16hi(u.z);
        k[8 * v + 6] = bf16lo(u.w); k[8 * v + 7] = bf16hi(u.w);
    }
    float acc = 0.f;
    for (int r = 0; r < R; ++r) {
        float s = 0.f;
#pragma unroll
        for (int v = 0; v < kD / 8; ++v) {
            uint4 u = qs[r * (kD / 8) + v];
            s = fmaf(k[8 * v + 0], bf16lo(u.x), s); s = fmaf(k[8 * v + 1], bf16hi(u.x), s);
            s = fmaf(k[8 * v + 2], bf16lo(u.y), s); s = fmaf(k[8 * v + 3], bf16hi(u.y), s);
            s = fmaf(k[8 * v + 4], bf16lo(u.z), s); s = fmaf(k[8 * v + 5], bf16hi(u.z), s);
            s = fmaf(k[8 * v + 6], bf16lo(u.w), s); s = fmaf(k[8 * v + 7], bf16hi(u.w), s);
        }
        acc += exp2f(fmaf(c, s, -Ms[r]));
    }
    scores[(size_t)kv * L + j] = acc;
}

}  // namespace

// Combine the partial (m, l) pairs of slots [0, nslot) of every head, in slot order.
// grid (Hkv); block >= R threads.
__global__ void merge_partials_uniform(const float2 *__restrict__ part, int R, int nslot, float c,
                                       float *__restrict__ Mrow)
{
    const int kv = blockIdx.x;
    for (int r = threadIdx.x; r < R; r += blockDim.x) {
        float m = -INFINITY, l = 0.f;
        for (int s = 0; s < nslot; ++s) {
            float2 p = part[((size_t)kv * kSlots + s) * R + r];
            if (p.y > 0.f) {
                float mn = fmaxf(m, p.x);
                l = l * exp2f(c * (m - mn)) + p.y * exp2f(c * (p.x - mn));
                m = mn;
            }
        }
        Mrow[(size_t)kv * R + r] = c * m + log2f(l);
    }
}

jq_status launch_score_fma(const void *K, const void *Q, const jq_shape &s, float *scores,
                           const Workspace &w, cudaStream_t st)
{
    const int R = s.group * s.w;
    const float c = 1.4426950408889634f / sqrtf((float)s.d);
    const int ntile = (s.L + kTileKeys - 1) / kTileKeys;
    const int nslot = ntile < kSlots ? ntile : kSlots;
    const int threads = (R + 31) / 32 * 32;
    score_fma_pass1<<<dim3(nslot, s.Hkv), threads, 0, st>>>((const uint16_t *)K, (const uint16_t *)Q,
                                                            s.L, R, nslot, c, w.part);
    merge_partials_uniform<<<s.Hkv, 256, 0, st>>>(w.part, R, nslot, c, w.Mrow);
    const size_t smem = (size_t)R * kD * 2 + (size_t)R * 4;
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(score_fma_pass2, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kMaxR * kD * 2 + kMaxR * 4) != cudaSuccess)
            return JQ_ERR_CUDA;
        attr_set = true;
    }
    score_fma_pass2<<<dim3((s.L + 127) / 128, s.Hkv), 128, smem, st>>>(
        (const uint16_t *)K, (const uint16_t *)Q, s.L, R, c, w.Mrow, scores);
    count_launch(3);
    return check_launch();
}

}  // namespace jq
