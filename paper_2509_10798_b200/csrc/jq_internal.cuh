// Internal declarations shared by the translation units of libjq (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "jq.h"

namespace jq {

constexpr int kD = 128;          // head dimension the kernels are built for
constexpr int kMaxR = 256;       // query rows per KV head (group * w)
constexpr int kSlots = 640;      // partial (reference, sum-exp) slots per KV head in the workspace (up to 4 per CTA)
constexpr int kStatusWords = 64; // first 256 bytes of the workspace

// Device status word values (sticky since jq_workspace_init): 0 ok, else a jq_status.
struct Workspace {
    int *status;        // [kStatusWords]
    float *Mrow;        // [Hkv][R]   log2-domain normaliser per query row: c*max + log2(sumexp)
    float2 *part;       // [Hkv][kSlots][R]   (raw max, sum of exp2(c*(s-max))) per contributing block
    float *scores;      // [Hkv][L]   pre-pool scores (jq_evict_layer keeps them here)
    uint32_t *keys;     // [Hkv][L]   order-preserving bit patterns of the pooled scores
    uint32_t *sel;      // select scratch
    size_t bytes;       // total
};

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Select scratch per KV head, in 32-bit words: histograms and counters (see jq_select.cu).
constexpr int kSelWordsPerHead = 4096 + 64;

static inline Workspace carve(void *base, const jq_shape &s)
{
    Workspace w;
    const size_t R = (size_t)s.group * s.w;
    char *p = (char *)base;
    size_t off = 0;
    w.status = (int *)(p + off);
    off += align_up(kStatusWords * sizeof(int), 256);
    w.Mrow = (float *)(p + off);
    off += align_up((size_t)s.Hkv * R * sizeof(float), 256);
    w.part = (float2 *)(p + off);
    off += align_up((size_t)s.Hkv * kSlots * R * sizeof(float2), 256);
    w.scores = (float *)(p + off);
    off += align_up((size_t)s.Hkv * s.L * sizeof(float), 256);
    w.keys = (uint32_t *)(p + off);
    off += align_up((size_t)s.Hkv * s.L * sizeof(uint32_t), 256);
    w.sel = (uint32_t *)(p + off);
    off += align_up((size_t)s.Hkv * kSelWordsPerHead * sizeof(uint32_t), 256);
    w.bytes = off;
    return w;
}

// Layers of equal shape living in buffers of their own (jq_evict_layers): tables in device memory, behind the
// workspace proper.  KV head kv of the stacked numbering belongs to layer kv / hpl and is head kv % hpl of it.
constexpr int kMaxLayers = 128;
constexpr size_t kTensorMapBytes = 128;
struct LayerTables {
    const void *maps = nullptr;          // device: [nlayers][2] TMA tensor maps (K, Qwin)
    const void *const *K = nullptr;      // device: [nlayers] base of K
    const void *const *V = nullptr;      // device: [nlayers] base of V
    int hpl = 0;                         // KV heads per layer (0: no tables, one buffer)
};
static inline size_t layer_tables_bytes(int nlayers)
{
    return align_up((size_t)nlayers * 2 * kTensorMapBytes, 256) + 2 * align_up((size_t)nlayers * sizeof(void *), 256);
}
// Fills host_maps ([nlayers][2] tensor maps) for K[l] [hpl][L][128] and Qwin[l] [hpl][R][128].
bool build_layer_maps(const void *const *K, const void *const *Qwin, int nlayers, const jq_shape &layer, void *host_maps);

// Host-side bookkeeping.
void count_launch(int n = 1);
jq_status check_launch();   // cudaGetLastError -> JQ_OK / JQ_ERR_CUDA

// Stage launchers (arguments already validated).
jq_status launch_score_fma(const void *K, const void *Q, const jq_shape &s, float *scores,
                           const Workspace &w, cudaStream_t st);
// Kwin, when not null: keys [Hkv][w][128] of the query positions themselves (window-inclusive softmax).
// With tables (s is then the stacked shape, K and Q those of the first layer) the tiles come from the layers' own buffers.
jq_status launch_score_tc(const void *K, const void *Q, const jq_shape &s, float *scores,
                          const Workspace &w, cudaStream_t st, const void *Kwin = nullptr,
                          const LayerTables *tables = nullptr);
// With K, V, Kout, Vout given, the kernel also copies the kept rows (the fused layer path).
jq_status launch_select(const float *scores, const jq_shape &s, int32_t *idx, float *pooled,
                        const Workspace &w, cudaStream_t st, const void *K = nullptr, const void *V = nullptr,
                        void *Kout = nullptr, void *Vout = nullptr, const LayerTables *tables = nullptr);
jq_status launch_gather(const void *K, const void *V, const int32_t *idx, const jq_shape &s,
                        void *Kout, void *Vout, cudaStream_t st);

}  // namespace jq
