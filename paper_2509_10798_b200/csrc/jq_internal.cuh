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

// Carve-up of a workspace for `heads` KV heads with R query rows each and `keys` prefix positions in total
// (heads x L for one shape; the sum over the units of a ragged call).
static inline Workspace carve(void *base, size_t heads, size_t R, size_t keys)
{
    Workspace w;
    char *p = (char *)base;
    size_t off = 0;
    w.status = (int *)(p + off);
    off += align_up(kStatusWords * sizeof(int), 256);
    w.Mrow = (float *)(p + off);
    off += align_up(heads * R * sizeof(float), 256);
    w.part = (float2 *)(p + off);
    off += align_up(heads * kSlots * R * sizeof(float2), 256);
    w.scores = (float *)(p + off);
    off += align_up(keys * sizeof(float), 256);
    w.keys = (uint32_t *)(p + off);
    off += align_up(keys * sizeof(uint32_t), 256);
    w.sel = (uint32_t *)(p + off);
    off += align_up(heads * kSelWordsPerHead * sizeof(uint32_t), 256);
    w.bytes = off;
    return w;
}
static inline Workspace carve(void *base, const jq_shape &s)
{
    return carve(base, (size_t)s.Hkv, (size_t)s.group * s.w, (size_t)s.Hkv * s.L);
}

// Units (layers, sequences) of one head geometry living in buffers of their own, with prefix lengths and
// budgets of their own (jq_evict_ragged, jq_evict_layers): tables in device memory, behind the workspace proper.
// KV heads are numbered through all units; unit u owns heads [u * hpu, (u + 1) * hpu).
constexpr int kMaxUnits = 4096;
constexpr size_t kTensorMapBytes = 128;
// A head group of the scoring kernel: consecutive KV heads of one prefix length whose keys fit a share of the
// L2.  A group may run over consecutive units of equal length (their scores are consecutive too).
struct GroupRec {
    int h0, nh;          // first KV head (global numbering) and number of heads
    int tph, L;          // tiles per head, prefix length
    int unit, c20;       // the unit of head h0, and the index of head h0 within it
    long long sbase;     // offset (floats) of head h0's scores in the scores array
    uint32_t tph_magic;  // div_magic(tph): the kernel divides tile numbers by tph with a multiplication
    uint32_t pad;
};
// ceil(2^32 / d) for 2 <= d < 2^31; 2^32 - 1 for d = 1 (the kernel's fast_div corrects the estimate either way).
static inline uint32_t div_magic(uint32_t d) { return d <= 1 ? 0xffffffffu : (uint32_t)((0x100000000ull + d - 1) / d); }
// A KV head as the selection kernel sees it.
struct HeadRec {
    int L, nkeep;
    int unit, kv_in;     // the unit and the head's index within it
    long long soff;      // offset (floats / keys) of the head's scores and select keys
    long long ooff;      // offset (rows) of the head's kept indices and compacted rows in the stacked outputs
};
struct UnitTables {
    const void *maps = nullptr;          // device: [nunits][2] TMA tensor maps (K, Qwin)
    const void *const *K = nullptr;      // device: [nunits] base of K
    const void *const *V = nullptr;      // device: [nunits] base of V
    const GroupRec *groups = nullptr;    // device: [ngroups]
    const HeadRec *heads = nullptr;      // device: [nunits * hpu]
    int ngroups = 0, hpu = 0;            // hpu: KV heads per unit
    int max_group_tiles = 0;             // most tiles in any group (sizes the grid)
    int max_L = 0;                       // longest prefix (sizes the selection kernel's shared memory)
    long long total_keys = 0;            // keys of all units (floats in the scores array)
    long long total_rows = 0;            // rows of the stacked outputs
};
static inline size_t unit_tables_bytes(int nunits, int hpu)
{
    return align_up((size_t)nunits * 2 * kTensorMapBytes, 256) + 2 * align_up((size_t)nunits * sizeof(void *), 256) +
           align_up((size_t)nunits * hpu * sizeof(GroupRec), 256) + align_up((size_t)nunits * hpu * sizeof(HeadRec), 256);
}
// One tensor map for a bf16 tensor [heads][rows][128], boxes of 64 columns x box_rows rows (host).
bool make_tensor_map(void *map, const void *ptr, int rows, int heads, int box_rows);
// Most KV heads of L keys that the scoring kernel takes as one group (tiles of a group are split over `sms` CTAs).
int heads_per_group(int L, int heads, int tiles_per_head, int sms);
int score_sms();   // CTAs of the scoring kernel on the current device; 0 on error

// Host-side bookkeeping.
void count_launch(int n = 1);
jq_status check_launch();   // cudaGetLastError -> JQ_OK / JQ_ERR_CUDA

// Stage launchers (arguments already validated).
jq_status launch_score_fma(const void *K, const void *Q, const jq_shape &s, float *scores,
                           const Workspace &w, cudaStream_t st);
// Kwin, when not null: keys [Hkv][w][128] of the query positions themselves (window-inclusive softmax).
// With tables, s holds the head geometry and the total head count (s.L, s.budget unused): tiles, lengths and
// score offsets come from the tables, K and Q are ignored.
// k_head_rows: rows between consecutive heads of K in memory when the heads are not packed (0: s.L).
jq_status launch_score_tc(const void *K, const void *Q, const jq_shape &s, float *scores,
                          const Workspace &w, cudaStream_t st, const void *Kwin = nullptr,
                          const UnitTables *tables = nullptr, int k_head_rows = 0);
// With K, V, Kout, Vout given, the kernel also copies the kept rows (the fused layer path).  With tables, every
// head has a length, a budget and offsets of its own (s.L, s.budget unused).
// src_head_rows: rows between consecutive heads of K and V in memory when the heads are not packed (0: s.L);
// out_head_rows: rows between consecutive heads of Kout and Vout when more than nkeep (0: nkeep).
jq_status launch_select(const float *scores, const jq_shape &s, int32_t *idx, float *pooled,
                        const Workspace &w, cudaStream_t st, const void *K = nullptr, const void *V = nullptr,
                        void *Kout = nullptr, void *Vout = nullptr, const UnitTables *tables = nullptr,
                        int src_head_rows = 0, int out_head_rows = 0);
jq_status launch_gather(const void *K, const void *V, const int32_t *idx, const jq_shape &s,
                        void *Kout, void *Vout, cudaStream_t st);

}  // namespace jq
