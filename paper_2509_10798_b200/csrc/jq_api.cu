// The C ABI: argument validation, workspace carve-up, stage sequencing.  See include/jq.h.
#include "jq_internal.cuh"
#include <atomic>
#include <vector>

namespace jq {

static std::atomic<unsigned long long> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }

jq_status check_launch() { return cudaGetLastError() == cudaSuccess ? JQ_OK : JQ_ERR_CUDA; }

static jq_status check_shape(const jq_shape *s)
{
    if (!s) return JQ_ERR_INVALID_ARG;
    if (s->Hkv < 1 || s->Hq < 1 || s->group < 1 || s->L < 1 || s->d < 1 || s->w < 1 || s->budget < 1 ||
        s->pool < 1)
        return JQ_ERR_INVALID_ARG;
    if ((long long)s->Hkv * s->group != (long long)s->Hq) return JQ_ERR_INVALID_ARG;
    if (s->pool % 2 == 0) return JQ_ERR_INVALID_ARG;
    if (s->d != kD) return JQ_ERR_UNSUPPORTED;
    if ((long long)s->group * s->w > kMaxR) return JQ_ERR_UNSUPPORTED;
    if (s->pool > 63) return JQ_ERR_UNSUPPORTED;
    if (s->L > (1 << 24)) return JQ_ERR_UNSUPPORTED;
    if (s->Hkv > 65535) return JQ_ERR_UNSUPPORTED;
    return JQ_OK;
}

static bool aligned16(const void *p) { return p && ((uintptr_t)p & 15u) == 0; }

static jq_status check_ws(const jq_shape *s, void *ws, size_t ws_bytes, Workspace *out)
{
    if (!aligned16(ws) || ((uintptr_t)ws & 255u)) return JQ_ERR_INVALID_ARG;
    *out = carve(ws, *s);
    return ws_bytes < out->bytes ? JQ_ERR_WORKSPACE : JQ_OK;
}

}  // namespace jq

using namespace jq;

extern "C" {

jq_status jq_check_shape(const jq_shape *s) { return check_shape(s); }

size_t jq_workspace_bytes(const jq_shape *s)
{
    if (check_shape(s) != JQ_OK) return 0;
    return carve(nullptr, *s).bytes;
}

int jq_num_kept(const jq_shape *s)
{
    if (check_shape(s) != JQ_OK) return 0;
    return s->budget < s->L ? s->budget : s->L;
}

jq_status jq_workspace_init(void *ws, size_t ws_bytes, jq_stream_t stream)
{
    if (!aligned16(ws) || ((uintptr_t)ws & 255u)) return JQ_ERR_INVALID_ARG;
    if (ws_bytes < 256) return JQ_ERR_WORKSPACE;
    return cudaMemsetAsync(ws, 0, 256, (cudaStream_t)stream) == cudaSuccess ? JQ_OK : JQ_ERR_CUDA;
}

jq_status jq_score(const void *K, const void *Qwin, const jq_shape *s, float *scores, void *ws,
                   size_t ws_bytes, jq_stream_t stream)
{
    jq_status rc = check_shape(s);
    if (rc != JQ_OK) return rc;
    if (!aligned16(K) || !aligned16(Qwin) || !aligned16(scores)) return JQ_ERR_INVALID_ARG;
    Workspace w;
    if ((rc = check_ws(s, ws, ws_bytes, &w)) != JQ_OK) return rc;
    return launch_score_tc(K, Qwin, *s, scores, w, (cudaStream_t)stream);
}

jq_status jq_score_windowed(const void *K, const void *Qwin, const void *Kwin, const jq_shape *s, float *scores,
                            void *ws, size_t ws_bytes, jq_stream_t stream)
{
    jq_status rc = check_shape(s);
    if (rc != JQ_OK) return rc;
    if (s->w > 128) return JQ_ERR_UNSUPPORTED;   // the window keys of a head must fit one tile
    if (!aligned16(K) || !aligned16(Qwin) || !aligned16(Kwin) || !aligned16(scores)) return JQ_ERR_INVALID_ARG;
    Workspace w;
    if ((rc = check_ws(s, ws, ws_bytes, &w)) != JQ_OK) return rc;
    return launch_score_tc(K, Qwin, *s, scores, w, (cudaStream_t)stream, Kwin);
}

jq_status jq_evict_layer_windowed(const void *K, const void *V, const void *Qwin, const void *Kwin, const jq_shape *s,
                                  void *Kout, void *Vout, int32_t *kept_idx, void *ws, size_t ws_bytes,
                                  jq_stream_t stream)
{
    jq_status rc = check_shape(s);
    if (rc != JQ_OK) return rc;
    if (s->w > 128) return JQ_ERR_UNSUPPORTED;   // the window keys of a head must fit one tile
    if (!aligned16(K) || !aligned16(V) || !aligned16(Qwin) || !aligned16(Kwin) || !aligned16(Kout) || !aligned16(Vout) ||
        !aligned16(kept_idx))
        return JQ_ERR_INVALID_ARG;
    Workspace w;
    if ((rc = check_ws(s, ws, ws_bytes, &w)) != JQ_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    if ((rc = launch_score_tc(K, Qwin, *s, w.scores, w, st, Kwin)) != JQ_OK) return rc;
    return launch_select(w.scores, *s, kept_idx, nullptr, w, st, K, V, Kout, Vout);
}

jq_status jq_evict_layer_window_kept(const void *K, const void *V, const void *Qwin, const void *Kwin, const void *Vwin,
                                     const jq_shape *s, void *Kout, void *Vout, int32_t *kept_idx, void *ws, size_t ws_bytes,
                                     jq_stream_t stream)
{
    jq_status rc = check_shape(s);
    if (rc != JQ_OK) return rc;
    if (s->w > 128) return JQ_ERR_UNSUPPORTED;                 // the window keys of a head must fit one tile
    if (s->budget <= s->w) return JQ_ERR_INVALID_ARG;          // the window alone would fill the budget
    if (!aligned16(K) || !aligned16(V) || !aligned16(Qwin) || !aligned16(Kwin) || !aligned16(Vwin) || !aligned16(Kout) ||
        !aligned16(Vout) || !aligned16(kept_idx))
        return JQ_ERR_INVALID_ARG;
    Workspace w;
    if ((rc = check_ws(s, ws, ws_bytes, &w)) != JQ_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    // prefix rows: the window-inclusive pass with budget - w; then the w window rows behind them, head by head
    jq_shape sp = *s;
    sp.budget = s->budget - s->w;
    const size_t row = (size_t)s->d * 2, np = (size_t)(sp.budget < s->L ? sp.budget : s->L), nt = np + (size_t)s->w;
    // the kept prefix rows of head kv go to rows [kv * nt, kv * nt + np) of the outputs, its window rows behind them
    if ((rc = launch_score_tc(K, Qwin, sp, w.scores, w, st, Kwin)) != JQ_OK) return rc;
    if ((rc = launch_select(w.scores, sp, kept_idx, nullptr, w, st, K, V, Kout, Vout, nullptr, 0, (int)nt)) != JQ_OK) return rc;
    if (cudaMemcpy2DAsync((char *)Kout + np * row, nt * row, Kwin, (size_t)s->w * row, (size_t)s->w * row, (size_t)s->Hkv, cudaMemcpyDeviceToDevice, st) != cudaSuccess ||
        cudaMemcpy2DAsync((char *)Vout + np * row, nt * row, Vwin, (size_t)s->w * row, (size_t)s->w * row, (size_t)s->Hkv, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        return JQ_ERR_CUDA;
    return JQ_OK;
}

jq_status jq_score_fma(const void *K, const void *Qwin, const jq_shape *s, float *scores, void *ws,
                       size_t ws_bytes, jq_stream_t stream)
{
    jq_status rc = check_shape(s);
    if (rc != JQ_OK) return rc;
    if (!aligned16(K) || !aligned16(Qwin) || !aligned16(scores)) return JQ_ERR_INVALID_ARG;
    Workspace w;
    if ((rc = check_ws(s, ws, ws_bytes, &w)) != JQ_OK) return rc;
    return launch_score_fma(K, Qwin, *s, scores, w, (cudaStream_t)stream);
}

jq_status jq_select_topk(const float *scores, const jq_shape *s, int32_t *kept_idx, float *pooled_or_null,
                         void *ws, size_t ws_bytes, jq_stream_t stream)
{
    jq_status rc = check_shape(s);
    if (rc != JQ_OK) return rc;
    if (!aligned16(scores) || !aligned16(kept_idx)) return JQ_ERR_INVALID_ARG;
    if (pooled_or_null && !aligned16(pooled_or_null)) return JQ_ERR_INVALID_ARG;
    Workspace w;
    if ((rc = check_ws(s, ws, ws_bytes, &w)) != JQ_OK) return rc;
    return launch_select(scores, *s, kept_idx, pooled_or_null, w, (cudaStream_t)stream);
}

jq_status jq_compact_kv(const void *K, const void *V, const int32_t *kept_idx, const jq_shape *s,
                        void *Kout, void *Vout, jq_stream_t stream)
{
    jq_status rc = check_shape(s);
    if (rc != JQ_OK) return rc;
    if (!aligned16(K) || !aligned16(V) || !aligned16(kept_idx) || !aligned16(Kout) || !aligned16(Vout))
        return JQ_ERR_INVALID_ARG;
    return launch_gather(K, V, kept_idx, *s, Kout, Vout, (cudaStream_t)stream);
}

jq_status jq_evict_layer(const void *K, const void *V, const void *Qwin, const jq_shape *s, void *Kout,
                         void *Vout, int32_t *kept_idx, void *ws, size_t ws_bytes, jq_stream_t stream)
{
    jq_status rc = check_shape(s);
    if (rc != JQ_OK) return rc;
    if (!aligned16(K) || !aligned16(V) || !aligned16(Qwin) || !aligned16(Kout) || !aligned16(Vout) ||
        !aligned16(kept_idx))
        return JQ_ERR_INVALID_ARG;
    Workspace w;
    if ((rc = check_ws(s, ws, ws_bytes, &w)) != JQ_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    if ((rc = launch_score_tc(K, Qwin, *s, w.scores, w, st)) != JQ_OK) return rc;
    return launch_select(w.scores, *s, kept_idx, nullptr, w, st, K, V, Kout, Vout);   // selects, then copies the kept rows
}

// ---- units of one head geometry in buffers of their own: lengths, budgets and offsets per unit

namespace {

struct RaggedPlan {
    jq_shape S;                 // head geometry with the total head count (L = longest prefix, budget = largest nkeep)
    size_t keys = 0;            // sum over units of Hkv * L
    long long rows = 0;         // sum over units of Hkv * nkeep
    int max_L = 0;
};

// Validates the arguments the two ragged entry points share and sums the sizes.  L and budget may be NULL
// (then every unit has common->L / common->budget).
jq_status plan_ragged(const jq_shape *common, int nunits, const int *L, const int *budget, RaggedPlan *out)
{
    if (!common) return JQ_ERR_INVALID_ARG;
    if (nunits < 1) return JQ_ERR_INVALID_ARG;
    if (nunits > kMaxUnits) return JQ_ERR_UNSUPPORTED;
    RaggedPlan pl;
    int max_keep = 0;
    for (int u = 0; u < nunits; ++u) {
        jq_shape su = *common;
        if (L) su.L = L[u];
        if (budget) su.budget = budget[u];
        const jq_status rc = check_shape(&su);
        if (rc != JQ_OK) return rc;
        const int nkeep = su.budget < su.L ? su.budget : su.L;
        pl.keys += (size_t)su.Hkv * su.L;
        pl.rows += (long long)su.Hkv * nkeep;
        if (su.L > pl.max_L) pl.max_L = su.L;
        if (nkeep > max_keep) max_keep = nkeep;
    }
    if ((long long)common->Hkv * nunits > 65535) return JQ_ERR_UNSUPPORTED;
    pl.S = *common;
    pl.S.Hkv = common->Hkv * nunits;
    pl.S.Hq = common->Hq * nunits;
    pl.S.L = pl.max_L;
    pl.S.budget = max_keep;
    *out = pl;
    return JQ_OK;
}

}  // namespace

size_t jq_ragged_workspace_bytes(const jq_shape *common, int nunits, const int *L)
{
    RaggedPlan pl;
    if (plan_ragged(common, nunits, L, nullptr, &pl) != JQ_OK) return 0;
    return carve(nullptr, (size_t)pl.S.Hkv, (size_t)common->group * common->w, pl.keys).bytes + unit_tables_bytes(nunits, common->Hkv);
}

long long jq_ragged_output_rows(const jq_shape *common, int nunits, const int *L, const int *budget)
{
    RaggedPlan pl;
    if (plan_ragged(common, nunits, L, budget, &pl) != JQ_OK) return 0;
    return pl.rows;
}

jq_status jq_evict_ragged(const void *const *K, const void *const *V, const void *const *Qwin, int nunits,
                          const jq_shape *common, const int *L, const int *budget, void *Kout, void *Vout,
                          int32_t *kept_idx, void *ws, size_t ws_bytes, jq_stream_t stream)
{
    RaggedPlan pl;
    jq_status rc = plan_ragged(common, nunits, L, budget, &pl);
    if (rc != JQ_OK) return rc;
    if (!K || !V || !Qwin || !aligned16(Kout) || !aligned16(Vout) || !aligned16(kept_idx)) return JQ_ERR_INVALID_ARG;
    for (int u = 0; u < nunits; ++u)
        if (!aligned16(K[u]) || !aligned16(V[u]) || !aligned16(Qwin[u])) return JQ_ERR_INVALID_ARG;
    if (!aligned16(ws) || ((uintptr_t)ws & 255u)) return JQ_ERR_INVALID_ARG;
    const int hpu = common->Hkv, R = common->group * common->w;
    const Workspace w = carve(ws, (size_t)pl.S.Hkv, (size_t)R, pl.keys);
    const size_t tab_bytes = unit_tables_bytes(nunits, hpu);
    if (ws_bytes < w.bytes + tab_bytes) return JQ_ERR_WORKSPACE;
    const int sms = score_sms();
    if (sms < 1) return JQ_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;

    // All tables are assembled in one host buffer of the library's own (so that the caller's arrays are only read
    // before the call returns, whatever memory they live in) and go to the device in one copy.
    static thread_local std::vector<unsigned char> staging;
    staging.assign(tab_bytes, 0);
    unsigned char *hb = staging.data();
    const size_t maps_bytes = align_up((size_t)nunits * 2 * kTensorMapBytes, 256), ptr_bytes = align_up((size_t)nunits * sizeof(void *), 256);
    const size_t grp_bytes = align_up((size_t)nunits * hpu * sizeof(GroupRec), 256);
    unsigned char *h_maps = hb;
    const void **h_K = (const void **)(hb + maps_bytes), **h_V = (const void **)(hb + maps_bytes + ptr_bytes);
    GroupRec *h_grp = (GroupRec *)(hb + maps_bytes + 2 * ptr_bytes);
    HeadRec *h_head = (HeadRec *)(hb + maps_bytes + 2 * ptr_bytes + grp_bytes);
    UnitTables t;
    long long soff = 0, ooff = 0;
    int ngroups = 0;
    for (int u = 0; u < nunits; ++u) {
        const int Lu = L ? L[u] : common->L, Bu = budget ? budget[u] : common->budget;
        const int nkeep = Bu < Lu ? Bu : Lu;
        if (!make_tensor_map(h_maps + (size_t)(2 * u) * kTensorMapBytes, K[u], Lu, hpu, 128) ||
            !make_tensor_map(h_maps + (size_t)(2 * u + 1) * kTensorMapBytes, Qwin[u], R, hpu, R <= 128 ? 128 : 256))
            return JQ_ERR_CUDA;
        h_K[u] = K[u]; h_V[u] = V[u];
        for (int h = 0; h < hpu; ++h) {
            HeadRec &r = h_head[u * hpu + h];
            r.L = Lu; r.nkeep = nkeep; r.unit = u; r.kv_in = h;
            r.soff = soff + (long long)h * Lu;
            r.ooff = ooff + (long long)h * nkeep;
        }
        soff += (long long)hpu * Lu;
        ooff += (long long)hpu * nkeep;
    }
    // head groups of the scoring kernel: every run of consecutive units of one length is cut into groups of
    // about 32 MiB of keys (short prefixes share a group across units, so that a group still has tiles for every CTA)
    for (int u0 = 0; u0 < nunits;) {
        const int Lu = L ? L[u0] : common->L, tph = (Lu + 127) / 128;
        int u1 = u0 + 1;
        while (u1 < nunits && (L ? L[u1] : common->L) == Lu) ++u1;
        const int heads = (u1 - u0) * hpu, hpg = heads_per_group(Lu, heads, tph, sms);
        for (int h0 = 0; h0 < heads; h0 += hpg) {
            GroupRec &g = h_grp[ngroups++];
            g.h0 = u0 * hpu + h0; g.nh = h0 + hpg <= heads ? hpg : heads - h0;
            g.tph = tph; g.L = Lu; g.unit = u0 + h0 / hpu; g.c20 = h0 % hpu;
            g.sbase = h_head[g.h0].soff; g.tph_magic = div_magic((uint32_t)tph); g.pad = 0;
            if (g.nh * tph > t.max_group_tiles) t.max_group_tiles = g.nh * tph;
        }
        u0 = u1;
    }
    char *tab = (char *)ws + w.bytes;
    if (cudaMemcpyAsync(tab, hb, tab_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return JQ_ERR_CUDA;
    t.maps = tab;
    t.K = (const void *const *)(tab + maps_bytes);
    t.V = (const void *const *)(tab + maps_bytes + ptr_bytes);
    t.groups = (const GroupRec *)(tab + maps_bytes + 2 * ptr_bytes);
    t.heads = (const HeadRec *)(tab + maps_bytes + 2 * ptr_bytes + grp_bytes);
    t.ngroups = ngroups; t.hpu = hpu; t.max_L = pl.max_L; t.total_keys = (long long)pl.keys; t.total_rows = pl.rows;
    if ((rc = launch_score_tc(nullptr, nullptr, pl.S, w.scores, w, st, nullptr, &t)) != JQ_OK) return rc;
    return launch_select(w.scores, pl.S, kept_idx, nullptr, w, st, nullptr, nullptr, Kout, Vout, &t);
}

size_t jq_layers_workspace_bytes(const jq_shape *layer, int nlayers)
{
    return jq_ragged_workspace_bytes(layer, nlayers, nullptr);
}

jq_status jq_evict_layers(const void *const *K, const void *const *V, const void *const *Qwin, int nlayers,
                          const jq_shape *layer, void *Kout, void *Vout, int32_t *kept_idx, void *ws, size_t ws_bytes,
                          jq_stream_t stream)
{
    return jq_evict_ragged(K, V, Qwin, nlayers, layer, nullptr, nullptr, Kout, Vout, kept_idx, ws, ws_bytes, stream);
}

// ---- streaming re-eviction: the pruned cache of a layer has grown during decoding

size_t jq_append_workspace_bytes(const jq_shape *s)
{
    if (check_shape(s) != JQ_OK) return 0;
    const size_t nkeep = (size_t)(s->budget < s->L ? s->budget : s->L);
    return carve(nullptr, *s).bytes + 2 * align_up((size_t)s->Hkv * nkeep * s->d * 2, 256);
}

jq_status jq_evict_append(void *Kc, void *Vc, int cap, int n_old, const void *Knew, const void *Vnew, int n_new,
                          const void *Qrecent, const jq_shape *s, int32_t *kept_idx, void *ws, size_t ws_bytes,
                          jq_stream_t stream)
{
    jq_status rc = check_shape(s);
    if (rc != JQ_OK) return rc;
    if (n_old < 0 || n_new < 0 || cap < 1 || (long long)n_old + n_new != (long long)s->L || s->L > cap) return JQ_ERR_INVALID_ARG;
    if (!aligned16(Kc) || !aligned16(Vc) || !aligned16(Qrecent) || !aligned16(kept_idx)) return JQ_ERR_INVALID_ARG;
    if (n_new > 0 && (!aligned16(Knew) || !aligned16(Vnew))) return JQ_ERR_INVALID_ARG;
    Workspace w;
    if ((rc = check_ws(s, ws, ws_bytes, &w)) != JQ_OK) return rc;
    if (ws_bytes < jq_append_workspace_bytes(s)) return JQ_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t row = (size_t)s->d * 2, nkeep = (size_t)(s->budget < s->L ? s->budget : s->L);
    char *Ktmp = (char *)ws + w.bytes, *Vtmp = Ktmp + align_up((size_t)s->Hkv * nkeep * row, 256);
    // 1. the new rows go behind the retained ones, head by head (the cache keeps `cap` rows per head)
    if (n_new > 0) {
        if (cudaMemcpy2DAsync((char *)Kc + (size_t)n_old * row, (size_t)cap * row, Knew, (size_t)n_new * row, (size_t)n_new * row,
                              (size_t)s->Hkv, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return JQ_ERR_CUDA;
        if (cudaMemcpy2DAsync((char *)Vc + (size_t)n_old * row, (size_t)cap * row, Vnew, (size_t)n_new * row, (size_t)n_new * row,
                              (size_t)s->Hkv, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return JQ_ERR_CUDA;
    }
    // 2. the pass over the L = n_old + n_new rows of every head, compacted into the workspace (a row may move
    //    onto a row that another thread still has to read, so the compaction cannot run in place)
    if ((rc = launch_score_tc(Kc, Qrecent, *s, w.scores, w, st, nullptr, nullptr, cap)) != JQ_OK) return rc;
    if ((rc = launch_select(w.scores, *s, kept_idx, nullptr, w, st, Kc, Vc, Ktmp, Vtmp, nullptr, cap)) != JQ_OK) return rc;
    // 3. back to the head of the cache
    if (cudaMemcpy2DAsync(Kc, (size_t)cap * row, Ktmp, nkeep * row, nkeep * row, (size_t)s->Hkv, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        return JQ_ERR_CUDA;
    if (cudaMemcpy2DAsync(Vc, (size_t)cap * row, Vtmp, nkeep * row, nkeep * row, (size_t)s->Hkv, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        return JQ_ERR_CUDA;
    return JQ_OK;
}

size_t jq_host_call_bytes(const jq_shape *s)
{
    if (check_shape(s) != JQ_OK) return 0;
    const size_t row = (size_t)s->d * 2;
    const size_t nkeep = (size_t)(s->budget < s->L ? s->budget : s->L);
    size_t b = 0;
    b += 2 * align_up((size_t)s->Hkv * s->L * row, 256);      // K, V
    b += align_up((size_t)s->Hq * s->w * row, 256);           // Qwin
    b += 2 * align_up((size_t)s->Hkv * nkeep * row, 256);     // Kout, Vout
    b += align_up((size_t)s->Hkv * nkeep * 4, 256);           // kept_idx
    b += carve(nullptr, *s).bytes;
    return b;
}

jq_status jq_evict_layer_host(const void *hK, const void *hV, const void *hQwin, const jq_shape *s,
                              void *hKout, void *hVout, int32_t *hkept_idx, void *dev_buf,
                              size_t dev_buf_bytes, jq_stream_t stream)
{
    jq_status rc = check_shape(s);
    if (rc != JQ_OK) return rc;
    if (!hK || !hV || !hQwin || !hKout || !hVout || !hkept_idx) return JQ_ERR_INVALID_ARG;
    if (!dev_buf || ((uintptr_t)dev_buf & 255u)) return JQ_ERR_INVALID_ARG;
    if (dev_buf_bytes < jq_host_call_bytes(s)) return JQ_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t row = (size_t)s->d * 2;
    const size_t nkeep = (size_t)(s->budget < s->L ? s->budget : s->L);
    const size_t kvb = (size_t)s->Hkv * s->L * row, qb = (size_t)s->Hq * s->w * row;
    const size_t ob = (size_t)s->Hkv * nkeep * row, ib = (size_t)s->Hkv * nkeep * 4;
    char *p = (char *)dev_buf;
    char *dK = p;          p += align_up(kvb, 256);
    char *dV = p;          p += align_up(kvb, 256);
    char *dQ = p;          p += align_up(qb, 256);
    char *dKo = p;         p += align_up(ob, 256);
    char *dVo = p;         p += align_up(ob, 256);
    char *dI = p;          p += align_up(ib, 256);
    char *ws = p;
    const size_t wsb = carve(nullptr, *s).bytes;
    if (cudaMemsetAsync(ws, 0, 256, st) != cudaSuccess) return JQ_ERR_CUDA;
    if (cudaMemcpyAsync(dQ, hQwin, qb, cudaMemcpyHostToDevice, st) != cudaSuccess) return JQ_ERR_CUDA;
    if (cudaMemcpyAsync(dK, hK, kvb, cudaMemcpyHostToDevice, st) != cudaSuccess) return JQ_ERR_CUDA;
    // V is read at the kept rows only.  A page-locked host buffer is mapped into the device's address space: the
    // selection kernel then fetches those rows from it directly and the copy of all of V is skipped.
    const void *v_src = dV;
    cudaPointerAttributes pa;
    if (cudaPointerGetAttributes(&pa, hV) == cudaSuccess && pa.type == cudaMemoryTypeHost && pa.devicePointer &&
        !((uintptr_t)pa.devicePointer & 15u)) {
        v_src = pa.devicePointer;
    } else {
        cudaGetLastError();
        if (cudaMemcpyAsync(dV, hV, kvb, cudaMemcpyHostToDevice, st) != cudaSuccess) return JQ_ERR_CUDA;
    }
    rc = jq_evict_layer(dK, v_src, dQ, s, dKo, dVo, (int32_t *)dI, ws, wsb, stream);
    if (rc != JQ_OK) return rc;
    if (cudaMemcpyAsync(hkept_idx, dI, ib, cudaMemcpyDeviceToHost, st) != cudaSuccess) return JQ_ERR_CUDA;
    if (cudaMemcpyAsync(hKout, dKo, ob, cudaMemcpyDeviceToHost, st) != cudaSuccess) return JQ_ERR_CUDA;
    if (cudaMemcpyAsync(hVout, dVo, ob, cudaMemcpyDeviceToHost, st) != cudaSuccess) return JQ_ERR_CUDA;
    return JQ_OK;
}

jq_status jq_last_device_status(const void *ws, jq_stream_t stream)
{
    if (!ws) return JQ_ERR_INVALID_ARG;
    int word = 0;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return JQ_ERR_CUDA;
    if (cudaMemcpy(&word, ws, sizeof word, cudaMemcpyDeviceToHost) != cudaSuccess) return JQ_ERR_CUDA;
    if (word < 0 || word > JQ_ERR_TIMEOUT) return JQ_ERR_CUDA;
    return (jq_status)word;
}

unsigned long long jq_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char *jq_status_string(jq_status s)
{
    switch (s) {
        case JQ_OK: return "ok";
        case JQ_ERR_INVALID_ARG: return "invalid argument";
        case JQ_ERR_UNSUPPORTED: return "unsupported shape";
        case JQ_ERR_WORKSPACE: return "workspace too small";
        case JQ_ERR_CUDA: return "CUDA error";
        case JQ_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

}  // extern "C"
