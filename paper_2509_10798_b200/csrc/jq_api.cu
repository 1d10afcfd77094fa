// The C ABI: argument validation, workspace carve-up, stage sequencing.  See include/jq.h.
#include "jq_internal.cuh"
#include <atomic>

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

// The shape of nlayers layers of shape `layer` stacked along the KV-head axis.
static jq_status stacked_shape(const jq_shape *layer, int nlayers, jq_shape *out)
{
    jq_status rc = check_shape(layer);
    if (rc != JQ_OK) return rc;
    if (nlayers < 1) return JQ_ERR_INVALID_ARG;
    if (nlayers > kMaxLayers) return JQ_ERR_UNSUPPORTED;
    *out = *layer;
    out->Hkv = layer->Hkv * nlayers;
    out->Hq = layer->Hq * nlayers;
    return check_shape(out);
}

size_t jq_layers_workspace_bytes(const jq_shape *layer, int nlayers)
{
    jq_shape S;
    if (stacked_shape(layer, nlayers, &S) != JQ_OK) return 0;
    return carve(nullptr, S).bytes + layer_tables_bytes(nlayers);
}

jq_status jq_evict_layers(const void *const *K, const void *const *V, const void *const *Qwin, int nlayers,
                          const jq_shape *layer, void *Kout, void *Vout, int32_t *kept_idx, void *ws, size_t ws_bytes,
                          jq_stream_t stream)
{
    jq_shape S;
    jq_status rc = stacked_shape(layer, nlayers, &S);
    if (rc != JQ_OK) return rc;
    if (!K || !V || !Qwin || !aligned16(Kout) || !aligned16(Vout) || !aligned16(kept_idx)) return JQ_ERR_INVALID_ARG;
    for (int l = 0; l < nlayers; ++l)
        if (!aligned16(K[l]) || !aligned16(V[l]) || !aligned16(Qwin[l])) return JQ_ERR_INVALID_ARG;
    if (!aligned16(ws) || ((uintptr_t)ws & 255u)) return JQ_ERR_INVALID_ARG;
    const Workspace w = carve(ws, S);
    if (ws_bytes < w.bytes + layer_tables_bytes(nlayers)) return JQ_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    // tables behind the workspace proper: tensor maps, then the K and the V base pointers
    char *tab = (char *)ws + w.bytes;
    const size_t maps_bytes = align_up((size_t)nlayers * 2 * kTensorMapBytes, 256), ptr_bytes = align_up((size_t)nlayers * sizeof(void *), 256);
    alignas(64) unsigned char host_maps[kMaxLayers * 2 * kTensorMapBytes];
    if (!build_layer_maps(K, Qwin, nlayers, *layer, host_maps)) return JQ_ERR_CUDA;
    // (copies from pageable host memory are staged before the call returns, so the sources may live on this stack)
    if (cudaMemcpyAsync(tab, host_maps, (size_t)nlayers * 2 * kTensorMapBytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return JQ_ERR_CUDA;
    if (cudaMemcpyAsync(tab + maps_bytes, K, (size_t)nlayers * sizeof(void *), cudaMemcpyHostToDevice, st) != cudaSuccess) return JQ_ERR_CUDA;
    if (cudaMemcpyAsync(tab + maps_bytes + ptr_bytes, V, (size_t)nlayers * sizeof(void *), cudaMemcpyHostToDevice, st) != cudaSuccess) return JQ_ERR_CUDA;
    LayerTables t;
    t.maps = tab;
    t.K = (const void *const *)(tab + maps_bytes);
    t.V = (const void *const *)(tab + maps_bytes + ptr_bytes);
    t.hpl = layer->Hkv;
    if ((rc = launch_score_tc(K[0], Qwin[0], S, w.scores, w, st, nullptr, &t)) != JQ_OK) return rc;
    return launch_select(w.scores, S, kept_idx, nullptr, w, st, nullptr, nullptr, Kout, Vout, &t);
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
