/*
 * jq.h -- C ABI of the B200 (sm_100a) library for the per-layer KV-cache eviction pass of
 * "Judge Q" (arXiv 2509.10798).
 *
 * The pass (inference section of the paper; Eq. 3 defines the attention map it uses): the queries
 * of the w soft tokens appended to the prompt score every prefix key of one layer,
 *     s[h,i,j]   = Qwin[h,i,:] . K[h/group, j, :] / sqrt(d)
 *     P[h,i,:]   = softmax over the L prefix keys of s[h,i,:]
 *     score[kv,j]= sum over the `group` query heads of KV head kv and the w soft tokens of P[h,i,j]
 *     pooled     = centred max of odd width `pool` over the key axis (same length, edges clipped)
 * the min(budget, L) positions with the largest pooled score are kept per KV head (equal values:
 * the lower index wins), reported in ascending order, and their K and V rows are copied into a
 * compacted cache.
 *
 * Conventions, for every entry point unless it says otherwise:
 *  - pointers named K, V, Qwin, scores, kept_idx, Kout, Vout, ws are DEVICE pointers owned by the
 *    caller, contiguous row-major, 16-byte aligned; the library allocates and frees nothing;
 *  - bf16 tensors are raw 16-bit patterns:  K, V [Hkv, L, d];  Qwin [Hq, w, d];
 *    Kout, Vout [Hkv, nkeep, d];  scores, pooled [Hkv, L] fp32;  kept_idx [Hkv, nkeep] int32,
 *    nkeep = jq_num_kept(shape) = min(budget, L);
 *  - all work is enqueued on `stream` (a cudaStream_t); the call returns without synchronising;
 *    outputs are valid once the stream reaches the end of the call's work;
 *  - outputs must not overlap inputs or the workspace; the same workspace may be reused by
 *    successive calls on ONE stream; calls on different streams need different workspaces;
 *  - inputs must be finite; NaN or Inf give unspecified kept sets (never a fault);
 *  - errors are return codes; argument errors are detected on the host before anything is
 *    launched and leave every output untouched.
 *
 * Supported shapes: d == 128;  Hq == Hkv * group;  1 <= group * w <= 256;  pool odd, 1..63;
 * budget >= 1;  1 <= L <= 2^24;  Hkv >= 1.
 */
#ifndef JQ_H_
#define JQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    JQ_OK = 0,
    JQ_ERR_INVALID_ARG = 1, /* null or misaligned pointer, inconsistent shape                 */
    JQ_ERR_UNSUPPORTED = 2, /* a legal shape the library has no kernel for (d != 128, ...)     */
    JQ_ERR_WORKSPACE = 3,   /* ws_bytes < jq_workspace_bytes(shape)                            */
    JQ_ERR_CUDA = 4,        /* a CUDA runtime / driver call or a launch failed                 */
    JQ_ERR_TIMEOUT = 5      /* a bounded device-side wait ran out (see jq_last_device_status)  */
} jq_status;

typedef struct {
    int Hkv;    /* KV heads                                             */
    int Hq;     /* query heads, = Hkv * group                           */
    int group;  /* GQA group size: query head h reads KV head h / group */
    int L;      /* prefix length (keys per KV head)                     */
    int d;      /* head dimension (128)                                 */
    int w;      /* soft-token queries per query head (the paper's n)    */
    int budget; /* positions to keep per KV head                        */
    int pool;   /* max-pool width (odd); 1 = no pooling                 */
} jq_shape;

/* A cudaStream_t, spelled so that this header needs no CUDA header. */
typedef struct CUstream_st *jq_stream_t;

/* Bytes of device workspace every call below needs for this shape (host-only, no CUDA call);
 * 0 if the shape is invalid or unsupported. */
size_t jq_workspace_bytes(const jq_shape *shape);

/*
 * Zeroes the status word at the head of a workspace.  Call once after allocating `ws` and before
 * its first use (on the stream that will use it); the status then accumulates over all later calls
 * until it is read with jq_last_device_status or cleared by calling this again.  The block also holds
 * the counters the scoring kernel's CTAs synchronise through; a call that ended in JQ_ERR_TIMEOUT
 * leaves them undefined, so call this again before reusing the workspace after such an error.
 */
jq_status jq_workspace_init(void *ws, size_t ws_bytes, jq_stream_t stream);

/* min(budget, L); 0 for an invalid shape. */
int jq_num_kept(const jq_shape *shape);

/* Why a shape is (not) accepted: JQ_OK, JQ_ERR_INVALID_ARG or JQ_ERR_UNSUPPORTED (host-only). */
jq_status jq_check_shape(const jq_shape *shape);

/*
 * Eq. 3 (summed, not averaged, over the soft tokens and over the GQA group): pre-pool scores.
 * Two streaming passes over K on the tensor cores: pass 1 finds each query row's running max
 * and sum of exponentials, pass 2 recomputes the logits and accumulates the normalised
 * probabilities per key (fp32 accumulation of bf16 products).
 *   K [Hkv,L,d] bf16, Qwin [Hq,w,d] bf16  ->  scores [Hkv,L] fp32.
 */
jq_status jq_score(const void *K, const void *Qwin, const jq_shape *shape, float *scores,
                   void *ws, size_t ws_bytes, jq_stream_t stream);

/*
 * Window-inclusive variants.  Eq. 3 can also be read as the attention the model itself computes for a soft
 * token: its softmax then runs over the prefix AND, causally, over the soft tokens up to itself; the same
 * holds for the last-window queries that the compared methods of the experimental section score with.
 * Kwin [Hkv, w, d] bf16 holds the keys of the w query positions; query i of every head of the group sees
 * Kwin[kv, 0..i] besides the L prefix keys.  These columns only enter the denominator: scores, pooling,
 * selection and compaction still run over the L prefix positions (a caller that wants the window kept
 * keeps it itself).  Needs w <= 128 (JQ_ERR_UNSUPPORTED otherwise).  Everything else as in jq_score /
 * jq_evict_layer.  The window keys are scored as one more tile of each head in pass 1, masked causally.
 */
jq_status jq_score_windowed(const void *K, const void *Qwin, const void *Kwin, const jq_shape *shape,
                            float *scores, void *ws, size_t ws_bytes, jq_stream_t stream);
jq_status jq_evict_layer_windowed(const void *K, const void *V, const void *Qwin, const void *Kwin,
                                  const jq_shape *shape, void *Kout, void *Vout, int32_t *kept_idx,
                                  void *ws, size_t ws_bytes, jq_stream_t stream);

/*
 * The window-inclusive pass with the window itself retained, the way the last-window methods of the paper's
 * experimental section use their budget: of `budget` rows per KV head, w are the query positions' own pairs
 * (always kept) and budget - w are chosen among the L prefix positions by jq_evict_layer_windowed's scores.
 * Vwin [Hkv, w, d] bf16: the values of the query positions.  Kout, Vout: bf16 [Hkv, np + w, d] with
 * np = min(budget - w, L): the kept prefix rows in ascending position, then the w window rows in order.
 * kept_idx [Hkv, np] int32: the kept prefix positions.  Needs w <= 128 and budget > w (JQ_ERR_INVALID_ARG).
 */
jq_status jq_evict_layer_window_kept(const void *K, const void *V, const void *Qwin, const void *Kwin, const void *Vwin,
                                     const jq_shape *shape, void *Kout, void *Vout, int32_t *kept_idx, void *ws,
                                     size_t ws_bytes, jq_stream_t stream);

/*
 * jq_score for callers that cannot allocate device memory: an inference server that has handed every
 * free byte of the GPU to its KV-cache pool, a plug-in running inside somebody else's memory budget, a
 * call site that must not touch the allocator.  (The paper has no counterpart; this is a property of
 * the library.)  Same inputs, same output and the same kernel as jq_score, but no workspace argument:
 * the scratch the kernel needs sits in a device array built into the library, about 10.5 MB that every
 * GPU using the library holds until the process exits.
 *  - Limit: Hkv * group * w <= 2048 query rows in total; a larger shape returns JQ_ERR_UNSUPPORTED and
 *    launches nothing.
 *  - The call allocates and frees nothing (no cudaMalloc, cudaFree or allocating library routine).
 *    Its first call on a device looks up the array's device address; make that first call outside any
 *    stream capture.
 *  - All calls share the one array, and it keeps the previous call's contents (the part that must start
 *    from zero is cleared on `stream` by every call).  Calls whose work can overlap on the GPU, from
 *    different streams or threads, race on it: keep them on one stream, or order them yourself.
 *  - A bounded device-side wait that runs out leaves its record inside the array, where
 *    jq_last_device_status cannot see it; callers that need that status use jq_score.
 */
jq_status jq_score_static(const void *K, const void *Qwin, const jq_shape *shape, float *scores,
                          jq_stream_t stream);

/*
 * The same scores computed with plain fp32 FMA on the CUDA cores.  A comparator for profiling the
 * tensor-core path against (the contraction is small and of low arithmetic intensity per key);
 * never used by jq_evict_layer.
 */
jq_status jq_score_fma(const void *K, const void *Qwin, const jq_shape *shape, float *scores,
                       void *ws, size_t ws_bytes, jq_stream_t stream);

/*
 * Max-pool (experimental setting: every method shares one pooling configuration) followed by the
 * top-k retention of the inference section.  scores [Hkv,L] fp32, all >= 0.
 *   -> kept_idx [Hkv,nkeep] int32 ascending; ties at the threshold go to the lower index.
 *   pooled_or_null, if not NULL, receives the pooled scores [Hkv,L] fp32.
 * Exact: with identical input scores the result is unique.
 */
jq_status jq_select_topk(const float *scores, const jq_shape *shape, int32_t *kept_idx,
                         float *pooled_or_null, void *ws, size_t ws_bytes, jq_stream_t stream);

/*
 * Compaction of the pruned cache (inference section): Kout[kv,t,:] = K[kv, kept_idx[kv,t], :] and
 * the same for V, bit for bit.  An index outside [0,L) is clamped into range (never a fault); such
 * an index cannot come from jq_select_topk.
 */
jq_status jq_compact_kv(const void *K, const void *V, const int32_t *kept_idx,
                        const jq_shape *shape, void *Kout, void *Vout, jq_stream_t stream);

/*
 * The whole pass for one layer, with the results of jq_score -> jq_select_topk -> jq_compact_kv, on one
 * stream in two launches (the selection kernel also copies the kept rows); the scores stay in the
 * workspace.  K may hold several layers of equal shape stacked along the KV-head axis (Hkv = layers x
 * heads per layer, Qwin stacked alike): heads are independent, so one call evicts them all.
 */
jq_status jq_evict_layer(const void *K, const void *V, const void *Qwin, const jq_shape *shape,
                         void *Kout, void *Vout, int32_t *kept_idx, void *ws, size_t ws_bytes,
                         jq_stream_t stream);

/*
 * The pass over several units in ONE call of two launches.  A unit is a layer of a cache, or a layer of one
 * sequence of a batch: K, V [Hkv, L_u, d] and Qwin [Hq, w, d] in buffers of its own, with a prefix length L_u
 * and a budget B_u of its own; all units share the head geometry of `common` (Hkv, Hq, group, d, w, pool).
 * (Every (unit, KV head) is an independent instance of the pass of the inference section; lengths that differ
 * are the 4K-32K contexts of the paper's length sweeps, budgets that differ per layer are the layer-wise
 * schedule its experimental-setting paragraph describes for one of the compared methods.)  The results are
 * those of one jq_evict_layer call per unit, bit for bit.
 *   K, V, Qwin: HOST arrays of nunits DEVICE pointers, each as jq_evict_layer takes it for unit u;
 *   L, budget:  HOST arrays of nunits ints, or NULL for "common->L / common->budget for every unit"
 *               (the corresponding field of `common` is ignored when the array is given);
 *   all five arrays are only read before the call returns;
 *   Kout, Vout: device, bf16 [rows, d];  kept_idx: device int32 [rows], where unit u's block of
 *               Hkv * nkeep_u rows (head-major, as jq_evict_layer writes them), nkeep_u = min(B_u, L_u),
 *               starts at row sum_{u' < u} Hkv * nkeep_u' and rows = jq_ragged_output_rows(...);
 *   ws: device, 256-byte aligned, at least jq_ragged_workspace_bytes(common, nunits, L) bytes (0 for arguments
 *       the call would reject), its first 256 bytes initialised by jq_workspace_init.
 * nunits <= 4096 and nunits * Hkv <= 65535, else JQ_ERR_UNSUPPORTED.  The call copies its tables (tensor maps,
 * base pointers, per-head lengths and offsets) from host memory of its own to the device on `stream`, so it
 * cannot be captured into a CUDA graph; capture calls of jq_evict_layer instead.
 */
size_t jq_ragged_workspace_bytes(const jq_shape *common, int nunits, const int *L);
long long jq_ragged_output_rows(const jq_shape *common, int nunits, const int *L, const int *budget);
jq_status jq_evict_ragged(const void *const *K, const void *const *V, const void *const *Qwin, int nunits,
                          const jq_shape *common, const int *L, const int *budget, void *Kout, void *Vout,
                          int32_t *kept_idx, void *ws, size_t ws_bytes, jq_stream_t stream);

/*
 * jq_evict_ragged for nlayers layers of ONE shape (the usual cache after a prefill): the same call with
 * L = budget = NULL.  Kout, Vout: device, bf16 [nlayers * Hkv, nkeep, d]; kept_idx: device [nlayers * Hkv, nkeep]
 * (layer l at rows l * Hkv ...).  ws: at least jq_layers_workspace_bytes(layer, nlayers) bytes.
 */
size_t jq_layers_workspace_bytes(const jq_shape *layer, int nlayers);
jq_status jq_evict_layers(const void *const *K, const void *const *V, const void *const *Qwin, int nlayers,
                          const jq_shape *layer, void *Kout, void *Vout, int32_t *kept_idx, void *ws, size_t ws_bytes,
                          jq_stream_t stream);

/*
 * jq_evict_layer for callers whose tensors live in HOST memory (pinned memory gives asynchronous
 * copies).  hK, hV, hQwin are copied to the device, the layer is evicted, and hKout, hVout,
 * hkept_idx are copied back, all on `stream`; the call returns without synchronising.  When hV is
 * page-locked memory only its kept rows cross to the device (the kernel reads them in place); hV must
 * then stay unchanged until the stream has passed the call, like every other host buffer.
 * dev_buf is a device buffer of at least jq_host_call_bytes(shape) bytes (it holds the device
 * copies and the workspace).
 */
size_t jq_host_call_bytes(const jq_shape *shape);
jq_status jq_evict_layer_host(const void *hK, const void *hV, const void *hQwin,
                              const jq_shape *shape, void *hKout, void *hVout, int32_t *hkept_idx,
                              void *dev_buf, size_t dev_buf_bytes, jq_stream_t stream);

/*
 * Eq. 6, the critical key-value hit rate: rate[kv] = |cur[kv] ^ ref[kv]| / nref, the share of a reference
 * kept set (in the paper: the one chosen with the queries of the actually decoded tokens) that another kept
 * set of the same head also holds.  cur [Hkv, ncur], ref [Hkv, nref] int32 device arrays whose rows are
 * strictly ascending (as jq_select_topk writes them); rate [Hkv] fp32 device array.
 */
jq_status jq_hit_rate(const int32_t *cur, const int32_t *ref, int Hkv, int ncur, int nref, float *rate,
                      jq_stream_t stream);

/*
 * The step after the pass (inference section: decoding continues from the end of the input with the retained
 * pairs only): attention of one new query position over the pruned cache,
 *     out[h,:] = softmax_j( q[h,:] . Kc[kv,j,:] / sqrt(d) ) Vc[kv,:,:],   kv = h / (Hq / Hkv),  d = 128.
 * Kc, Vc: device, bf16 [Hkv, n, 128] (what jq_evict_layer wrote), 16-byte aligned.  q: device, bf16 [Hq, 128].
 * out: device, fp32 [Hq, 128], 16-byte aligned.  workspace: device, 16-byte aligned, at least
 * jq_decode_workspace_bytes(Hkv, Hq, n) bytes (0 for arguments the call would reject); no initialisation
 * needed, contents undefined afterwards.  Hq / Hkv <= 8.  Asynchronous on `stream`; one launch (and a memset
 * of Hkv counters in the workspace).
 */
size_t jq_decode_workspace_bytes(int Hkv, int Hq, int n);
jq_status jq_decode_attention(const void *Kc, const void *Vc, const void *q, int Hkv, int Hq, int n, float *out,
                              void *workspace, size_t workspace_bytes, jq_stream_t stream);

/*
 * Re-eviction while decoding (the paper's limitations / future-work paragraph: eviction is done once, after
 * the prefill, and extending it to the decoding stage is left open; the pass itself is the one of the
 * inference section, run again on the grown cache with the queries of recent positions as judges).
 * Kc, Vc: the layer's cache, device, bf16 [Hkv, cap, d]: `cap` rows per head of which the first n_old are
 * retained pairs.  Knew, Vnew: device, bf16 [Hkv, n_new, d], the pairs decoded since (may be NULL when
 * n_new == 0).  Qrecent: device, bf16 [Hq, w, d], the queries that score (e.g. those of the last w decoded
 * positions).  shape->L must equal n_old + n_new and be <= cap; shape->budget is the new size.
 * The call appends the new rows behind the retained ones, runs the pass of jq_evict_layer over the
 * L rows of every head, and leaves the min(budget, L) kept rows, in ascending order of their position in
 * that concatenation, in rows [0, nkeep) of Kc and Vc; kept_idx [Hkv, nkeep] holds those positions (values
 * below n_old are old rows).  Rows [nkeep, cap) are unspecified afterwards.  Same results as jq_evict_layer on
 * the concatenated tensors.  ws: at least jq_append_workspace_bytes(shape) bytes (it also holds the compacted
 * rows before they are moved to the head of the cache), first 256 bytes initialised by jq_workspace_init.
 * Two launches and up to six strided device copies, all on `stream`.
 */
size_t jq_append_workspace_bytes(const jq_shape *shape);
jq_status jq_evict_append(void *Kc, void *Vc, int cap, int n_old, const void *Knew, const void *Vnew, int n_new,
                          const void *Qrecent, const jq_shape *shape, int32_t *kept_idx, void *ws, size_t ws_bytes,
                          jq_stream_t stream);

/*
 * Synchronises `stream` and reads the status word kernels of earlier calls left in the workspace:
 * JQ_OK, JQ_ERR_TIMEOUT (a bounded wait inside a kernel gave up; outputs are invalid),
 * JQ_ERR_INVALID_ARG (an out-of-range index was met), or JQ_ERR_CUDA.
 */
jq_status jq_last_device_status(const void *ws, jq_stream_t stream);

/* Number of kernels the library has launched in this process (for benchmarks' launch counts). */
unsigned long long jq_launch_count(void);

const char *jq_status_string(jq_status s);

#ifdef __cplusplus
}
#endif
#endif /* JQ_H_ */
