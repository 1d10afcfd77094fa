"""B200 (sm_100a) library for the per-layer KV-cache eviction pass of Judge Q (arXiv 2509.10798).

Thin ctypes binding over libjq.so (C ABI in include/jq.h).  The functions here only marshal
arguments: torch tensors supply device memory and the current CUDA stream, every step of the pass
runs in the library's own kernels.  There is no CPU or PyTorch fallback: if libjq.so is missing or
no CUDA device is present, the calls raise.
"""
import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libjq.so")

JQ_OK, JQ_ERR_INVALID_ARG, JQ_ERR_UNSUPPORTED, JQ_ERR_WORKSPACE, JQ_ERR_CUDA, JQ_ERR_TIMEOUT = range(6)

EXPORTS = (
    "jq_workspace_bytes", "jq_workspace_init", "jq_num_kept", "jq_check_shape", "jq_score",
    "jq_score_fma", "jq_select_topk", "jq_compact_kv", "jq_evict_layer", "jq_host_call_bytes",
    "jq_evict_layer_host", "jq_last_device_status", "jq_launch_count", "jq_status_string",
    "jq_score_static", "jq_score_windowed", "jq_evict_layer_windowed", "jq_hit_rate",
    "jq_decode_workspace_bytes", "jq_decode_attention", "jq_layers_workspace_bytes", "jq_evict_layers",
    "jq_ragged_workspace_bytes", "jq_ragged_output_rows", "jq_evict_ragged",
    "jq_append_workspace_bytes", "jq_evict_append", "jq_evict_layer_window_kept",
)


class JqShape(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in ("Hkv", "Hq", "group", "L", "d", "w", "budget", "pool")]


class JqError(RuntimeError):
    def __init__(self, where, code):
        self.code = int(code)
        super().__init__("%s: %s (jq_status %d)" % (where, status_string(code), code))


_lib = None


def lib():
    """Loads libjq.so (never builds it; see build.py) and declares the prototypes."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libjq.so is not built: run `python -m paper_2509_10798_b200.build` "
                               "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, sz, ci = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
        sp = ctypes.POINTER(JqShape)
        L.jq_workspace_bytes.argtypes = [sp]
        L.jq_workspace_bytes.restype = sz
        L.jq_host_call_bytes.argtypes = [sp]
        L.jq_host_call_bytes.restype = sz
        L.jq_num_kept.argtypes = [sp]
        L.jq_num_kept.restype = ci
        L.jq_check_shape.argtypes = [sp]
        L.jq_check_shape.restype = ci
        L.jq_workspace_init.argtypes = [vp, sz, vp]
        L.jq_score.argtypes = [vp, vp, sp, vp, vp, sz, vp]
        L.jq_score_fma.argtypes = [vp, vp, sp, vp, vp, sz, vp]
        L.jq_score_static.argtypes = [vp, vp, sp, vp, vp]
        L.jq_decode_workspace_bytes.argtypes = [ci, ci, ci]
        L.jq_decode_workspace_bytes.restype = ctypes.c_size_t
        L.jq_decode_attention.argtypes = [vp, vp, vp, ci, ci, ci, vp, vp, ctypes.c_size_t, vp]
        L.jq_layers_workspace_bytes.argtypes = [sp, ci]
        L.jq_layers_workspace_bytes.restype = ctypes.c_size_t
        L.jq_evict_layers.argtypes = [vp, vp, vp, ci, sp, vp, vp, vp, vp, sz, vp]
        L.jq_ragged_workspace_bytes.argtypes = [sp, ci, vp]
        L.jq_ragged_workspace_bytes.restype = ctypes.c_size_t
        L.jq_ragged_output_rows.argtypes = [sp, ci, vp, vp]
        L.jq_ragged_output_rows.restype = ctypes.c_longlong
        L.jq_evict_ragged.argtypes = [vp, vp, vp, ci, sp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.jq_evict_layer_window_kept.argtypes = [vp, vp, vp, vp, vp, sp, vp, vp, vp, vp, sz, vp]
        L.jq_append_workspace_bytes.argtypes = [sp]
        L.jq_append_workspace_bytes.restype = ctypes.c_size_t
        L.jq_evict_append.argtypes = [vp, vp, ci, ci, vp, vp, ci, vp, sp, vp, vp, sz, vp]
        L.jq_hit_rate.argtypes = [vp, vp, ci, ci, ci, vp, vp]
        L.jq_score_windowed.argtypes = [vp, vp, vp, sp, vp, vp, sz, vp]
        L.jq_evict_layer_windowed.argtypes = [vp, vp, vp, vp, sp, vp, vp, vp, vp, sz, vp]
        L.jq_select_topk.argtypes = [vp, sp, vp, vp, vp, sz, vp]
        L.jq_compact_kv.argtypes = [vp, vp, vp, sp, vp, vp, vp]
        L.jq_evict_layer.argtypes = [vp, vp, vp, sp, vp, vp, vp, vp, sz, vp]
        L.jq_evict_layer_host.argtypes = [vp, vp, vp, sp, vp, vp, vp, vp, sz, vp]
        L.jq_last_device_status.argtypes = [vp, vp]
        L.jq_launch_count.argtypes = []
        L.jq_launch_count.restype = ctypes.c_ulonglong
        L.jq_status_string.argtypes = [ci]
        L.jq_status_string.restype = ctypes.c_char_p
        for name in EXPORTS:
            getattr(L, name)          # AttributeError if the library lacks a declared entry point
        _lib = L
    return _lib


def status_string(code):
    return lib().jq_status_string(int(code)).decode()


def shape(Hkv, Hq, L, w, budget, pool=7, d=128, group=None):
    return JqShape(int(Hkv), int(Hq), int(Hq // Hkv if group is None else group), int(L), int(d), int(w),
                   int(budget), int(pool))


def check_shape(s):
    return int(lib().jq_check_shape(ctypes.byref(s)))


def workspace_bytes(s):
    return int(lib().jq_workspace_bytes(ctypes.byref(s)))


def host_call_bytes(s):
    return int(lib().jq_host_call_bytes(ctypes.byref(s)))


def num_kept(s):
    return int(lib().jq_num_kept(ctypes.byref(s)))


def launch_count():
    return int(lib().jq_launch_count())


def _torch():
    import torch
    if not torch.cuda.is_available():
        raise RuntimeError("paper_2509_10798_b200 needs a CUDA device; there is no CPU path")
    return torch


def _stream(stream):
    if stream is None:
        stream = _torch().cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _raise(where, rc):
    if rc != JQ_OK:
        raise JqError(where, rc)


def new_workspace(s, device="cuda", stream=None):
    """Allocates and initialises a workspace tensor (uint8) for shape `s`."""
    torch = _torch()
    n = workspace_bytes(s)
    if n == 0:
        raise JqError("jq_workspace_bytes", check_shape(s) or JQ_ERR_INVALID_ARG)
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    _raise("jq_workspace_init", lib().jq_workspace_init(_ptr(ws), n, _stream(stream)))
    return ws


def score(K, Qwin, s, scores, ws, stream=None, fma=False):
    fn = lib().jq_score_fma if fma else lib().jq_score
    _raise("jq_score_fma" if fma else "jq_score",
           fn(_ptr(K), _ptr(Qwin), ctypes.byref(s), _ptr(scores), _ptr(ws), ws.numel(), _stream(stream)))


def score_static(K, Qwin, s, scores, stream=None):
    """jq_score without a workspace, for callers that may not allocate device memory: the scratch is a
    fixed array inside the library (at most 2048 query rows over all KV heads; calls share it, so keep
    them on one stream)."""
    _raise("jq_score_static",
           lib().jq_score_static(_ptr(K), _ptr(Qwin), ctypes.byref(s), _ptr(scores), _stream(stream)))


def score_windowed(K, Qwin, Kwin, s, scores, ws, stream=None):
    """jq_score with the causal window keys Kwin [Hkv, w, d] in the softmax denominator."""
    _raise("jq_score_windowed", lib().jq_score_windowed(_ptr(K), _ptr(Qwin), _ptr(Kwin), ctypes.byref(s), _ptr(scores),
                                                        _ptr(ws), ws.numel(), _stream(stream)))


def evict_layer_windowed(K, V, Qwin, Kwin, s, Kout, Vout, kept_idx, ws, stream=None):
    _raise("jq_evict_layer_windowed",
           lib().jq_evict_layer_windowed(_ptr(K), _ptr(V), _ptr(Qwin), _ptr(Kwin), ctypes.byref(s), _ptr(Kout), _ptr(Vout),
                                         _ptr(kept_idx), _ptr(ws), ws.numel(), _stream(stream)))


def evict_layer_window_kept(K, V, Qwin, Kwin, Vwin, s, Kout, Vout, kept_idx, ws, stream=None):
    """jq_evict_layer_window_kept: budget - w prefix rows chosen by the window-inclusive scores, then the w window rows."""
    _raise("jq_evict_layer_window_kept",
           lib().jq_evict_layer_window_kept(_ptr(K), _ptr(V), _ptr(Qwin), _ptr(Kwin), _ptr(Vwin), ctypes.byref(s), _ptr(Kout),
                                            _ptr(Vout), _ptr(kept_idx), _ptr(ws), ws.numel(), _stream(stream)))


def select_topk(scores, s, kept_idx, ws, pooled=None, stream=None):
    _raise("jq_select_topk", lib().jq_select_topk(_ptr(scores), ctypes.byref(s), _ptr(kept_idx), _ptr(pooled),
                                                  _ptr(ws), ws.numel(), _stream(stream)))


def compact_kv(K, V, kept_idx, s, Kout, Vout, stream=None):
    _raise("jq_compact_kv", lib().jq_compact_kv(_ptr(K), _ptr(V), _ptr(kept_idx), ctypes.byref(s), _ptr(Kout),
                                                _ptr(Vout), _stream(stream)))


def evict_layer(K, V, Qwin, s, Kout, Vout, kept_idx, ws, stream=None):
    _raise("jq_evict_layer", lib().jq_evict_layer(_ptr(K), _ptr(V), _ptr(Qwin), ctypes.byref(s), _ptr(Kout),
                                                  _ptr(Vout), _ptr(kept_idx), _ptr(ws), ws.numel(),
                                                  _stream(stream)))


def evict_layer_host(hK, hV, hQwin, s, hKout, hVout, hkept_idx, dev_buf, stream=None):
    """Host-tensor variant: all h* are CPU tensors (pinned for asynchronous copies)."""
    _raise("jq_evict_layer_host",
           lib().jq_evict_layer_host(_ptr(hK), _ptr(hV), _ptr(hQwin), ctypes.byref(s), _ptr(hKout), _ptr(hVout),
                                     _ptr(hkept_idx), _ptr(dev_buf), dev_buf.numel(), _stream(stream)))


def layers_workspace_bytes(s, nlayers):
    return int(lib().jq_layers_workspace_bytes(ctypes.byref(s), int(nlayers)))


def new_layers_workspace(s, nlayers, device="cuda", stream=None):
    """Allocates and initialises a workspace tensor (uint8) for evict_layers on nlayers layers of shape `s`."""
    torch = _torch()
    n = layers_workspace_bytes(s, nlayers)
    if n == 0:
        raise JqError("jq_layers_workspace_bytes", check_shape(s) or JQ_ERR_UNSUPPORTED)
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    _raise("jq_workspace_init", lib().jq_workspace_init(_ptr(ws), ws.numel(), _stream(stream)))
    return ws


def evict_layers(Ks, Vs, Qwins, s, Kout, Vout, kept_idx, ws, stream=None):
    """jq_evict_layers: Ks, Vs, Qwins are lists of per-layer CUDA tensors of shape `s`; the outputs are stacked."""
    n = len(Ks)
    arr = lambda ts: (ctypes.c_void_p * n)(*[t.data_ptr() for t in ts])
    _raise("jq_evict_layers",
           lib().jq_evict_layers(arr(Ks), arr(Vs), arr(Qwins), n, ctypes.byref(s), _ptr(Kout), _ptr(Vout), _ptr(kept_idx),
                                 _ptr(ws), ws.numel(), _stream(stream)))


def _ints(xs):
    return None if xs is None else (ctypes.c_int * len(xs))(*[int(x) for x in xs])


def ragged_workspace_bytes(s, nunits, L=None):
    return int(lib().jq_ragged_workspace_bytes(ctypes.byref(s), int(nunits), _ints(L)))


def ragged_output_rows(s, nunits, L=None, budget=None):
    return int(lib().jq_ragged_output_rows(ctypes.byref(s), int(nunits), _ints(L), _ints(budget)))


def new_ragged_workspace(s, nunits, L=None, device="cuda", stream=None):
    """Allocates and initialises a workspace tensor (uint8) for evict_ragged on nunits units of geometry `s`."""
    torch = _torch()
    n = ragged_workspace_bytes(s, nunits, L)
    if n == 0:
        raise JqError("jq_ragged_workspace_bytes", check_shape(s) or JQ_ERR_UNSUPPORTED)
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    _raise("jq_workspace_init", lib().jq_workspace_init(_ptr(ws), ws.numel(), _stream(stream)))
    return ws


def evict_ragged(Ks, Vs, Qwins, s, L, budget, Kout, Vout, kept_idx, ws, stream=None):
    """jq_evict_ragged: Ks, Vs, Qwins are lists of per-unit CUDA tensors; L, budget lists of ints (or None for
    s.L / s.budget everywhere); the outputs hold the units' blocks of Hkv * nkeep_u rows one after the other."""
    n = len(Ks)
    arr = lambda ts: (ctypes.c_void_p * n)(*[t.data_ptr() for t in ts])
    _raise("jq_evict_ragged",
           lib().jq_evict_ragged(arr(Ks), arr(Vs), arr(Qwins), n, ctypes.byref(s), _ints(L), _ints(budget), _ptr(Kout),
                                 _ptr(Vout), _ptr(kept_idx), _ptr(ws), ws.numel(), _stream(stream)))


def new_append_workspace(s, device="cuda", stream=None):
    torch = _torch()
    n = int(lib().jq_append_workspace_bytes(ctypes.byref(s)))
    if n == 0:
        raise JqError("jq_append_workspace_bytes", check_shape(s) or JQ_ERR_UNSUPPORTED)
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    _raise("jq_workspace_init", lib().jq_workspace_init(_ptr(ws), ws.numel(), _stream(stream)))
    return ws


def evict_append(Kc, Vc, n_old, Knew, Vnew, Qrecent, s, kept_idx, ws, stream=None):
    """jq_evict_append: Kc, Vc [Hkv, cap, d] hold n_old retained rows per head; Knew, Vnew [Hkv, n_new, d] are appended and
    the cache is evicted again to s.budget rows (s.L = n_old + n_new), in place."""
    n_new = 0 if Knew is None else int(Knew.shape[1])
    _raise("jq_evict_append",
           lib().jq_evict_append(_ptr(Kc), _ptr(Vc), int(Kc.shape[1]), int(n_old), _ptr(Knew), _ptr(Vnew), n_new, _ptr(Qrecent),
                                 ctypes.byref(s), _ptr(kept_idx), _ptr(ws), ws.numel(), _stream(stream)))


def decode_workspace_bytes(Hkv, Hq, n):
    return int(lib().jq_decode_workspace_bytes(int(Hkv), int(Hq), int(n)))


def decode_attention(Kc, Vc, q, out, ws, stream=None):
    """One decoding step over the pruned cache: Kc, Vc [Hkv,n,128] bf16, q [Hq,128] bf16 -> out [Hq,128] fp32."""
    _raise("jq_decode_attention", lib().jq_decode_attention(_ptr(Kc), _ptr(Vc), _ptr(q), int(Kc.shape[0]), int(q.shape[0]),
                                                            int(Kc.shape[1]), _ptr(out), _ptr(ws), ws.numel() * ws.element_size(), _stream(stream)))


def hit_rate(cur_idx, ref_idx, rate, stream=None):
    """Eq. 6 per KV head: the share of ref_idx's rows that cur_idx's rows also hold (rows ascending)."""
    _raise("jq_hit_rate", lib().jq_hit_rate(_ptr(cur_idx), _ptr(ref_idx), int(cur_idx.shape[0]), int(cur_idx.shape[1]),
                                            int(ref_idx.shape[1]), _ptr(rate), _stream(stream)))


def last_device_status(ws, stream=None):
    return int(lib().jq_last_device_status(_ptr(ws), _stream(stream)))
