"""ctypes front end of the fp64 CPU oracle (oracle/jq_oracle.c).

TEST INFRASTRUCTURE ONLY.  The oracle is the plain definition of the Judge Q
eviction pass (Eq. 3 scores -> max-pool -> top-k -> gather) that the CUDA
library is checked against.  Nothing in the product package imports this
module; only tests, the smoke check and the benchmark's CPU-baseline leg do.

All tensors are numpy arrays; bf16 data travels as uint16 bit patterns.
"""
import ctypes
import numpy as np

from .build import build as _build

_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build())
        c_int = ctypes.c_int
        vp = ctypes.c_void_p
        lib.jq_oracle_threads.argtypes = [c_int]
        lib.jq_oracle_threads.restype = c_int
        lib.jq_oracle_score_f64.argtypes = [vp, vp, c_int, c_int, c_int, c_int, c_int, vp, vp]
        lib.jq_oracle_score.argtypes = [vp, vp, c_int, c_int, c_int, c_int, c_int, vp, vp]
        lib.jq_oracle_score_windowed_f64.argtypes = [vp, vp, vp, c_int, c_int, c_int, c_int, c_int, vp, vp]
        lib.jq_oracle_score_windowed.argtypes = [vp, vp, vp, c_int, c_int, c_int, c_int, c_int, vp, vp]
        lib.jq_oracle_hit_rate.argtypes = [vp, vp, c_int, c_int, c_int, vp]
        lib.jq_oracle_decode_attention.argtypes = [vp, vp, vp, c_int, c_int, c_int, c_int, vp]
        lib.jq_oracle_pool.argtypes = [vp, c_int, c_int, c_int, vp]
        lib.jq_oracle_select.argtypes = [vp, c_int, c_int, c_int, vp]
        lib.jq_oracle_select_f32.argtypes = [vp, c_int, c_int, c_int, c_int, vp, vp]
        lib.jq_oracle_compact.argtypes = [vp, vp, vp, c_int, c_int, c_int, c_int, vp, vp]
        lib.jq_oracle_evict_layer.argtypes = [vp, vp, vp] + [c_int] * 7 + [vp] * 5
        _lib = lib
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _chk(a, dtype, shape=None):
    a = np.ascontiguousarray(a, dtype=dtype)
    if shape is not None and tuple(a.shape) != tuple(shape):
        raise ValueError("shape %s, expected %s" % (a.shape, shape))
    return a


def threads(units):
    """Threads the oracle uses for `units` KV heads (it parallelises over KV heads only)."""
    return int(_load().jq_oracle_threads(int(units)))


def score(K, Q, return_probs=False):
    """Eq. 3 pre-pool scores.  K [Hkv,L,d] uint16 (bf16 bits) or float64; Q [Hq,w,d] likewise.
    Returns score [Hkv,L] float64 (and the softmax rows [Hq,w,L] if asked)."""
    lib = _load()
    Hkv, L, d = K.shape
    Hq, w, d2 = Q.shape
    if d2 != d:
        raise ValueError("head dims differ")
    out = np.empty((Hkv, L), np.float64)
    probs = np.empty((Hq, w, L), np.float64) if return_probs else None
    if K.dtype == np.uint16:
        K, Q = _chk(K, np.uint16), _chk(Q, np.uint16)
        rc = lib.jq_oracle_score(_p(K), _p(Q), Hkv, Hq, L, d, w, _p(out), _p(probs))
    else:
        K, Q = _chk(K, np.float64), _chk(Q, np.float64)
        rc = lib.jq_oracle_score_f64(_p(K), _p(Q), Hkv, Hq, L, d, w, _p(out), _p(probs))
    if rc:
        raise ValueError("jq_oracle_score: bad arguments")
    return (out, probs) if return_probs else out


def score_windowed(K, Q, Kw, return_probs=False):
    """Window-inclusive scores: query i also attends, causally, to the window keys Kw[kv, i' <= i]; only the
    mass on the prefix keys is scored.  K [Hkv,L,d], Q [Hq,w,d], Kw [Hkv,w,d], all uint16 (bf16 bits) or all
    float64.  Returns score [Hkv,L] float64 (and the prefix part of the softmax rows [Hq,w,L] if asked)."""
    lib = _load()
    Hkv, L, d = K.shape
    Hq, w, _ = Q.shape
    if Kw.shape != (Hkv, w, d) or Q.shape[2] != d:
        raise ValueError("shapes of K, Q, Kw do not fit")
    out = np.empty((Hkv, L), np.float64)
    probs = np.empty((Hq, w, L), np.float64) if return_probs else None
    if K.dtype == np.uint16:
        K, Q, Kw = _chk(K, np.uint16), _chk(Q, np.uint16), _chk(Kw, np.uint16)
        rc = lib.jq_oracle_score_windowed(_p(K), _p(Q), _p(Kw), Hkv, Hq, L, d, w, _p(out), _p(probs))
    else:
        K, Q, Kw = _chk(K, np.float64), _chk(Q, np.float64), _chk(Kw, np.float64)
        rc = lib.jq_oracle_score_windowed_f64(_p(K), _p(Q), _p(Kw), Hkv, Hq, L, d, w, _p(out), _p(probs))
    if rc:
        raise ValueError("jq_oracle_score_windowed: bad arguments")
    return (out, probs) if return_probs else out


def pool(scores, p):
    """Centred max of odd width p over the key axis, same length.  scores [Hkv,L] float64."""
    s = _chk(scores, np.float64)
    Hkv, L = s.shape
    out = np.empty_like(s)
    if _load().jq_oracle_pool(_p(s), Hkv, L, int(p), _p(out)):
        raise ValueError("jq_oracle_pool: bad arguments")
    return out


def select(pooled, budget):
    """Top-min(budget,L) per head, ties to the lower index, ascending.  Returns int32 [Hkv,nkeep]."""
    s = _chk(pooled, np.float64)
    Hkv, L = s.shape
    nkeep = min(int(budget), L)
    idx = np.empty((Hkv, max(nkeep, 0)), np.int32)
    if _load().jq_oracle_select(_p(s), Hkv, L, int(budget), _p(idx)):
        raise ValueError("jq_oracle_select: bad arguments")
    return idx


def select_f32(scores_f32, budget, p):
    """pool + select on fp32 scores (stage isolation).  Returns (idx int32, pooled float32)."""
    s = _chk(scores_f32, np.float32)
    Hkv, L = s.shape
    nkeep = min(int(budget), L)
    idx = np.empty((Hkv, max(nkeep, 0)), np.int32)
    pooled = np.empty_like(s)
    if _load().jq_oracle_select_f32(_p(s), Hkv, L, int(budget), int(p), _p(idx), _p(pooled)):
        raise ValueError("jq_oracle_select_f32: bad arguments")
    return idx, pooled


def hit_rate(cur, ref):
    """Eq. 6: per KV head, the share of the reference kept set `ref` [Hkv,nref] that `cur` [Hkv,ncur] also keeps."""
    cur, ref = _chk(cur, np.int32), _chk(ref, np.int32)
    out = np.empty(cur.shape[0], np.float64)
    if _load().jq_oracle_hit_rate(_p(cur), _p(ref), cur.shape[0], cur.shape[1], ref.shape[1], _p(out)):
        raise ValueError("jq_oracle_hit_rate: bad arguments")
    return out


def decode_attention(Kc, Vc, q):
    """One decoding step over the pruned cache: Kc, Vc [Hkv,n,d], q [Hq,d] bf16 bits -> out [Hq,d] float64."""
    Kc, Vc, q = _chk(Kc, np.uint16), _chk(Vc, np.uint16, Kc.shape), _chk(q, np.uint16)
    Hkv, n, d = Kc.shape
    out = np.empty((q.shape[0], d), np.float64)
    if q.shape[1] != d or _load().jq_oracle_decode_attention(_p(Kc), _p(Vc), _p(q), Hkv, q.shape[0], n, d, _p(out)):
        raise ValueError("jq_oracle_decode_attention: bad arguments")
    return out


def compact(K, V, idx):
    """Gather rows.  K,V [Hkv,L,d] uint16; idx [Hkv,nkeep] int32."""
    K, V = _chk(K, np.uint16), _chk(V, np.uint16, K.shape)
    idx = _chk(idx, np.int32)
    Hkv, L, d = K.shape
    nkeep = idx.shape[1]
    Ko = np.empty((Hkv, nkeep, d), np.uint16)
    Vo = np.empty_like(Ko)
    if _load().jq_oracle_compact(_p(K), _p(V), _p(idx), Hkv, L, d, nkeep, _p(Ko), _p(Vo)):
        raise ValueError("jq_oracle_compact: bad arguments")
    return Ko, Vo


def evict_layer(K, V, Q, budget, p, return_scores=False):
    """The whole pass.  Returns (Kout, Vout, idx[, score, pooled])."""
    K, V, Q = _chk(K, np.uint16), _chk(V, np.uint16, K.shape), _chk(Q, np.uint16)
    Hkv, L, d = K.shape
    Hq, w, _ = Q.shape
    nkeep = min(int(budget), L)
    Ko = np.empty((Hkv, max(nkeep, 0), d), np.uint16)
    Vo = np.empty_like(Ko)
    idx = np.empty((Hkv, max(nkeep, 0)), np.int32)
    sc = np.empty((Hkv, L), np.float64) if return_scores else None
    po = np.empty((Hkv, L), np.float64) if return_scores else None
    rc = _load().jq_oracle_evict_layer(_p(K), _p(V), _p(Q), Hkv, Hq, L, d, w, int(budget), int(p),
                                       _p(Ko), _p(Vo), _p(idx), _p(sc), _p(po))
    if rc:
        raise ValueError("jq_oracle_evict_layer: bad arguments")
    return (Ko, Vo, idx, sc, po) if return_scores else (Ko, Vo, idx)
