"""Seeded synthetic KV caches and soft-token queries for the five benchmark configurations.

Only input generation lives here (no part of the eviction method's arithmetic), so both the
CPU oracle's tests and the CUDA library's tests and benchmark can draw the very same bits.
The shapes, lengths and budgets follow the paper's workloads (Llama-3.1-8B-Instruct and
Mistral-7B-Instruct-v0.3 caches of 4K-32K tokens, 32 soft tokens, budgets 128-3072; Tables
2-5 and the needle experiment); the values are stand-ins for the LongBench / RULER /
needle-in-a-haystack caches, which need model weights and datasets that are not available.

All tensors are numpy uint16 arrays holding bf16 bit patterns (fp32 values rounded to
nearest-even once):  K, V [Hkv, L, d];  Qwin [Hq, w, d].
Seeds: 1000*config + layer (+ 100000*sequence for the ragged batch).
"""
from dataclasses import dataclass, replace
import numpy as np

D = 128
POOL = 7


@dataclass(frozen=True)
class Workload:
    name: str
    config: int
    Hkv: int
    Hq: int
    L: int
    w: int
    budget: int
    pool: int = POOL
    d: int = D
    layers: int = 1          # layer calls that make up one pass over the model
    distinct_layers: int = 1  # how many of them have their own tensors

    @property
    def group(self):
        return self.Hq // self.Hkv

    @property
    def R(self):
        return self.group * self.w

    @property
    def nkeep(self):
        return min(self.budget, self.L)

    def with_budget(self, budget):
        return replace(self, budget=int(budget))

    def with_L(self, L):
        return replace(self, L=int(L))


CFG1 = Workload("cfg1-tiny", 1, Hkv=2, Hq=8, L=2048, w=16, budget=256)
CFG2 = Workload("cfg2-llama8b-8k", 2, Hkv=8, Hq=32, L=8192, w=32, budget=1024)
CFG3 = Workload("cfg3-llama8b-32k-32layers", 3, Hkv=8, Hq=32, L=32768, w=32, budget=512,
                layers=32, distinct_layers=32)
CFG3_BUDGETS = (128, 512, 2048)
CFG4_LENGTHS = (4096, 12000, 20480, 32768)
CFG4 = tuple(Workload("cfg4-mistral7b-ragged-L%d" % L, 4, Hkv=8, Hq=32, L=L, w=32, budget=1024,
                      layers=32, distinct_layers=32) for L in CFG4_LENGTHS)
CFG5 = Workload("cfg5-llama8b-128k", 5, Hkv=8, Hq=32, L=131072, w=64, budget=1024,
                layers=32, distinct_layers=1)
CFG5_BUDGETS = (256, 1024, 2048, 4096)


def bf16_bits(x):
    """float32 array -> uint16 bf16 bit patterns, round to nearest even (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def bf16_to_f32(b):
    """uint16 bf16 bit patterns -> float32 (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(seed, stream):
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([int(seed), int(stream)])))


def _normal(rng, shape):
    return rng.standard_normal(shape, dtype=np.float32)


def make_v(wl, seed):
    """V ~ N(0,1) from a stream of its own (V never influences the selection)."""
    return bf16_bits(_normal(_rng(seed, 2), (wl.Hkv, wl.L, wl.d)))


def _q_from_planted(rng, wl, Kf, planted):
    """Row rho of KV head kv = 0.7 N(0,1) + 0.3 K[kv, planted[kv][rho mod len]]."""
    g, w, d = wl.group, wl.w, wl.d
    Q = 0.7 * _normal(rng, (wl.Hq, w, d))
    for kv in range(wl.Hkv):
        pl = planted[kv]
        for hl in range(g):
            rho = hl * w + np.arange(w)
            Q[kv * g + hl] += 0.3 * Kf[kv, pl[rho % len(pl)], :]
    return Q


def _gen_tiny(wl, seed):
    """Config 1: N(0,1) keys, 8 duplicated key rows per head (tie-break exercise), 24 planted rows."""
    rng = _rng(seed, 1)
    K = bf16_to_f32(bf16_bits(_normal(rng, (wl.Hkv, wl.L, wl.d))))
    planted, dups = [], []
    n_pl = min(24, wl.L)
    n_dup = 8 if wl.L >= 64 else 0
    for kv in range(wl.Hkv):
        pl = rng.choice(wl.L, size=n_pl, replace=False)
        planted.append(pl)
        pairs = []
        taken = set(int(x) for x in pl)
        for t in range(n_dup):
            src = int(pl[t]) if t < n_dup // 2 else int(rng.integers(wl.L))
            while True:
                dst = int(rng.integers(wl.L))
                if abs(dst - src) > wl.pool and dst not in taken:
                    break
            taken.add(dst)
            K[kv, dst, :] = K[kv, src, :]
            pairs.append((src, dst))
        dups.append(pairs)
    Q = _q_from_planted(rng, wl, K, planted)
    return bf16_bits(K), bf16_bits(Q), {"planted": planted, "dups": dups}


def _gen_outlier(wl, seed):
    """Configs 2, 3, 5: N(0,1) keys with 4 outlier channels x8 per head; 64 planted heavy keys spread
    over the context plus 16 in the last 256 positions."""
    rng = _rng(seed, 1)
    K = _normal(rng, (wl.Hkv, wl.L, wl.d))
    for kv in range(wl.Hkv):
        ch = rng.choice(wl.d, size=4, replace=False)
        K[kv, :, ch] *= 8.0
    K = bf16_to_f32(bf16_bits(K))
    planted = []
    n_spread = min(64, wl.L)
    tail = min(256, wl.L)
    for kv in range(wl.Hkv):
        u = rng.random(n_spread)
        spread = np.minimum(((np.arange(n_spread) + u) * wl.L / n_spread).astype(np.int64), wl.L - 1)
        recent = wl.L - tail + rng.choice(tail, size=min(16, tail), replace=False)
        planted.append(np.concatenate([spread, recent]))
    Q = _q_from_planted(rng, wl, K, planted)
    return bf16_bits(K), bf16_bits(Q), {"planted": planted}


def _gen_clusters(wl, seed):
    """Config 4: topic-like keys from 16 Gaussian clusters in contiguous segments, 32 isolated needles;
    queries aligned to 3 clusters plus the needles."""
    rng = _rng(seed, 1)
    Hkv, L, d, g, w = wl.Hkv, wl.L, wl.d, wl.group, wl.w
    K = np.empty((Hkv, L, d), np.float32)
    Q = 0.5 * _normal(rng, (wl.Hq, w, d))
    needles_all = []
    R = wl.R
    n_needle = min(32, L)
    n_cluster_rows = max(R - n_needle, 0)
    for kv in range(Hkv):
        centres = _normal(rng, (16, d))
        pos = 0
        lab = np.empty(L, np.int64)
        while pos < L:
            seg = int(rng.integers(64, 1025))
            lab[pos:pos + seg] = int(rng.integers(16))
            pos += seg
        K[kv] = centres[lab] + 0.5 * _normal(rng, (L, d))
        needles = rng.choice(L, size=n_needle, replace=False)
        K[kv, needles, :] = 1.5 * _normal(rng, (n_needle, d))
        needles_all.append(needles)
        chosen = rng.choice(16, size=3, replace=False)
        Kh = bf16_to_f32(bf16_bits(K[kv]))
        noise = _normal(rng, (R, d))
        for rho in range(R):
            h, i = kv * g + rho // w, rho % w
            if rho < n_cluster_rows:
                Q[h, i] += 0.5 * centres[chosen[rho % 3]]
            else:
                Q[h, i] = 0.7 * noise[rho] + 0.3 * Kh[needles[(rho - n_cluster_rows) % n_needle]]
    return bf16_bits(K), bf16_bits(Q), {"needles": needles_all}


def seed_of(wl, layer=0, seq=0):
    return 1000 * wl.config + int(layer) + 100000 * int(seq)


def make_layer(wl, layer=0, seq=0, with_v=True):
    """Returns (K, V, Qwin, info) as uint16 bf16 bit patterns; V is None if with_v is False."""
    seed = seed_of(wl, layer, seq)
    if wl.config == 1:
        K, Q, info = _gen_tiny(wl, seed)
    elif wl.config == 4:
        K, Q, info = _gen_clusters(wl, seed)
    else:
        K, Q, info = _gen_outlier(wl, seed)
    V = make_v(wl, seed) if with_v else None
    return K, V, Q, info


def make_window_keys(wl, Q, layer=0, seq=0):
    """Keys of the w query positions themselves, [Hkv, w, d] bf16 bits, for the window-inclusive mode:
    N(0,1) plus 0.3 x the mean query of the position over the GQA group (a token's key resembles its
    query a little, so that the window takes a visible but not dominant share of the attention)."""
    rng = _rng(seed_of(wl, layer, seq), 3)
    Qf = bf16_to_f32(Q).reshape(wl.Hkv, wl.group, wl.w, wl.d)
    return bf16_bits(_normal(rng, (wl.Hkv, wl.w, wl.d)) + 0.3 * Qf.mean(axis=1))


def formula_bytes(wl):
    """Algorithmic HBM bytes of one layer call: two reads of K, one read of the kept V rows, the
    writes of the compacted K and V and of the int32 indices."""
    row = wl.d * 2
    return 2 * wl.Hkv * wl.L * row + wl.Hkv * wl.nkeep * row + 2 * wl.Hkv * wl.nkeep * row + wl.Hkv * wl.nkeep * 4
