"""Pins for the fp64 CPU oracle: what the paper's definitions and plain mathematics fix.

The paper prints no worked numeric example of the eviction pass, so the oracle is pinned by
invariants, closed forms, library special cases and brute force, chosen so that a dropped term,
a wrong scale, a transposed operand, a wrong GQA mapping or a wrong tie rule fails at least one.
"""
import math

import numpy as np
import pytest
import torch

import oracle
import jq_workloads as W


def rnd_bf16(rng, shape, scale=1.0):
    return W.bf16_bits(scale * rng.standard_normal(shape, dtype=np.float32))


def as_f64(bits):
    return W.bf16_to_f32(bits).astype(np.float64)


# ---------------------------------------------------------------- softmax / Eq. 3

def test_rows_sum_to_one_and_mass_is_w_times_group():
    rng = np.random.default_rng(1)
    Hkv, g, w, L, d = 3, 2, 5, 97, 16
    K = rnd_bf16(rng, (Hkv, L, d))
    Q = rnd_bf16(rng, (Hkv * g, w, d), 2.0)
    score, probs = oracle.score(K, Q, return_probs=True)
    assert probs.shape == (Hkv * g, w, L)
    assert np.all(probs >= 0)
    np.testing.assert_allclose(probs.sum(-1), 1.0, atol=1e-12, rtol=0)
    np.testing.assert_allclose(score.sum(-1), w * g, atol=1e-9, rtol=0)
    # the score is the sum of the rows of the heads that share the KV head (contiguous groups)
    np.testing.assert_allclose(score, probs.reshape(Hkv, g * w, L).sum(1), atol=1e-12, rtol=0)


def test_single_query_equals_library_softmax():
    rng = np.random.default_rng(2)
    L, d = 301, 128
    K = rnd_bf16(rng, (1, L, d))
    Q = rnd_bf16(rng, (1, 1, d))
    got = oracle.score(K, Q)[0]
    logits = torch.from_numpy(as_f64(K)[0]) @ torch.from_numpy(as_f64(Q)[0, 0]) / math.sqrt(d)
    want = torch.softmax(logits, dim=0).numpy()
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-15)


def test_gqa_against_library_softmax_asymmetric_shapes():
    """Hkv, g, w, L, d all different so that a swapped axis or a wrong head->KV map shows."""
    rng = np.random.default_rng(3)
    Hkv, g, w, L, d = 2, 3, 4, 53, 8
    K = rnd_bf16(rng, (Hkv, L, d))
    Q = rnd_bf16(rng, (Hkv * g, w, d), 1.5)
    got = oracle.score(K, Q)
    Kt, Qt = torch.from_numpy(as_f64(K)), torch.from_numpy(as_f64(Q))
    want = np.zeros((Hkv, L))
    for h in range(Hkv * g):
        logits = Qt[h] @ Kt[h // g].T / math.sqrt(d)       # [w, L]
        want[h // g] += torch.softmax(logits, dim=-1).sum(0).numpy()
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-15)


def test_key_shift_invariance():
    """Adding one vector u to every key adds q.u/sqrt(d) to a whole row: softmax is unchanged."""
    rng = np.random.default_rng(4)
    Hkv, g, w, L, d = 2, 2, 3, 40, 16
    K = rng.standard_normal((Hkv, L, d))
    Q = rng.standard_normal((Hkv * g, w, d))
    u = rng.standard_normal((Hkv, 1, d))
    a = oracle.score(K, Q)
    b = oracle.score(K + u, Q)
    np.testing.assert_allclose(a, b, rtol=1e-10, atol=1e-14)


def test_key_permutation_permutes_scores():
    rng = np.random.default_rng(5)
    K = rnd_bf16(rng, (2, 64, 32))
    Q = rnd_bf16(rng, (4, 3, 32))
    perm = rng.permutation(64)
    a = oracle.score(K, Q)
    b = oracle.score(K[:, perm, :], Q)
    np.testing.assert_allclose(a[:, perm], b, rtol=1e-12, atol=1e-15)


def test_duplicate_key_rows_score_identically():
    rng = np.random.default_rng(6)
    K = rnd_bf16(rng, (1, 50, 16))
    K[0, 37] = K[0, 5]
    Q = rnd_bf16(rng, (2, 4, 16))
    s = oracle.score(K, Q)
    assert s[0, 37] == s[0, 5]


def test_zero_queries_uniform_scores_and_lowest_indices_kept():
    """Q = 0: every probability is 1/L, every score R/L, all tied -> the first nkeep indices."""
    Hkv, g, w, L, d, B = 2, 4, 3, 100, 8, 17
    rng = np.random.default_rng(7)
    K = rnd_bf16(rng, (Hkv, L, d))
    V = rnd_bf16(rng, (Hkv, L, d))
    Q = np.zeros((Hkv * g, w, d), np.uint16)
    Ko, Vo, idx, sc, po = oracle.evict_layer(K, V, Q, B, 7, return_scores=True)
    np.testing.assert_allclose(sc, g * w / L, rtol=1e-13)
    assert np.array_equal(idx, np.tile(np.arange(B, dtype=np.int32), (Hkv, 1)))
    assert np.array_equal(Ko, K[:, :B]) and np.array_equal(Vo, V[:, :B])


def test_one_hot_closed_form():
    """Queries alpha*e_a, one key beta*e_a, all other keys 0:  P(j*) = e^t / (e^t + L - 1) with
    t = alpha*beta/sqrt(d); every other key gets 1/(e^t + L - 1).  Pins the 1/sqrt(d) scale."""
    L, d, g, w = 200, 64, 2, 3
    alpha, beta, a, jstar = 3.0, 2.5, 11, 123
    Kf = np.zeros((1, L, d), np.float32)
    Kf[0, jstar, a] = beta
    Qf = np.zeros((g, w, d), np.float32)
    Qf[:, :, a] = alpha
    s = oracle.score(W.bf16_bits(Kf), W.bf16_bits(Qf))[0]
    t = alpha * beta / math.sqrt(d)
    z = math.exp(t) + L - 1
    np.testing.assert_allclose(s[jstar], g * w * math.exp(t) / z, rtol=1e-13)
    np.testing.assert_allclose(np.delete(s, jstar), g * w / z, rtol=1e-13)
    # a wrong scale (1/d, or none) must miss this value by far more than the tolerance
    for wrong in (alpha * beta / d, alpha * beta):
        assert abs(g * w * math.exp(wrong) / (math.exp(wrong) + L - 1) - s[jstar]) > 1e-3


def test_multi_needle_kept_set():
    """Three needles on distinct axes with distinct strengths, one per KV-head-specific position:
    pooled plateaus around each needle; the kept set is plateau(s) in strength order, then the
    lowest remaining indices."""
    L, d, p, r = 300, 32, 7, 3
    Hkv, g, w = 2, 2, 4
    needles = {0: [(40, 1, 6.0), (150, 2, 5.0), (260, 3, 4.0)],
               1: [(10, 4, 4.0), (200, 5, 6.0), (297, 6, 5.0)]}
    Kf = np.zeros((Hkv, L, d), np.float32)
    Qf = np.zeros((Hkv * g, w, d), np.float32)
    for kv, lst in needles.items():
        for (j, ax, strength) in lst:
            Kf[kv, j, ax] = strength
            Qf[kv * g:(kv + 1) * g, :, ax] = 4.0
    K, Q = W.bf16_bits(Kf), W.bf16_bits(Qf)
    V = np.arange(Hkv * L * d, dtype=np.uint32).astype(np.uint16).reshape(Hkv, L, d)

    def plateau(j):
        return set(range(max(0, j - r), min(L, j + r + 1)))

    for B in (1, 3, 7, 9, 14, 18, 21, 30):
        _, _, idx = oracle.evict_layer(K, V, Q, B, p)
        for kv, lst in needles.items():
            ranked = []                       # positions in (strength desc, index asc) order
            for (j, _, _) in sorted(lst, key=lambda t: -t[2]):
                ranked += sorted(plateau(j))
            rest = [j for j in range(L) if j not in set(ranked)]
            want = sorted((ranked + rest)[:B])
            assert idx[kv].tolist() == want, (B, kv)


# ---------------------------------------------------------------- pooling

def brute_pool(s, p):
    L = len(s)
    r = (p - 1) // 2
    out = []
    for j in range(L):
        best = None
        for u in range(j - r, j + r + 1):
            if 0 <= u < L and (best is None or s[u] > best):
                best = s[u]
        out.append(best)
    return np.array(out)


@pytest.mark.parametrize("L", [1, 2, 3, 6, 7, 8, 33])
@pytest.mark.parametrize("p", [1, 3, 7, 9])
def test_pool_brute_force_and_library(L, p):
    rng = np.random.default_rng(100 * L + p)
    s = rng.random((2, L))
    got = oracle.pool(s, p)
    for kv in range(2):
        assert np.array_equal(got[kv], brute_pool(s[kv], p))
    lib = torch.nn.functional.max_pool1d(torch.from_numpy(s)[None], kernel_size=p, stride=1,
                                         padding=(p - 1) // 2)[0].numpy()
    assert np.array_equal(got, lib)
    assert np.all(got >= s)
    assert np.array_equal(got.max(-1), s.max(-1))
    if p == 1:
        assert np.array_equal(got, s)


def test_pool_rejects_even_width():
    with pytest.raises(ValueError):
        oracle.pool(np.zeros((1, 8)), 4)


# ---------------------------------------------------------------- selection

@pytest.mark.parametrize("L,B", [(1, 1), (5, 9), (64, 1), (64, 63), (64, 64), (257, 40), (1000, 333)])
def test_select_matches_library_stable_sort(L, B):
    rng = np.random.default_rng(L * 7 + B)
    # few distinct values -> ties everywhere, the normal case after max-pooling
    pooled = rng.integers(0, 6, size=(3, L)).astype(np.float64) / 8.0
    idx = oracle.select(pooled, B)
    nkeep = min(B, L)
    assert idx.shape == (3, nkeep) and idx.dtype == np.int32
    for kv in range(3):
        order = np.argsort(-pooled[kv], kind="stable")[:nkeep]
        assert idx[kv].tolist() == sorted(order.tolist())
        kept = np.zeros(L, bool)
        kept[idx[kv]] = True
        assert np.all(np.diff(idx[kv]) > 0)
        if nkeep < L:
            tau = pooled[kv][kept].min()
            assert tau >= pooled[kv][~kept].max()
            at_tau = np.flatnonzero(pooled[kv] == tau)
            k_tau, e_tau = at_tau[kept[at_tau]], at_tau[~kept[at_tau]]
            if len(k_tau) and len(e_tau):
                assert k_tau.max() < e_tau.min()      # lower index wins a tie


def test_select_f32_pool_is_exact_and_consistent():
    rng = np.random.default_rng(11)
    s = rng.random((2, 500), dtype=np.float32)
    idx, pooled = oracle.select_f32(s, 50, 7)
    assert np.array_equal(pooled.astype(np.float64), oracle.pool(s.astype(np.float64), 7))
    assert np.array_equal(idx, oracle.select(pooled.astype(np.float64), 50))


# ---------------------------------------------------------------- compaction / whole pass

def test_compact_copies_rows_bitwise():
    Hkv, L, d = 2, 40, 8
    K = (np.arange(Hkv * L * d) % 65521).astype(np.uint16).reshape(Hkv, L, d)
    V = ((np.arange(Hkv * L * d) * 7 + 3) % 65521).astype(np.uint16).reshape(Hkv, L, d)
    idx = np.array([[0, 3, 39], [1, 2, 38]], np.int32)
    Ko, Vo = oracle.compact(K, V, idx)
    for kv in range(Hkv):
        for t in range(3):
            assert np.array_equal(Ko[kv, t], K[kv, idx[kv, t]])
            assert np.array_equal(Vo[kv, t], V[kv, idx[kv, t]])
    with pytest.raises(ValueError):
        oracle.compact(K, V, np.array([[0, 1, 40], [0, 1, 2]], np.int32))


def test_evict_layer_is_the_composition_and_budget_ge_L_keeps_all():
    rng = np.random.default_rng(12)
    Hkv, g, w, L, d = 2, 2, 3, 90, 16
    K, V = rnd_bf16(rng, (Hkv, L, d)), rnd_bf16(rng, (Hkv, L, d))
    Q = rnd_bf16(rng, (Hkv * g, w, d), 3.0)
    Ko, Vo, idx, sc, po = oracle.evict_layer(K, V, Q, 20, 7, return_scores=True)
    assert np.array_equal(sc, oracle.score(K, Q))
    assert np.array_equal(po, oracle.pool(sc, 7))
    assert np.array_equal(idx, oracle.select(po, 20))
    Ko2, Vo2 = oracle.compact(K, V, idx)
    assert np.array_equal(Ko, Ko2) and np.array_equal(Vo, Vo2)
    Ko, Vo, idx = oracle.evict_layer(K, V, Q, 1000, 7)
    assert np.array_equal(idx, np.tile(np.arange(L, dtype=np.int32), (Hkv, 1)))
    assert np.array_equal(Ko, K) and np.array_equal(Vo, V)


def test_mean_instead_of_sum_keeps_the_same_set():
    """Eq. 3 averages over the n soft tokens; the oracle sums.  A positive rescale changes no rank."""
    rng = np.random.default_rng(13)
    K = rnd_bf16(rng, (1, 128, 16))
    Q = rnd_bf16(rng, (2, 8, 16), 3.0)
    s = oracle.score(K, Q)
    assert np.array_equal(oracle.select(oracle.pool(s, 7), 16), oracle.select(oracle.pool(s / 8.0, 7), 16))


def test_config1_planted_and_duplicates():
    """Config 1 recipe: duplicated key rows tie exactly; planted rows dominate the kept set."""
    wl = W.CFG1
    K, V, Q, info = W.make_layer(wl)
    assert K.shape == (wl.Hkv, wl.L, wl.d) and Q.shape == (wl.Hq, wl.w, wl.d)
    Ko, Vo, idx, sc, po = oracle.evict_layer(K, V, Q, wl.budget, wl.pool, return_scores=True)
    np.testing.assert_allclose(sc.sum(-1), wl.R, atol=1e-9)
    for kv in range(wl.Hkv):
        for (src, dst) in info["dups"][kv]:
            assert np.array_equal(K[kv, src], K[kv, dst])
            assert sc[kv, src] == sc[kv, dst]
        kept = set(idx[kv].tolist())
        hit = sum(int(j) in kept for j in info["planted"][kv])
        assert hit >= 20, hit                     # 24 planted heavy keys, budget 256


# ---------------------------------------------------------------- window-inclusive scores

def _rand_kqw(Hkv, g, w, L, d=16, seed=0):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((Hkv, L, d)), rng.standard_normal((Hkv * g, w, d)), rng.standard_normal((Hkv, w, d)))


def test_windowed_equals_library_softmax_over_masked_concatenation():
    """Each row against torch.softmax over [prefix logits, window logits] with the causal mask, prefix part kept."""
    import torch
    Hkv, g, w, L, d = 2, 3, 5, 37, 16
    K, Q, Kw = _rand_kqw(Hkv, g, w, L, d, seed=3)
    score, probs = oracle.score_windowed(K, Q, Kw, return_probs=True)
    want = np.zeros((Hkv, L))
    for h in range(Hkv * g):
        kv = h // g
        keys = torch.from_numpy(np.concatenate([K[kv], Kw[kv]], 0))                     # [L+w, d]
        logits = torch.from_numpy(Q[h]) @ keys.T / np.sqrt(d)                            # [w, L+w]
        mask = torch.zeros((w, L + w), dtype=torch.bool)
        for i in range(w):
            mask[i, L + i + 1:] = True                                                   # window keys after the query
        p = torch.softmax(logits.masked_fill(mask, float("-inf")), dim=-1).numpy()
        np.testing.assert_allclose(probs[h], p[:, :L], rtol=1e-12, atol=1e-15)
        want[kv] += p[:, :L].sum(0)
    np.testing.assert_allclose(score, want, rtol=1e-12)
    assert np.all(score.sum(-1) < g * w)          # some mass went to the window


def test_windowed_zero_queries_closed_form_pins_the_mask_direction():
    Hkv, g, w, L, d = 1, 2, 6, 50, 8
    K, Q, Kw = _rand_kqw(Hkv, g, w, L, d, seed=4)
    _, probs = oracle.score_windowed(K, np.zeros_like(Q), Kw, return_probs=True)
    for i in range(w):      # query i sees L prefix keys and i + 1 window keys, all with logit 0
        np.testing.assert_allclose(probs[:, i, :], 1.0 / (L + i + 1), rtol=1e-13)


def test_window_that_attracts_no_mass_gives_the_plain_scores():
    Hkv, g, w, L, d = 2, 2, 4, 64, 16
    K, Q, _ = _rand_kqw(Hkv, g, w, L, d, seed=5)
    u = np.ones(d) / np.sqrt(d)
    Q = Q * 0.1 + 3.0 * u                      # every query has a large component along u ...
    Kw = np.tile(-200.0 * u, (Hkv, w, 1))      # ... and every window key points the other way: logits near -150
    np.testing.assert_allclose(oracle.score_windowed(K, Q, Kw), oracle.score(K, Q), rtol=1e-12)


def test_windowed_bf16_entry_matches_double_entry():
    Hkv, g, w, L = 2, 2, 3, 40
    rng = np.random.default_rng(6)
    K = W.bf16_bits(rng.standard_normal((Hkv, L, 128), dtype=np.float32))
    Q = W.bf16_bits(rng.standard_normal((Hkv * g, w, 128), dtype=np.float32))
    Kw = W.bf16_bits(rng.standard_normal((Hkv, w, 128), dtype=np.float32))
    f = lambda b: W.bf16_to_f32(b).astype(np.float64)
    np.testing.assert_allclose(oracle.score_windowed(K, Q, Kw), oracle.score_windowed(f(K), f(Q), f(Kw)), rtol=1e-14)


# ---------------------------------------------------------------- Eq. 6, hit rate

def test_hit_rate_special_cases_and_library_intersection():
    rng = np.random.default_rng(8)
    a = np.stack([np.sort(rng.choice(500, 64, replace=False)) for _ in range(3)]).astype(np.int32)
    np.testing.assert_array_equal(oracle.hit_rate(a, a), 1.0)                        # a set against itself
    np.testing.assert_array_equal(oracle.hit_rate(a, a + 1000), 0.0)                  # disjoint sets
    b = np.stack([np.sort(rng.choice(500, 40, replace=False)) for _ in range(3)]).astype(np.int32)
    want = [len(np.intersect1d(a[k], b[k])) / 40.0 for k in range(3)]                 # library set intersection
    np.testing.assert_allclose(oracle.hit_rate(a, b), want, rtol=0, atol=0)
    half = np.concatenate([a[:, :32], a[:, 32:] + 1000], axis=1).astype(np.int32)    # exactly half shared
    np.testing.assert_array_equal(oracle.hit_rate(half, a), 0.5)


# ---------------------------------------------------------------- decoding step over the pruned cache

def _decode_case(Hkv, group, n, seed, d=128):
    rng = np.random.default_rng(seed)
    Kc = W.bf16_bits(rng.standard_normal((Hkv, n, d)).astype(np.float32))
    Vc = W.bf16_bits(rng.standard_normal((Hkv, n, d)).astype(np.float32))
    q = W.bf16_bits((2.0 * rng.standard_normal((Hkv * group, d))).astype(np.float32))
    return Kc, Vc, q


def test_decode_attention_matches_library_softmax_and_matmul():
    Kc, Vc, q = _decode_case(3, 4, 257, 5)
    got = oracle.decode_attention(Kc, Vc, q)
    Kf, Vf, qf = (torch.from_numpy(W.bf16_to_f32(x).astype(np.float64)) for x in (Kc, Vc, q))
    for h in range(q.shape[0]):
        kv = h // 4
        p = torch.softmax(Kf[kv] @ qf[h] / math.sqrt(128.0), dim=0)
        np.testing.assert_allclose(got[h], (p @ Vf[kv]).numpy(), rtol=1e-12, atol=1e-14)


def test_decode_attention_closed_forms():
    Kc, Vc, q = _decode_case(2, 2, 64, 6)
    Vf = W.bf16_to_f32(Vc).astype(np.float64)
    # q = 0: uniform weights, the mean of the head's V rows (and of the RIGHT head: GQA mapping h -> h // group)
    got = oracle.decode_attention(Kc, Vc, np.zeros_like(q))
    for h in range(4):
        np.testing.assert_allclose(got[h], Vf[h // 2].mean(0), rtol=1e-13, atol=1e-15)
    # one key aligned with the query and scaled up takes all the mass: the output is its V row
    Kf = W.bf16_to_f32(Kc).copy()
    qf = W.bf16_to_f32(q)
    Kf[1, 17] = 64.0 * qf[3]                       # head 3 -> KV head 1
    got = oracle.decode_attention(W.bf16_bits(Kf), Vc, q)
    np.testing.assert_allclose(got[3], Vf[1, 17], rtol=0, atol=1e-9)
    # n = 1: the single V row, whatever the logits
    got = oracle.decode_attention(Kc[:, :1], Vc[:, :1], q)
    for h in range(4):
        np.testing.assert_array_equal(got[h], Vf[h // 2, 0])
    # the order of the keys does not matter when V is permuted alike
    perm = np.random.default_rng(0).permutation(64)
    np.testing.assert_allclose(oracle.decode_attention(Kc[:, perm], Vc[:, perm], q), oracle.decode_attention(Kc, Vc, q),
                               rtol=1e-12, atol=1e-14)
    # scaling: logits are divided by sqrt(d) (a query scaled by 4 with d = 128 is not the same as one with d = 8)
    Kc8, Vc8, q8 = _decode_case(1, 1, 9, 7, d=8)
    s = W.bf16_to_f32(Kc8)[0].astype(np.float64) @ W.bf16_to_f32(q8)[0].astype(np.float64) / math.sqrt(8.0)
    p = np.exp(s - s.max()); p /= p.sum()
    np.testing.assert_allclose(oracle.decode_attention(Kc8, Vc8, q8)[0], p @ W.bf16_to_f32(Vc8)[0].astype(np.float64), rtol=1e-12)
