"""GPU parity: the CUDA library (through its C ABI) against the fp64 CPU oracle, element by element.

Agreement rules: integer / byte / index work is bit-exact when fed identical scores; pre-pool and
pooled scores agree within 2e-3 relative + 1e-6 absolute (fp32 accumulation of bf16 products);
end to end, kept sets may differ only at positions whose oracle pooled score lies within 1e-4
relative of the k-th pooled score.
"""
import numpy as np
import pytest
import torch

import oracle
import jq_workloads as W
import paper_2509_10798_b200 as jq
from gpu_util import (assert_kept_sets_agree, assert_scores_close, dev_bf16, gpu_evict, gpu_score,
                      gpu_select, host_bits, shape_of)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    import __graft_entry__ as entry
    entry.build()


def small_wl(Hkv, g, w, L, budget, pool=7, config=2):
    return W.Workload("t", config, Hkv=Hkv, Hq=Hkv * g, L=L, w=w, budget=budget, pool=pool)


# ------------------------------------------------------------------ scores (steps 1-3)

SCORE_CASES = [
    # Hkv, g, w, L : tiles of 128 keys -> below one tile, exact tiles, ragged tails, several tiles
    (1, 1, 1, 1), (1, 1, 1, 7), (2, 1, 3, 8), (1, 2, 5, 127), (2, 4, 16, 128), (2, 4, 16, 129),
    (3, 4, 32, 300), (2, 4, 32, 1000), (1, 4, 64, 777), (2, 4, 64, 2049), (8, 4, 32, 1536),
    (2, 8, 32, 515), (1, 3, 11, 4000),
]


@pytest.mark.parametrize("fma", [False, True], ids=["tensor", "fma"])
@pytest.mark.parametrize("Hkv,g,w,L", SCORE_CASES)
def test_score_small_shapes(Hkv, g, w, L, fma):
    wl = small_wl(Hkv, g, w, L, 1)
    K, _, Q, _ = W.make_layer(wl, with_v=False)
    want = oracle.score(K, Q)
    got = gpu_score(K, Q, shape_of(wl), fma=fma)
    assert_scores_close(got, want)
    np.testing.assert_allclose(got.sum(-1), wl.R, rtol=1e-3)


@pytest.mark.parametrize("fma", [False, True], ids=["tensor", "fma"])
@pytest.mark.parametrize("wl", [W.CFG1, W.CFG2, W.CFG4[1].with_L(3000)], ids=lambda w: w.name)
def test_score_configs(wl, fma):
    K, _, Q, _ = W.make_layer(wl, with_v=False)
    assert_scores_close(gpu_score(K, Q, shape_of(wl), fma=fma), oracle.score(K, Q))


def test_score_zero_queries_is_uniform():
    wl = small_wl(2, 4, 16, 999, 1)
    K, _, Q, _ = W.make_layer(wl, with_v=False)
    got = gpu_score(K, np.zeros_like(Q), shape_of(wl))
    np.testing.assert_allclose(got, wl.R / wl.L, rtol=1e-5)


def test_score_large_logits_do_not_overflow():
    """Strongly peaked rows (logit range of several hundred) must stay finite and normalised."""
    wl = small_wl(1, 2, 8, 640, 1)
    K, _, Q, _ = W.make_layer(wl, with_v=False)
    Qs = W.bf16_bits(W.bf16_to_f32(Q) * 24.0)
    got = gpu_score(K, Qs, shape_of(wl))
    assert np.all(np.isfinite(got))
    assert_scores_close(got, oracle.score(K, Qs))


def test_score_rising_logits_raise_the_running_reference():
    """Keys whose logits climb by hundreds from tile to tile: pass 1 must raise its reference and stay exact."""
    wl = small_wl(1, 2, 8, 1500, 1)
    rng = np.random.default_rng(5)
    u = rng.standard_normal(128).astype(np.float32)
    u /= np.linalg.norm(u)
    ramp = np.linspace(-40.0, 40.0, wl.L, dtype=np.float32)[:, None]
    Kf = ramp * u[None, :] + 0.1 * rng.standard_normal((wl.L, 128)).astype(np.float32)
    Qf = 300.0 * u[None, None, :] + rng.standard_normal((wl.Hq, wl.w, 128)).astype(np.float32)
    K, Q = W.bf16_bits(Kf[None]), W.bf16_bits(Qf)
    got = gpu_score(K, Q, shape_of(wl))
    assert np.all(np.isfinite(got))
    assert_scores_close(got, oracle.score(K, Q))
    np.testing.assert_allclose(got.sum(-1), wl.R, rtol=1e-3)


# ------------------------------------------------------------------ pool + select (steps 4-5), bit-exact

SELECT_CASES = [(1, 1, 1, 7), (1, 5, 9, 7), (2, 6, 3, 7), (2, 64, 64, 7), (3, 257, 40, 7), (2, 1000, 333, 3),
                (2, 4096, 1024, 7), (1, 5000, 4999, 9), (2, 33000, 2048, 7), (1, 70001, 4096, 1),
                (8, 8192, 1024, 7)]


@pytest.mark.parametrize("Hkv,L,B,p", SELECT_CASES)
@pytest.mark.parametrize("kind", ["random", "ties", "oracle_scores"])
def test_select_bit_exact(Hkv, L, B, p, kind):
    rng = np.random.default_rng(L * 31 + B)
    if kind == "random":
        s32 = rng.random((Hkv, L), dtype=np.float32)
    elif kind == "ties":
        s32 = (rng.integers(0, 5, size=(Hkv, L)) / 4.0).astype(np.float32)
    else:
        wl = small_wl(Hkv, 2, 4, L, B, p)
        K, _, Q, _ = W.make_layer(wl, with_v=False)
        s32 = oracle.score(K, Q).astype(np.float32)
    want_idx, want_pooled = oracle.select_f32(s32, B, p)
    s = jq.shape(Hkv, Hkv, L, 1, B, p)
    got_idx, got_pooled = gpu_select(s32, s)
    assert np.array_equal(got_pooled.view(np.uint32), want_pooled.view(np.uint32))
    assert np.array_equal(got_idx, want_idx)


# With many heads the selection runs smaller clusters (4 or 2 CTAs per head instead of 8) and, from 128 heads on, the
# kernel that gives every head one CTA of 512 or 1024 threads (1024 in the last case): same results.
# The tied inputs put more keys into the winning histogram bin than its candidate list holds.
@pytest.mark.parametrize("Hkv,L,B,p", [(64, 4096, 512, 7), (160, 5000, 700, 7), (300, 1000, 100, 5), (148, 40000, 2048, 7),
                                       (200, 1, 1, 7), (200, 5, 9, 7), (100, 33, 10, 3), (256, 70001, 300, 1),
                                       (130, 4001, 4001, 9), (129, 1023, 77, 9), (400, 70000, 500, 7), (128, 200001, 1000, 9)])
@pytest.mark.parametrize("kind", ["random", "ties"])
def test_select_many_heads_bit_exact(Hkv, L, B, p, kind):
    rng = np.random.default_rng(Hkv * 7 + L)
    if kind == "random":
        s32 = rng.random((Hkv, L), dtype=np.float32)
    else:
        s32 = (rng.integers(0, 5, size=(Hkv, L)) / 4.0).astype(np.float32)
    want_idx, want_pooled = oracle.select_f32(s32, B, p)
    got_idx, got_pooled = gpu_select(s32, jq.shape(Hkv, Hkv, L, 1, B, p))
    assert np.array_equal(got_pooled.view(np.uint32), want_pooled.view(np.uint32))
    assert np.array_equal(got_idx, want_idx)


@pytest.mark.parametrize("Hkv", [2, 150])
def test_select_all_equal_keeps_lowest_indices(Hkv):
    s32 = np.full((Hkv, 5000), 0.25, np.float32)
    idx, _ = gpu_select(s32, jq.shape(Hkv, Hkv, 5000, 1, 777, 7))
    assert np.array_equal(idx, np.tile(np.arange(777, dtype=np.int32), (Hkv, 1)))


# ------------------------------------------------------------------ compaction (step 6), bit-exact

@pytest.mark.parametrize("Hkv,L,n", [(1, 1, 1), (2, 100, 7), (8, 4096, 1024), (3, 5000, 4999)])
def test_compact_bit_exact(Hkv, L, n):
    rng = np.random.default_rng(L + n)
    K = rng.integers(0, 65536, size=(Hkv, L, 128), dtype=np.uint16)
    V = rng.integers(0, 65536, size=(Hkv, L, 128), dtype=np.uint16)
    idx = np.stack([np.sort(rng.choice(L, size=n, replace=False)) for _ in range(Hkv)]).astype(np.int32)
    s = jq.shape(Hkv, Hkv, L, 1, n, 7)
    Ko = torch.zeros((Hkv, n, 128), dtype=torch.bfloat16, device="cuda")
    Vo = torch.zeros_like(Ko)
    jq.compact_kv(dev_bf16(K), dev_bf16(V), torch.from_numpy(idx).cuda(), s, Ko, Vo)
    wK, wV = oracle.compact(K, V, idx)
    assert np.array_equal(host_bits(Ko), wK) and np.array_equal(host_bits(Vo), wV)


# ------------------------------------------------------------------ whole pass

def run_e2e(wl, K, V, Q, pooled=None):
    s = shape_of(wl)
    gKo, gVo, gidx = gpu_evict(K, V, Q, s)
    if pooled is None:
        pooled = oracle.pool(oracle.score(K, Q), wl.pool)
    oidx = oracle.select(pooled, wl.budget)
    swaps = assert_kept_sets_agree(gidx, oidx, pooled, wl.nkeep)
    for kv in range(wl.Hkv):           # gathered bytes are exactly the rows the GPU chose
        assert np.array_equal(gKo[kv], K[kv][gidx[kv]]) and np.array_equal(gVo[kv], V[kv][gidx[kv]])
    if swaps == 0:
        oKo, oVo = oracle.compact(K, V, oidx)
        assert np.array_equal(gKo, oKo) and np.array_equal(gVo, oVo)
    return swaps


@pytest.mark.parametrize("wl", [W.CFG1, W.CFG2, W.CFG2.with_budget(100000), W.CFG4[0], W.CFG4[1],
                                small_wl(2, 4, 16, 5, 3), small_wl(1, 4, 64, 1, 1), small_wl(160, 1, 4, 5000, 700)],
                         ids=lambda w: "%s-L%d-B%d" % (w.name, w.L, w.budget))
def test_evict_layer_end_to_end(wl):
    K, V, Q, _ = W.make_layer(wl)
    run_e2e(wl, K, V, Q)


def test_evict_layer_zero_queries_ties_everywhere():
    wl = small_wl(2, 4, 16, 3000, 500)
    K, V, Q, _ = W.make_layer(wl)
    _, _, gidx = gpu_evict(K, V, np.zeros_like(Q), shape_of(wl))
    # all scores tie (up to fp32 noise the oracle rule tolerates); the structure must still be valid
    assert gidx.shape == (2, 500) and np.all(np.diff(gidx, axis=1) > 0)


def test_evict_layer_is_deterministic_and_workspace_reusable():
    wl = W.CFG2.with_L(5000)
    K, V, Q, _ = W.make_layer(wl)
    s = shape_of(wl)
    ws = jq.new_workspace(s)
    dK, dV, dQ = dev_bf16(K), dev_bf16(V), dev_bf16(Q)
    outs = []
    for _ in range(3):
        Ko = torch.zeros((s.Hkv, wl.nkeep, s.d), dtype=torch.bfloat16, device="cuda")
        Vo = torch.zeros_like(Ko)
        idx = torch.zeros((s.Hkv, wl.nkeep), dtype=torch.int32, device="cuda")
        jq.evict_layer(dK, dV, dQ, s, Ko, Vo, idx, ws)
        outs.append((host_bits(Ko), host_bits(Vo), idx.cpu().numpy()))
    assert jq.last_device_status(ws) == jq.JQ_OK
    for o in outs[1:]:
        for a, b in zip(outs[0], o):
            assert np.array_equal(a, b)


def test_host_entry_matches_device_entry():
    wl = W.CFG2.with_L(3000)
    K, V, Q, _ = W.make_layer(wl)
    s = shape_of(wl)
    gKo, gVo, gidx = gpu_evict(K, V, Q, s)
    pin = lambda a: torch.from_numpy(a.view(np.int16)).pin_memory()
    hK, hV, hQ = pin(K), pin(V), pin(Q)
    hKo = torch.zeros((s.Hkv, wl.nkeep, s.d), dtype=torch.int16).pin_memory()
    hVo = torch.zeros_like(hKo).pin_memory()
    hidx = torch.zeros((s.Hkv, wl.nkeep), dtype=torch.int32).pin_memory()
    buf = torch.empty(jq.host_call_bytes(s), dtype=torch.uint8, device="cuda")
    # page-locked V (only the kept rows cross to the device) and pageable V (copied whole): same results
    for v_in in (hV, torch.from_numpy(V.view(np.int16).copy())):
        hKo.zero_(); hVo.zero_(); hidx.zero_()
        jq.evict_layer_host(hK, v_in, hQ, s, hKo, hVo, hidx, buf)
        torch.cuda.synchronize()
        assert np.array_equal(hidx.numpy(), gidx)
        assert np.array_equal(hKo.numpy().view(np.uint16), gKo) and np.array_equal(hVo.numpy().view(np.uint16), gVo)


# ------------------------------------------------------------------ full-size workloads (bench launch configuration)

def test_cfg3_full_size_layer_budget_sweep():
    K, V, Q, _ = W.make_layer(W.CFG3, layer=7)
    pooled = oracle.pool(oracle.score(K, Q), W.CFG3.pool)     # scores do not depend on the budget
    for budget in W.CFG3_BUDGETS:
        run_e2e(W.CFG3.with_budget(budget), K, V, Q, pooled)


@pytest.mark.parametrize("seq", [2, 3])
def test_cfg4_long_sequences(seq):
    wl = W.CFG4[seq]                                           # L = 20480 and 32768 (0 and 1 run in test_evict_layer_end_to_end)
    K, V, Q, _ = W.make_layer(wl, layer=1, seq=seq)
    run_e2e(wl, K, V, Q)


def test_cfg5_full_size_all_heads():
    """L = 131072, R = 256: the whole layer, all eight KV heads, against the oracle, for every budget of
    the sweep."""
    wl = W.CFG5
    K, V, Q, _ = W.make_layer(wl)
    s = shape_of(wl)
    heads = list(range(wl.Hkv))
    g = wl.group
    qrows = np.concatenate([np.arange(kv * g, kv * g + g) for kv in heads])
    sc = oracle.score(K[heads], Q[qrows])
    got = gpu_score(K, Q, s)
    assert_scores_close(got[heads], sc)
    np.testing.assert_allclose(got.sum(-1), wl.R, rtol=1e-3)
    po = oracle.pool(sc, wl.pool)
    for budget in W.CFG5_BUDGETS:
        wb = wl.with_budget(budget)
        gKo, gVo, gidx = gpu_evict(K, V, Q, shape_of(wb))
        oidx = oracle.select(po, budget)
        assert_kept_sets_agree(gidx[heads], oidx, po, wb.nkeep)
        for kv in range(wl.Hkv):
            assert np.all(np.diff(gidx[kv]) > 0)
            assert np.array_equal(gKo[kv], K[kv][gidx[kv]]) and np.array_equal(gVo[kv], V[kv][gidx[kv]])


# ------------------------------------------------------------------ bounded waits (failure is made on the host)

def test_wait_that_nothing_ends_times_out_and_leaves_the_context_usable():
    """A grid counter the kernel waits for is set, from the host, to a value it can never reach.  Every wait
    in the kernel is bounded, so the call must come back with JQ_ERR_TIMEOUT in the status word (no trap,
    no hang), and the same workspace must work again after jq_workspace_init."""
    wl = small_wl(2, 4, 16, 700, 1)
    K, _, Q, _ = W.make_layer(wl, with_v=False)
    s = shape_of(wl)
    ws = jq.new_workspace(s)
    torch.cuda.synchronize()
    ws.view(torch.int32)[8] = -(1 << 28)            # first pass-1 completion counter: unreachable
    out = torch.zeros((s.Hkv, s.L), dtype=torch.float32, device="cuda")
    jq.score(dev_bf16(K), dev_bf16(Q), s, out, ws)
    assert jq.last_device_status(ws) == jq.JQ_ERR_TIMEOUT
    lib = jq.lib()
    import ctypes
    assert lib.jq_workspace_init(ctypes.c_void_p(ws.data_ptr()), ws.numel(), ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)) == jq.JQ_OK
    jq.score(dev_bf16(K), dev_bf16(Q), s, out, ws)
    assert jq.last_device_status(ws) == jq.JQ_OK
    assert_scores_close(out.cpu().numpy(), oracle.score(K, Q))


def test_score_full_size_is_bitwise_repeatable():
    """The 128K-key, 256-row workload three times in a row: every launch must give the same bits (all
    reductions have a fixed order; the two additions per key of the wide mode commute)."""
    wl = W.CFG5
    K, _, Q, _ = W.make_layer(wl, with_v=False)
    s = shape_of(wl)
    ws = jq.new_workspace(s)
    dK, dQ = dev_bf16(K), dev_bf16(Q)
    outs = []
    for _ in range(3):
        out = torch.full((s.Hkv, s.L), -1.0, dtype=torch.float32, device="cuda")
        jq.score(dK, dQ, s, out, ws)
        assert jq.last_device_status(ws) == jq.JQ_OK
        outs.append(out.cpu().numpy())
    assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[0], outs[2])


def test_layers_stacked_along_the_head_axis_equal_separate_calls():
    """Every (layer, KV head) is an independent unit: one call on K, V, Qwin of several layers stacked along
    the head axis must give, bit for bit, what one call per layer gives."""
    wl = small_wl(2, 4, 32, 2500, 300)
    layers = [W.make_layer(wl, layer=i) for i in range(3)]
    K = np.concatenate([l[0] for l in layers]); V = np.concatenate([l[1] for l in layers]); Q = np.concatenate([l[2] for l in layers])
    sS = jq.shape(wl.Hkv * 3, wl.Hq * 3, wl.L, wl.w, wl.budget, wl.pool, wl.d)
    gKo, gVo, gidx = gpu_evict(K, V, Q, sS)
    for i, (Ki, Vi, Qi, _) in enumerate(layers):
        Ko, Vo, idx = gpu_evict(Ki, Vi, Qi, shape_of(wl))
        sl = slice(i * wl.Hkv, (i + 1) * wl.Hkv)
        assert np.array_equal(idx, gidx[sl]) and np.array_equal(Ko, gKo[sl]) and np.array_equal(Vo, gVo[sl])


# ------------------------------------------------------------------ the benchmark's launch configuration

def _stacked_call(K_layers, V_layers, Q_layers, wl):
    """One jq_evict_layer call on layers stacked along the KV-head axis, tensors built on the device."""
    n = len(K_layers)
    dK = torch.cat([dev_bf16(k) for k in K_layers], 0)
    dV = torch.cat([dev_bf16(v) for v in V_layers], 0)
    dQ = torch.cat([dev_bf16(q) for q in Q_layers], 0)
    s = jq.shape(wl.Hkv * n, wl.Hq * n, wl.L, wl.w, wl.budget, wl.pool, wl.d)
    ws = jq.new_workspace(s)
    Ko = torch.zeros((s.Hkv, wl.nkeep, s.d), dtype=torch.bfloat16, device="cuda")
    Vo = torch.zeros_like(Ko)
    idx = torch.full((s.Hkv, wl.nkeep), -1, dtype=torch.int32, device="cuda")
    jq.evict_layer(dK, dV, dQ, s, Ko, Vo, idx, ws)
    assert jq.last_device_status(ws) == jq.JQ_OK
    return Ko, Vo, idx.cpu().numpy()


def test_cfg3_all_32_layers_in_one_stacked_call_sampled_heads():
    """The benchmark's call for the 32K workload: 32 distinct layers, 256 stacked KV heads, one launch of each
    kernel.  The oracle recomputes sampled (layer, head) units in full; every unit's structure is checked."""
    wl = W.CFG3
    layers = [W.make_layer(wl, layer=i) for i in range(wl.layers)]
    Ko, Vo, idx = _stacked_call([l[0] for l in layers], [l[1] for l in layers], [l[2] for l in layers], wl)
    g = wl.group
    for layer, kv in ((0, 0), (13, 5), (31, 7)):
        K, V, Q, _ = layers[layer]
        po = oracle.pool(oracle.score(K[kv:kv + 1], Q[kv * g:(kv + 1) * g]), wl.pool)
        oidx = oracle.select(po, wl.budget)
        u = layer * wl.Hkv + kv
        assert_kept_sets_agree(idx[u:u + 1], oidx, po, wl.nkeep)
        assert np.array_equal(host_bits(Ko[u]), K[kv][idx[u]]) and np.array_equal(host_bits(Vo[u]), V[kv][idx[u]])
    assert np.all(np.diff(idx, axis=1) > 0) and idx.min() >= 0 and idx.max() < wl.L


def test_cfg5_32_copies_in_one_stacked_call_sampled_heads():
    """The benchmark's call for the 128K workload: one layer copied 32 times (16 GiB of K and V), 256 stacked
    KV heads.  Copies must agree with one another bit for bit and a sampled head with the oracle."""
    wl = W.CFG5
    K, V, Q, _ = W.make_layer(wl)
    Ko, Vo, idx = _stacked_call([K] * wl.layers, [V] * wl.layers, [Q] * wl.layers, wl)
    for c in range(1, wl.layers):
        assert np.array_equal(idx[:wl.Hkv], idx[c * wl.Hkv:(c + 1) * wl.Hkv])
    kv, g = 3, wl.group
    po = oracle.pool(oracle.score(K[kv:kv + 1], Q[kv * g:(kv + 1) * g]), wl.pool)
    oidx = oracle.select(po, wl.budget)
    for c in (0, 17, 31):
        u = c * wl.Hkv + kv
        assert_kept_sets_agree(idx[u:u + 1], oidx, po, wl.nkeep)
        assert np.array_equal(host_bits(Ko[u]), K[kv][idx[u]]) and np.array_equal(host_bits(Vo[u]), V[kv][idx[u]])


# ------------------------------------------------------------------ window-inclusive mode

def gpu_score_windowed(K, Q, Kw, s):
    ws = jq.new_workspace(s)
    out = torch.full((s.Hkv, s.L), -1.0, dtype=torch.float32, device="cuda")
    jq.score_windowed(dev_bf16(K), dev_bf16(Q), dev_bf16(Kw), s, out, ws)
    assert jq.last_device_status(ws) == jq.JQ_OK
    return out.cpu().numpy()


@pytest.mark.parametrize("Hkv,g,w,L", [(1, 1, 1, 5), (2, 4, 16, 129), (3, 4, 32, 1000), (2, 4, 64, 2049), (1, 3, 11, 4000),
                                       (8, 4, 32, 8192)])
def test_score_windowed_matches_oracle(Hkv, g, w, L):
    wl = small_wl(Hkv, g, w, L, 1)
    K, _, Q, _ = W.make_layer(wl, with_v=False)
    Kw = W.make_window_keys(wl, Q)
    want = oracle.score_windowed(K, Q, Kw)
    got = gpu_score_windowed(K, Q, Kw, shape_of(wl))
    assert_scores_close(got, want)
    plain = oracle.score(K, Q)
    assert np.all(want.sum(-1) < plain.sum(-1))           # the window did take mass (the case is not vacuous)


def test_score_windowed_with_dominant_window_keys():
    """Window keys far more attractive than any prefix key: nearly all mass leaves the prefix; still exact."""
    wl = small_wl(2, 2, 8, 700, 1)
    K, _, Q, _ = W.make_layer(wl, with_v=False)
    Kw = W.bf16_bits(3.0 * W.bf16_to_f32(Q).reshape(2, 2, 8, 128).mean(axis=1))
    want = oracle.score_windowed(K, Q, Kw)
    got = gpu_score_windowed(K, Q, Kw, shape_of(wl))
    assert_scores_close(got, want)
    assert want.sum() < 0.5 * wl.R * wl.Hkv


def test_evict_layer_windowed_end_to_end():
    wl = W.CFG2.with_L(5000)
    K, V, Q, _ = W.make_layer(wl)
    Kw = W.make_window_keys(wl, Q)
    s = shape_of(wl)
    ws = jq.new_workspace(s)
    Ko = torch.zeros((s.Hkv, wl.nkeep, s.d), dtype=torch.bfloat16, device="cuda")
    Vo = torch.zeros_like(Ko)
    idx = torch.full((s.Hkv, wl.nkeep), -1, dtype=torch.int32, device="cuda")
    jq.evict_layer_windowed(dev_bf16(K), dev_bf16(V), dev_bf16(Q), dev_bf16(Kw), s, Ko, Vo, idx, ws)
    assert jq.last_device_status(ws) == jq.JQ_OK
    gidx = idx.cpu().numpy()
    pooled = oracle.pool(oracle.score_windowed(K, Q, Kw), wl.pool)
    assert_kept_sets_agree(gidx, oracle.select(pooled, wl.budget), pooled, wl.nkeep)
    gK, gV = host_bits(Ko), host_bits(Vo)
    for kv in range(wl.Hkv):
        assert np.array_equal(gK[kv], K[kv][gidx[kv]]) and np.array_equal(gV[kv], V[kv][gidx[kv]])


# ------------------------------------------------------------------ Eq. 6

@pytest.mark.parametrize("Hkv,L,na,nb", [(1, 10, 3, 3), (8, 8192, 1024, 1024), (3, 70000, 4096, 512), (2, 300, 300, 1)])
def test_hit_rate_matches_oracle(Hkv, L, na, nb):
    rng = np.random.default_rng(L + na)
    a = np.stack([np.sort(rng.choice(L, na, replace=False)) for _ in range(Hkv)]).astype(np.int32)
    b = np.stack([np.sort(rng.choice(L, nb, replace=False)) for _ in range(Hkv)]).astype(np.int32)
    out = torch.full((Hkv,), -1.0, dtype=torch.float32, device="cuda")
    jq.hit_rate(torch.from_numpy(a).cuda(), torch.from_numpy(b).cuda(), out)
    np.testing.assert_allclose(out.cpu().numpy(), oracle.hit_rate(a, b), rtol=1e-7)


# ------------------------------------------------------------------ the step after the pass: decoding over the pruned cache

def gpu_decode(Kc, Vc, q):
    dKc, dVc, dq = dev_bf16(Kc), dev_bf16(Vc), dev_bf16(q)
    out = torch.full((q.shape[0], 128), float("nan"), dtype=torch.float32, device="cuda")
    ws = torch.empty(jq.decode_workspace_bytes(Kc.shape[0], q.shape[0], Kc.shape[1]), dtype=torch.uint8, device="cuda")
    jq.decode_attention(dKc, dVc, dq, out, ws)
    torch.cuda.synchronize()
    return out.cpu().numpy()


# fp32 sums of at most a few thousand products of bf16 values of unit size, weights from exp2f: absolute error of the
# output (a convex combination of V values of size ~1) stays below 2e-5
@pytest.mark.parametrize("Hkv,group,n", [(1, 1, 1), (2, 4, 63), (2, 4, 64), (3, 8, 65), (8, 4, 512), (8, 4, 1024), (2, 2, 5000),
                                         (8, 4, 4096)])
def test_decode_attention_matches_oracle(Hkv, group, n):
    rng = np.random.default_rng(n * 13 + group)
    Kc = W.bf16_bits(rng.standard_normal((Hkv, n, 128)).astype(np.float32))
    Vc = W.bf16_bits(rng.standard_normal((Hkv, n, 128)).astype(np.float32))
    q = W.bf16_bits((3.0 * rng.standard_normal((Hkv * group, 128))).astype(np.float32))
    np.testing.assert_allclose(gpu_decode(Kc, Vc, q), oracle.decode_attention(Kc, Vc, q), rtol=1e-4, atol=2e-5)


def test_decode_attention_large_logits_stay_finite():
    rng = np.random.default_rng(3)
    u = rng.standard_normal(128).astype(np.float32)
    Kc = W.bf16_bits((30.0 * u[None, None, :] * rng.standard_normal((2, 300, 1))).astype(np.float32))
    Vc = W.bf16_bits(rng.standard_normal((2, 300, 128)).astype(np.float32))
    q = W.bf16_bits(np.tile(30.0 * u, (8, 1)).astype(np.float32))
    got = gpu_decode(Kc, Vc, q)
    assert np.all(np.isfinite(got))
    np.testing.assert_allclose(got, oracle.decode_attention(Kc, Vc, q), rtol=1e-4, atol=2e-5)


def test_evict_then_decode_then_evict_again():
    """Streaming use: evict, decode over the pruned cache, append new rows, evict again - every step against the oracle."""
    wl = small_wl(2, 4, 16, 3000, 400)
    K, V, Q, _ = W.make_layer(wl)
    run_e2e(wl, K, V, Q)
    Kc, Vc, _ = gpu_evict(K, V, Q, shape_of(wl))
    q = np.ascontiguousarray(Q[:, -1, :])                    # the last soft token's queries stand in for a decoding step
    np.testing.assert_allclose(gpu_decode(Kc, Vc, q), oracle.decode_attention(Kc, Vc, q), rtol=1e-4, atol=2e-5)
    # 200 newly decoded positions join the pruned cache, which is evicted again to the budget
    K2, V2, Q2, _ = W.make_layer(small_wl(2, 4, 16, 200, 400), layer=1)
    Kn, Vn = np.concatenate([Kc, K2], axis=1), np.concatenate([Vc, V2], axis=1)
    run_e2e(small_wl(2, 4, 16, Kn.shape[1], 400), Kn, Vn, Q2)


# ------------------------------------------------------------------ several layers in buffers of their own, one call

@pytest.mark.parametrize("Hkv,g,w,L,B,nl", [(2, 4, 16, 3000, 400, 5), (2, 4, 64, 2049, 300, 3), (8, 4, 32, 8192, 1024, 32),
                                            (1, 1, 1, 5, 3, 2), (3, 2, 8, 130, 1000, 7)])
def test_evict_layers_matches_calls_per_layer(Hkv, g, w, L, B, nl):
    wl = small_wl(Hkv, g, w, L, B)
    s = shape_of(wl)
    layers = [W.make_layer(wl, layer=i) for i in range(nl)]
    pad = torch.empty(1000, dtype=torch.uint8, device="cuda")     # keeps the layers' buffers from being neighbours
    dK, dV, dQ = [], [], []
    for K, V, Q, _ in layers:
        dK.append(dev_bf16(K)); dV.append(dev_bf16(V)); dQ.append(dev_bf16(Q))
        pad = torch.empty(pad.numel() + 4096, dtype=torch.uint8, device="cuda")
    nkeep = wl.nkeep
    Ko = torch.zeros((nl * Hkv, nkeep, 128), dtype=torch.bfloat16, device="cuda")
    Vo = torch.zeros_like(Ko)
    idx = torch.full((nl * Hkv, nkeep), -1, dtype=torch.int32, device="cuda")
    ws = jq.new_layers_workspace(s, nl)
    for _ in range(2):                                            # twice: the workspace is reusable as it is left
        Ko.zero_(); Vo.zero_(); idx.fill_(-1)
        jq.evict_layers(dK, dV, dQ, s, Ko, Vo, idx, ws)
        assert jq.last_device_status(ws) == jq.JQ_OK
        gK, gV, gi = host_bits(Ko), host_bits(Vo), idx.cpu().numpy()
        for i, (K, V, Q, _) in enumerate(layers):
            wK, wV, wi = gpu_evict(K, V, Q, s)
            sl = slice(i * Hkv, (i + 1) * Hkv)
            assert np.array_equal(gi[sl], wi) and np.array_equal(gK[sl], wK) and np.array_equal(gV[sl], wV)
    # and one layer of it against the oracle, under the end-to-end rule
    K, V, Q, _ = layers[nl - 1]
    pooled = oracle.pool(oracle.score(K, Q), wl.pool)
    assert_kept_sets_agree(gi[(nl - 1) * Hkv:], oracle.select(pooled, wl.budget), pooled, nkeep)


def _layers_call(layers, wl, ws=None):
    """jq_evict_layers on the given (K, V, Q) host layers of workload wl, each in a device buffer of its own."""
    nl = len(layers)
    dK, dV, dQ = [dev_bf16(l[0]) for l in layers], [dev_bf16(l[1]) for l in layers], [dev_bf16(l[2]) for l in layers]
    s = shape_of(wl)
    Ko = torch.zeros((nl * wl.Hkv, wl.nkeep, 128), dtype=torch.bfloat16, device="cuda")
    Vo = torch.zeros_like(Ko)
    idx = torch.full((nl * wl.Hkv, wl.nkeep), -1, dtype=torch.int32, device="cuda")
    if ws is None:
        ws = jq.new_layers_workspace(s, nl)
    jq.evict_layers(dK, dV, dQ, s, Ko, Vo, idx, ws)
    assert jq.last_device_status(ws) == jq.JQ_OK
    return host_bits(Ko), host_bits(Vo), idx.cpu().numpy()


def test_evict_layers_workspace_reused_with_other_buffers_and_shapes():
    """One workspace, three calls in a row on different layer buffers, layer counts and shapes: the per-layer
    tensor maps the call leaves in the workspace are rewritten every time, and the kernel must read the new
    ones (the first call's buffers are freed before the second runs)."""
    wa, wb = small_wl(2, 4, 32, 3000, 400), small_wl(4, 4, 64, 1500, 200)
    need = max(jq.layers_workspace_bytes(shape_of(wa), 6), jq.layers_workspace_bytes(shape_of(wb), 3))
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    jq._raise("jq_workspace_init", jq.lib().jq_workspace_init(jq._ptr(ws), ws.numel(), jq._stream(None)))
    for wl, nl, first in ((wa, 6, 0), (wb, 3, 10), (wa, 4, 20), (wb, 2, 30)):
        layers = [W.make_layer(wl, layer=first + i) for i in range(nl)]
        gK, gV, gi = _layers_call(layers, wl, ws)
        for i, (K, V, Q, _) in enumerate(layers):
            wK, wV, wi = gpu_evict(K, V, Q, shape_of(wl))
            sl = slice(i * wl.Hkv, (i + 1) * wl.Hkv)
            assert np.array_equal(gi[sl], wi) and np.array_equal(gK[sl], wK) and np.array_equal(gV[sl], wV)
        torch.cuda.empty_cache()


def test_evict_layers_cfg5_shape_against_the_oracle():
    """The benchmark's default call at the 128K-key shape (three distinct layers here), compared with the oracle
    directly on sampled (layer, head) units."""
    wl = W.CFG5
    layers = [W.make_layer(wl, layer=i) for i in range(3)]
    gK, gV, gi = _layers_call(layers, wl)
    g = wl.group
    for layer, kv in ((0, 1), (1, 6), (2, 3), (2, 7)):
        K, V, Q, _ = layers[layer]
        po = oracle.pool(oracle.score(K[kv:kv + 1], Q[kv * g:(kv + 1) * g]), wl.pool)
        u = layer * wl.Hkv + kv
        assert_kept_sets_agree(gi[u:u + 1], oracle.select(po, wl.budget), po, wl.nkeep)
        assert np.array_equal(gK[u], K[kv][gi[u]]) and np.array_equal(gV[u], V[kv][gi[u]])
    assert np.all(np.diff(gi, axis=1) > 0) and gi.min() >= 0 and gi.max() < wl.L


# ------------------------------------------------------------------ ragged units: lengths and budgets of their own, one call

def _ragged_call(units, s_common, Ls, Bs, ws=None):
    """jq_evict_ragged on host units (K, V, Q); returns per-unit (Kout bits, Vout bits, idx) slices of the stacked outputs."""
    n = len(units)
    dK, dV, dQ = [dev_bf16(u[0]) for u in units], [dev_bf16(u[1]) for u in units], [dev_bf16(u[2]) for u in units]
    rows = jq.ragged_output_rows(s_common, n, Ls, Bs)
    Hkv = s_common.Hkv
    keeps = [min(b, l) for b, l in zip(Bs, Ls)]
    assert rows == Hkv * sum(keeps)
    Ko = torch.zeros((rows, 128), dtype=torch.bfloat16, device="cuda")
    Vo = torch.zeros_like(Ko)
    idx = torch.full((rows,), -1, dtype=torch.int32, device="cuda")
    if ws is None:
        ws = jq.new_ragged_workspace(s_common, n, Ls)
    jq.evict_ragged(dK, dV, dQ, s_common, Ls, Bs, Ko, Vo, idx, ws)
    assert jq.last_device_status(ws) == jq.JQ_OK
    gK, gV, gi = host_bits(Ko), host_bits(Vo), idx.cpu().numpy()
    out, r0 = [], 0
    for k in keeps:
        r1 = r0 + Hkv * k
        out.append((gK[r0:r1].reshape(Hkv, k, 128), gV[r0:r1].reshape(Hkv, k, 128), gi[r0:r1].reshape(Hkv, k)))
        r0 = r1
    return out


@pytest.mark.parametrize("Hkv,g,w,Ls,Bs", [
    (2, 4, 32, [3000, 130, 5000, 1, 2049], [400, 1000, 64, 3, 2049]),        # tails, L = 1, budget >= L, budget == L
    (2, 4, 64, [2049, 700, 4096], [300, 300, 10]),                           # 256 query rows per KV head
    (8, 4, 32, [4096, 12000, 20480, 8192], [1024, 900, 800, 700]),           # the ragged batch's lengths (shortened), decreasing budgets
    (1, 1, 1, [5, 7], [3, 2]),
])
def test_evict_ragged_matches_calls_per_unit(Hkv, g, w, Ls, Bs):
    """Units of different lengths and budgets in one call: bit for bit what one jq_evict_layer call per unit gives,
    and one unit against the oracle under the end-to-end rule."""
    base = small_wl(Hkv, g, w, max(Ls), max(Bs))
    units = [W.make_layer(base.with_L(l).with_budget(b), layer=i) for i, (l, b) in enumerate(zip(Ls, Bs))]
    got = _ragged_call(units, shape_of(base), Ls, Bs)
    for (K, V, Q, _), (gK, gV, gi), l, b in zip(units, got, Ls, Bs):
        wK, wV, wi = gpu_evict(K, V, Q, shape_of(base.with_L(l).with_budget(b)))
        assert np.array_equal(gi, wi) and np.array_equal(gK, wK) and np.array_equal(gV, wV)
    K, V, Q, _ = units[0]
    pooled = oracle.pool(oracle.score(K, Q), base.pool)
    assert_kept_sets_agree(got[0][2], oracle.select(pooled, Bs[0]), pooled, min(Bs[0], Ls[0]))


def test_evict_ragged_per_layer_budget_schedule_against_the_oracle():
    """A layer-wise decreasing budget (the pyramid-shaped schedule of the experimental-setting paragraph) over the
    layers of one cache, one call; every layer against the oracle."""
    wl = small_wl(4, 4, 32, 6000, 1024)
    nl = 6
    Bs = [1024, 768, 512, 384, 256, 128]
    units = [W.make_layer(wl, layer=i) for i in range(nl)]
    got = _ragged_call(units, shape_of(wl), [wl.L] * nl, Bs)
    for (K, V, Q, _), (gK, gV, gi), b in zip(units, got, Bs):
        pooled = oracle.pool(oracle.score(K, Q), wl.pool)
        assert_kept_sets_agree(gi, oracle.select(pooled, b), pooled, b)
        for kv in range(wl.Hkv):
            assert np.array_equal(gK[kv], K[kv][gi[kv]]) and np.array_equal(gV[kv], V[kv][gi[kv]])


def test_evict_ragged_whole_batch_of_config_4_in_one_call():
    """The ragged batch at full size: four sequences (4096, 12000, 20480, 32768 keys) x 4 layers each, 16 units, one
    call; one sampled layer per sequence against the oracle, every unit against its own jq_evict_layer call."""
    nl = 4
    units, Ls, Bs, meta = [], [], [], []
    for seq, wl in enumerate(W.CFG4):
        for layer in range(nl):
            units.append(W.make_layer(wl, layer=layer, seq=seq)); Ls.append(wl.L); Bs.append(wl.budget); meta.append((seq, layer, wl))
    got = _ragged_call(units, shape_of(W.CFG4[3]), Ls, Bs)
    for (K, V, Q, _), (gK, gV, gi), (seq, layer, wl) in zip(units, got, meta):
        wK, wV, wi = gpu_evict(K, V, Q, shape_of(wl))
        assert np.array_equal(gi, wi) and np.array_equal(gK, wK) and np.array_equal(gV, wV)
        if layer == seq:                                       # one layer per sequence
            pooled = oracle.pool(oracle.score(K, Q), wl.pool)
            assert_kept_sets_agree(gi, oracle.select(pooled, wl.budget), pooled, wl.nkeep)


def test_evict_ragged_rejects_bad_arguments():
    wl = small_wl(2, 4, 16, 500, 10)
    s = shape_of(wl)
    assert jq.ragged_workspace_bytes(s, 2, [500, 0]) == 0           # a unit without keys
    assert jq.ragged_workspace_bytes(s, 0) == 0
    assert jq.ragged_output_rows(s, 2, [500, 300], [10, -1]) == 0
    assert jq.ragged_output_rows(s, 2, [500, 300], [10, 1000]) == 2 * (10 + 300)


def test_evict_layer_window_kept_keeps_the_window_and_fills_the_rest():
    """budget rows per head = the w window pairs (always) + budget - w prefix rows chosen by the window-inclusive
    scores; expected: the oracle's windowed scores, pooled, top-(budget - w), then the window rows."""
    wl = small_wl(3, 4, 32, 3000, 500)
    K, V, Q, _ = W.make_layer(wl)
    Kw = W.make_window_keys(wl, Q)
    Vw = W.make_v(small_wl(3, 4, 32, wl.w, 1), 777)
    s = shape_of(wl)
    np_ = wl.budget - wl.w
    Ko = torch.zeros((wl.Hkv, wl.budget, 128), dtype=torch.bfloat16, device="cuda"); Vo = torch.zeros_like(Ko)
    idx = torch.full((wl.Hkv, np_), -1, dtype=torch.int32, device="cuda")
    ws = jq.new_workspace(s)
    jq.evict_layer_window_kept(dev_bf16(K), dev_bf16(V), dev_bf16(Q), dev_bf16(Kw), dev_bf16(Vw), s, Ko, Vo, idx, ws)
    assert jq.last_device_status(ws) == jq.JQ_OK
    gi, gK, gV = idx.cpu().numpy(), host_bits(Ko), host_bits(Vo)
    pooled = oracle.pool(oracle.score_windowed(K, Q, Kw), wl.pool)
    assert_kept_sets_agree(gi, oracle.select(pooled, np_), pooled, np_)
    for kv in range(wl.Hkv):
        assert np.array_equal(gK[kv, :np_], K[kv][gi[kv]]) and np.array_equal(gV[kv, :np_], V[kv][gi[kv]])
        assert np.array_equal(gK[kv, np_:], Kw[kv]) and np.array_equal(gV[kv, np_:], Vw[kv])
    with pytest.raises(jq.JqError):
        jq.evict_layer_window_kept(dev_bf16(K), dev_bf16(V), dev_bf16(Q), dev_bf16(Kw), dev_bf16(Vw), shape_of(wl.with_budget(32)), Ko, Vo, idx, ws)


# ------------------------------------------------------------------ streaming re-eviction

@pytest.mark.parametrize("Hkv,g,w,n_old,n_new,budget,cap", [(2, 4, 16, 512, 100, 512, 640), (2, 4, 64, 300, 1, 200, 301),
                                                             (3, 2, 32, 1000, 0, 400, 1500), (1, 1, 8, 10, 30, 64, 40)])
def test_evict_append_matches_the_pass_on_the_concatenation(Hkv, g, w, n_old, n_new, budget, cap):
    """The cache of a layer holds n_old retained rows per head in a buffer of `cap` rows; n_new rows are appended and the
    cache is evicted again, in place.  Expected: the oracle's pass over the concatenated rows (end-to-end rule), and the
    rows the indices name, bit for bit, at the head of the cache."""
    wl = small_wl(Hkv, g, w, n_old + n_new, budget)
    K, V, Q, _ = W.make_layer(wl, layer=3)
    s = shape_of(wl)
    Kc = torch.zeros((Hkv, cap, 128), dtype=torch.bfloat16, device="cuda")
    Vc = torch.zeros_like(Kc)
    Kc[:, :n_old] = dev_bf16(K[:, :n_old]); Vc[:, :n_old] = dev_bf16(V[:, :n_old])
    Kn = dev_bf16(K[:, n_old:]) if n_new else None
    Vn = dev_bf16(V[:, n_old:]) if n_new else None
    idx = torch.full((Hkv, wl.nkeep), -1, dtype=torch.int32, device="cuda")
    ws = jq.new_append_workspace(s)
    jq.evict_append(Kc, Vc, n_old, Kn, Vn, dev_bf16(Q), s, idx, ws)
    assert jq.last_device_status(ws) == jq.JQ_OK
    gi = idx.cpu().numpy()
    pooled = oracle.pool(oracle.score(K, Q), wl.pool)
    assert_kept_sets_agree(gi, oracle.select(pooled, budget), pooled, wl.nkeep)
    gK, gV = host_bits(Kc), host_bits(Vc)
    for kv in range(Hkv):
        assert np.array_equal(gK[kv, :wl.nkeep], K[kv][gi[kv]]) and np.array_equal(gV[kv, :wl.nkeep], V[kv][gi[kv]])
    # and bit for bit what jq_evict_layer gives on the packed concatenation
    wK, wV, wi = gpu_evict(K, V, Q, s)
    assert np.array_equal(gi, wi) and np.array_equal(gK[:, :wl.nkeep], wK) and np.array_equal(gV[:, :wl.nkeep], wV)


def test_evict_append_twice_in_a_row_then_decode():
    """Evict after the prefill, then two rounds of: decode over the pruned cache, append rows, evict again."""
    wl = small_wl(2, 4, 16, 2000, 256)
    K, V, Q, _ = W.make_layer(wl)
    cap = 256 + 64
    Ko, Vo, gidx = gpu_evict(K, V, Q, shape_of(wl))
    Kc = torch.zeros((wl.Hkv, cap, 128), dtype=torch.bfloat16, device="cuda"); Vc = torch.zeros_like(Kc)
    Kc[:, :256] = dev_bf16(Ko); Vc[:, :256] = dev_bf16(Vo)
    hostK, hostV = Ko.copy(), Vo.copy()
    for rnd in range(2):
        extra = small_wl(2, 4, 16, 64, 256)
        Kn, Vn, Qn, _ = W.make_layer(extra, layer=50 + rnd)
        allK, allV = np.concatenate([hostK, Kn], 1), np.concatenate([hostV, Vn], 1)
        s2 = shape_of(small_wl(2, 4, 16, 320, 256))
        idx = torch.full((wl.Hkv, 256), -1, dtype=torch.int32, device="cuda")
        ws = jq.new_append_workspace(s2)
        jq.evict_append(Kc, Vc, 256, dev_bf16(Kn), dev_bf16(Vn), dev_bf16(Qn), s2, idx, ws)
        assert jq.last_device_status(ws) == jq.JQ_OK
        gi = idx.cpu().numpy()
        pooled = oracle.pool(oracle.score(allK, Qn), wl.pool)
        assert_kept_sets_agree(gi, oracle.select(pooled, 256), pooled, 256)
        hostK = np.stack([allK[kv][gi[kv]] for kv in range(wl.Hkv)]); hostV = np.stack([allV[kv][gi[kv]] for kv in range(wl.Hkv)])
        assert np.array_equal(host_bits(Kc)[:, :256], hostK) and np.array_equal(host_bits(Vc)[:, :256], hostV)
