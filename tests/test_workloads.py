"""Seeded input generators: shapes, determinism, recipe structure, and the stored config-1 fixture."""
import os
import zlib

import numpy as np

import oracle
import jq_workloads as W

GOLD = os.path.join(os.path.dirname(__file__), "golden", "cfg1_kept_idx.txt")


def test_bf16_round_trip_and_rne():
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 0.0, 3.0e-5], np.float32)
    b = W.bf16_bits(x)
    # 1 + 2^-8 is a tie between 1.0 and 1 + 2^-7: ties go to the even mantissa (1.0)
    assert b[1] == b[0]
    # 1 + 3*2^-8 is a tie between 1+2^-7 (odd) and 1+2^-6 (even)
    assert W.bf16_to_f32(b[2:3])[0] == np.float32(1.015625)
    y = W.bf16_to_f32(b)
    assert np.array_equal(W.bf16_bits(y), b)
    assert np.all(np.abs(y - x) <= np.abs(x) * 2.0 ** -8)


def test_generators_are_deterministic_and_shaped():
    for wl in (W.CFG1, W.CFG2.with_L(1024), W.CFG4[0].with_L(1500), W.CFG5.with_L(2048)):
        a = W.make_layer(wl, layer=3)
        b = W.make_layer(wl, layer=3)
        c = W.make_layer(wl, layer=4)
        for x, y in zip(a[:3], b[:3]):
            assert x.dtype == np.uint16 and np.array_equal(x, y)
        assert not np.array_equal(a[0], c[0])
        assert a[0].shape == (wl.Hkv, wl.L, wl.d) and a[1].shape == a[0].shape
        assert a[2].shape == (wl.Hq, wl.w, wl.d)
        assert np.all(np.isfinite(W.bf16_to_f32(a[0]))) and np.all(np.isfinite(W.bf16_to_f32(a[2])))


def test_outlier_channels_and_planted_rows_are_heavy():
    wl = W.CFG2.with_L(2048).with_budget(256)
    K, V, Q, info = W.make_layer(wl)
    Kf = W.bf16_to_f32(K)
    var = Kf.var(axis=1)                      # [Hkv, d]
    assert np.all((var > 30).sum(-1) == 4)    # four channels scaled x8 per head
    sc = oracle.score(K, Q)
    for kv in range(wl.Hkv):
        # the planted keys carry far more attention mass than a typical key (uniform level R/L)
        pl = np.unique(info["planted"][kv])
        assert np.median(sc[kv, pl]) > 2 * np.median(sc[kv])
        assert sc[kv, pl].mean() > 2 * wl.R / wl.L


def test_formula_bytes_matches_hand_computed_numbers():
    assert abs(W.formula_bytes(W.CFG2) / 1e6 - 39.9) < 0.1
    assert abs(W.formula_bytes(W.CFG3) / 1e6 - 137.4) < 0.1
    assert abs(W.formula_bytes(W.CFG5) / 1e6 - 543.2) < 0.1


def test_config1_fixture():
    with open(GOLD) as f:
        lines = f.read().strip().split("\n")
    wl = W.CFG1
    K, V, Q, _ = W.make_layer(wl)
    crc = [int(t) for t in lines[0].split()[1:]]
    assert [zlib.crc32(a.tobytes()) for a in (K, V, Q)] == crc, "seeded generator drifted"
    want = np.array([[int(t) for t in ln.split()] for ln in lines[1:]], np.int32)
    _, _, idx = oracle.evict_layer(K, V, Q, wl.budget, wl.pool)
    assert np.array_equal(idx, want)
