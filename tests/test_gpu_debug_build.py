"""The bounds-checked build of the kernels (libjq_debug.so, -DJQ_DEBUG): a sweep of small and awkward shapes through
every kernel of the hot path with all computed indices checked against the extents of what they index.  No memory
checker is available where this suite runs, so the library carries its own: a violation would be counted in a device
record (and the access skipped, never a trap); the sweep must end with the count at zero and every status JQ_OK.
The sweep runs in a process of its own because a process binds one copy of the library.
"""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SWEEP = r'''
import ctypes, os, sys
import numpy as np, torch
sys.path.insert(0, %(root)r)
sys.path.insert(0, os.path.join(%(root)r, "tests"))
import paper_2509_10798_b200 as jq
from paper_2509_10798_b200 import build
jq.LIB_PATH = build.build(debug=True)
import jq_workloads as W
from gpu_util import dev_bf16, shape_of
lib = jq.lib()
rec = (ctypes.c_longlong * 5)()
assert lib.jq_debug_reset() == 0

def wl_of(Hkv, g, w, L, B, p=7):
    return W.Workload("t", 2, Hkv=Hkv, Hq=Hkv * g, L=L, w=w, budget=B, pool=p)

def whole_pass(wl, layer=0):
    K, V, Q, _ = W.make_layer(wl, layer=layer)
    s = shape_of(wl)
    ws = jq.new_workspace(s)
    dK, dV, dQ = dev_bf16(K), dev_bf16(V), dev_bf16(Q)
    sc = torch.empty((s.Hkv, s.L), dtype=torch.float32, device="cuda")
    jq.score(dK, dQ, s, sc, ws)
    idx = torch.zeros((s.Hkv, wl.nkeep), dtype=torch.int32, device="cuda")
    pooled = torch.empty_like(sc)
    jq.select_topk(sc, s, idx, ws, pooled=pooled)
    Ko = torch.zeros((s.Hkv, wl.nkeep, 128), dtype=torch.bfloat16, device="cuda"); Vo = torch.zeros_like(Ko)
    jq.compact_kv(dK, dV, idx, s, Ko, Vo)
    jq.evict_layer(dK, dV, dQ, s, Ko, Vo, idx, ws)
    assert jq.last_device_status(ws) == jq.JQ_OK, wl
    if wl.w <= 128:
        Kw = dev_bf16(W.make_window_keys(wl, Q, layer=layer))
        jq.evict_layer_windowed(dK, dV, dQ, Kw, s, Ko, Vo, idx, ws)
        assert jq.last_device_status(ws) == jq.JQ_OK, wl
    if wl.group <= 8:
        q1 = dQ[:, -1, :].contiguous()
        od = torch.empty((wl.Hq, 128), dtype=torch.float32, device="cuda")
        wsd = torch.empty(jq.decode_workspace_bytes(wl.Hkv, wl.Hq, wl.nkeep), dtype=torch.uint8, device="cuda")
        jq.decode_attention(Ko, Vo, q1, od, wsd)
    return K, V, Q

# scores: one tile, tails, L = 1, many heads, 256 query rows, odd row counts; selection: budgets around L, pool widths
cases = [(1, 1, 1, 1, 1, 1), (1, 1, 1, 5, 3, 3), (2, 4, 16, 129, 7, 7), (2, 4, 16, 2048, 256, 7), (3, 4, 32, 1000, 1000, 5),
         (2, 4, 64, 2049, 300, 7), (1, 3, 11, 4000, 4001, 9), (5, 2, 64, 640, 64, 1), (160, 1, 4, 5000, 700, 7),
         (2, 4, 32, 40000, 2048, 7), (1, 8, 32, 12000, 1024, 63), (2, 2, 40, 3333, 33, 7)]
for c in cases:
    whole_pass(wl_of(*c))

# selection over many heads (one CTA of 512 or 1024 threads per head): odd lengths, ties, budgets at and above L
for Hkv, L, B, p in [(129, 1023, 77, 9), (130, 4001, 4001, 7), (300, 70000, 500, 7), (128, 200001, 1000, 5)]:
    s = jq.shape(Hkv, Hkv, L, 1, B, p)
    ws = jq.new_workspace(s)
    for sc in (torch.rand((Hkv, L), device="cuda"), torch.randint(0, 5, (Hkv, L), device="cuda").float()):
        idx = torch.zeros((Hkv, min(B, L)), dtype=torch.int32, device="cuda")
        jq.select_topk(sc, s, idx, ws, pooled=torch.empty_like(sc))
        assert jq.last_device_status(ws) == jq.JQ_OK

# several units in one call: lengths and budgets of their own, groups that run over units of one length
base = wl_of(2, 4, 32, 5000, 400)
Ls, Bs = [3000, 130, 130, 5000, 1, 2049, 2049, 2049], [400, 1000, 7, 64, 3, 2049, 100, 5]
units = [W.make_layer(base.with_L(l).with_budget(b), layer=i) for i, (l, b) in enumerate(zip(Ls, Bs))]
s = shape_of(base)
rows = jq.ragged_output_rows(s, len(units), Ls, Bs)
Ko = torch.zeros((rows, 128), dtype=torch.bfloat16, device="cuda"); Vo = torch.zeros_like(Ko)
idx = torch.zeros((rows,), dtype=torch.int32, device="cuda")
ws = jq.new_ragged_workspace(s, len(units), Ls)
jq.evict_ragged([dev_bf16(u[0]) for u in units], [dev_bf16(u[1]) for u in units], [dev_bf16(u[2]) for u in units], s, Ls, Bs, Ko, Vo, idx, ws)
assert jq.last_device_status(ws) == jq.JQ_OK

# a cache that grows and is evicted again in place
wl = wl_of(2, 4, 16, 612, 512)
K, V, Q, _ = W.make_layer(wl)
Kc = torch.zeros((2, 700, 128), dtype=torch.bfloat16, device="cuda"); Vc = torch.zeros_like(Kc)
Kc[:, :512] = dev_bf16(K[:, :512]); Vc[:, :512] = dev_bf16(V[:, :512])
idx = torch.zeros((2, 512), dtype=torch.int32, device="cuda")
ws = jq.new_append_workspace(shape_of(wl))
jq.evict_append(Kc, Vc, 512, dev_bf16(K[:, 512:]), dev_bf16(V[:, 512:]), dev_bf16(Q), shape_of(wl), idx, ws)
assert jq.last_device_status(ws) == jq.JQ_OK

assert lib.jq_debug_read(rec) == 0
print("DEBUG-SWEEP violations=%%d kernel=%%d site=%%d index=%%d extent=%%d" %% tuple(rec))
'''


def test_no_index_leaves_its_array_in_the_bounds_checked_build():
    out = subprocess.run([sys.executable, "-c", SWEEP % {"root": ROOT}], capture_output=True, text=True, timeout=900)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-4000:]
    line = [ln for ln in out.stdout.splitlines() if ln.startswith("DEBUG-SWEEP")]
    assert line, out.stdout[-2000:]
    assert line[0].startswith("DEBUG-SWEEP violations=0 "), line[0]
