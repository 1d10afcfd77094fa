"""jq_score_static: scoring for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is off limits: a serving process that gave all free GPU
memory to its KV-cache pool at start-up, or code that lives inside another component's memory budget.
For them the library carries its own fixed scratch array, and jq_score_static uses it instead of a
caller-provided workspace.  The test calls it through the C ABI twice in a row (the array keeps the
previous call's contents, so the second call is the one that shows stale state) and compares with
jq_score and with the CPU oracle on the same inputs, within the score tolerance of the parity tests; one
case sits exactly at the 2048-row limit of the built-in array.  This file sorts last on
purpose: a run that stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

import jq_workloads as W
import oracle
import paper_2509_10798_b200 as jq
from gpu_util import SCORE_ATOL, SCORE_RTOL, dev_bf16, shape_of

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def built():
    import __graft_entry__ as entry
    entry.build()


def scores_both_ways(wl, layer):
    K, _, Q, _ = W.make_layer(wl, layer=layer, with_v=False)
    s = shape_of(wl)
    dK, dQ = dev_bf16(K), dev_bf16(Q)
    ws = jq.new_workspace(s)
    want = torch.full((s.Hkv, s.L), -1.0, dtype=torch.float32, device="cuda")
    jq.score(dK, dQ, s, want, ws)
    assert jq.last_device_status(ws) == jq.JQ_OK
    got = torch.full((s.Hkv, s.L), -2.0, dtype=torch.float32, device="cuda")   # allocated by the test, not the call
    jq.score_static(dK, dQ, s, got)
    torch.cuda.synchronize()
    return got.cpu().numpy().astype(np.float64), want.cpu().numpy().astype(np.float64), oracle.score(K, Q)


def test_static_scratch_matches_workspace_path_on_two_calls_in_a_row():
    # two different shapes back to back: 128 and 256 query rows per KV head, ragged tails, several head groups
    # the third uses the array to its last byte: 8 heads x 256 query rows = 2048 rows
    cases = [W.Workload("t", 2, Hkv=8, Hq=32, L=3000, w=32, budget=1), W.Workload("t", 2, Hkv=4, Hq=16, L=1300, w=64, budget=1),
             W.Workload("t", 2, Hkv=8, Hq=32, L=1500, w=64, budget=1)]
    for rep, wl in enumerate(cases + cases):
        got, want, exact = scores_both_ways(wl, layer=rep)
        assert np.all(np.abs(got - want) <= SCORE_RTOL * np.abs(want) + SCORE_ATOL), "call %d differs from jq_score" % rep
        assert np.all(np.abs(got - exact) <= SCORE_RTOL * np.abs(exact) + SCORE_ATOL), "call %d differs from the oracle" % rep
        np.testing.assert_allclose(got.sum(-1), wl.R, rtol=1e-3)


def test_shapes_beyond_the_built_in_scratch_are_refused():
    wl = W.Workload("t", 2, Hkv=16, Hq=64, L=256, w=64, budget=1)     # 16 * 256 = 4096 query rows > 2048
    s = shape_of(wl)
    K = torch.zeros((s.Hkv, s.L, s.d), dtype=torch.bfloat16, device="cuda")
    Q = torch.zeros((s.Hq, s.w, s.d), dtype=torch.bfloat16, device="cuda")
    out = torch.full((s.Hkv, s.L), 7.0, dtype=torch.float32, device="cuda")
    with pytest.raises(jq.JqError) as e:
        jq.score_static(K, Q, s, out)
    assert e.value.code == jq.JQ_ERR_UNSUPPORTED
    assert float(out.min()) == 7.0 and float(out.max()) == 7.0      # nothing was launched
