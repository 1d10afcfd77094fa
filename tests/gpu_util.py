"""Helpers for the GPU parity tests: numpy bit patterns <-> device tensors, and the agreement rules."""
import numpy as np
import torch

import paper_2509_10798_b200 as jq

SCORE_RTOL, SCORE_ATOL = 2e-3, 1e-6     # fp32 accumulation of bf16 products vs the fp64 oracle
KTH_RTOL = 1e-4                         # kept sets may differ only this close to the k-th pooled score


def dev_bf16(bits):
    """uint16 bit patterns -> CUDA bf16 tensor with the same bits."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def host_bits(t):
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def shape_of(wl):
    return jq.shape(wl.Hkv, wl.Hq, wl.L, wl.w, wl.budget, wl.pool, wl.d)


def gpu_score(K, Q, s, fma=False):
    ws = jq.new_workspace(s)
    out = torch.full((s.Hkv, s.L), -1.0, dtype=torch.float32, device="cuda")
    jq.score(dev_bf16(K), dev_bf16(Q), s, out, ws, fma=fma)
    assert jq.last_device_status(ws) == jq.JQ_OK
    return out.cpu().numpy()


def gpu_select(scores_f32, s, want_pooled=True):
    ws = jq.new_workspace(s)
    nkeep = jq.num_kept(s)
    idx = torch.full((s.Hkv, nkeep), -1, dtype=torch.int32, device="cuda")
    pooled = torch.full((s.Hkv, s.L), -1.0, dtype=torch.float32, device="cuda") if want_pooled else None
    jq.select_topk(torch.from_numpy(np.ascontiguousarray(scores_f32)).cuda(), s, idx, ws, pooled=pooled)
    assert jq.last_device_status(ws) == jq.JQ_OK
    return idx.cpu().numpy(), (pooled.cpu().numpy() if want_pooled else None)


def gpu_evict(K, V, Q, s):
    ws = jq.new_workspace(s)
    nkeep = jq.num_kept(s)
    dK, dV, dQ = dev_bf16(K), dev_bf16(V), dev_bf16(Q)
    Ko = torch.zeros((s.Hkv, nkeep, s.d), dtype=torch.bfloat16, device="cuda")
    Vo = torch.zeros_like(Ko)
    idx = torch.full((s.Hkv, nkeep), -1, dtype=torch.int32, device="cuda")
    jq.evict_layer(dK, dV, dQ, s, Ko, Vo, idx, ws)
    assert jq.last_device_status(ws) == jq.JQ_OK
    return host_bits(Ko), host_bits(Vo), idx.cpu().numpy()


def assert_scores_close(got, want):
    err = np.abs(got.astype(np.float64) - want)
    tol = SCORE_RTOL * np.abs(want) + SCORE_ATOL
    bad = err > tol
    assert not bad.any(), "scores off at %d positions, worst rel err %.3g" % (
        bad.sum(), (err / np.maximum(np.abs(want), 1e-30)).max())


def assert_kept_sets_agree(idx_gpu, idx_oracle, pooled_oracle, nkeep):
    """Same sets, except for positions whose oracle pooled score is within KTH_RTOL of the k-th one."""
    Hkv, L = pooled_oracle.shape
    assert idx_gpu.shape == (Hkv, nkeep)
    swaps = 0
    for kv in range(Hkv):
        g = idx_gpu[kv]
        assert np.all(np.diff(g) > 0) and g[0] >= 0 and g[-1] < L, "kept indices not strictly ascending in range"
        kth = np.sort(pooled_oracle[kv])[L - nkeep]
        diff = np.setxor1d(g, idx_oracle[kv])
        swaps += len(diff)
        if len(diff):
            assert np.all(np.abs(pooled_oracle[kv][diff] - kth) <= KTH_RTOL * kth), (
                "kept sets differ away from the threshold, head %d" % kv)
    return swaps
