"""Host-side checks of the C ABI that need no GPU: the library loads, exports every entry point the
header declares, and rejects bad arguments before touching CUDA."""
import ctypes
import os
import re

import pytest

import __graft_entry__ as entry
import paper_2509_10798_b200 as jq

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    entry.build()


def declared_symbols():
    with open(os.path.join(ROOT, "include", "jq.h")) as f:
        text = re.sub(r"/\*.*?\*/", "", f.read(), flags=re.S)
    return sorted(set(re.findall(r"\b(jq_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_symbols()
    assert len(names) >= 12
    lib = ctypes.CDLL(jq.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(jq.EXPORTS)


def test_shape_validation_and_sizes():
    ok = jq.shape(8, 32, 32768, 32, 512)
    assert jq.check_shape(ok) == jq.JQ_OK
    assert jq.num_kept(ok) == 512
    assert jq.num_kept(jq.shape(8, 32, 100, 32, 512)) == 100
    ws = jq.workspace_bytes(ok)
    assert ws >= 2 * 8 * 32768 * 4 and ws % 256 == 0
    assert jq.host_call_bytes(ok) >= ws + 2 * 8 * 32768 * 256
    bad = [
        jq.shape(8, 32, 32768, 32, 512, pool=6),          # even pool width
        jq.shape(8, 32, 32768, 32, 0),                    # budget < 1
        jq.shape(8, 32, 0, 32, 512),                      # L < 1
        jq.shape(8, 32, 32768, 0, 512),                   # w < 1
        jq.shape(8, 33, 32768, 32, 512, group=4),         # Hq != Hkv * group
    ]
    for s in bad:
        assert jq.check_shape(s) == jq.JQ_ERR_INVALID_ARG
        assert jq.workspace_bytes(s) == 0 and jq.num_kept(s) == 0
    unsupported = [
        jq.shape(8, 32, 32768, 32, 512, d=64),            # head dim
        jq.shape(8, 32, 32768, 65, 512),                  # group * w > 256
        jq.shape(8, 32, 32768, 32, 512, pool=65),
    ]
    for s in unsupported:
        assert jq.check_shape(s) == jq.JQ_ERR_UNSUPPORTED
        assert jq.workspace_bytes(s) == 0


def test_pointer_errors_are_caught_on_the_host():
    lib = jq.lib()
    s = jq.shape(2, 8, 2048, 16, 256)
    ref = ctypes.byref(s)
    n = jq.workspace_bytes(s)
    a = ctypes.c_void_p(0x1000)        # aligned, never dereferenced: every call below fails first
    odd = ctypes.c_void_p(0x1008)
    assert lib.jq_score(None, a, ref, a, a, n, None) == jq.JQ_ERR_INVALID_ARG
    assert lib.jq_score(odd, a, ref, a, a, n, None) == jq.JQ_ERR_INVALID_ARG
    assert lib.jq_score(a, a, ref, a, a, n - 1, None) == jq.JQ_ERR_WORKSPACE
    assert lib.jq_score_fma(a, a, ref, a, a, 0, None) == jq.JQ_ERR_WORKSPACE
    assert lib.jq_select_topk(a, ref, None, None, a, n, None) == jq.JQ_ERR_INVALID_ARG
    assert lib.jq_compact_kv(a, a, a, ref, a, odd, None) == jq.JQ_ERR_INVALID_ARG
    assert lib.jq_evict_layer(a, a, a, ref, a, a, a, a, 16, None) == jq.JQ_ERR_WORKSPACE
    assert lib.jq_evict_layer_host(a, a, a, ref, a, a, a, a, 16, None) == jq.JQ_ERR_WORKSPACE
    assert lib.jq_evict_layer(a, a, a, None, a, a, a, a, n, None) == jq.JQ_ERR_INVALID_ARG
    assert lib.jq_decode_attention(a, a, a, 2, 8, 100, None, a, 1 << 20, None) == jq.JQ_ERR_INVALID_ARG
    assert lib.jq_decode_attention(a, a, a, 2, 7, 100, a, a, 1 << 20, None) == jq.JQ_ERR_INVALID_ARG      # Hq % Hkv
    assert lib.jq_decode_attention(a, a, a, 1, 16, 100, a, a, 1 << 20, None) == jq.JQ_ERR_UNSUPPORTED     # group > 8
    assert lib.jq_decode_attention(a, a, a, 2, 8, 100, a, a, 16, None) == jq.JQ_ERR_WORKSPACE
    assert jq.decode_workspace_bytes(2, 8, 100) >= 8 * 2 * 130 * 4 and jq.decode_workspace_bytes(2, 7, 100) == 0
    ptrs = (ctypes.c_void_p * 2)(0x1000, 0x2000)
    assert lib.jq_evict_layers(ptrs, ptrs, ptrs, 2, ref, a, a, a, a, 16, None) == jq.JQ_ERR_WORKSPACE
    assert lib.jq_evict_layers(ptrs, ptrs, ptrs, 0, ref, a, a, a, a, 1 << 40, None) == jq.JQ_ERR_INVALID_ARG
    assert lib.jq_evict_layers(ptrs, ptrs, ptrs, 4097, ref, a, a, a, a, 1 << 40, None) == jq.JQ_ERR_UNSUPPORTED
    two = (ctypes.c_int * 2)
    assert lib.jq_evict_ragged(ptrs, ptrs, ptrs, 2, ref, two(100, 200), two(10, 10), a, a, a, a, 16, None) == jq.JQ_ERR_WORKSPACE
    assert lib.jq_evict_ragged(ptrs, ptrs, ptrs, 2, ref, two(100, 0), two(10, 10), a, a, a, a, 1 << 40, None) == jq.JQ_ERR_INVALID_ARG
    assert lib.jq_evict_ragged(ptrs, ptrs, ptrs, 2, ref, two(100, 200), two(10, 0), a, a, a, a, 1 << 40, None) == jq.JQ_ERR_INVALID_ARG
    assert lib.jq_evict_ragged(ptrs, ptrs, ptrs, 2, ref, None, None, a, a, odd, a, 1 << 40, None) == jq.JQ_ERR_INVALID_ARG
    assert jq.ragged_workspace_bytes(s, 2, [100, 200]) < jq.ragged_workspace_bytes(s, 2, [100, 300])
    assert jq.ragged_output_rows(s, 3, [100, 200, 5], [10, 300, 7]) == 2 * (10 + 200 + 5)
    assert lib.jq_evict_layers(None, ptrs, ptrs, 2, ref, a, a, a, a, 1 << 40, None) == jq.JQ_ERR_INVALID_ARG
    odd_ptrs = (ctypes.c_void_p * 2)(0x1000, 0x2008)
    assert lib.jq_evict_layers(odd_ptrs, ptrs, ptrs, 2, ref, a, a, a, a, 1 << 40, None) == jq.JQ_ERR_INVALID_ARG
    assert jq.layers_workspace_bytes(s, 2) > jq.workspace_bytes(jq.shape(4, 16, 2048, 16, 256)) and jq.layers_workspace_bytes(s, 0) == 0
    assert lib.jq_hit_rate(a, a, 0, 4, 4, a, None) == jq.JQ_ERR_INVALID_ARG
    # jq_evict_append: s.L = 2048 must equal n_old + n_new and fit the cache's rows per head
    assert lib.jq_evict_append(a, a, 4096, 2000, a, a, 47, a, ref, a, a, 1 << 40, None) == jq.JQ_ERR_INVALID_ARG
    assert lib.jq_evict_append(a, a, 2047, 2000, a, a, 48, a, ref, a, a, 1 << 40, None) == jq.JQ_ERR_INVALID_ARG
    assert lib.jq_evict_append(a, a, 4096, 2000, None, a, 48, a, ref, a, a, 1 << 40, None) == jq.JQ_ERR_INVALID_ARG
    assert lib.jq_evict_append(a, a, 4096, 2000, a, a, 48, a, ref, a, a, n, None) == jq.JQ_ERR_WORKSPACE
    assert lib.jq_append_workspace_bytes(ref) > n
    assert lib.jq_last_device_status(None, None) == jq.JQ_ERR_INVALID_ARG
    assert jq.status_string(jq.JQ_ERR_TIMEOUT) and jq.status_string(99)
    assert jq.launch_count() == 0      # nothing above reached a launch
