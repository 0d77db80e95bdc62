"""CPU-side checks of the C-ABI library: it loads, exports every symbol the header declares,
and rejects bad arguments on the host before anything is launched (no GPU needed)."""
import ctypes as C
import os
import re

import pytest

from paper_2510_07651_b200 import api, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    build.build()
    return api.lib()


def test_exports_every_declared_symbol(L):
    hdr = open(os.path.join(ROOT, "include", "obcache.h")).read()
    declared = set(re.findall(r"\b(obc_[a-z_0-9]+)\s*\(", hdr))
    assert declared == set(api.EXPORTS)
    for name in declared:
        assert hasattr(L, name), name


def test_status_strings_and_version(L):
    assert L.obc_status_string(0) == b"ok"
    for s in range(-7, 0):
        assert len(L.obc_status_string(s)) > 3
    assert L.obc_version() >= 100


def _sp(**kw):
    base = dict(batch=1, n_q_heads=4, n_kv_heads=2, head_dim=128, window=8, max_len=256, seq_lens=None,
                scale=0.0, causal=1, variants=4, path=0)
    base.update(kw)
    return api.obc_score_params(C.sizeof(api.obc_score_params), *[base[k] for k in
                                ("batch", "n_q_heads", "n_kv_heads", "head_dim", "window", "max_len", "seq_lens",
                                 "scale", "causal", "variants", "path")])


def test_score_workspace_and_validation(L):
    n = C.c_size_t(0)
    assert L.obc_score_workspace(C.byref(_sp()), C.byref(n)) == 0 and n.value > 0 and n.value % 256 == 0
    assert L.obc_score_workspace(C.byref(_sp(head_dim=64)), C.byref(n)) == -3
    assert L.obc_score_workspace(C.byref(_sp(n_q_heads=3)), C.byref(n)) == -2
    assert L.obc_score_workspace(C.byref(_sp(window=0)), C.byref(n)) == -2
    assert L.obc_score_workspace(C.byref(_sp(window=512)), C.byref(n)) == -2
    assert L.obc_score_workspace(C.byref(_sp(variants=0)), C.byref(n)) == -3
    assert L.obc_score_workspace(C.byref(_sp(variants=64)), C.byref(n)) == -3
    assert L.obc_score_workspace(C.byref(_sp()), None) == -1
    bad = _sp()
    bad.struct_size = 8
    assert L.obc_score_workspace(C.byref(bad), C.byref(n)) == -3


def test_score_rejects_null_and_misaligned_before_launch(L):
    t = lambda ptr, dt=1: api.obc_tensor(ptr, dt, 0, 256 * 128, 128)
    p = _sp()
    assert L.obc_score(C.byref(p), t(None), t(4096), t(4096), 4096, 4096, 1 << 30, None) == -1
    assert L.obc_score(C.byref(p), t(4096), t(4096), t(4096), None, 4096, 1 << 30, None) == -1
    assert L.obc_score(C.byref(p), t(4104), t(4096), t(4096), 4096, 4096, 1 << 30, None) == -4
    assert L.obc_score(C.byref(p), t(4096), t(4096, 0), t(4096), 4096, 4096, 1 << 30, None) == -3
    assert L.obc_score(C.byref(p), t(4096), t(4096), t(4096), 4096, 4096, 16, None) == -5
    assert L.obc_score(C.byref(p), t(4096), t(4096), t(4096), 4096, None, 1 << 30, None) == -5
    assert L.obc_score(C.byref(_sp(path=2, window=1)), t(4096), t(4096), t(4096), 4096, 4096, 1 << 30, None) == -3


def _selp(**kw):
    base = dict(batch=1, n_kv_heads=2, max_len=256, seq_lens=None, budget=64, budgets=None, idx_stride=64,
                n_sink=0, n_recent=8, pool_mode=2, pool_kernel=7)
    base.update(kw)
    return api.obc_select_params(C.sizeof(api.obc_select_params), *[base[k] for k in
                                 ("batch", "n_kv_heads", "max_len", "seq_lens", "budget", "budgets", "idx_stride",
                                  "n_sink", "n_recent", "pool_mode", "pool_kernel")])


def test_select_validation(L):
    n = C.c_size_t(0)
    assert L.obc_select_workspace(C.byref(_selp()), C.byref(n)) == 0 and n.value >= 2 * 256 * 4
    assert L.obc_select_workspace(C.byref(_selp(pool_kernel=4)), C.byref(n)) == -2
    assert L.obc_select_workspace(C.byref(_selp(budget=4)), C.byref(n)) == -2
    assert L.obc_select_workspace(C.byref(_selp(budget=300, idx_stride=300)), C.byref(n)) == -2
    assert L.obc_select_workspace(C.byref(_selp(pool_mode=5)), C.byref(n)) == -3
    assert L.obc_select(C.byref(_selp()), None, 4096, 4096, 1 << 20, None) == -1
    assert L.obc_select(C.byref(_selp()), 4096, 4096, 4096, 16, None) == -5


def test_given_and_adaptive_validation(L):
    t = lambda ptr, dt=1: api.obc_tensor(ptr, dt, 0, 256 * 128, 128)
    p = _sp()
    # the attention outputs and their log-sum-exp are both required; o may be fp32 next to a bf16 cache
    assert L.obc_score_given(C.byref(p), t(4096), t(4096), t(4096), t(4096), None, 4096, 4096, 1 << 30, None) == -1
    assert L.obc_score_given(C.byref(p), t(4096), t(4096), t(4096), t(None), 4096, 4096, 4096, 1 << 30, None) == -1
    assert L.obc_score_given(C.byref(p), t(4096), t(4096), t(4096), t(4096, 0), 4096, 4096, 4096, 16, None) == -5
    assert L.obc_score_given(C.byref(_sp(variants=16)), t(4096), t(4096), t(4096), t(4104), 4096, 4096, 4096, 1 << 30, None) == -4
    n = C.c_size_t(0)
    assert L.obc_select_adaptive_workspace(C.byref(_selp()), 0.2, C.byref(n)) == 0 and n.value >= 2 * 256 * 4
    assert L.obc_select_adaptive_workspace(C.byref(_selp()), 1.5, C.byref(n)) == -2
    assert L.obc_select_adaptive_workspace(C.byref(_selp()), -0.1, C.byref(n)) == -2
    assert L.obc_select_adaptive_workspace(C.byref(_selp(budgets=4096)), 0.2, C.byref(n)) == -3
    assert L.obc_select_adaptive(C.byref(_selp()), 0.2, 4096, 4096, None, 4096, 1 << 20, None) == -1
    assert L.obc_select_adaptive(C.byref(_selp()), 0.2, 4096, 4096, 4096, 4096, 16, None) == -5
    d1, d2 = C.c_double(0), C.c_double(0)
    assert L.obc_score_kernel_spans(None, None, C.byref(d1), C.byref(d2)) == -1


def test_token_shard_calls_validation(L):
    t = lambda ptr, dt=1: api.obc_tensor(ptr, dt, 0, 256 * 128, 128)
    n = C.c_size_t(0)
    # a window longer than the cache is only meaningful for a shard of a longer sequence (mask_lens given)
    long_w = _sp(window=300)
    assert L.obc_score_workspace(C.byref(long_w), C.byref(n)) == -2
    long_w.mask_lens = 4096
    assert L.obc_score_workspace(C.byref(long_w), C.byref(n)) == 0
    p = _sp()
    assert L.obc_window_attention(C.byref(p), t(4096), t(4096), t(4096), None, 4096, 4096, 1 << 30, None) == -1
    assert L.obc_window_attention(C.byref(p), t(4096), t(4096), t(4096), 4096, None, 4096, 1 << 30, None) == -1
    assert L.obc_window_attention(C.byref(p), t(4096), t(4096), t(4096), 4100, 4096, 4096, 1 << 30, None) == -4
    assert L.obc_window_attention(C.byref(p), t(4096), t(4096), t(4096), 4096, 4096, 4096, 16, None) == -5
    assert L.obc_window_attention(C.byref(p), t(4096), t(4096, 0), t(4096), 4096, 4096, 4096, 1 << 30, None) == -3
    assert L.obc_merge_attention(0, 64, 128, 4096, 4096, 4096, 4096, None) == -2
    assert L.obc_merge_attention(2, 0, 128, 4096, 4096, 4096, 4096, None) == -2
    assert L.obc_merge_attention(2, 64, 64, 4096, 4096, 4096, 4096, None) == -3
    assert L.obc_merge_attention(2, 64, 128, None, 4096, 4096, 4096, None) == -1
    assert L.obc_merge_attention(2, 64, 128, 4100, 4096, 4096, 4096, None) == -4
    assert L.obc_shard_indices(1, 2, 64, 4096, 0, 0, 8192, 4096, None) == -2        # an empty shard
    assert L.obc_shard_indices(1, 2, 64, 4096, -1, 10, 8192, 4096, None) == -2
    assert L.obc_shard_indices(1, 2, 64, None, 0, 10, 8192, 4096, None) == -1
    assert L.obc_shard_indices(1, 2, 64, 4096, 0, 10, 4096, 4096, None) == -2       # in place


def test_compact_and_decode_validation(L):
    t = lambda ptr: api.obc_tensor(ptr, 1, 0, 256 * 128, 128)
    assert L.obc_compact(1, 2, 64, 16, 256, t(4096), t(4096), 4096, t(4096), t(4096), None, None, None) == -3
    assert L.obc_compact(1, 2, 128, 16, 256, t(4096), t(4096), None, t(4096), t(4096), None, None, None) == -1
    assert L.obc_compact(1, 2, 128, 16, 256, t(None), t(4096), 4096, t(4096), t(4096), None, None, None) == -1
    dp = api.obc_decode_params(C.sizeof(api.obc_decode_params), 2, 8, 2, 128, 65, 64, 4, 16, 4, 0.0)
    n = C.c_size_t(0)
    assert L.obc_decode_workspace(C.byref(dp), C.byref(n)) == 0 and n.value > 0
    dp.capacity = 64
    assert L.obc_decode_workspace(C.byref(dp), C.byref(n)) == -2
    dp.capacity, dp.variant = 65, 3
    assert L.obc_decode_workspace(C.byref(dp), C.byref(n)) == -3
    dp.variant, dp.acc_window = 4, -1                          # accumulation window: 0..4096 steps
    assert L.obc_decode_workspace(C.byref(dp), C.byref(n)) == -2
    dp.acc_window = 4097
    assert L.obc_decode_workspace(C.byref(dp), C.byref(n)) == -2
    dp.acc_window = 8                                          # a window needs its ring of per-step scores
    assert L.obc_decode_workspace(C.byref(dp), C.byref(n)) == 0
    assert L.obc_decode_step(C.byref(dp), t(4096), t(4096), t(4096), t(4096), t(4096), 4096, 4096, 4096, 70,
                             4096, n.value, None) == -1


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(api, "_lib", None)
    monkeypatch.setattr(api, "LIB_PATH", "/nonexistent/libobcache.so")
    with pytest.raises(OSError):
        api.lib()
