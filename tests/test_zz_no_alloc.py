"""obc_select_noalloc: the selection entry point for callers that cannot allocate device memory
(a plug-in inside an engine that owns the heap, a serving loop with a fixed memory budget).  Its
key scratch is a fixed array inside the library, shared by all calls.  Called through the C ABI
twice in a row, on different problems, it must give exactly the indices obc_select gives with a
caller-owned workspace, and exactly the CPU checker's pool + select (selection is integer work: the
bar is bit-exact, as in the other select tests; the checker pins the one-CTA-per-head kernel that
only this entry point reaches at these sizes); the second, smaller call runs over the keys the
first one left behind.

This file sorts last on purpose: a run that stops at the first failure has then run all others.
"""
import numpy as np
import pytest
import torch

from oracle import reference as ref
from paper_2510_07651_b200 import api

pytestmark = pytest.mark.gpu


def _both(scores_np, **kw):
    scores = torch.from_numpy(scores_np).cuda()
    stride = kw.pop("idx_stride")
    want = api.obc_select(scores, idx_stride=stride, **kw)
    idx = torch.full((scores.shape[0], scores.shape[1], stride), -7, dtype=torch.int32, device="cuda")
    got = api.obc_select_noalloc(scores, idx, **kw)
    torch.cuda.synchronize()
    return got.cpu().numpy(), want.cpu().numpy()


def test_two_calls_in_a_row_match_obc_select():
    rng = np.random.default_rng(11)
    big = (rng.random((1, 8, 32768), dtype=np.float32) ** 8 * 1e-3).astype(np.float32)
    got, want = _both(big, budget=2048, idx_stride=2048, n_recent=32, pool="max", pool_kernel=7)
    assert np.array_equal(got, want)
    assert np.array_equal(got, ref.select_pipeline(big, [32768], [2048], 0, 32, "max", 7, 2048))
    # second call: smaller, ragged, heavy ties, other pooling; stale keys of the first call lie beyond it
    small = (rng.integers(0, 5, (3, 2, 3000)) / 4).astype(np.float32)
    lens = torch.tensor([3000, 517, 2300], dtype=torch.int32, device="cuda")
    budgets = torch.tensor([300, 60, 230], dtype=torch.int32, device="cuda")
    got, want = _both(small, budgets=budgets, idx_stride=300, seq_lens=lens, n_sink=4, n_recent=32,
                      pool="avg", pool_kernel=5)
    assert np.array_equal(got, want)
    assert np.array_equal(got, ref.select_pipeline(small, [3000, 517, 2300], [300, 60, 230], 4, 32, "avg", 5, 300))
    assert (got[1, :, 60:] == -1).all()


def test_rejects_problems_beyond_the_fixed_capacity():
    n = api.SELECT_NOALLOC_MAX_KEYS // 8 + 1
    scores = torch.zeros((1, 8, n), dtype=torch.float32, device="cuda")
    idx = torch.empty((1, 8, 64), dtype=torch.int32, device="cuda")
    with pytest.raises(api.ObcError) as e:
        api.obc_select_noalloc(scores, idx, budget=64, n_recent=8)
    assert e.value.status == -8
