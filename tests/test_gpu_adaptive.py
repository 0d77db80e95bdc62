"""Bit-exact parity of obc_select_adaptive (head-adaptive budgets: ranking across the heads of a layer with a
per-head safeguard) with the CPU checker fed the same fp32 scores, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import reference as ref
from paper_2510_07651_b200 import api, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _both(scores, seq_lens, budget, n_sink, n_recent, pool, kern, safeguard, stride):
    B, Hkv, Nmax = scores.shape
    want_idx, want_cnt = ref.select_adaptive_pipeline(scores, seq_lens, [budget] * B, n_sink, n_recent, pool, kern,
                                                      safeguard, stride)
    ld = None if (np.asarray(seq_lens) == Nmax).all() else torch.from_numpy(np.asarray(seq_lens, np.int32)).cuda()
    idx, cnt = api.obc_select_adaptive(torch.from_numpy(scores).cuda(), budget=budget, safeguard=safeguard,
                                       idx_stride=stride, seq_lens=ld, n_sink=n_sink, n_recent=n_recent, pool=pool,
                                       pool_kernel=kern)
    torch.cuda.synchronize()
    return idx.cpu().numpy(), cnt.cpu().numpy(), want_idx, want_cnt


@pytest.mark.parametrize("safeguard", [0.0, 0.2, 0.55, 1.0])
@pytest.mark.parametrize("pool,kern", [("none", 1), ("max", 7), ("avg", 5)])
def test_adaptive_bit_exact_with_ties(safeguard, pool, kern):
    rng = np.random.default_rng(int(safeguard * 100) + kern)
    B, Hkv, N = 2, 4, 3000
    scores = (rng.integers(0, 40, (B, Hkv, N)) / 16).astype(np.float32)       # ties within and across heads
    scores[:, 1] *= 3.0                                                        # one head scores higher overall
    scores[:, 2] *= 0.25
    idx, cnt, want_idx, want_cnt = _both(scores, [N, N], 300, 4, 32, pool, kern, safeguard, 1100)
    assert np.array_equal(cnt, want_cnt) and np.array_equal(idx, want_idx)
    assert (cnt.sum(axis=1) == Hkv * 300).all()


def test_adaptive_ragged_lengths_and_random_scores():
    rng = np.random.default_rng(5)
    lens = np.array([5000, 777, 2300], np.int32)
    scores = (rng.random((3, 3, 5000), dtype=np.float32) ** 6).astype(np.float32)
    scores[:, 0] *= 4.0
    idx, cnt, want_idx, want_cnt = _both(scores, lens, 200, 2, 16, "max", 7, 0.2, 570)
    assert np.array_equal(cnt, want_cnt) and np.array_equal(idx, want_idx)


def test_adaptive_degenerate_budgets():
    rng = np.random.default_rng(6)
    scores = rng.random((1, 2, 400), dtype=np.float32)
    # nothing to choose: only the protected tokens
    idx, cnt, want_idx, want_cnt = _both(scores, [400], 36, 4, 32, "none", 1, 0.2, 40)
    assert np.array_equal(cnt, want_cnt) and np.array_equal(idx, want_idx)
    # everything is kept
    idx, cnt, want_idx, want_cnt = _both(scores, [400], 400, 0, 16, "none", 1, 0.2, 400)
    assert np.array_equal(cnt, want_cnt) and np.array_equal(idx, want_idx)
    # a safeguard so small that no head has a guaranteed token
    idx, cnt, want_idx, want_cnt = _both(scores, [400], 50, 0, 8, "max", 5, 0.01, 100)
    assert np.array_equal(cnt, want_cnt) and np.array_equal(idx, want_idx)


def test_a_head_that_outgrows_its_row_is_flagged():
    # head 0 scores far higher and takes nearly all of the layer's slots; its row holds only 40 of them
    scores = np.ones((1, 3, 500), np.float32)
    scores[0, 0] = 50.0
    idx, cnt = api.obc_select_adaptive(torch.from_numpy(scores).cuda(), budget=30, safeguard=0.2, idx_stride=40, n_recent=4)
    torch.cuda.synchronize()
    idx, cnt = idx.cpu().numpy(), cnt.cpu().numpy()
    assert cnt[0, 0] == -1 and (idx[0, 0] == -1).all()
    # n_hh = 26, 5 guaranteed per head; heads 1 and 2 keep 5 + 4 recent tokens
    assert cnt[0, 1] == 9 and cnt[0, 2] == 9 and (idx[0, 1, :5] == np.arange(5)).all()
    assert (idx[0, 1, 5:9] == np.arange(496, 500)).all() and (idx[0, 1, 9:] == -1).all()
    with pytest.raises(api.ObcError):                     # one budget per call
        api.lib()
        p = api.select_params(torch.from_numpy(scores).cuda(), budget=30, budgets=torch.zeros(1, dtype=torch.int32, device="cuda"),
                              idx_stride=40)
        n = api.C.c_size_t(0)
        api._check(api.lib().obc_select_adaptive_workspace(api.C.byref(p), 0.2, api.C.byref(n)), "workspace")


def test_adaptive_then_compact_on_a_scored_layer():
    # the whole path on a Llama-shaped layer: scores from obc_score, adaptive budgets, ragged gather
    case, run = synth.config(2, shrink=4)                                   # N = 8192, 8 KV heads
    q, k, v = H.upload(case)
    scores = api.obc_score(q, k, v, variants=["VK"])
    budget, stride = run["budget"], 4 * run["budget"]
    idx, cnt = api.obc_select_adaptive(scores[0], budget=budget, safeguard=0.2, idx_stride=stride,
                                       n_recent=run["n_recent"], pool="max", pool_kernel=7)
    ko = torch.full((case.B, case.Hkv, stride, 128), 1.5, dtype=torch.bfloat16, device="cuda")
    vo = torch.full_like(ko, 1.5)
    api.obc_compact(k, v, idx, k_out=ko, v_out=vo)
    torch.cuda.synchronize()
    s = scores[0].cpu().numpy()
    want_idx, want_cnt = ref.select_adaptive_pipeline(s, case.seq_lens, [budget], 0, run["n_recent"], "max", 7, 0.2, stride)
    idx, cnt = idx.cpu().numpy(), cnt.cpu().numpy()
    assert np.array_equal(cnt, want_cnt) and np.array_equal(idx, want_idx)
    assert cnt.sum() == case.Hkv * budget and cnt.min() >= int(0.2 * (budget - run["n_recent"])) + run["n_recent"]
    kb = ko.view(torch.int16).cpu().numpy()
    pad = torch.full((1,), 1.5, dtype=torch.bfloat16).view(torch.int16).numpy()[0]
    for h in range(case.Hkv):
        n = int(cnt[0, h])
        assert np.array_equal(kb[0, h, :n], case.k_bits.view(np.int16)[0, h][want_idx[0, h, :n]])
        assert (kb[0, h, n:] == pad).all()
