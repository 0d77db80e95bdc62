"""Bit-exact parity of obc_select / obc_compact with the CPU checker when both are fed the
same fp32 scores."""
import numpy as np
import pytest
import torch

from oracle import reference as ref
from paper_2510_07651_b200 import api, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _select_both(scores, seq_lens, budgets, n_sink, n_recent, pool, kern, stride=None):
    B, Hkv, Nmax = scores.shape
    budgets = np.asarray(budgets, np.int32)
    stride = int(budgets.max()) if stride is None else stride
    want = ref.select_pipeline(scores, seq_lens, budgets, n_sink, n_recent, pool, kern, stride)
    sd = torch.from_numpy(scores).cuda()
    uniform = (budgets == budgets[0]).all()
    ld = None if (np.asarray(seq_lens) == Nmax).all() else torch.from_numpy(np.asarray(seq_lens, np.int32)).cuda()
    got = api.obc_select(sd, budget=int(budgets[0]) if uniform else 0,
                         budgets=None if uniform else torch.from_numpy(budgets).cuda(), idx_stride=stride,
                         seq_lens=ld, n_sink=n_sink, n_recent=n_recent, pool=pool, pool_kernel=kern)
    torch.cuda.synchronize()
    return got, want


@pytest.mark.parametrize("pool,kern", [("none", 1), ("max", 7), ("avg", 5)])
@pytest.mark.parametrize("N,budget,n_sink,n_recent", [(1024, 256, 0, 16), (5000, 700, 4, 32), (33000, 2048, 0, 32),
                                                        (100, 100, 0, 0), (100, 20, 4, 16), (70000, 4096, 0, 64)])
def test_select_bit_exact_on_random_scores(pool, kern, N, budget, n_sink, n_recent):
    rng = np.random.default_rng(N + kern)
    scores = (rng.random((2, 3, N), dtype=np.float32) ** 8 * 1e-3).astype(np.float32)
    got, want = _select_both(scores, [N, N], [budget, budget], n_sink, n_recent, pool, kern)
    assert np.array_equal(got.cpu().numpy(), want)


def test_select_ties_keep_lowest_index_and_all_equal_scores():
    N = 3000
    rng = np.random.default_rng(0)
    scores = (rng.integers(0, 6, (1, 4, N)) / 4).astype(np.float32)     # heavy ties
    scores[0, 1] = 0.5                                                  # all equal
    scores[0, 2] = 0.0
    scores[0, 3, ::2] = -0.0                                            # -0.0 ranks equal to +0.0
    scores[0, 3, 1::2] = 0.0
    got, want = _select_both(scores, [N], [777], 4, 32, "none", 1, stride=800)
    g = got.cpu().numpy()
    assert np.array_equal(g, want)
    assert (g[..., 777:] == -1).all()


@pytest.mark.parametrize("N,budget", [(40000, 3000), (33000, 2048)])
def test_select_when_the_first_radix_pass_leaves_too_many_survivors(N, budget):
    """Scores that share their top 11 key bits (all equal; five distinct values; a narrow range with distinct low
    bits): the survivor lists of the first pass do not fit their slots, and the cluster settles the remaining bits
    with two more exchanged passes instead of on gathered lists."""
    rng = np.random.default_rng(N)
    scores = np.empty((1, 4, N), np.float32)
    scores[0, 0] = 0.25                                                     # all equal: ties -> lowest indices
    scores[0, 1] = (1.0 + rng.integers(0, 5, N) * 2.0 ** -20).astype(np.float32)   # five values in one bin, heavy ties
    scores[0, 2] = (1.0 + rng.random(N) * 2.0 ** -12).astype(np.float32)    # one bin, distinct low bits
    scores[0, 3] = (rng.random(N, dtype=np.float32) ** 8 * 1e-3)            # an ordinary head beside them
    for pool, kern in (("none", 1), ("max", 7)):
        got, want = _select_both(scores, [N], [budget], 4, 32, pool, kern)
        assert np.array_equal(got.cpu().numpy(), want), (pool, kern)


def test_select_ragged_lengths_and_per_sequence_budgets():
    rng = np.random.default_rng(1)
    lens = np.array([4096, 517, 2300], np.int32)
    scores = rng.random((3, 2, 4096), dtype=np.float32)
    budgets = [max(33, int(n) // 10) for n in lens]
    got, want = _select_both(scores, lens, budgets, 0, 32, "max", 7)
    assert np.array_equal(got.cpu().numpy(), want)


def test_select_budget_equals_protected_tokens():
    rng = np.random.default_rng(2)
    scores = rng.random((1, 2, 500), dtype=np.float32)
    got, want = _select_both(scores, [500], [36], 4, 32, "max", 7)
    assert np.array_equal(got.cpu().numpy(), want)


def test_bad_device_side_budget_gives_minus_one_row():
    scores = torch.rand((2, 1, 256), device="cuda")
    budgets = torch.tensor([64, 9999], dtype=torch.int32, device="cuda")
    idx = api.obc_select(scores, budgets=budgets, idx_stride=64, n_recent=8)
    torch.cuda.synchronize()
    assert (idx[1] == -1).all() and (idx[0] >= 0).all()


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_compact_bit_exact(dtype):
    case = synth.make_prefill("cmp", B=2, Hq=4, Hkv=2, d=128, W=8, N=[900, 411], dtype=dtype, seed=21)
    q, k, v = H.upload(case)
    rng = np.random.default_rng(3)
    scores = rng.random((2, 2, 900), dtype=np.float32)
    budgets = np.array([90, 41], np.int32)
    got_idx, want_idx = _select_both(scores, case.seq_lens, budgets, 0, 8, "none", 1)
    assert np.array_equal(got_idx.cpu().numpy(), want_idx)
    ko, vo, so = api.obc_compact(k, v, got_idx, scores_in=torch.from_numpy(scores).cuda())
    torch.cuda.synchronize()
    kb = ko.view(torch.int16).cpu().numpy() if dtype == "bf16" else ko.cpu().numpy()
    vb = vo.view(torch.int16).cpu().numpy() if dtype == "bf16" else vo.cpu().numpy()
    src_k = case.k_bits.view(np.int16) if dtype == "bf16" else case.k
    src_v = case.v_bits.view(np.int16) if dtype == "bf16" else case.v
    for b in range(2):
        for h in range(2):
            n = budgets[b]
            assert np.array_equal(kb[b, h, :n], ref.compact(src_k[b, h], want_idx[b, h], n))
            assert np.array_equal(vb[b, h, :n], ref.compact(src_v[b, h], want_idx[b, h], n))
            assert (kb[b, h, n:] == 0).all() and (vb[b, h, n:] == 0).all()
            assert np.array_equal(so[b, h, :n].cpu().numpy(), scores[b, h][want_idx[b, h, :n]])


def test_whole_prefill_path_config1():
    # score -> select -> compact end to end; selection compared on the GPU's own fp32 scores
    case, run = synth.config(1)
    q, k, v = H.upload(case)
    ko, vo, idx, scores = api.evict_prefill(q, k, v, budget=run["budget"], variant="VK", n_recent=run["n_recent"])
    torch.cuda.synchronize()
    s = scores[0].cpu().numpy()
    want_idx = ref.select_pipeline(s, case.seq_lens, [run["budget"]], 0, run["n_recent"], "none", 1, run["budget"])
    assert np.array_equal(idx.cpu().numpy(), want_idx)
    assert np.array_equal(ko.cpu().numpy()[0, 0], case.k[0, 0][want_idx[0, 0]])
    assert np.array_equal(vo.cpu().numpy()[0, 0], case.v[0, 0][want_idx[0, 0]])
    # and the kept set agrees with the one the double-precision scores select, except near ties
    ref_s = H.oracle_scores(case, ["VK"])["VK"].astype(np.float32)
    ref_idx = ref.select_pipeline(ref_s, case.seq_lens, [run["budget"]], 0, run["n_recent"], "none", 1, run["budget"])
    overlap = len(set(ref_idx[0, 0].tolist()) & set(want_idx[0, 0].tolist()))
    assert overlap >= run["budget"] - 2
