"""Pins for the CPU checker's pool / select / compact / decode-evict functions (Algorithm 2):
library pooling routines, sort-based brute force, and numpy indexing."""
import numpy as np
import pytest
import torch

from oracle import reference as ref


def test_max_pool_matches_library_routine():
    rng = np.random.default_rng(0)
    s = rng.random(200).astype(np.float32)
    for kern in (3, 5, 7):
        lo, hi = 4, 180
        got = ref.pool(s, lo, hi, "max", kern)
        want = torch.nn.functional.max_pool1d(torch.from_numpy(s[lo:hi])[None, None], kern, 1, kern // 2)[0, 0].numpy()
        assert (got[lo:hi] == want).all()
        assert (got[:lo] == s[:lo]).all() and (got[hi:] == s[hi:]).all()


def test_avg_pool_matches_sequential_fp32_adds_and_library():
    rng = np.random.default_rng(1)
    s = (rng.random(120) * 1e-3).astype(np.float32)
    lo, hi, kern = 0, 100, 5
    got = ref.pool(s, lo, hi, "avg", kern)
    want = np.empty(hi - lo, np.float32)
    for p in range(lo, hi):
        acc = np.float32(0)
        for t in range(p - 2, p + 3):
            if lo <= t < hi:
                acc = np.float32(acc + s[t])
        want[p - lo] = np.float32(acc / np.float32(kern))
    assert (got[lo:hi] == want).all()
    lib = torch.nn.functional.avg_pool1d(torch.from_numpy(s[lo:hi])[None, None], kern, 1, 2,
                                         count_include_pad=True)[0, 0].numpy()
    np.testing.assert_allclose(got[lo:hi], lib, rtol=3e-7)


def test_pool_none_is_identity():
    s = np.arange(10, dtype=np.float32)
    assert (ref.pool(s, 2, 8, "none", 1) == s).all()
    assert (ref.pool(s, 2, 8, "max", 1) == s).all()


def brute_select(s, budget, n_sink, n_recent):
    N = len(s)
    lo, hi = n_sink, N - n_recent
    order = sorted(range(lo, hi), key=lambda p: (-float(s[p]), p))
    keep = sorted(order[:budget - n_sink - n_recent])
    return np.array(list(range(n_sink)) + keep + list(range(hi, N)), np.int32)


@pytest.mark.parametrize("seed", range(4))
def test_select_matches_sort_brute_force_with_ties(seed):
    rng = np.random.default_rng(seed)
    N = 300
    s = rng.integers(0, 12, N).astype(np.float32) / 8     # many exact ties
    for budget, n_sink, n_recent in [(40, 0, 8), (64, 4, 16), (N, 0, 0), (24, 4, 20), (100, 0, 0)]:
        got = ref.select(s, budget, n_sink, n_recent, idx_len=budget + 3)
        want = brute_select(s, budget, n_sink, n_recent)
        assert (got[:budget] == want).all()
        assert (got[budget:] == -1).all()
        assert (np.diff(got[:budget]) > 0).all()


def test_select_agrees_with_library_topk_when_scores_are_distinct():
    rng = np.random.default_rng(9)
    s = rng.permutation(500).astype(np.float32)
    got = ref.select(s, 50, 0, 10)
    top = torch.topk(torch.from_numpy(s[:490]), 40).indices.sort().values.numpy()
    assert (got[:40] == top).all() and (got[40:] == np.arange(490, 500)).all()


def test_select_rejects_bad_budgets():
    s = np.zeros(10, np.float32)
    with pytest.raises(ValueError):
        ref.select(s, 11, 0, 0)
    with pytest.raises(ValueError):
        ref.select(s, 3, 2, 2)


def test_compact_is_a_row_gather():
    rng = np.random.default_rng(2)
    src = rng.integers(0, 65535, (50, 16)).astype(np.uint16)
    idx = np.array([0, 3, 7, 49], np.int32)
    assert (ref.compact(src, idx, 4) == src[idx]).all()
    src32 = rng.standard_normal((50, 8)).astype(np.float32)
    assert (ref.compact(src32, idx, 3) == src32[idx[:3]]).all()


def test_decode_scores_match_a_single_query_prefill_problem():
    # the live slots, in any slot order, are a W = 1 cache: same scores as the prefill scorer
    rng = np.random.default_rng(3)
    G, d, cap, n = 4, 16, 40, 29
    qg = rng.standard_normal((G, d)).astype(np.float32)
    kc = rng.standard_normal((cap, d)).astype(np.float32)
    vc = rng.standard_normal((cap, d)).astype(np.float32)
    pos = np.full(cap, -1, np.int32)
    slots = rng.permutation(36)[:n]
    pos[slots] = rng.permutation(100)[:n]
    for var in ("V", "K", "VK", "ATTN"):
        got = ref.decode_scores(qg, kc, vc, pos, 36, var)
        live = np.sort(slots)
        want = ref.score(qg[None, :, None, :], kc[live][None, None], vc[live][None, None], want=(var,))[var][0, 0]
        np.testing.assert_allclose(got[live], want, rtol=1e-12)
        dead = np.setdiff1d(np.arange(cap), live)
        assert (got[dead] == 0).all()


def test_decode_evict_brute_force():
    rng = np.random.default_rng(4)
    for trial in range(20):
        cap = 30
        pos = np.full(cap, -1, np.int32)
        live = rng.permutation(cap)[:22]
        pos[live] = rng.permutation(60)[:22]
        s = (rng.integers(0, 4, cap) / 4).astype(np.float32)
        step_pos, n_sink, n_recent = 60, 4, 10
        cands = [p for p in range(cap) if pos[p] >= n_sink and pos[p] <= step_pos - n_recent]
        want = min(cands, key=lambda p: (float(s[p]), -int(pos[p]))) if cands else -1
        assert ref.decode_evict(s, pos, cap, step_pos, n_sink, n_recent) == want


def test_decode_state_keeps_sinks_and_recents_and_respects_budget():
    rng = np.random.default_rng(5)
    G, d, n0, budget, n_sink, n_recent = 2, 8, 12, 12, 2, 4
    st = ref.DecodeState(rng.standard_normal((n0, d)).astype(np.float32),
                         rng.standard_normal((n0, d)).astype(np.float32), cap=budget + 1)
    for t in range(30):
        step_pos = n0 + t
        st.append(rng.standard_normal(d).astype(np.float32), rng.standard_normal(d).astype(np.float32), step_pos)
        st.s_acc += st.scores(rng.standard_normal((G, d)).astype(np.float32)).astype(np.float32)
        st.evict(step_pos, budget, n_sink, n_recent)
        assert st.live == budget
        livepos = st.pos[st.pos >= 0]
        assert len(set(livepos.tolist())) == budget
        assert set(range(n_sink)) <= set(livepos.tolist())
        assert set(range(step_pos - n_recent + 1, step_pos + 1)) <= set(livepos.tolist())


@pytest.mark.parametrize("window", [1, 3, 7, 64])
def test_decode_window_accumulator_matches_a_log_kept_per_token(window):
    """Accumulation within a recent window (App. B): the state's ring, indexed by slot and step mod w, must
    give every live token the sum of the scores it received in the last w steps, as read off a plain log
    keyed by (token position, step) that knows nothing of slots or rings."""
    rng = np.random.default_rng(40 + window)
    G, d, n0, budget, n_sink, n_recent, steps = 2, 8, 10, 12, 2, 3, 40
    k0 = rng.standard_normal((n0, d)).astype(np.float32)
    v0 = rng.standard_normal((n0, d)).astype(np.float32)
    st = ref.DecodeState(k0, v0, cap=budget + 1, window=window)
    full = ref.DecodeState(k0, v0, cap=budget + 1)                       # accumulates over every step
    log = {}                                                             # (position, step) -> score
    for t in range(steps):
        step_pos = n0 + t
        k_t, v_t = rng.standard_normal(d).astype(np.float32), rng.standard_normal(d).astype(np.float32)
        q_t = rng.standard_normal((G, d)).astype(np.float32)
        st.append(k_t, v_t, step_pos)
        sc = st.scores(q_t)
        for slot in np.flatnonzero(st.pos >= 0):
            log[(int(st.pos[slot]), t)] = float(sc[slot])
        acc = st.accumulate(sc, step_pos)
        for slot in np.flatnonzero(st.pos >= 0):
            want = sum(log.get((int(st.pos[slot]), u), 0.0) for u in range(max(0, t - window + 1), t + 1))
            assert abs(acc[slot] - want) <= 1e-12 * max(1.0, abs(want))
        if window == 1:                                                  # only this step's scores
            np.testing.assert_array_equal(acc[st.pos >= 0], sc[st.pos >= 0])
        st.s_acc[:] = acc.astype(np.float32)
        st.evict(step_pos, budget, n_sink, n_recent)
        if window >= steps:                                              # never slides: the plain accumulation
            full.append(k_t, v_t, step_pos)
            facc = full.accumulate(full.scores(q_t), step_pos)
            full.s_acc[:] = facc.astype(np.float32)
            full.evict(step_pos, budget, n_sink, n_recent)
            assert np.array_equal(full.pos, st.pos)
            np.testing.assert_allclose(acc[st.pos >= 0], facc[st.pos >= 0], rtol=1e-6, atol=1e-12)


# ---- head-adaptive budgets (global ranking across heads with a per-head safeguard) ----------------
def brute_adaptive(pooled, budget, n_sink, n_recent, safeguard):
    """Plain-Python statement: every head's s best candidates, then the best of the rest of all heads."""
    H, N = pooled.shape
    lo, hi, n_hh = n_sink, N - n_recent, budget - n_sink - n_recent
    s = int(np.floor(float(np.float32(safeguard)) * n_hh))
    kept = [set() for _ in range(H)]
    rest = []
    for h in range(H):
        order = sorted(range(lo, hi), key=lambda p: (-float(pooled[h, p]), p))
        kept[h].update(order[:s])
        rest += [(-float(pooled[h, p]), h, p) for p in order[s:]]
    for _, h, p in sorted(rest)[:H * (n_hh - s)]:
        kept[h].add(p)
    return [np.array(list(range(n_sink)) + sorted(k) + list(range(hi, N)), np.int32) for k in kept]


@pytest.mark.parametrize("seed", range(3))
@pytest.mark.parametrize("safeguard", [0.0, 0.2, 0.5, 1.0])
def test_adaptive_select_matches_brute_force_with_ties(seed, safeguard):
    rng = np.random.default_rng(100 + seed)
    H, N = 3, 120
    pooled = rng.integers(0, 9, (H, N)).astype(np.float32) / 4          # many ties, within and across heads
    pooled[1] *= 2.0                                                     # one head scores higher overall
    for budget, n_sink, n_recent in [(30, 0, 8), (40, 4, 16), (N, 0, 0), (25, 4, 20)]:
        idx_len = n_sink + n_recent + H * (budget - n_sink - n_recent)
        idx_len = min(idx_len, N)
        idx, counts = ref.select_adaptive(pooled, budget, n_sink, n_recent, safeguard, idx_len)
        want = brute_adaptive(pooled, budget, n_sink, n_recent, safeguard)
        assert counts.sum() == H * budget
        for h in range(H):
            assert counts[h] == len(want[h])
            assert (idx[h, :counts[h]] == want[h]).all() and (idx[h, counts[h]:] == -1).all()


def test_adaptive_select_limits():
    rng = np.random.default_rng(7)
    H, N, budget, n_sink, n_recent = 4, 200, 50, 2, 10
    pooled = rng.random((H, N), dtype=np.float32)
    # safeguard 1: every head keeps exactly its own top budget, i.e. the per-head selection
    idx, counts = ref.select_adaptive(pooled, budget, n_sink, n_recent, 1.0, budget)
    for h in range(H):
        assert counts[h] == budget and (idx[h] == ref.select(pooled[h], budget, n_sink, n_recent)).all()
    # safeguard 0 with distinct scores: the library's top-k over all heads' candidates at once
    idx, counts = ref.select_adaptive(pooled, budget, n_sink, n_recent, 0.0, N)
    n_hh = budget - n_sink - n_recent
    flat = torch.from_numpy(pooled[:, n_sink:N - n_recent].copy()).reshape(-1)
    top = torch.topk(flat, H * n_hh).indices.numpy()
    n = N - n_sink - n_recent
    for h in range(H):
        want = np.sort(top[top // n == h] % n + n_sink)
        got = idx[h, n_sink:counts[h] - n_recent]
        assert (got == want).all()
        assert (idx[h, :n_sink] == np.arange(n_sink)).all() and (idx[h, counts[h] - n_recent:counts[h]] == np.arange(N - n_recent, N)).all()


def test_adaptive_select_moves_budget_to_the_head_that_scores_higher():
    # head 0 scores 10 everywhere, head 1 scores 1: with a quarter safeguarded (1 of 4 slots), head 1 keeps
    # its one guaranteed token and head 0 takes the other seven
    pooled = np.stack([np.full(12, 10.0, np.float32), np.full(12, 1.0, np.float32)])
    idx, counts = ref.select_adaptive(pooled, 4, 0, 0, 0.25, 8)
    assert counts.tolist() == [7, 1]
    assert idx[0, :7].tolist() == list(range(7)) and idx[1, 0] == 0 and (idx[1, 1:] == -1).all()
    # a head may not outgrow the index buffer
    with pytest.raises(ValueError):
        ref.select_adaptive(pooled, 4, 0, 0, 0.25, 6)


def test_adaptive_pipeline_pools_each_head_before_ranking():
    rng = np.random.default_rng(11)
    scores = rng.random((2, 3, 90), dtype=np.float32)
    lens = np.array([90, 61], np.int32)
    idx, counts = ref.select_adaptive_pipeline(scores, lens, [20, 15], 1, 6, "max", 5, 0.2, 60)
    for b in range(2):
        n = int(lens[b])
        pooled = np.stack([ref.pool(scores[b, h, :n], 1, n - 6, "max", 5) for h in range(3)])
        want = brute_adaptive(pooled, [20, 15][b], 1, 6, 0.2)
        for h in range(3):
            assert (idx[b, h, :counts[b, h]] == want[h]).all() and (idx[b, h, counts[b, h]:] == -1).all()
