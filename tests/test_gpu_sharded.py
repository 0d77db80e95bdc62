"""A cache sharded by token range (context parallelism), on one GPU: the shards are scored one after another
through obc_window_attention -> obc_merge_attention -> obc_score_given, exactly the calls each rank of a
multi-GPU job makes (the all-gather between them is a stack here), and the concatenated scores are compared
with the CPU checker's scores of the whole, unsharded cache."""
import numpy as np
import pytest
import torch

from paper_2510_07651_b200 import api, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _sharded_scores(case, cuts, variants, path):
    q, k, v = H.upload(case)
    N, B = case.Nmax, case.B
    bounds = [0] + list(cuts) + [N]
    shards = [(lo, hi) for lo, hi in zip(bounds[:-1], bounds[1:])]
    masks = [torch.full((B,), N - lo, dtype=torch.int32, device="cuda") for lo, _ in shards]
    parts = [api.obc_window_attention(q, k[:, :, lo:hi], v[:, :, lo:hi], mask_lens=m, path=path)
             for (lo, hi), m in zip(shards, masks)]
    o_all, lse_all = api.obc_merge_attention(torch.stack([p[0] for p in parts]), torch.stack([p[1] for p in parts]))
    order = [n for n in H.VARIANT_ORDER if n in variants]
    out = []
    for (lo, hi), m in zip(shards, masks):
        ks, vs = k[:, :, lo:hi], v[:, :, lo:hi]
        p = api.score_params(q, ks, variants=order, path=path, mask_lens=m)
        ws = torch.empty(api.obc_score_workspace(p), dtype=torch.uint8, device="cuda")
        s = api.obc_score_given(q, ks, vs, o_all, lse_all, variants=order, path=path, mask_lens=m, workspace=ws)
        api.obc_score_status(ws)
        out.append(s)
    torch.cuda.synchronize()
    s = torch.cat(out, dim=-1).cpu().numpy()
    return {n: s[i] for i, n in enumerate(order)}, o_all, lse_all


@pytest.mark.parametrize("N,W,Hq,Hkv,dtype,path,cuts", [
    (3000, 64, 8, 2, "bf16", "tc", (1100, 2950)),        # R = 256 (row chunks of 64); the last shard (50 tokens) is shorter than the window
    (2500, 32, 8, 2, "bf16", "auto", (777, 1500, 2490)), # R = 128: the single-chunk kernels; uneven shards, one of 10 tokens
    (900, 16, 4, 2, "f32", "auto", (300, 640)),          # CUDA-core kernels, fp32
    (1500, 24, 6, 2, "bf16", "simt", (1490,)),           # CUDA-core kernels, bf16; the second shard lies inside the window
])
def test_token_sharded_cache_scores_like_the_whole(N, W, Hq, Hkv, dtype, path, cuts):
    case = synth.make_prefill("sharded", B=2, Hq=Hq, Hkv=Hkv, d=128, W=W, N=N, dtype=dtype, seed=500 + N, hh_frac=0.02)
    variants = ["V", "K", "VK", "ATTN"]
    got, o_all, lse_all = _sharded_scores(case, cuts, variants, path)
    want = H.oracle_scores(case, variants)
    mx = max(np.abs(want[n]).max() for n in ("V", "K", "VK"))
    for n in variants:
        H.assert_scores_close(got[n], want[n], dtype, tight=2e-2 if dtype == "bf16" else None,
                              what=f"sharded {n} {path}", mx=None if n == "ATTN" else mx)
    # the merged attention is the attention over the whole cache
    from oracle import reference as ref
    att = ref.score(case.q, case.k, case.v, want=("ATTN",), return_attention=True)
    o_ref = att["O"].reshape(case.B, Hq, W, 128)
    lse_ref = (att["m"] + np.log(att["l"])).reshape(case.B, Hq, W)
    tol = 2e-2 if dtype == "bf16" else 1e-4
    assert np.abs(lse_all.cpu().numpy() - lse_ref).max() <= tol
    assert np.abs(o_all.cpu().numpy() - o_ref).max() <= tol * max(1.0, np.abs(o_ref).max())


def test_window_attention_with_one_cta_per_row_chunk():
    """2560 window rows per KV head in 20 chunks: pass 1 has one CTA per (unit, chunk), writes the merged results
    itself and no merge kernel runs; in the second shard the early rows see no token at all (their output is 0 and
    their log-sum-exp -inf, which the merge of the shards must weigh as nothing)."""
    N, W, Hq, Hkv = 1024, 640, 32, 8
    case = synth.make_prefill("direct", B=1, Hq=Hq, Hkv=Hkv, d=128, W=W, N=N, dtype="bf16", seed=77, hh_frac=0.02)
    q, k, v = H.upload(case)
    shards = [(0, 700), (700, N)]
    parts = [api.obc_window_attention(q, k[:, :, lo:hi], v[:, :, lo:hi],
                                      mask_lens=torch.full((1,), N - lo, dtype=torch.int32, device="cuda"), path="tc")
             for lo, hi in shards]
    lse1 = parts[1][1].cpu().numpy()
    assert np.isneginf(lse1[0, :, : 700 - (N - W)]).all() and np.isfinite(lse1[0, :, 700 - (N - W):]).all()
    o_all, lse_all = api.obc_merge_attention(torch.stack([p[0] for p in parts]), torch.stack([p[1] for p in parts]))
    torch.cuda.synchronize()
    from oracle import reference as ref
    att = ref.score(case.q, case.k, case.v, want=("ATTN",), return_attention=True)
    o_ref = att["O"].reshape(1, Hq, W, 128)
    lse_ref = (att["m"] + np.log(att["l"])).reshape(1, Hq, W)
    assert np.abs(lse_all.cpu().numpy() - lse_ref).max() <= 2e-2
    assert np.abs(o_all.cpu().numpy() - o_ref).max() <= 2e-2 * max(1.0, np.abs(o_ref).max())
    # the unsharded call takes the same path
    o_one, lse_one = api.obc_window_attention(q, k, v, path="tc")
    torch.cuda.synchronize()
    assert np.abs(lse_one.cpu().numpy() - lse_ref).max() <= 2e-2
    assert np.abs(o_one.cpu().numpy() - o_ref).max() <= 2e-2 * max(1.0, np.abs(o_ref).max())


def test_merge_attention_weights_and_empty_shards():
    """lse = log sum exp(lse_s), o = sum exp(lse_s - lse) o_s; a shard that saw nothing (lse = -inf) weighs 0."""
    g = torch.Generator(device="cpu").manual_seed(3)
    P, rows = 4, 37
    o = torch.randn((P, rows, 128), generator=g)
    lse = torch.randn((P, rows), generator=g) * 3
    lse[2, :10] = float("-inf")
    lse[:, 5] = float("-inf"); lse[1, 5] = 0.25                  # only one shard saw row 5
    want_lse = torch.logsumexp(lse.double(), dim=0)
    want_o = (torch.exp(lse.double() - want_lse).unsqueeze(-1) * o.double()).sum(0)
    got_o, got_lse = api.obc_merge_attention(o.cuda(), lse.cuda())
    assert torch.allclose(got_lse.cpu().double(), want_lse, rtol=1e-5, atol=1e-5)
    assert torch.allclose(got_o.cpu().double(), want_o, rtol=1e-4, atol=1e-5)
    assert torch.equal(got_o[5].cpu(), o[1, 5])


def test_shard_indices_and_local_compaction():
    """Every shard gathers the kept rows it owns; put side by side the shards' compacted rows are the compacted cache."""
    case = synth.make_prefill("shardidx", B=2, Hq=4, Hkv=2, d=128, W=8, N=[1000, 640], dtype="bf16", seed=9)
    q, k, v = H.upload(case)
    lens = H.lens_dev(case)
    s = api.obc_score(q, k, v, seq_lens=lens, variants=["VK"])
    budgets = torch.tensor([100, 64], dtype=torch.int32, device="cuda")
    idx = api.obc_select(s[0], budget=0, budgets=budgets, idx_stride=100, seq_lens=lens, n_recent=8, pool="max", pool_kernel=7)
    k_all, v_all = api.obc_compact(k, v, idx)
    torch.cuda.synchronize()
    idx_h = idx.cpu().numpy()
    cuts = [0, 300, 310, 900, 1000]                           # a shard of ten tokens; the last one holds the recent tail
    filled = np.zeros((2, 2), np.int64)
    for lo, hi in zip(cuts[:-1], cuts[1:]):
        loc, cnt = api.obc_shard_indices(idx, lo, hi - lo)
        ko = torch.zeros((2, 2, 100, 128), dtype=torch.bfloat16, device="cuda")
        vo = torch.zeros_like(ko)
        api.obc_compact(k[:, :, lo:hi], v[:, :, lo:hi], loc, k_out=ko, v_out=vo)
        torch.cuda.synchronize()
        loc_h, cnt_h = loc.cpu().numpy(), cnt.cpu().numpy()
        for b in range(2):
            for h in range(2):
                row = idx_h[b, h]
                want = row[(row >= lo) & (row < hi)] - lo
                assert cnt_h[b, h] == len(want)
                assert np.array_equal(loc_h[b, h, :len(want)], want) and (loc_h[b, h, len(want):] == -1).all()
                f = int(filled[b, h])
                assert torch.equal(ko[b, h, :len(want)], k_all[b, h, f:f + len(want)])
                assert torch.equal(vo[b, h, :len(want)], v_all[b, h, f:f + len(want)])
                filled[b, h] += len(want)
    assert (filled == np.array([[100, 100], [64, 64]])).all()


def test_llama_32k_layer_sharded_over_two_ranks_full():
    """The 32k Llama layer at full size, its tokens split evenly over two shards: scores against the checker's
    scores of the whole cache, then the selection on the gathered scores and every shard's own compaction against
    the checker's selection and gather."""
    from oracle import reference as ref
    case, run = synth.config(2)
    got, _, _ = _sharded_scores(case, (case.Nmax // 2,), ["VK"], "auto")
    want = H.oracle_scores(case, ["VK"])["VK"]
    H.assert_scores_close(got["VK"], want, "bf16", tight=2e-2, what="sharded config 2")
    scores = torch.from_numpy(got["VK"]).cuda()
    budget = run["budget"]
    idx = api.obc_select(scores, budget=budget, n_sink=run["n_sink"], n_recent=run["n_recent"], pool=run["pool_mode"],
                         pool_kernel=run["pool_kernel"])
    torch.cuda.synchronize()
    want_idx = ref.select_pipeline(got["VK"], case.seq_lens, [budget], run["n_sink"], run["n_recent"], run["pool_mode"],
                                   run["pool_kernel"], budget)
    assert np.array_equal(idx.cpu().numpy(), want_idx)
    q, k, v = H.upload(case)
    half = case.Nmax // 2
    filled = np.zeros((case.B, case.Hkv), np.int64)
    for lo, hi in ((0, half), (half, case.Nmax)):
        loc, cnt = api.obc_shard_indices(idx, lo, hi - lo)
        ko, vo = api.obc_compact(k[:, :, lo:hi], v[:, :, lo:hi], loc)
        torch.cuda.synchronize()
        kb, vb, c = ko.view(torch.int16).cpu().numpy(), vo.view(torch.int16).cpu().numpy(), cnt.cpu().numpy()
        for h in range(case.Hkv):
            f, n = int(filled[0, h]), int(c[0, h])
            rows = want_idx[0, h, f:f + n]
            assert ((rows >= lo) & (rows < hi)).all()
            assert np.array_equal(kb[0, h, :n], case.k_bits[0, h].view(np.int16)[rows])
            assert np.array_equal(vb[0, h, :n], case.v_bits[0, h].view(np.int16)[rows])
            filled[0, h] += n
    assert (filled == budget).all()


@pytest.mark.parametrize("W,Hq,Hkv,path", [(32, 8, 2, "auto"), (64, 8, 2, "tc"), (16, 4, 2, "simt")])
def test_context_parallel_scores_with_the_library_ops(W, Hq, Hkv, path):
    """multirank.context_parallel_scores, the function every rank of a token-sharded job runs, with the library's own
    calls and no process group (a job of one rank: the all-gather is skipped, everything else is the code the ranks
    execute).  Once over the whole cache, and once per shard with the other shards' attention merged in by hand,
    against the checker's scores of the unsharded cache."""
    from paper_2510_07651_b200 import multirank
    N = 2100
    case = synth.make_prefill("cp", B=2, Hq=Hq, Hkv=Hkv, d=128, W=W, N=N, dtype="bf16", seed=77 + W, hh_frac=0.02)
    q, k, v = H.upload(case)
    variants = ["K", "VK", "ATTN"]
    want = H.oracle_scores(case, variants)
    mx = max(np.abs(want[n]).max() for n in ("K", "VK"))
    s = multirank.context_parallel_scores(q, k, v, offset=0, total_len=N, variants=variants, path=path)
    torch.cuda.synchronize()
    s = s.cpu().numpy()
    for i, n in enumerate(variants):
        H.assert_scores_close(s[i], want[n], "bf16", tight=2e-2, what=f"one rank {n} {path}", mx=None if n == "ATTN" else mx)

    # two shards: each rank's call, with an `ops` object whose merge folds in the peer's attention (what the
    # all-gather would have delivered); window attention and scoring are the library's
    cut = 1300
    shards = [(0, cut), (cut, N)]
    parts = [api.obc_window_attention(q, k[:, :, lo:hi], v[:, :, lo:hi],
                                      mask_lens=torch.full((case.B,), N - lo, dtype=torch.int32, device="cuda"), path=path)
             for lo, hi in shards]

    class Ops:
        def __init__(self, me): self.me = me
        obc_window_attention = staticmethod(api.obc_window_attention)
        obc_score_given = staticmethod(api.obc_score_given)
        def obc_merge_attention(self, o_parts, lse_parts):
            peer = parts[1 - self.me]
            return api.obc_merge_attention(torch.cat([o_parts, peer[0].unsqueeze(0)]), torch.cat([lse_parts, peer[1].unsqueeze(0)]))
    got = []
    for r, (lo, hi) in enumerate(shards):
        got.append(multirank.context_parallel_scores(q, k[:, :, lo:hi], v[:, :, lo:hi], offset=lo, total_len=N,
                                                     variants=variants, path=path, ops=Ops(r)))
    torch.cuda.synchronize()
    s2 = torch.cat(got, dim=-1).cpu().numpy()
    for i, n in enumerate(variants):
        H.assert_scores_close(s2[i], want[n], "bf16", tight=2e-2, what=f"two ranks {n} {path}", mx=None if n == "ATTN" else mx)
