"""The multi-GPU path on CPU: two gloo ranks each take their share of the KV heads of one layer,
run score -> select -> compact on it (here with the CPU checker standing in for the kernels), and
the gathered result must equal the unsharded one bit for bit: the units are independent, so the
sharded job needs no data-path collective.  Also the step-time reduction bench.py uses."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2510_07651_b200 import multirank, synth


def test_partition_is_contiguous_balanced_and_complete():
    for n, w in [(8, 1), (8, 2), (8, 3), (4, 8), (7, 4), (256, 8)]:
        parts = multirank.partition_units(n, w)
        assert len(parts) == w and parts[0][0] == 0 and parts[-1][1] == n
        assert all(parts[i][1] == parts[i + 1][0] for i in range(w - 1))
        sizes = [hi - lo for lo, hi in parts]
        assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)
    kv, qh = multirank.kv_head_shard(8, 4, 1, 2)
    assert (kv, qh) == (slice(4, 8), slice(16, 32))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    from oracle import reference as ref
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        case = synth.make_prefill("mr", B=2, Hq=12, Hkv=3, d=128, W=8, N=[600, 411], dtype="bf16", seed=31)
        G, budgets = case.G, np.array([60, 41], np.int32)
        kv, qh = multirank.kv_head_shard(case.Hkv, G, rank, world)

        def pipeline(q, k, v, k_bits):
            s = ref.score(q, k, v, seq_lens=case.seq_lens, want=("VK",))["VK"].astype(np.float32)
            idx = ref.select_pipeline(s, case.seq_lens, budgets, 0, 8, "max", 7, 60)
            kept = np.zeros(idx.shape + (128,), np.int16)
            for b in range(idx.shape[0]):
                for h in range(idx.shape[1]):
                    kept[b, h, :budgets[b]] = ref.compact(k_bits[b, h].view(np.int16), idx[b, h], budgets[b])
            return idx, kept

        idx_l, kept_l = pipeline(case.q[:, qh], case.k[:, kv], case.v[:, kv], case.k_bits[:, kv])
        idx_all = multirank.gather_head_shards(torch.from_numpy(idx_l), case.Hkv).numpy()
        kept_all = multirank.gather_head_shards(torch.from_numpy(kept_l), case.Hkv).numpy()
        slow = multirank.max_over_ranks(10.0 + rank)
        if rank == 0:
            idx_ref, kept_ref = pipeline(case.q, case.k, case.v, case.k_bits)
            out.put((np.array_equal(idx_all, idx_ref), np.array_equal(kept_all, kept_ref), slow))
    finally:
        dist.destroy_process_group()


def test_two_ranks_sharded_by_kv_head_match_the_unsharded_job():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    same_idx, same_kept, slow = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert same_idx and same_kept
    assert slow == pytest.approx(11.0)


# ---- cache sharded by token range: the exchange of the window attention -------------------------------
class _CpuOps:
    """Stand-ins for the three library calls, in plain double-precision tensor code, with the library's
    conventions: natural-log lse, -inf and a zero row where a shard shows a window row no token, and
    `mask_lens` = sequence length minus the position of the shard's first token."""

    @staticmethod
    def _logits(q, k, mask_lens, causal, scale):
        B, Hq, W, d = q.shape
        Hkv, n = k.shape[1], k.shape[2]
        G = Hq // Hkv
        z = torch.einsum("bhwd,bhnd->bhwn", q.double(), k.double().repeat_interleave(G, dim=1)) * (scale or d ** -0.5)
        if causal:
            last = mask_lens.view(B, 1, 1, 1).double() - W + torch.arange(W).view(1, 1, W, 1)
            z = z.masked_fill(torch.arange(n).view(1, 1, 1, n) > last, float("-inf"))
        return z, G

    @classmethod
    def obc_window_attention(cls, q, k, v, *, mask_lens, scale=0.0, causal=True, path="auto"):
        z, G = cls._logits(q, k, mask_lens, causal, scale)
        lse = torch.logsumexp(z, dim=-1)
        a = torch.exp(z - torch.where(torch.isinf(lse), torch.zeros_like(lse), lse).unsqueeze(-1))
        o = torch.einsum("bhwn,bhnd->bhwd", a, v.double().repeat_interleave(G, dim=1))
        return o.float(), lse.float()

    @staticmethod
    def obc_merge_attention(o_parts, lse_parts):
        lse = torch.logsumexp(lse_parts.double(), dim=0)
        w = torch.exp(lse_parts.double() - lse)
        return (w.unsqueeze(-1) * o_parts.double()).sum(0).float(), lse.float()

    @classmethod
    def obc_score_given(cls, q, k, v, o, lse, *, mask_lens, variants=("ATTN",), causal=True, scale=0.0, path="auto"):
        # the attention-only plane sum_r A_rp (Sec. 4.3) is enough to show which lse and which mask were used
        z, G = cls._logits(q, k, mask_lens, causal, scale)
        a = torch.exp(z - lse.double().unsqueeze(-1))
        B, Hq, W, n = a.shape
        return a.view(B, Hq // G, G * W, n).sum(2).unsqueeze(0).float()


def _cp_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        case = synth.make_prefill("cp", B=2, Hq=4, Hkv=2, d=128, W=40, N=107, dtype="f32", seed=77)
        q, k, v = (torch.from_numpy(x) for x in (case.q, case.k, case.v))
        N = case.Nmax
        lo, hi = multirank.token_shards(N, world)[rank]          # world 3: the last shard is shorter than the window
        s_loc = multirank.context_parallel_scores(q, k[:, :, lo:hi], v[:, :, lo:hi], offset=lo, total_len=N,
                                                  variants=("ATTN",), ops=_CpuOps)
        s_all = multirank.gather_token_shards(s_loc, N)
        if rank == 0:
            full = _CpuOps.obc_window_attention(q, k, v, mask_lens=torch.full((2,), N, dtype=torch.int32))
            want = _CpuOps.obc_score_given(q, k, v, *full, mask_lens=torch.full((2,), N, dtype=torch.int32))
            out.put((tuple(s_all.shape), float((s_all - want).abs().max()), float(s_all.sum())))
    finally:
        dist.destroy_process_group()


def test_token_shards_exchange_the_window_attention():
    """Three gloo ranks, each with a third of the tokens: after the all-gather and merge of the shards' (o, lse)
    every rank's attention weights are those of the whole sequence, so the gathered attention-only scores
    equal the unsharded ones and sum to the number of window rows."""
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_cp_worker, args=(r, 3, port, out)) for r in range(3)]
    for p in procs:
        p.start()
    shape, err, total = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert shape == (1, 2, 2, 107)
    assert err < 1e-5
    assert total == pytest.approx(2 * 4 * 40, rel=1e-5)       # every softmax row sums to 1
