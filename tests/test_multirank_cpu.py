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
