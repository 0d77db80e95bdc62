"""The five workloads at full size, in the launch configuration bench.py times (one obc_score /
obc_select / obc_compact call per layer cache, default path), against the CPU checker.

Scores: every element against the double-precision checker.  Selection and compaction: bit-exact
against the checker fed with the GPU's own fp32 scores (both sides then take the same decisions in
the same precision), plus the overlap of the kept sets with what the double-precision scores select.
The decode workload is checked on a sample of (batch item, KV head) units over all steps.
"""
import numpy as np
import pytest
import torch

from oracle import reference as ref
from paper_2510_07651_b200 import api, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _prefill_full(idx):
    case, run = synth.config(idx)
    q, k, v = H.upload(case)
    lens_d = H.lens_dev(case)
    order = [n for n in ("V", "K", "VK") if n in run["variants"]]
    p = api.score_params(q, k, seq_lens=lens_d, variants=order)
    ws = torch.empty(api.obc_score_workspace(p), dtype=torch.uint8, device="cuda")
    scores = api.obc_score(q, k, v, seq_lens=lens_d, variants=order, workspace=ws)
    api.obc_score_status(ws)
    got = scores.cpu().numpy()
    want = H.oracle_scores(case, order)
    mx = max(np.abs(want[n]).max() for n in order)
    for i, n in enumerate(order):
        H.assert_scores_close(got[i], want[n], case.dtype, tight=2e-2, what=f"{case.name}/{n}", mx=mx)

    budgets = np.asarray(run["budget"] if isinstance(run["budget"], list) else [run["budget"]] * case.B, np.int32)
    stride = int(budgets.max())
    uniform = bool((budgets == budgets[0]).all())
    plane = len(order) - 1                                     # select on the last requested variant (VK)
    idx_d = api.obc_select(scores[plane], budget=int(budgets[0]) if uniform else 0,
                           budgets=None if uniform else torch.from_numpy(budgets).cuda(), idx_stride=stride,
                           seq_lens=lens_d, n_sink=run["n_sink"], n_recent=run["n_recent"],
                           pool=run["pool_mode"], pool_kernel=run["pool_kernel"])
    k_out, v_out = api.obc_compact(k, v, idx_d)
    torch.cuda.synchronize()
    gi = idx_d.cpu().numpy()
    want_idx = ref.select_pipeline(got[plane], case.seq_lens, budgets, run["n_sink"], run["n_recent"],
                                   run["pool_mode"], run["pool_kernel"], stride)
    assert np.array_equal(gi, want_idx)
    ref_idx = ref.select_pipeline(want[order[plane]].astype(np.float32), case.seq_lens, budgets, run["n_sink"],
                                  run["n_recent"], run["pool_mode"], run["pool_kernel"], stride)
    kb, vb = k_out.view(torch.int16).cpu().numpy(), v_out.view(torch.int16).cpu().numpy()
    worst_overlap, worst_rel_top, worst_rel_max = 1.0, 0.0, 0.0
    gp, wp = got[plane], want[order[plane]]
    for b in range(case.B):
        nb = int(budgets[b])
        for h in range(case.Hkv):
            assert np.array_equal(kb[b, h, :nb], ref.compact(case.k_bits[b, h].view(np.int16), want_idx[b, h], nb))
            assert np.array_equal(vb[b, h, :nb], ref.compact(case.v_bits[b, h].view(np.int16), want_idx[b, h], nb))
            kept, kept_ref = set(gi[b, h, :nb].tolist()), set(ref_idx[b, h, :nb].tolist())
            assert len(kept & kept_ref) >= 0.97 * nb, (b, h, len(kept & kept_ref), nb)
            worst_overlap = min(worst_overlap, len(kept & kept_ref) / nb)
            # relative error on the tokens the double-precision scores rank in the top budget (unpooled scores)
            n = int(case.seq_lens[b])
            top = np.argsort(-wp[b, h, :n], kind="stable")[:nb]
            worst_rel_top = max(worst_rel_top, float(np.max(np.abs(gp[b, h, top] - wp[b, h, top]) / wp[b, h, top])))
            worst_rel_max = max(worst_rel_max, float(np.abs(gp[b, h, :n] - wp[b, h, :n]).max() / wp[b, h, :n].max()))
    # reported (the bound asserted above is the tolerance; these say how far inside it the kernels are)
    print(f"\n[{case.name}] kept-set overlap with the double-precision selection >= {worst_overlap:.4f}; "
          f"max relative error on the checker's top-budget tokens {worst_rel_top:.2e}; max error / max score {worst_rel_max:.2e}")


def test_config2_llama_32k_full():
    _prefill_full(2)


def test_config3_qwen_128k_full():
    _prefill_full(3)


def test_config4_ragged_batch_full():
    _prefill_full(4)


def test_whole_sequence_window_llama_shapes_1k():
    # Llama shapes with every one of 1024 query positions as a window row (R = 4096 rows per KV head): shared row
    # chunks, skipped tile pairs and the warp-per-row merge, every element against the checker
    case, run = synth.full_history(1024)
    got = H.gpu_scores(case, ["K", "VK"])
    want = H.oracle_scores(case, ["K", "VK"])
    mx = max(np.abs(want[n]).max() for n in ("K", "VK"))
    for n in ("K", "VK"):
        H.assert_scores_close(got[n], want[n], "bf16", tight=2e-2, what=f"history1k/{n}", mx=mx)


def test_config5_decode_full_shapes_sampled_units():
    # Llama shapes, batch 32, 256 steps in steady state (live 4096 -> 4097 -> 4096 per step); the
    # checker replays 6 sampled units teacher-forced on the GPU's own accumulators.
    B, Hq, Hkv, n0, budget, steps = 32, 32, 8, 4096, 4096, 256
    cap, n_sink, n_recent, G = budget + 1, 4, 256, 4
    dc = synth.make_decode(B=B, Hq=Hq, Hkv=Hkv, d=128, n0=n0, steps=steps, seed=1239)
    kc = torch.zeros((B, Hkv, cap, 128), dtype=torch.bfloat16, device="cuda")
    vc = torch.zeros_like(kc)
    kc[:, :, :n0] = H.dev_bf16(dc.k0_bits); vc[:, :, :n0] = H.dev_bf16(dc.v0_bits)
    pos = torch.full((B, Hkv, cap), -1, dtype=torch.int32, device="cuda")
    pos[:, :, :n0] = torch.arange(n0, dtype=torch.int32, device="cuda")
    s_acc = torch.zeros((B, Hkv, cap), dtype=torch.float32, device="cuda")
    state = torch.zeros((B, Hkv, 4), dtype=torch.int32, device="cuda")
    state[..., 0] = n0; state[..., 1] = n0; state[..., 2] = n0
    units = [(0, 0), (3, 5), (17, 2), (31, 7), (9, 1), (22, 6)]
    sts = {u: ref.DecodeState(dc.k0[u[0], u[1]], dc.v0[u[0], u[1]], cap) for u in units}
    qd, kd, vd = H.dev_bf16(dc.q_t_bits), H.dev_bf16(dc.k_t_bits), H.dev_bf16(dc.v_t_bits)
    ws = None
    for t in range(steps):
        step_pos = n0 + t
        ws = api.obc_decode_step(qd[t].unsqueeze(2), kd[t].unsqueeze(2), vd[t].unsqueeze(2), kc, vc, s_acc, pos,
                                 state, step_pos, budget=budget, n_sink=n_sink, n_recent=n_recent, variant="VK",
                                 workspace=ws)
        for (b, h), st in sts.items():
            g_acc, g_pos, g_state = s_acc[b, h].cpu().numpy(), pos[b, h].cpu().numpy(), state[b, h].cpu().numpy()
            st.append(dc.k_t[t, b, h], dc.v_t[t, b, h], step_pos)
            if t % 16 == 0 or t == steps - 1:                  # double-precision scores on a subset of the steps
                sc = st.scores(dc.q_t[t, b, h * G:(h + 1) * G], "VK")
                live = st.pos >= 0
                H.assert_scores_close(g_acc[live], (st.s_acc.astype(np.float64) + sc)[live], "bf16", tight=2e-2,
                                      what=f"step {t} unit {b},{h}")
            st.s_acc[:] = np.where(st.pos >= 0, g_acc, st.s_acc)    # teacher forcing
            st.evict(step_pos, budget, n_sink, n_recent)
            assert np.array_equal(g_pos, st.pos), f"step {t} unit {b},{h}"
            assert tuple(g_state[:3]) == (st.live, st.next_slot, st.hi) and g_state[3] == 0
    torch.cuda.synchronize()
    assert int(state[..., 0].max()) == budget and int(state[..., 0].min()) == budget
