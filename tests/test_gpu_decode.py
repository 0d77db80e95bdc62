"""GPU parity of obc_decode_step with the CPU checker.  Each step is compared teacher-forced:
the checker scores the same pre-step cache in double precision (scores within tolerance), then
takes the eviction decision from the GPU's own fp32 accumulators (slot, pos, state and cache
contents bit-exact)."""
import numpy as np
import pytest
import torch

from oracle import reference as ref
from paper_2510_07651_b200 import api, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _run(B, Hq, Hkv, n0, budget, cap, n_sink, n_recent, steps, variant="VK", seed=55, s_acc0=False, window=0,
         strided=False):
    G = Hq // Hkv
    dc = synth.make_decode(B=B, Hq=Hq, Hkv=Hkv, d=128, n0=n0, steps=steps, seed=seed)
    dev = "cuda"
    if strided:      # caches that are views of larger allocations: rows 272 bytes apart, spare slots after every head, NaN between
        kbig = torch.full((B, Hkv + 1, cap + 5, 136), float("nan"), dtype=torch.bfloat16, device=dev)
        vbig = torch.full((B, Hkv + 1, cap + 5, 136), float("nan"), dtype=torch.bfloat16, device=dev)
        kc, vc = kbig[:, :Hkv, :cap, :128], vbig[:, :Hkv, :cap, :128]
        kc.zero_(); vc.zero_()
    else:
        kc = torch.zeros((B, Hkv, cap, 128), dtype=torch.bfloat16, device=dev)
        vc = torch.zeros_like(kc)
    kc[:, :, :n0] = H.dev_bf16(dc.k0_bits)
    vc[:, :, :n0] = H.dev_bf16(dc.v0_bits)
    pos = torch.full((B, Hkv, cap), -1, dtype=torch.int32, device=dev)
    pos[:, :, :n0] = torch.arange(n0, dtype=torch.int32, device=dev)
    s_acc = torch.zeros((B, Hkv, cap), dtype=torch.float32, device=dev)
    init = None
    if s_acc0:
        init = np.random.default_rng(seed).random((B, Hkv, n0), dtype=np.float32) * 1e-3
        s_acc[:, :, :n0] = torch.from_numpy(init).cuda()
    state = torch.zeros((B, Hkv, 4), dtype=torch.int32, device=dev)
    state[..., 0] = n0; state[..., 1] = n0; state[..., 2] = n0
    sts = [[ref.DecodeState(dc.k0[b, h], dc.v0[b, h], cap, None if init is None else init[b, h], window=window)
            for h in range(Hkv)] for b in range(B)]
    hist = torch.zeros((B, Hkv, window, cap), dtype=torch.float32, device=dev) if window else None
    qd, kd, vd = H.dev_bf16(dc.q_t_bits), H.dev_bf16(dc.k_t_bits), H.dev_bf16(dc.v_t_bits)
    ws = None
    n_evicted = 0
    for t in range(steps):
        step_pos = n0 + t
        ws = api.obc_decode_step(qd[t].unsqueeze(2), kd[t].unsqueeze(2), vd[t].unsqueeze(2), kc, vc, s_acc, pos,
                                 state, step_pos, budget=budget, n_sink=n_sink, n_recent=n_recent, variant=variant,
                                 workspace=ws, acc_window=window, s_hist=hist)
        torch.cuda.synchronize()
        g_acc, g_pos, g_state = s_acc.cpu().numpy(), pos.cpu().numpy(), state.cpu().numpy()
        for b in range(B):
            for h in range(Hkv):
                st = sts[b][h]
                st.append(dc.k_t[t, b, h], dc.v_t[t, b, h], step_pos)
                sc = st.scores(dc.q_t[t, b, h * G:(h + 1) * G], variant)
                want_acc = st.accumulate(sc, step_pos)
                livemask = st.pos >= 0
                H.assert_scores_close(g_acc[b, h][livemask], want_acc[livemask], "bf16", tight=2e-2,
                                      what=f"step {t} unit {b},{h}")
                st.s_acc[livemask] = g_acc[b, h][livemask]          # teacher forcing
                e = st.evict(step_pos, budget, n_sink, n_recent)
                n_evicted += e >= 0
                assert np.array_equal(g_pos[b, h], st.pos), f"step {t} unit {b},{h}"
                assert tuple(g_state[b, h][:3]) == (st.live, st.next_slot, st.hi)
                assert g_state[b, h][3] == 0
    kb, vb = kc.contiguous().view(torch.int16).cpu().numpy(), vc.contiguous().view(torch.int16).cpu().numpy()
    if strided:      # nothing outside the views was written
        assert torch.isnan(kbig[:, Hkv]).all() and torch.isnan(kbig[:, :, cap:]).all() and torch.isnan(kbig[..., 128:]).all()
        assert torch.isnan(vbig[:, Hkv]).all() and torch.isnan(vbig[:, :, cap:]).all() and torch.isnan(vbig[..., 128:]).all()
    for b in range(B):
        for h in range(Hkv):
            st = sts[b][h]
            live = st.pos >= 0
            assert np.array_equal(kb[b, h][live], synth.bf16_round(st.k[live])[1].view(np.int16))
            assert np.array_equal(vb[b, h][live], synth.bf16_round(st.v[live])[1].view(np.int16))
    return n_evicted


def test_decode_small_single_chunk():
    ev = _run(B=2, Hq=8, Hkv=2, n0=40, budget=48, cap=64, n_sink=4, n_recent=8, steps=30)
    assert ev == 2 * 2 * (30 - 8)


def test_decode_multi_chunk_steady_state():
    # capacity = budget + 1: after the cache fills, every step evicts and reuses the freed slot
    ev = _run(B=1, Hq=4, Hkv=1, n0=600, budget=640, cap=641, n_sink=4, n_recent=256, steps=60, s_acc0=True)
    assert ev == 20


@pytest.mark.parametrize("variant", ["V", "K", "ATTN"])
def test_decode_other_variants(variant):
    _run(B=1, Hq=7, Hkv=1, n0=300, budget=310, cap=330, n_sink=2, n_recent=16, steps=20, variant=variant)


@pytest.mark.parametrize("G", [1, 2, 3, 5, 6, 8])
def test_decode_every_group_size(G):
    # the MMA tiles pad the query heads of a group to 8 columns: every group size, two chunks, an odd extent
    _run(B=1, Hq=2 * G, Hkv=2, n0=290, budget=300, cap=301, n_sink=3, n_recent=20, steps=24)


@pytest.mark.parametrize("window", [1, 5, 16])
def test_decode_accumulation_window(window):
    """Scores accumulated over the last `window` steps only: steady-state eviction with slot reuse, several
    chunks, a window shorter and longer than a token's usual stay beyond the protected recents."""
    ev = _run(B=2, Hq=8, Hkv=2, n0=280, budget=290, cap=291, n_sink=4, n_recent=12, steps=40, window=window)
    assert ev == 2 * 2 * 30


def test_decode_caches_that_are_views_of_larger_buffers():
    """Strided caches (the tensor maps of the bulk copies carry the strides); capacity not a multiple of the chunk, so the
    last chunk's rows beyond it must read as zeros although the memory behind them holds NaN."""
    assert _run(B=2, Hq=8, Hkv=2, n0=300, budget=280, cap=333, n_sink=4, n_recent=8, steps=6, strided=True) > 0

