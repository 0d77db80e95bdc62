"""GPU parity of obc_score against the CPU checker, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

from paper_2510_07651_b200 import api, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _check(case, variants, causal=True, path="auto", tight=None):
    want = H.oracle_scores(case, variants, causal)
    got = H.gpu_scores(case, variants, causal, path)
    own = ("ATTN", "VATP")                            # not on the scale of the three OBCache scores
    mx = max(np.abs(want[n]).max() for n in variants if n not in own) if any(n not in own for n in variants) else None
    for n in variants:
        H.assert_scores_close(got[n], want[n], case.dtype, tight=tight, what=f"{case.name}/{n}/{path}",
                              mx=None if n in own else mx)
        for b in range(case.B):                      # padding beyond each sequence is written as 0
            assert (got[n][b, :, case.seq_lens[b]:] == 0).all()


def test_config1_fp32_all_variants():
    case, run = synth.config(1)
    _check(case, run["variants"] + ["ATTN", "VATP"], tight=2e-5)


@pytest.mark.parametrize("path", ["simt", "auto"])
def test_config2_shape_reduced_length(path):
    case, run = synth.config(2, shrink=8)            # N = 4096: several tiles per split
    _check(case, ["V", "K", "VK"], path=path, tight=2e-2)


@pytest.mark.parametrize("path", ["simt", "auto"])
def test_config3_shape_reduced_length(path):
    case, run = synth.config(3, shrink=32)           # R = 448, N = 4096
    _check(case, run["variants"], path=path, tight=2e-2)


@pytest.mark.parametrize("path", ["simt", "auto"])
def test_config4_ragged_batch_reduced(path):
    case, run = synth.config(4, shrink=16)           # lengths in [512, 4096], ragged tails
    _check(case, run["variants"], path=path, tight=2e-2)


@pytest.mark.parametrize("N,W,Hq,Hkv,dtype,causal", [
    (1, 1, 1, 1, "f32", True),            # single cached token
    (16, 16, 2, 1, "f32", True),          # window == whole cache
    (65, 3, 7, 1, "bf16", True),          # ragged tile tail, odd group
    (200, 1, 4, 1, "bf16", True),         # W = 1 (decode-like), R = 4
    (333, 5, 8, 2, "f32", False),         # non-causal
    (1000, 40, 4, 2, "bf16", True),       # R = 80: not a multiple of the row chunk
])
def test_small_and_degenerate_shapes(N, W, Hq, Hkv, dtype, causal):
    case = synth.make_prefill("edge", B=2, Hq=Hq, Hkv=Hkv, d=128, W=W, N=N, dtype=dtype, seed=77 + N,
                              hh_frac=0.05)
    _check(case, ["V", "K", "VK", "ATTN", "VATP"], causal=causal, tight=2e-2 if dtype == "bf16" else None)


@pytest.mark.parametrize("lens,W,Hq,Hkv", [
    ([1100, 333], 64, 14, 2),      # R = 448 (row chunks of 64), odd tile counts: the second tile of the last pair is past the end
    ([2900], 40, 5, 1),            # R = 200: padded to 256 rows, 23 tiles
    ([129, 4000, 640], 48, 12, 3), # R = 192, ragged, a unit with two tiles of which the second holds one token
])
def test_more_than_128_window_rows(lens, W, Hq, Hkv):
    case = synth.make_prefill("rows", B=len(lens), Hq=Hq, Hkv=Hkv, d=128, W=W, N=lens, dtype="bf16", seed=101 + W,
                              hh_frac=0.02)
    _check(case, ["V", "K", "VK", "ATTN", "VATP"], tight=2e-2)
    _check(case, ["K", "VK"], tight=2e-2)
    _check(case, ["VK"], tight=2e-2)


@pytest.mark.parametrize("N,W,Hq,Hkv", [(5000, 64, 1, 1), (3001, 16, 8, 2), (257, 128, 1, 1), (4224, 24, 4, 1)])
def test_tensor_core_row_counts(N, W, Hq, Hkv):
    # R = 64, 64, 128, 96 (chunks of 64 / 64 / 128 / 96 rows), token counts with and without a ragged last tile
    case = synth.make_prefill("tc", B=1, Hq=Hq, Hkv=Hkv, d=128, W=W, N=N, dtype="bf16", seed=7 + N, hh_frac=0.02)
    _check(case, ["VK"], path="tc", tight=2e-2)
    _check(case, ["V", "K", "VK", "ATTN", "VATP"], path="tc", tight=2e-2)


@pytest.mark.parametrize("N,Hq,Hkv,dtype,path", [
    (96, 2, 1, "f32", "auto"),            # R = 192 on CUDA cores
    (384, 2, 2, "bf16", "simt"),
    (384, 4, 2, "bf16", "auto"),          # R = 768: twelve row chunks of 64 on tensor cores
    (640, 1, 1, "bf16", "tc"),            # R = 640, five token tiles, every tile needs the mask
])
def test_full_history_window(N, Hq, Hkv, dtype, path):
    """The perturbation window is the whole sequence (w = 1 in Sec. 4.3, the accumulation H2O uses): every
    query position is a window row and row i sees the tokens p <= i."""
    case = synth.make_prefill("history", B=1, Hq=Hq, Hkv=Hkv, d=128, W=N, N=N, dtype=dtype, seed=311 + N,
                              hh_frac=0.02)
    _check(case, ["V", "K", "VK", "ATTN", "VATP"], path=path, tight=2e-2 if dtype == "bf16" else None)


def test_peaky_attention_cancellation_case():
    # some attention weights approach 1, so ||v_p - o_i||^2 cancels heavily
    case = synth.make_prefill("peaky", B=1, Hq=8, Hkv=2, d=128, W=16, N=2048, dtype="bf16", seed=5,
                              hh_frac=0.01, peaky=True)
    _check(case, ["V", "K", "VK"], path="simt")
    _check(case, ["V", "K", "VK"], path="auto")


def test_strided_views_and_split_invariance():
    # K/V given as non-contiguous views (token stride 2d) must score like their contiguous copies
    case = synth.make_prefill("strided", B=1, Hq=4, Hkv=2, d=128, W=8, N=700, dtype="bf16", seed=9)
    q, k, v = H.upload(case)
    wide_k = torch.zeros((1, 2, 700, 256), dtype=torch.bfloat16, device="cuda")
    wide_v = torch.zeros_like(wide_k)
    wide_k[..., :128] = k
    wide_v[..., :128] = v
    a = api.obc_score(q, k, v, variants=["VK"])
    b = api.obc_score(q, wide_k[..., :128], wide_v[..., :128], variants=["VK"])
    torch.cuda.synchronize()
    assert torch.equal(a, b)


def test_workspace_poison_does_not_leak():
    case = synth.make_prefill("poison", B=1, Hq=4, Hkv=1, d=128, W=4, N=300, dtype="f32", seed=3)
    q, k, v = H.upload(case)
    p = api.score_params(q, k, variants=["VK"])
    ws = torch.full((api.obc_score_workspace(p),), 0xFF, dtype=torch.uint8, device="cuda")   # NaN pattern
    s = api.obc_score(q, k, v, variants=["VK"], workspace=ws)
    want = H.oracle_scores(case, ["VK"])["VK"]
    H.assert_scores_close(s[0].cpu().numpy(), want, "f32", tight=2e-5)


@pytest.mark.parametrize("path", ["simt", "tc"])
def test_ragged_batch_with_poisoned_workspace(path):
    """Splits past the end of a shorter sequence run nothing and write nothing: whatever the workspace held
    there (here a NaN pattern) must not reach the scores."""
    case = synth.make_prefill("ragpoison", B=3, Hq=8, Hkv=2, d=128, W=16, N=[9000, 700, 2500], dtype="bf16", seed=21)
    q, k, v = H.upload(case)
    lens = H.lens_dev(case)
    p = api.score_params(q, k, seq_lens=lens, variants=["VK"], path=path)
    ws = torch.full((api.obc_score_workspace(p),), 0xFF, dtype=torch.uint8, device="cuda")
    s = api.obc_score(q, k, v, seq_lens=lens, variants=["VK"], path=path, workspace=ws)
    api.obc_score_status(ws)
    want = H.oracle_scores(case, ["VK"])["VK"]
    H.assert_scores_close(s[0].cpu().numpy(), want, "bf16", tight=2e-2, what=f"ragged poison {path}")


def test_kernel_spans_are_recorded_and_cleared():
    """Both tensor-core kernels leave a plausible device-side extent in the workspace header; reading
    it zeroes it; the CUDA-core path leaves nothing."""
    case, run = synth.config(2, shrink=8)
    q, k, v = H.upload(case)
    p = api.score_params(q, k, variants=["VK"])
    ws = torch.zeros(api.obc_score_workspace(p), dtype=torch.uint8, device="cuda")
    api.obc_score(q, k, v, variants=["VK"], workspace=ws)
    p1, p2 = api.obc_score_kernel_spans(ws)
    assert 1.0 < p1 < 1e4 and 1.0 < p2 < 1e4
    assert api.obc_score_kernel_spans(ws) == (0.0, 0.0)
    ps = api.score_params(q, k, variants=["VK"], path="simt")
    ws2 = torch.zeros(api.obc_score_workspace(ps), dtype=torch.uint8, device="cuda")
    api.obc_score(q, k, v, variants=["VK"], path="simt", workspace=ws2)
    assert api.obc_score_kernel_spans(ws2) == (0.0, 0.0)
