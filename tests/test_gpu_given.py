"""GPU parity of obc_score_given (scores from attention outputs the caller supplies) against the CPU
checker fed the same O and LSE, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

from paper_2510_07651_b200 import api, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu
OWN = ("ATTN", "VATP")


def _check(case, variants, causal=True, path="auto", tight=None, perturb=False):
    want, got = H.given_scores(case, variants, causal, path, perturb)
    mx = max(np.abs(want[n]).max() for n in variants if n not in OWN) if any(n not in OWN for n in variants) else None
    for n in variants:
        H.assert_scores_close(got[n], want[n], case.dtype, tight=tight, what=f"{case.name}/{n}/{path}/given",
                              mx=None if n in OWN else mx)
        for b in range(case.B):
            assert (got[n][b, :, case.seq_lens[b]:] == 0).all()


def test_fp32_all_variants():
    case, run = synth.config(1)
    _check(case, ["V", "K", "VK", "ATTN", "VATP"], tight=2e-5)
    _check(case, ["V", "K", "VK", "ATTN", "VATP"], tight=2e-5, perturb=True)


@pytest.mark.parametrize("path", ["simt", "auto"])
def test_config2_shape_reduced_length(path):
    case, run = synth.config(2, shrink=8)            # R = 128, N = 4096
    _check(case, ["VK"], path=path, tight=2e-2)
    _check(case, ["K", "VK"], path=path, tight=2e-2)
    _check(case, ["V", "K", "VK", "ATTN", "VATP"], path=path, tight=2e-2)


def test_supplied_values_are_used_not_recomputed():
    # O and LSE that are not the true attention of (q, k, v): the result must follow them
    case, run = synth.config(2, shrink=16)
    _check(case, ["V", "K", "VK", "ATTN", "VATP"], tight=2e-2, perturb=True)
    want_true, _ = H.given_scores(case, ["VK"], perturb=False)
    want_pert, got_pert = H.given_scores(case, ["VK"], perturb=True)
    assert np.abs(want_true["VK"] - want_pert["VK"]).max() > 0.1 * np.abs(want_true["VK"]).max()


@pytest.mark.parametrize("path", ["simt", "auto"])
def test_config3_shape_more_than_128_rows(path):
    case, run = synth.config(3, shrink=32)           # R = 448: row chunks of 64
    _check(case, run["variants"], path=path, tight=2e-2)


def test_ragged_batch_and_odd_tile_counts():
    case = synth.make_prefill("given-ragged", B=3, Hq=8, Hkv=2, d=128, W=16, N=[129, 4000, 641], dtype="bf16",
                              seed=211, hh_frac=0.02)                      # R = 64
    _check(case, ["V", "K", "VK", "ATTN", "VATP"], tight=2e-2)
    case = synth.make_prefill("given-rows", B=2, Hq=14, Hkv=2, d=128, W=64, N=[1100, 333], dtype="bf16",
                              seed=212, hh_frac=0.02)                      # R = 448
    _check(case, ["V", "K", "VK", "ATTN", "VATP"], tight=2e-2)


@pytest.mark.parametrize("causal", [True, False])
def test_small_shapes_cuda_core_path(causal):
    case = synth.make_prefill("given-small", B=2, Hq=6, Hkv=2, d=128, W=5, N=[77, 300], dtype="bf16", seed=213,
                              hh_frac=0.05)                                # R = 15: CUDA-core kernels
    _check(case, ["V", "K", "VK", "ATTN", "VATP"], causal=causal, tight=2e-2)


def test_output_dtype_may_differ_from_the_cache():
    # bf16 cache with fp32 attention outputs
    case, run = synth.config(2, shrink=16)
    o, lse, _, lse_dev = H.given_attention(case)
    from oracle import reference as ref
    out = ref.score(case.q, case.k, case.v, want=("ATTN",), return_attention=True)
    o32 = out["O"].reshape(case.B, case.Hq, case.W, case.d).astype(np.float32)
    want = ref.score(case.q, case.k, case.v, want=("VK",), given=(o32, lse))["VK"]
    q, k, v = H.upload(case)
    got = api.obc_score_given(q, k, v, torch.from_numpy(o32).cuda(), lse_dev, variants=["VK"])[0].cpu().numpy()
    H.assert_scores_close(got, want, "bf16", tight=2e-2, what="f32 o with bf16 cache")
