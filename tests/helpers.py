"""Shared helpers of the GPU parity tests: upload seeded cases, tolerances, comparisons."""
import numpy as np
import torch

from oracle import reference as ref
from paper_2510_07651_b200 import api, synth

# spec tolerances: |gpu - ref| <= atol + rtol * |ref|
BF16_RTOL, BF16_ATOL = 2e-2, 1e-4
F32_RTOL = 1e-5            # fp32 caches: atol = 1e-5 * max|ref|


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def upload(case: synth.PrefillCase):
    if case.dtype == "bf16":
        return dev_bf16(case.q_bits), dev_bf16(case.k_bits), dev_bf16(case.v_bits)
    return torch.from_numpy(case.q).cuda(), torch.from_numpy(case.k).cuda(), torch.from_numpy(case.v).cuda()


def lens_dev(case):
    if (case.seq_lens == case.Nmax).all():
        return None
    return torch.from_numpy(case.seq_lens).cuda()


def assert_scores_close(got: np.ndarray, want: np.ndarray, dtype: str, *, tight: float | None = None, what="",
                        mx: float | None = None):
    """Spec tolerance, plus (tight) a relative bound normalised by the largest reference
    score, which stays meaningful when scores are far below the absolute tolerance.  `mx` is the
    magnitude the fp32 absolute tolerance scales with (default: the largest reference value of
    this plane; callers pass the largest OBCache score of the case so that a plane that is
    identically zero, e.g. the key score of a single-token cache, is judged on the same scale)."""
    want = np.asarray(want, np.float64)
    got = np.asarray(got, np.float64)
    assert np.isfinite(got).all(), what
    mx = np.abs(want).max() if mx is None else max(mx, np.abs(want).max())
    if dtype == "bf16":
        bound = BF16_ATOL + BF16_RTOL * np.abs(want)
    else:
        bound = F32_RTOL * mx + F32_RTOL * np.abs(want)
    err = np.abs(got - want)
    worst = np.argmax(err - bound)
    assert (err <= bound).all(), f"{what}: |err|={err.flat[worst]:.3e} ref={want.flat[worst]:.3e} at {worst}"
    if tight is not None:
        b2 = tight * (np.abs(want) + 1e-3 * mx)
        w2 = np.argmax(err - b2)
        assert (err <= b2).all(), f"{what} (tight): |err|={err.flat[w2]:.3e} ref={want.flat[w2]:.3e} max={mx:.3e}"


def oracle_scores(case, variants, causal=True):
    lens = None if (case.seq_lens == case.Nmax).all() else case.seq_lens
    return ref.score(case.q, case.k, case.v, seq_lens=lens, causal=causal, want=tuple(variants))


def gpu_scores(case, variants, causal=True, path="auto"):
    q, k, v = upload(case)
    order = [n for n in ("V", "K", "VK", "ATTN") if n in variants]
    p = api.score_params(q, k, seq_lens=lens_dev(case), causal=causal, variants=order, path=path)
    ws = torch.empty(api.obc_score_workspace(p), dtype=torch.uint8, device="cuda")
    s = api.obc_score(q, k, v, seq_lens=lens_dev(case), causal=causal, variants=order, path=path, workspace=ws)
    api.obc_score_status(ws)
    torch.cuda.synchronize()
    s = s.cpu().numpy()
    return {n: s[i] for i, n in enumerate(order)}
