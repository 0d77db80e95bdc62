"""Shared helpers of the GPU parity tests: upload seeded cases, tolerances, comparisons."""
import numpy as np
import torch

from oracle import reference as ref
from paper_2510_07651_b200 import api, synth

# tolerances of the parity tests: |gpu - ref| <= atol + rtol * |ref|
BF16_RTOL, BF16_ATOL = 2e-2, 1e-4
F32_RTOL = 1e-5            # fp32 caches: atol = 1e-5 * max|ref|
VARIANT_ORDER = ("V", "K", "VK", "ATTN", "VATP")     # plane order of the scores buffer


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
    """The stated tolerance, plus (tight) a relative bound normalised by the largest reference
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
    order = [n for n in VARIANT_ORDER if n in variants]
    p = api.score_params(q, k, seq_lens=lens_dev(case), causal=causal, variants=order, path=path)
    ws = torch.empty(api.obc_score_workspace(p), dtype=torch.uint8, device="cuda")
    s = api.obc_score(q, k, v, seq_lens=lens_dev(case), causal=causal, variants=order, path=path, workspace=ws)
    api.obc_score_status(ws)
    torch.cuda.synchronize()
    s = s.cpu().numpy()
    return {n: s[i] for i, n in enumerate(order)}


def given_attention(case, causal=True, perturb=False):
    """Window attention outputs to hand to obc_score_given, from the CPU checker: o [B,Hq,W,d] rounded to the
    case's storage dtype and lse fp32 [B,Hq,W] (natural log).  With `perturb` they are deliberately not the
    true attention (shifted lse, scaled and offset o), to show that the supplied values are what is used."""
    lens = None if (case.seq_lens == case.Nmax).all() else case.seq_lens
    out = ref.score(case.q, case.k, case.v, seq_lens=lens, causal=causal, want=("ATTN",), return_attention=True)
    o = out["O"].reshape(case.B, case.Hq, case.W, case.d).astype(np.float32)
    lse = (out["m"] + np.log(out["l"])).reshape(case.B, case.Hq, case.W).astype(np.float32)
    if perturb:
        o = (0.5 * o + 0.25).astype(np.float32)
        lse = (lse + np.float32(0.7)).astype(np.float32)
    if case.dtype == "bf16":
        o, o_bits = synth.bf16_round(o)
        o_dev = dev_bf16(o_bits)
    else:
        o_dev = torch.from_numpy(o).cuda()
    return o, lse, o_dev, torch.from_numpy(lse).cuda()


def given_scores(case, variants, causal=True, path="auto", perturb=False):
    """(checker, GPU) scores from the same supplied attention outputs."""
    o, lse, o_dev, lse_dev = given_attention(case, causal, perturb)
    lens = None if (case.seq_lens == case.Nmax).all() else case.seq_lens
    order = [n for n in VARIANT_ORDER if n in variants]
    want = ref.score(case.q, case.k, case.v, seq_lens=lens, causal=causal, want=tuple(order), given=(o, lse))
    q, k, v = upload(case)
    p = api.score_params(q, k, seq_lens=lens_dev(case), causal=causal, variants=order, path=path)
    ws = torch.empty(api.obc_score_workspace(p), dtype=torch.uint8, device="cuda")
    s = api.obc_score_given(q, k, v, o_dev, lse_dev, seq_lens=lens_dev(case), causal=causal, variants=order,
                            path=path, workspace=ws)
    api.obc_score_status(ws)
    torch.cuda.synchronize()
    s = s.cpu().numpy()
    return want, {n: s[i] for i, n in enumerate(order)}
