"""Pins for the CPU checker's scores: each test compares oracle/obc_oracle.c with something
the paper or the mathematics fixes independently of it (brute-force row zeroing per Def. 3.1 /
Eq. 1, finite-difference limits of that same definition, hand-worked closed forms, special
cases, structural identities)."""
import os

import numpy as np
import pytest

from oracle import reference as ref

GOLD = os.path.join(os.path.dirname(__file__), "golden")


# ---- independent numpy statement of windowed GQA attention (Sec. 3, Eq. 9) -----------------
def window_outputs(q, k, v, scale, causal=True):
    """q [G,W,d], k,v [N,d] -> (A [G,W,N], Z [G,W,N], O [G,W,d]) in float64."""
    G, W, d = q.shape
    N = k.shape[0]
    Z = scale * np.einsum("gwd,nd->gwn", q, k)
    mask = np.ones((W, N), bool)
    if causal:
        for i in range(W):
            mask[i, N - W + i + 1:] = False
    Zm = np.where(mask[None], Z, -np.inf)
    E = np.exp(Zm - Zm.max(-1, keepdims=True))
    A = E / E.sum(-1, keepdims=True)
    return A, Z, A @ v


def pruning_error(q, k, v, scale, p, t_k, t_v, causal=True):
    """|| O(K - t_k e_p k_p, V - t_v e_p v_p) - O(K, V) ||_F^2 summed over the group (Eq. 1/9)."""
    _, _, O = window_outputs(q, k, v, scale, causal)
    k2, v2 = k.copy(), v.copy()
    k2[p] *= (1.0 - t_k)
    v2[p] *= (1.0 - t_v)
    _, _, O2 = window_outputs(q, k2, v2, scale, causal)
    return float(((O2 - O) ** 2).sum())


def tiny(seed=0, G=2, W=4, N=24, d=8, spread=1.5):
    rng = np.random.default_rng(seed)
    q = (spread * rng.standard_normal((G, W, d))).astype(np.float32)
    k = (spread * rng.standard_normal((N, d))).astype(np.float32)
    v = rng.standard_normal((N, d)).astype(np.float32)
    return q, k, v


def run_oracle(q, k, v, **kw):
    """q [G,W,d], k,v [N,d] -> dict of [N] arrays (one KV head, batch 1)."""
    out = ref.score(q[None], k[None, None], v[None, None], **kw)
    return {n: (a[0, 0] if a.ndim == 3 else a[0, 0]) for n, a in out.items()}


# ---- pins -----------------------------------------------------------------------------------
def test_golden_two_token_closed_form():
    rows = [l.split() for l in open(os.path.join(GOLD, "two_token_closed_form.txt")) if l[0] != "#"]
    gold = np.array([[float(x) for x in r[1:]] for r in rows])
    q = np.array([[[1.0]]], np.float32)
    k = np.log(np.array([[2.0], [3.0]])).astype(np.float32)
    v = np.array([[1.0], [2.0]], np.float32)
    # the keys are fp32 roundings of ln 2, ln 3: allow that much
    for form in ("eq", "alg1"):
        s = run_oracle(q, k, v, scale=1.0, causal=False, formulation=form)
        np.testing.assert_allclose(s["V"], gold[:, 0], rtol=1e-6)
        np.testing.assert_allclose(s["K"], gold[:, 1], rtol=1e-6)
        np.testing.assert_allclose(s["VK"], gold[:, 2], rtol=1e-6)


@pytest.mark.parametrize("causal", [True, False])
def test_value_score_equals_exact_value_zeroing(causal):
    # O is linear in V, so zeroing v_p changes O by exactly -A_ip v_p: Eq. 4 is exact (App. A.2)
    q, k, v = tiny(1)
    scale = 1 / np.sqrt(q.shape[-1])
    s = run_oracle(q, k, v, causal=causal)
    brute = [pruning_error(q.astype(float), k.astype(float), v.astype(float), scale, p, 0.0, 1.0, causal)
             for p in range(k.shape[0])]
    np.testing.assert_allclose(s["V"], brute, rtol=1e-11, atol=1e-300)


@pytest.mark.parametrize("which,tk,tv", [("K", 1.0, 0.0), ("VK", 1.0, 1.0), ("V", 0.0, 1.0)])
def test_scores_are_the_second_order_limit_of_the_pruning_error(which, tk, tv):
    # L(t)/t^2 -> S as t -> 0 along K - t e_p k_p, V - t e_p v_p (Theorem, Eq. 2-3); the
    # symmetric quotient (L(t)+L(-t))/(2 t^2) cancels the cubic term, leaving O(t^2)
    q, k, v = tiny(2)
    qd, kd, vd = q.astype(float), k.astype(float), v.astype(float)
    scale = 1 / np.sqrt(q.shape[-1])
    s = run_oracle(q, k, v)[which]
    t = 1e-3
    lim = np.array([(pruning_error(qd, kd, vd, scale, p, tk * t, tv * t)
                     + pruning_error(qd, kd, vd, scale, p, -tk * t, -tv * t)) / (2 * t * t)
                    for p in range(k.shape[0])])
    assert s.max() > 0
    np.testing.assert_allclose(s, lim, rtol=2e-4, atol=1e-9 * s.max())
    # one-sided quotient converges linearly: its error shrinks ~10x per decade of t
    errs = []
    for t1 in (1e-2, 1e-3):
        one = np.array([pruning_error(qd, kd, vd, scale, p, tk * t1, tv * t1) / (t1 * t1)
                        for p in range(k.shape[0])])
        errs.append(np.abs(one - s).max())
    assert errs[1] < errs[0] * 0.2 or errs[0] < 1e-12


def test_joint_score_is_one_squared_norm():
    # d o_i / dt = -A_ip [ v_p + Z_ip (v_p - o_i) ]  =>  S_joint = sum A^2 ||(1+Z) v_p - Z o_i||^2
    q, k, v = tiny(3)
    scale = 1 / np.sqrt(q.shape[-1])
    A, Z, O = window_outputs(q.astype(float), k.astype(float), v.astype(float), scale)
    vec = (1 + Z)[..., None] * v[None, None].astype(float) - Z[..., None] * O[:, :, None, :]
    expect = (A ** 2 * (vec ** 2).sum(-1)).sum((0, 1))
    s = run_oracle(q, k, v)
    np.testing.assert_allclose(s["VK"], expect, rtol=1e-11)
    assert (s["VK"] >= 0).all() and (s["K"] >= 0).all() and (s["V"] >= 0).all()


def test_equation_and_algorithm1_formulations_agree():
    q, k, v = tiny(4, G=3, W=5, N=40, d=16)
    a = run_oracle(q, k, v, formulation="eq")
    b = run_oracle(q, k, v, formulation="alg1")
    for n in ("V", "K", "VK"):
        np.testing.assert_allclose(a[n], b[n], rtol=1e-10, atol=1e-14 * a[n].max())


def test_attention_statistics():
    q, k, v = tiny(5)
    G, W, d = q.shape
    out = ref.score(q[None], k[None, None], v[None, None], want=("ATTN",), return_attention=True)
    # every softmax row sums to one, so the attention-only scores sum to the number of rows
    np.testing.assert_allclose(out["ATTN"].sum(), G * W, rtol=1e-12)
    A, Z, O = window_outputs(q.astype(float), k.astype(float), v.astype(float), 1 / np.sqrt(d))
    np.testing.assert_allclose(out["O"][0, 0].reshape(G, W, d), O, rtol=1e-11, atol=1e-14)
    np.testing.assert_allclose(out["ATTN"][0, 0], A.sum((0, 1)), rtol=1e-11)
    np.testing.assert_allclose(out["m"][0, 0].reshape(G, W), np.where(A > 0, Z, -np.inf).max(-1), rtol=1e-12)


def test_zero_queries_give_uniform_attention():
    # q = 0 => Z = 0, A = 1/N (non-causal): S_key = 0 and S_joint = S_value = R ||v_p||^2 / N^2
    _, k, v = tiny(6)
    G, W, N = 2, 3, k.shape[0]
    q = np.zeros((G, W, k.shape[1]), np.float32)
    s = run_oracle(q, k, v, causal=False)
    nv = (v.astype(float) ** 2).sum(-1)
    np.testing.assert_allclose(s["V"], G * W * nv / N ** 2, rtol=1e-12)
    np.testing.assert_allclose(s["K"], 0, atol=1e-300)
    np.testing.assert_allclose(s["VK"], s["V"], rtol=1e-12)


def test_single_token_cache():
    # N = 1 => A = 1 and o = v, so the key score vanishes and joint == value == G ||v||^2
    rng = np.random.default_rng(7)
    q = rng.standard_normal((3, 1, 8)).astype(np.float32)
    k = rng.standard_normal((1, 8)).astype(np.float32)
    v = rng.standard_normal((1, 8)).astype(np.float32)
    s = run_oracle(q, k, v)
    nv = float((v.astype(float) ** 2).sum())
    np.testing.assert_allclose(s["V"], [3 * nv], rtol=1e-12)
    np.testing.assert_allclose(s["K"], [0.0], atol=1e-25)
    np.testing.assert_allclose(s["VK"], [3 * nv], rtol=1e-12)


def test_zero_value_token():
    # v_p = 0 => S_value = 0, cross term = 0, so S_joint = S_key = sum A^2 Z^2 ||o_i||^2
    q, k, v = tiny(8)
    v[5] = 0
    s = run_oracle(q, k, v)
    A, Z, O = window_outputs(q.astype(float), k.astype(float), v.astype(float), 1 / np.sqrt(q.shape[-1]))
    assert s["V"][5] == 0
    np.testing.assert_allclose(s["K"][5], (A[..., 5] ** 2 * Z[..., 5] ** 2 * (O ** 2).sum(-1)).sum(), rtol=1e-11)
    np.testing.assert_allclose(s["VK"][5], s["K"][5], rtol=1e-12)


def test_gqa_is_the_sum_of_independent_heads():
    # App. A.5: the per-KV-head score is the sum of the per-query-head scores
    q, k, v = tiny(9, G=4, W=3)
    full = run_oracle(q, k, v)
    for n in ("V", "K", "VK"):
        parts = sum(run_oracle(q[g:g + 1], k, v)[n] for g in range(4))
        np.testing.assert_allclose(full[n], parts, rtol=1e-12)


def test_window_is_the_sum_of_single_query_problems():
    # causal window row i is a decode-style problem (W = 1) over the first N - W + i + 1 tokens
    q, k, v = tiny(10, G=2, W=5, N=30)
    N, W = 30, 5
    full = run_oracle(q, k, v, causal=True)
    for n in ("V", "K", "VK"):
        acc = np.zeros(N)
        for i in range(W):
            n_i = N - W + i + 1
            acc[:n_i] += run_oracle(q[:, i:i + 1], k[:n_i], v[:n_i], causal=True)[n]
        np.testing.assert_allclose(full[n], acc, rtol=1e-12)
    # and without the mask every row sees every token
    full_nc = run_oracle(q, k, v, causal=False)
    acc = sum(run_oracle(q[:, i:i + 1], k, v, causal=False)["VK"] for i in range(W))
    np.testing.assert_allclose(full_nc["VK"], acc, rtol=1e-12)
    assert np.abs(full_nc["VK"] - full["VK"]).max() > 0


def test_value_scaling_and_token_permutation():
    q, k, v = tiny(11, N=32, W=4)
    s = run_oracle(q, k, v)
    s4 = run_oracle(q, k, 2 * v)               # power-of-two scaling is exact in fp32 inputs
    for n in ("V", "K", "VK"):
        np.testing.assert_allclose(s4[n], 4 * s[n], rtol=1e-12)
    # permuting tokens that every window row sees permutes their scores the same way
    rng = np.random.default_rng(0)
    perm = np.arange(32)
    perm[:28] = rng.permutation(28)
    sp = run_oracle(q, k[perm], v[perm])
    for n in ("V", "K", "VK"):
        np.testing.assert_allclose(sp[n], s[n][perm], rtol=1e-11)


def test_batched_ragged_lengths_match_per_sequence_runs():
    rng = np.random.default_rng(12)
    B, Hq, Hkv, W, d, Nmax = 3, 4, 2, 3, 8, 20
    lens = np.array([20, 7, 13], np.int32)
    q = rng.standard_normal((B, Hq, W, d)).astype(np.float32)
    k = rng.standard_normal((B, Hkv, Nmax, d)).astype(np.float32)
    v = rng.standard_normal((B, Hkv, Nmax, d)).astype(np.float32)
    full = ref.score(q, k, v, seq_lens=lens)
    for b in range(B):
        n = lens[b]
        one = ref.score(q[b:b + 1], k[b:b + 1, :, :n], v[b:b + 1, :, :n])
        for name in ("V", "K", "VK"):
            np.testing.assert_allclose(full[name][b, :, :n], one[name][0], rtol=1e-12)
            assert (full[name][b, :, n:] == 0).all()


def test_thread_count_does_not_change_results():
    q, k, v = tiny(13, N=600, W=4)
    a = run_oracle(q, k, v, n_threads=1)
    b = run_oracle(q, k, v, n_threads=5)
    for n in ("V", "K", "VK"):
        assert (a[n] == b[n]).all()


def test_peaky_attention_is_finite_and_nonnegative():
    from paper_2510_07651_b200 import synth
    c = synth.make_prefill("peaky", B=1, Hq=2, Hkv=1, d=32, W=4, N=96, dtype="bf16", seed=5,
                           hh_frac=0.05, peaky=True)
    out = ref.score(c.q, c.k, c.v)
    for n in ("V", "K", "VK"):
        assert np.isfinite(out[n]).all() and (out[n] >= 0).all()


# ---- scores from attention outputs the caller supplies; the l1 value-aware variant -------------
def test_given_attention_outputs_reproduce_the_recompute():
    # O and LSE from the independent numpy attention above, laid out [B,Hq,W,d] / [B,Hq,W] with two KV
    # heads of two query heads each: the given-statistics path must land on the recomputed scores
    rng = np.random.default_rng(21)
    Hkv, G, W, N, d = 2, 2, 3, 19, 8
    q = rng.standard_normal((1, Hkv * G, W, d)).astype(np.float32)
    k = rng.standard_normal((1, Hkv, N, d)).astype(np.float32)
    v = rng.standard_normal((1, Hkv, N, d)).astype(np.float32)
    o = np.zeros((1, Hkv * G, W, d)); lse = np.zeros((1, Hkv * G, W))
    for g in range(Hkv):
        A, Z, O = window_outputs(q[0, g * G:(g + 1) * G].astype(float), k[0, g].astype(float),
                                 v[0, g].astype(float), 1 / np.sqrt(d))
        o[0, g * G:(g + 1) * G] = O
        lse[0, g * G:(g + 1) * G] = np.log(np.where(A > 0, np.exp(Z), 0.0).sum(-1))
    names = ("V", "K", "VK", "ATTN", "VATP")
    want = ref.score(q, k, v, want=names)
    got = ref.score(q, k, v, want=names, given=(o, lse))
    for n in names:      # O and LSE pass through fp32 on the way in
        np.testing.assert_allclose(got[n], want[n], rtol=2e-5, atol=1e-7 * want[n].max())


def test_given_statistics_are_used_as_supplied():
    # one query, one key: z = q.k/sqrt(d); lse = z - ln a forces A = a whatever softmax would say, and
    # the supplied o (not the true output v) enters the key and cross terms
    d, a = 4, 0.3
    q = np.array([[[[1.0, 2.0, 0.0, -1.0]]]], np.float32)
    k = np.array([[[[0.5, -1.0, 3.0, 2.0]]]], np.float32)
    v = np.array([[[[3.0, -4.0, 0.0, 1.0]]]], np.float32)
    o = np.array([[[[1.0, 1.0, -2.0, 0.5]]]], np.float32)
    z = (1.0 * 0.5 - 2.0 * 1.0 - 1.0 * 2.0) / 2.0                     # = -1.75
    lse = np.array([[[z - np.log(a)]]])
    s = ref.score(q, k, v, want=("V", "K", "VK", "ATTN", "VATP"), given=(o, lse))
    nv, vo, dvo = 26.0, 3.0 - 4.0 + 0.5, 4.0 + 25.0 + 4.0 + 0.25       # |v|^2, v.o, |v-o|^2
    tol = dict(rtol=1e-6)                                              # lse is rounded to fp32
    np.testing.assert_allclose(s["ATTN"].ravel(), [a], **tol)
    np.testing.assert_allclose(s["V"].ravel(), [a * a * nv], **tol)
    np.testing.assert_allclose(s["K"].ravel(), [(a * z) ** 2 * dvo], **tol)
    np.testing.assert_allclose(s["VK"].ravel(), [a * a * nv + (a * z) ** 2 * dvo + 2 * a * a * z * (nv - vo)], **tol)
    np.testing.assert_allclose(s["VATP"].ravel(), [a * 8.0], **tol)   # |v|_1 = 8, not |v|^2 = 26
    # doubling exp(lse) halves every A: value score / 4, attention / 2
    s2 = ref.score(q, k, v, want=("V", "ATTN"), given=(o, lse + np.log(2.0)))
    np.testing.assert_allclose(s2["V"].ravel(), [a * a * nv / 4], **tol)
    np.testing.assert_allclose(s2["ATTN"].ravel(), [a / 2], **tol)


def test_l1_value_aware_score():
    # sum_i |A_ip| ||v_p||_1: the attention-only score (pinned above by its row sums) times the l1 norm;
    # unchanged by flipping signs of value channels, linear (not quadratic) in the value scale
    q, k, v = tiny(31)
    s = run_oracle(q, k, v, want=("ATTN", "VATP"))
    np.testing.assert_allclose(s["VATP"], s["ATTN"] * np.abs(v.astype(float)).sum(-1), rtol=1e-12)
    flip = v * np.where(np.arange(v.shape[1]) % 2, -1.0, 1.0).astype(np.float32)
    np.testing.assert_allclose(run_oracle(q, k, flip, want=("VATP",))["VATP"], s["VATP"], rtol=1e-12)
    np.testing.assert_allclose(run_oracle(q, k, 2 * v, want=("VATP",))["VATP"], 2 * s["VATP"], rtol=1e-12)
    # uniform attention (q = 0, non-causal): every token gets R / N times its l1 norm
    G, W, N = 2, 3, k.shape[0]
    u = run_oracle(np.zeros((G, W, k.shape[1]), np.float32), k, v, want=("VATP",), causal=False)
    np.testing.assert_allclose(u["VATP"], G * W / N * np.abs(v.astype(float)).sum(-1), rtol=1e-12)


def test_maskout_diagnostic_equals_brute_force_removal():
    """Masking token p out of the softmax (the other reading of "pruning", kept as a diagnostic): the closed form
    sum_r (A/(1-A))^2 ||v_p - o_r||^2 must equal the output change of an attention recomputed without p."""
    q, k, v = tiny(seed=21, G=2, W=4, N=20, d=8)
    scale = 1.0 / np.sqrt(8.0)
    got = ref.maskout_scores(q, k, v)
    G, W, _ = q.shape
    N = k.shape[0]
    _, _, O = window_outputs(q.astype(np.float64), k.astype(np.float64), v.astype(np.float64), scale)
    for p in range(N):
        keep = [j for j in range(N) if j != p]
        # the same window positions, token p absent: row i still sees original tokens <= N - W + i
        Z = scale * np.einsum("gwd,nd->gwn", q.astype(np.float64), k[keep].astype(np.float64))
        vis = np.array([[j <= N - W + i for j in keep] for i in range(W)])
        Zm = np.where(vis[None], Z, -np.inf)
        E = np.exp(Zm - Zm.max(-1, keepdims=True))
        O2 = (E / E.sum(-1, keepdims=True)) @ v[keep].astype(np.float64)
        want = float(((O2 - O) ** 2).sum())
        assert abs(got[p] - want) <= 1e-12 * max(1.0, want), (p, got[p], want)


def test_rank_agreement_fixture_is_what_the_script_writes():
    """tests/golden/rank_agreement.txt (reported in the results table, nothing is asserted about its values) is
    reproducible from tests/golden/make_rank_agreement.py, which calls only the checker."""
    from tests.golden import make_rank_agreement as mk
    stored = open(os.path.join(GOLD, "rank_agreement.txt")).read()
    assert mk.render(mk.compute()) == stored
