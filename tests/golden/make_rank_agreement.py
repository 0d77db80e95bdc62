"""Writes rank_agreement.txt: how well the second-order joint score (Eq. 6) ranks the tokens of a small cache
compared with the exact pruning error of Def. 3.1 / Eq. 1 (rows p of K and V set to zero, attention recomputed).
Sec. 4.4 claims agreement of the rankings, not of the values.  Everything here comes from the CPU checker
(oracle/): its scores, and its attention outputs before and after the rows are zeroed.

    python -m tests.golden.make_rank_agreement
"""
import os

import numpy as np

from oracle import reference as ref

HERE = os.path.dirname(os.path.abspath(__file__))
CASES = [(0, 1.0), (1, 1.0), (2, 2.0), (3, 0.5)]            # (seed, spread of q and k)


def _ranks(x):
    order = np.argsort(-x, kind="stable")
    r = np.empty(len(x)); r[order] = np.arange(len(x))
    return r


def compute():
    G, W, N, d = 2, 8, 64, 16
    rows = []
    for seed, spread in CASES:
        rng = np.random.default_rng(seed)
        q = (spread * rng.standard_normal((1, G, W, d))).astype(np.float32)
        k = (spread * rng.standard_normal((1, 1, N, d))).astype(np.float32)
        v = rng.standard_normal((1, 1, N, d)).astype(np.float32)
        base = ref.score(q, k, v, want=("V", "K", "VK"), return_attention=True)
        exact = np.zeros(N)
        for p in range(N):
            k2, v2 = k.copy(), v.copy()
            k2[0, 0, p] = 0.0; v2[0, 0, p] = 0.0
            o2 = ref.score(q, k2, v2, want=("ATTN",), return_attention=True)["O"]
            exact[p] = float(((o2 - base["O"]) ** 2).sum())
        cand = slice(0, N - W)                               # tokens the selection may evict
        row = [seed, spread]
        for name in ("VK", "K", "V"):
            s = base[name][0, 0]
            rs, re_ = _ranks(s[cand]), _ranks(exact[cand])
            rho = float(np.corrcoef(rs, re_)[0, 1])          # Spearman: Pearson of the ranks
            kk = (N - W) // 4
            top = len(set(np.argsort(-s[cand], kind="stable")[:kk]) & set(np.argsort(-exact[cand], kind="stable")[:kk])) / kk
            row += [rho, top]
        rows.append(row)
    return rows


def render(rows):
    out = ["# Rank agreement of the second-order scores with the exact pruning error (Def. 3.1 / Eq. 1; Sec. 4.4), reported.",
           "# One KV head, G=2 query heads, W=8 window rows, N=64 tokens, d=16; candidates = tokens before the window.",
           "# Columns: seed, spread, then for the joint (Eq. 6), key (Eq. 5) and value (Eq. 4) scores: Spearman rho, overlap of the top quarter.",
           "# Written by tests/golden/make_rank_agreement.py (calls only the CPU checker)."]
    for r in rows:
        out.append(f"{r[0]:d} {r[1]:.1f} " + " ".join(f"{x:.6f}" for x in r[2:]))
    return "\n".join(out) + "\n"


if __name__ == "__main__":
    text = render(compute())
    open(os.path.join(HERE, "rank_agreement.txt"), "w").write(text)
    print(text)
