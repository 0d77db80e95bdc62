"""ctypes front end of the CPU checker in obc_oracle.c.

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's CPU-baseline leg use
this module; the product package never imports it.  It shares nothing with the CUDA path.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "obc_oracle.c")
_LIB = os.path.join(_HERE, "libobc_oracle.so")
_lib = None

VARIANT_BITS = {"V": 1, "K": 2, "VK": 4, "ATTN": 8, "VATP": 16}


def build(force: bool = False) -> str:
    """Compile the checker with gcc (-O2, no FMA contraction) if it is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-ffp-contract=off", "-fPIC", "-shared",
                               "-pthread", "-o", _LIB, _SRC, "-lm"])
    return _LIB


def host_threads() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def lib():
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(_LIB)
        fp, dp, ip = C.POINTER(C.c_float), C.POINTER(C.c_double), C.POINTER(C.c_int32)
        L.obc_oracle_score.argtypes = [fp, fp, fp, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, ip,
                                       C.c_double, C.c_int, C.c_int, dp, dp, dp, dp, dp, dp, dp, dp, C.c_int]
        L.obc_oracle_score_given.argtypes = [fp, fp, fp, fp, fp, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, ip,
                                             C.c_double, C.c_int, C.c_int, dp, dp, dp, dp, dp, C.c_int]
        L.obc_oracle_pool.argtypes = [fp, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, fp]
        L.obc_oracle_select.argtypes = [fp, C.c_int, C.c_int, C.c_int, C.c_int, ip, C.c_int]
        L.obc_oracle_select_adaptive.argtypes = [fp, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_float, ip, ip, C.c_int]
        L.obc_oracle_compact.argtypes = [C.c_void_p, C.c_int, C.c_int, ip, C.c_int, C.c_void_p]
        L.obc_oracle_decode_scores.argtypes = [fp, fp, fp, ip, C.c_int, C.c_int, C.c_int, C.c_int,
                                               C.c_double, C.c_int, dp]
        L.obc_oracle_decode_evict.argtypes = [fp, ip, C.c_int, C.c_int, C.c_int, C.c_int]
        _lib = L
    return _lib


def _f(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a, a.ctypes.data_as(C.POINTER(C.c_float))


def _i(a):
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a, a.ctypes.data_as(C.POINTER(C.c_int32))


def _d(a):
    return a.ctypes.data_as(C.POINTER(C.c_double))


def score(q, k, v, *, seq_lens=None, scale=0.0, causal=True, formulation="eq",
          want=("V", "K", "VK"), return_attention=False, n_threads=None, given=None):
    """Scores for q [B,Hq,W,d], k/v [B,Hkv,Nmax,d] -> dict name -> float64 [B,Hkv,Nmax].

    formulation "eq" follows Eq. 4-6, "alg1" follows Algorithm 1's expanded norms.
    With return_attention the dict also holds "O" [B,Hkv,R,d], "m" and "l" [B,Hkv,R].
    given = (o [B,Hq,W,d], lse [B,Hq,W]) evaluates the formulas with the caller's attention outputs
    (A = exp(Z - lse), natural log) instead of recomputing the window attention.
    """
    q, qp = _f(q); k, kp = _f(k); v, vp = _f(v)
    B, Hq, W, d = q.shape
    _, Hkv, Nmax, _ = k.shape
    R = (Hq // Hkv) * W
    outs = {n: np.zeros((B, Hkv, Nmax), dtype=np.float64) for n in want}
    null = C.POINTER(C.c_double)()
    ptr = lambda n: _d(outs[n]) if n in outs else null
    slp = C.POINTER(C.c_int32)()
    if seq_lens is not None:
        sl, slp = _i(seq_lens)
    o = m = l = None
    op = mp = lp = null
    if return_attention:
        o = np.zeros((B, Hkv, R, d)); m = np.zeros((B, Hkv, R)); l = np.zeros((B, Hkv, R))
        op, mp, lp = _d(o), _d(m), _d(l)
    form = {"eq": 0, "alg1": 1}[formulation]
    if given is not None:
        if return_attention:
            raise ValueError("return_attention has nothing to return when O and LSE are given")
        og, ogp = _f(given[0]); lg, lgp = _f(given[1])
        if og.shape != (B, Hq, W, d) or lg.shape != (B, Hq, W):
            raise ValueError("given O must be [B,Hq,W,d] and LSE [B,Hq,W]")
        rc = lib().obc_oracle_score_given(qp, kp, vp, ogp, lgp, B, Hq, Hkv, d, W, Nmax, slp, float(scale),
                                          int(bool(causal)), form, ptr("V"), ptr("K"), ptr("VK"), ptr("ATTN"),
                                          ptr("VATP"), n_threads or host_threads())
    else:
        rc = lib().obc_oracle_score(qp, kp, vp, B, Hq, Hkv, d, W, Nmax, slp, float(scale), int(bool(causal)),
                                    form, ptr("V"), ptr("K"), ptr("VK"), ptr("ATTN"), ptr("VATP"),
                                    op, mp, lp, n_threads or host_threads())
    if rc != 0:
        raise ValueError("obc_oracle_score rejected its arguments")
    if return_attention:
        outs.update(O=o, m=m, l=l)
    return outs


def maskout_scores(q, k, v, *, scale=0.0, causal=True):
    """Diagnostic, not one of the paper's scores: the exact output perturbation when token p is MASKED OUT of the
    softmax (instead of having its row zeroed, as Def. 3.1 prunes).  Removing p rescales the other weights of row r
    by 1/(1 - A_rp), which gives the closed form  sum_r (A_rp / (1 - A_rp))^2 ||v_p - o_r||^2.
    q [G,W,d], k, v [N,d] (one KV head) -> float64 [N].  A and O come from the checker's own attention."""
    q = np.asarray(q, np.float32); k = np.asarray(k, np.float32); v = np.asarray(v, np.float32)
    G, W, d = q.shape
    N = k.shape[0]
    att = score(q[None], k[None, None], v[None, None], scale=scale, causal=causal, want=("ATTN",), return_attention=True)
    O, m, l = att["O"][0, 0], att["m"][0, 0], att["l"][0, 0]                     # [R,d], [R], [R]
    sc = scale if scale > 0 else 1.0 / np.sqrt(d)
    out = np.zeros(N)
    for r in range(G * W):
        i = r % W
        last = N - W + i if causal else N - 1
        for p in range(last + 1):
            z = sc * float(np.dot(q[r // W, i].astype(np.float64), k[p].astype(np.float64)))
            a = np.exp(z - m[r]) / l[r]
            diff = v[p].astype(np.float64) - O[r]
            out[p] += (a / (1.0 - a)) ** 2 * float(np.dot(diff, diff))
    return out


def pool(s, lo, hi, mode, kernel):
    """fp32 pooling of one head's scores over [lo, hi).  mode: "none" | "avg" | "max"."""
    s, sp = _f(s)
    out = np.empty_like(s)
    rc = lib().obc_oracle_pool(sp, s.shape[0], lo, hi, {"none": 0, "avg": 1, "max": 2}[mode], kernel,
                               out.ctypes.data_as(C.POINTER(C.c_float)))
    if rc != 0:
        raise ValueError("obc_oracle_pool rejected its arguments")
    return out


def select(pooled, budget, n_sink, n_recent, idx_len=None):
    """Kept indices of one head (ascending, padded with -1 to idx_len)."""
    s, sp = _f(pooled)
    idx_len = budget if idx_len is None else idx_len
    idx = np.empty(idx_len, dtype=np.int32)
    rc = lib().obc_oracle_select(sp, s.shape[0], budget, n_sink, n_recent,
                                 idx.ctypes.data_as(C.POINTER(C.c_int32)), idx_len)
    if rc != 0:
        raise ValueError("obc_oracle_select rejected its arguments")
    return idx


def compact(src, idx, budget):
    """Gather rows of one head: src [N,d] (any 2- or 4-byte dtype) -> [budget,d]."""
    src = np.ascontiguousarray(src)
    idx, ip = _i(idx)
    out = np.zeros((budget, src.shape[1]), dtype=src.dtype)
    rc = lib().obc_oracle_compact(src.ctypes.data, src.shape[1], src.dtype.itemsize, ip, budget,
                                  out.ctypes.data)
    if rc != 0:
        raise ValueError("obc_oracle_compact rejected its arguments")
    return out


def select_pipeline(scores, seq_lens, budgets, n_sink, n_recent, pool_mode, pool_kernel, idx_len):
    """pool + select for scores [B,Hkv,Nmax] (fp32) -> idx [B,Hkv,idx_len]."""
    B, H, _ = scores.shape
    idx = np.full((B, H, idx_len), -1, dtype=np.int32)
    for b in range(B):
        n = int(seq_lens[b])
        for h in range(H):
            s = np.ascontiguousarray(scores[b, h, :n], dtype=np.float32)
            pooled = pool(s, n_sink, n - n_recent, pool_mode, pool_kernel)
            idx[b, h] = select(pooled, int(budgets[b]), n_sink, n_recent, idx_len)
    return idx


def select_adaptive(pooled, budget, n_sink, n_recent, safeguard, idx_len):
    """Head-adaptive selection for one batch item: pooled [H,N] -> (idx [H,idx_len], counts [H])."""
    s, sp = _f(pooled)
    H, N = s.shape
    idx = np.empty((H, idx_len), dtype=np.int32)
    counts = np.empty(H, dtype=np.int32)
    rc = lib().obc_oracle_select_adaptive(sp, H, N, budget, n_sink, n_recent, float(safeguard),
                                          idx.ctypes.data_as(C.POINTER(C.c_int32)),
                                          counts.ctypes.data_as(C.POINTER(C.c_int32)), idx_len)
    if rc != 0:
        raise ValueError("obc_oracle_select_adaptive rejected its arguments")
    return idx, counts


def select_adaptive_pipeline(scores, seq_lens, budgets, n_sink, n_recent, pool_mode, pool_kernel, safeguard, idx_len):
    """pool + head-adaptive select for scores [B,Hkv,Nmax] -> (idx [B,Hkv,idx_len], counts [B,Hkv])."""
    B, H, _ = scores.shape
    idx = np.full((B, H, idx_len), -1, dtype=np.int32)
    counts = np.zeros((B, H), dtype=np.int32)
    for b in range(B):
        n = int(seq_lens[b])
        pooled = np.stack([pool(np.ascontiguousarray(scores[b, h, :n], dtype=np.float32), n_sink, n - n_recent,
                                pool_mode, pool_kernel) for h in range(H)])
        idx[b], counts[b] = select_adaptive(pooled, int(budgets[b]), n_sink, n_recent, safeguard, idx_len)
    return idx, counts


def decode_scores(qg, kc, vc, pos, hi, variant="VK", scale=0.0):
    """W=1 scores of one KV head's slots: qg [G,d], kc/vc [cap,d], pos [cap] -> float64 [cap]."""
    qg, qp = _f(qg); kc, kp = _f(kc); vc, vp = _f(vc); pos, pp = _i(pos)
    out = np.zeros(kc.shape[0], dtype=np.float64)
    rc = lib().obc_oracle_decode_scores(qp, kp, vp, pp, qg.shape[0], qg.shape[1], kc.shape[0], hi,
                                        float(scale), VARIANT_BITS[variant], _d(out))
    if rc != 0:
        raise ValueError("obc_oracle_decode_scores rejected its arguments")
    return out


def decode_evict(s_acc, pos, hi, step_pos, n_sink, n_recent):
    s, sp = _f(s_acc); pos, pp = _i(pos)
    return int(lib().obc_oracle_decode_evict(sp, pp, hi, step_pos, n_sink, n_recent))


class DecodeState:
    """Slot-based decode cache of one (batch item, KV head), mirroring the library's layout.

    Step order: append the new (k, v) into `next_slot` -> score every live slot with the newest
    queries -> s_acc += score -> if live > budget, evict one slot (it becomes next_slot).
    """

    def __init__(self, k0, v0, cap, s_acc0=None, window=0):
        """`window` = w > 0: the accumulator is the sum of a token's scores over the last w steps only
        (App. B, accumulation within a recent window); 0: over every step since the token entered."""
        n0, d = k0.shape
        self.window = int(window)
        self.hist = np.zeros((self.window, cap), np.float64)      # ring of per-step scores, row = step_pos mod w
        self.k = np.zeros((cap, d), np.float32); self.v = np.zeros((cap, d), np.float32)
        self.k[:n0] = k0; self.v[:n0] = v0
        self.pos = np.full(cap, -1, np.int32); self.pos[:n0] = np.arange(n0)
        self.s_acc = np.zeros(cap, np.float32)
        if s_acc0 is not None:
            self.s_acc[:n0] = s_acc0
        self.live, self.next_slot, self.hi, self.cap = n0, n0, n0, cap

    def append(self, k_t, v_t, step_pos):
        s = self.next_slot
        self.k[s] = k_t; self.v[s] = v_t; self.pos[s] = step_pos; self.s_acc[s] = 0.0
        if self.window:
            self.hist[:, s] = 0.0
        self.live += 1
        self.hi = max(self.hi, s + 1)

    def scores(self, qg, variant="VK"):
        return decode_scores(qg, self.k, self.v, self.pos, self.hi, variant)

    def accumulate(self, sc, step_pos):
        """The accumulator after this step's scores `sc` [cap] (float64; the state's own s_acc is left to the
        caller, who may store a rounded or a teacher-forced value)."""
        if not self.window:
            return self.s_acc.astype(np.float64) + sc
        self.hist[step_pos % self.window] = np.where(self.pos >= 0, sc, 0.0)
        return self.hist.sum(axis=0)

    def evict(self, step_pos, budget, n_sink, n_recent):
        """Evict per the fp32 accumulator if over budget; returns the evicted slot or -1."""
        if self.live <= budget:
            self.next_slot = self.hi
            return -1
        e = decode_evict(self.s_acc, self.pos, self.hi, step_pos, n_sink, n_recent)
        if e >= 0:
            self.pos[e] = -1
            self.live -= 1
            self.next_slot = e
        else:
            self.next_slot = self.hi
        return e
