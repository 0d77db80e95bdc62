"""Seeded synthetic KV caches shaped like long-context LLaMA-3-8B / Qwen2.5-7B layers.

This module only draws random inputs.  It holds none of the scoring, selection or
compaction arithmetic, so both the CUDA path and the CPU checker can be fed from it.

Every tensor is drawn from a Philox counter-based stream keyed by (seed, tensor tag), so a
tensor's values do not depend on which other tensors were generated before it.

Value recipe (stand-in for real model activations):
  * Q, K, V i.i.d. N(0, 1);
  * a Bernoulli(hh_frac) subset of cached tokens per KV head are "heavy hitters": their key is
    shifted by `hh_shift` along the unit vector of the mean of that KV head's window queries,
    which raises their logits for every window row;
  * optionally token 0 gets the same shift (an attention sink);
  * per-token value norms are scaled by lognormal(0, v_sigma);
  * values are rounded to the storage dtype (bf16 round-to-nearest-even, or fp32) and returned
    as float32 arrays that hold exactly the rounded values, plus the raw bf16 bit patterns.
"""
from __future__ import annotations

import dataclasses
import numpy as np
from numpy.random import Generator, Philox

_TAGS = {"q": 1, "k": 2, "v": 3, "hh": 4, "vscale": 5, "lens": 6, "dq": 7, "dk": 8, "dv": 9}


def _rng(seed: int, tag: str, sub: int = 0) -> Generator:
    return Generator(Philox(key=[(int(seed) << 8) | _TAGS[tag], int(sub)]))


def bf16_round(x: np.ndarray) -> tuple[np.ndarray, np.ndarray]:
    """Round float32 to bfloat16 (nearest, ties to even).

    Returns (float32 array holding the rounded values, uint16 array of bf16 bit patterns).
    """
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    r = (u + bias) >> np.uint32(16)
    bits = r.astype(np.uint16)
    back = (r << np.uint32(16)).astype(np.uint32).view(np.float32)
    return back, bits


@dataclasses.dataclass
class PrefillCase:
    """One prefill-eviction problem.  Layouts: q [B,Hq,W,d]; k, v [B,Hkv,Nmax,d]."""
    name: str
    dtype: str                  # "bf16" | "f32"
    B: int
    Hq: int
    Hkv: int
    d: int
    W: int
    Nmax: int
    seq_lens: np.ndarray        # int32 [B]
    q: np.ndarray               # float32, exactly representable in `dtype`
    k: np.ndarray
    v: np.ndarray
    q_bits: np.ndarray | None   # uint16 bf16 patterns (None for f32)
    k_bits: np.ndarray | None
    v_bits: np.ndarray | None
    heavy: np.ndarray           # bool [B,Hkv,Nmax], which tokens were shifted

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    @property
    def R(self) -> int:
        return self.G * self.W


def _normal(seed, tag, shape, sub=0):
    return _rng(seed, tag, sub).standard_normal(shape, dtype=np.float32)


def make_prefill(name: str, *, B: int, Hq: int, Hkv: int, d: int, W: int, N, dtype: str,
                 seed: int, hh_frac: float = 0.01, hh_shift: float = 3.0, sink0: bool = False,
                 v_sigma: float = 0.5, peaky: bool = False) -> PrefillCase:
    """Draw one prefill case.  `N` is an int (all sequences equal) or a list of B lengths.

    `peaky=True` multiplies the heavy-hitter shift by sqrt(d), so that some attention weights
    approach 1 (a stress case for cancellation in ||v_p - o_i||^2).
    """
    seq_lens = np.full(B, N, dtype=np.int32) if np.isscalar(N) else np.asarray(N, dtype=np.int32)
    assert seq_lens.shape == (B,)
    Nmax = int(seq_lens.max())
    G = Hq // Hkv
    q = _normal(seed, "q", (B, Hq, W, d))
    k = _normal(seed, "k", (B, Hkv, Nmax, d))
    v = _normal(seed, "v", (B, Hkv, Nmax, d))
    # mean window-query direction per KV head
    qbar = q.reshape(B, Hkv, G * W, d).mean(axis=2)
    u = qbar / np.maximum(np.linalg.norm(qbar, axis=-1, keepdims=True), 1e-20)
    heavy = _rng(seed, "hh").random((B, Hkv, Nmax), dtype=np.float32) < np.float32(hh_frac)
    if sink0:
        heavy[:, :, 0] = True
    shift = np.float32(hh_shift * (np.sqrt(d) if peaky else 1.0))
    k += heavy[..., None].astype(np.float32) * (shift * u[:, :, None, :]).astype(np.float32)
    if v_sigma > 0:
        vs = np.exp(np.float32(v_sigma) * _normal(seed, "vscale", (B, Hkv, Nmax)))
        v *= vs[..., None]
    for b in range(B):          # the padding beyond each sequence is zero
        k[b, :, seq_lens[b]:] = 0
        v[b, :, seq_lens[b]:] = 0
        heavy[b, :, seq_lens[b]:] = False
    if dtype == "bf16":
        q, qb = bf16_round(q)
        k, kb = bf16_round(k)
        v, vb = bf16_round(v)
    elif dtype == "f32":
        qb = kb = vb = None
    else:
        raise ValueError(dtype)
    return PrefillCase(name, dtype, B, Hq, Hkv, d, W, Nmax, seq_lens, q, k, v, qb, kb, vb, heavy)


def ragged_lengths(B: int, lo: int, hi: int, seed: int) -> list[int]:
    """B sequence lengths uniform in [lo, hi] (inclusive)."""
    return [int(x) for x in _rng(seed, "lens").integers(lo, hi + 1, size=B)]


# The five workloads.  `scale` < 1 shrinks N (and the budget) for quick runs.
def config(idx: int, *, shrink: int = 1, seed: int | None = None) -> tuple[PrefillCase, dict]:
    """Return (case, run parameters) for prefill workloads 1-4.

    Run parameters: variants (list of "V","K","VK"), budget (int or per-sequence list),
    pool_mode ("none"|"avg"|"max"), pool_kernel, n_sink, n_recent.
    """
    seed = 1234 + idx if seed is None else seed
    if idx == 1:
        n = 1024 // shrink
        c = make_prefill("cfg1", B=1, Hq=1, Hkv=1, d=128, W=16, N=n, dtype="f32", seed=seed,
                         hh_frac=0.0, sink0=True, v_sigma=0.0)
        run = dict(variants=["V", "K", "VK"], budget=256 // shrink, pool_mode="none",
                   pool_kernel=1, n_sink=0, n_recent=16)
    elif idx == 2:
        n = 32768 // shrink
        c = make_prefill("cfg2", B=1, Hq=32, Hkv=8, d=128, W=32, N=n, dtype="bf16", seed=seed)
        run = dict(variants=["VK"], budget=2048 // shrink, pool_mode="max", pool_kernel=7,
                   n_sink=0, n_recent=32)
    elif idx == 3:
        n = 131072 // shrink
        c = make_prefill("cfg3", B=1, Hq=28, Hkv=4, d=128, W=64, N=n, dtype="bf16", seed=seed)
        run = dict(variants=["K", "VK"], budget=4096 // shrink, pool_mode="max", pool_kernel=7,
                   n_sink=0, n_recent=64)
    elif idx == 4:
        lens = ragged_lengths(8, 8192 // shrink, 65536 // shrink, seed)
        c = make_prefill("cfg4", B=8, Hq=32, Hkv=8, d=128, W=32, N=lens, dtype="bf16", seed=seed)
        run = dict(variants=["VK"], budget=[max(33, n // 10) for n in lens], pool_mode="none",
                   pool_kernel=1, n_sink=0, n_recent=32)
    else:
        raise ValueError("prefill configs are 1..4; config 5 is make_decode()")
    return c, run


def full_history(n: int = 4096, *, seed: int = 1240) -> tuple[PrefillCase, dict]:
    """Llama-3-8B-shaped layer scored with the whole sequence as the perturbation window (W = N): every
    query position is a window row, as in the w = 1 accumulation the paper attributes to H2O (Sec. 4.3)."""
    c = make_prefill("history", B=1, Hq=32, Hkv=8, d=128, W=n, N=n, dtype="bf16", seed=seed)
    run = dict(variants=["VK"], budget=n // 8, pool_mode="max", pool_kernel=7, n_sink=0, n_recent=32)
    return c, run


@dataclasses.dataclass
class DecodeCase:
    """Decode-time rescoring problem: an initial cache plus per-step (q, k, v)."""
    B: int
    Hq: int
    Hkv: int
    d: int
    cap: int
    n0: int                     # tokens in the initial cache (slots 0..n0-1, positions 0..n0-1)
    steps: int
    k0: np.ndarray              # float32 [B,Hkv,n0,d] (bf16-exact)
    v0: np.ndarray
    k0_bits: np.ndarray
    v0_bits: np.ndarray
    q_t: np.ndarray             # float32 [steps,B,Hq,d]
    k_t: np.ndarray             # float32 [steps,B,Hkv,d]
    v_t: np.ndarray
    q_t_bits: np.ndarray
    k_t_bits: np.ndarray
    v_t_bits: np.ndarray


def make_decode(*, B: int, Hq: int, Hkv: int, d: int, n0: int, steps: int, seed: int,
                hh_frac: float = 0.01, hh_shift: float = 3.0, v_sigma: float = 0.5) -> DecodeCase:
    """Initial cache of n0 tokens with the same structure as the prefill cases, then `steps`
    i.i.d. N(0,1) (q, k, v) triples.  Heavy-hitter keys are shifted toward the mean of all
    decode queries of the KV head's group."""
    G = Hq // Hkv
    q_t = _normal(seed, "dq", (steps, B, Hq, d))
    k_t = _normal(seed, "dk", (steps, B, Hkv, d))
    v_t = _normal(seed, "dv", (steps, B, Hkv, d))
    k0 = _normal(seed, "k", (B, Hkv, n0, d))
    v0 = _normal(seed, "v", (B, Hkv, n0, d))
    qbar = q_t.reshape(steps, B, Hkv, G, d).mean(axis=(0, 3))
    u = qbar / np.maximum(np.linalg.norm(qbar, axis=-1, keepdims=True), 1e-20)
    heavy = _rng(seed, "hh").random((B, Hkv, n0), dtype=np.float32) < np.float32(hh_frac)
    k0 += heavy[..., None].astype(np.float32) * (np.float32(hh_shift) * u[:, :, None, :])
    if v_sigma > 0:
        v0 *= np.exp(np.float32(v_sigma) * _normal(seed, "vscale", (B, Hkv, n0)))[..., None]
    k0, k0b = bf16_round(k0)
    v0, v0b = bf16_round(v0)
    q_t, qtb = bf16_round(q_t)
    k_t, ktb = bf16_round(k_t)
    v_t, vtb = bf16_round(v_t)
    return DecodeCase(B, Hq, Hkv, d, 0, n0, steps, k0, v0, k0b, v0b, q_t, k_t, v_t, qtb, ktb, vtb)
