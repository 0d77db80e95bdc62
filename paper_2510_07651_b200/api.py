"""Thin ctypes binding over libobcache.so.  Same names as include/obcache.h; argument
marshalling only: every step of the path runs in the library's CUDA kernels.

torch is used for device memory (`data_ptr()`), strides and the current stream, nothing else.
There is no fallback: if the shared library is missing or cannot be loaded, importing the
functions raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libobcache.so")

OBC_F32, OBC_BF16 = 0, 1
OBC_VAR_V, OBC_VAR_K, OBC_VAR_VK, OBC_VAR_ATTN, OBC_VAR_VATP = 1, 2, 4, 8, 16
OBC_POOL_NONE, OBC_POOL_AVG, OBC_POOL_MAX = 0, 1, 2
OBC_PATH_AUTO, OBC_PATH_SIMT, OBC_PATH_TC = 0, 1, 2
VARIANTS = {"V": OBC_VAR_V, "K": OBC_VAR_K, "VK": OBC_VAR_VK, "ATTN": OBC_VAR_ATTN, "VATP": OBC_VAR_VATP}
POOLS = {"none": OBC_POOL_NONE, "avg": OBC_POOL_AVG, "max": OBC_POOL_MAX}
PATHS = {"auto": OBC_PATH_AUTO, "simt": OBC_PATH_SIMT, "tc": OBC_PATH_TC}

EXPORTS = ["obc_score_workspace", "obc_score", "obc_score_given", "obc_window_attention", "obc_merge_attention", "obc_shard_indices", "obc_score_status", "obc_score_kernel_spans", "obc_select_workspace", "obc_select",
           "obc_select_noalloc", "obc_select_adaptive_workspace", "obc_select_adaptive", "obc_compact",
           "obc_decode_workspace", "obc_decode_step", "obc_profile_begin", "obc_profile_end",
           "obc_status_string", "obc_last_cuda_error", "obc_version"]


class ObcError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().obc_status_string(status).decode()
        if status == -6:
            msg += f" [cudaError {lib().obc_last_cuda_error()}]"
        super().__init__(f"{where}: {msg} ({status})")


class obc_tensor(C.Structure):
    _fields_ = [("ptr", C.c_void_p), ("dtype", C.c_int32), ("stride_b", C.c_int64),
                ("stride_h", C.c_int64), ("stride_t", C.c_int64)]


class obc_score_params(C.Structure):
    _fields_ = [("struct_size", C.c_size_t), ("batch", C.c_int32), ("n_q_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("window", C.c_int32),
                ("max_len", C.c_int32), ("seq_lens", C.c_void_p), ("scale", C.c_float),
                ("causal", C.c_int32), ("variants", C.c_uint32), ("path", C.c_int32), ("mask_lens", C.c_void_p)]


class obc_select_params(C.Structure):
    _fields_ = [("struct_size", C.c_size_t), ("batch", C.c_int32), ("n_kv_heads", C.c_int32),
                ("max_len", C.c_int32), ("seq_lens", C.c_void_p), ("budget", C.c_int32),
                ("budgets", C.c_void_p), ("idx_stride", C.c_int32), ("n_sink", C.c_int32),
                ("n_recent", C.c_int32), ("pool_mode", C.c_int32), ("pool_kernel", C.c_int32)]


class obc_decode_params(C.Structure):
    _fields_ = [("struct_size", C.c_size_t), ("batch", C.c_int32), ("n_q_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("capacity", C.c_int32),
                ("budget", C.c_int32), ("n_sink", C.c_int32), ("n_recent", C.c_int32),
                ("variant", C.c_uint32), ("scale", C.c_float), ("acc_window", C.c_int32), ("s_hist", C.c_void_p)]


class obc_kernel_time(C.Structure):
    _fields_ = [("name", C.c_char * 48), ("launches", C.c_int32), ("ms_total", C.c_float)]


_lib = None


def lib():
    """Load libobcache.so (raises OSError if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise OSError(f"{LIB_PATH} is missing: build it with `python -m paper_2510_07651_b200.build` "
                          "(there is no CPU or PyTorch fallback)")
        L = C.CDLL(LIB_PATH)
        vp, sz = C.c_void_p, C.POINTER(C.c_size_t)
        L.obc_score_workspace.argtypes = [C.POINTER(obc_score_params), sz]
        L.obc_score.argtypes = [C.POINTER(obc_score_params), obc_tensor, obc_tensor, obc_tensor, vp, vp, C.c_size_t, vp]
        L.obc_score_given.argtypes = [C.POINTER(obc_score_params), obc_tensor, obc_tensor, obc_tensor, obc_tensor, vp, vp, vp, C.c_size_t, vp]
        L.obc_window_attention.argtypes = [C.POINTER(obc_score_params), obc_tensor, obc_tensor, obc_tensor, vp, vp, vp, C.c_size_t, vp]
        L.obc_merge_attention.argtypes = [C.c_int32, C.c_int64, C.c_int32, vp, vp, vp, vp, vp]
        L.obc_shard_indices.argtypes = [C.c_int32, C.c_int32, C.c_int32, vp, C.c_int32, C.c_int32, vp, vp, vp]
        L.obc_score_status.argtypes = [vp, vp]
        L.obc_score_kernel_spans.argtypes = [vp, vp, C.POINTER(C.c_double), C.POINTER(C.c_double)]
        L.obc_select_workspace.argtypes = [C.POINTER(obc_select_params), sz]
        L.obc_select.argtypes = [C.POINTER(obc_select_params), vp, vp, vp, C.c_size_t, vp]
        L.obc_select_noalloc.argtypes = [C.POINTER(obc_select_params), vp, vp, vp]
        L.obc_select_adaptive_workspace.argtypes = [C.POINTER(obc_select_params), C.c_float, sz]
        L.obc_select_adaptive.argtypes = [C.POINTER(obc_select_params), C.c_float, vp, vp, vp, vp, C.c_size_t, vp]
        L.obc_compact.argtypes = [C.c_int32] * 5 + [obc_tensor, obc_tensor, vp, obc_tensor, obc_tensor, vp, vp, vp]
        L.obc_decode_workspace.argtypes = [C.POINTER(obc_decode_params), sz]
        L.obc_decode_step.argtypes = [C.POINTER(obc_decode_params)] + [obc_tensor] * 5 + [vp, vp, vp, C.c_int32, vp, C.c_size_t, vp]
        L.obc_profile_begin.argtypes = []
        L.obc_profile_end.argtypes = [C.POINTER(obc_kernel_time), C.c_int32, C.POINTER(C.c_int32)]
        L.obc_status_string.argtypes = [C.c_int]
        L.obc_status_string.restype = C.c_char_p
        for n in EXPORTS:
            if n not in ("obc_status_string",):
                getattr(L, n).restype = C.c_int
        _lib = L
    return _lib


def _check(st: int, where: str):
    if st != 0:
        raise ObcError(st, where)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return OBC_F32
    if t.dtype == torch.bfloat16:
        return OBC_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def as_tensor4(t: torch.Tensor) -> obc_tensor:
    """View of a 4-D [batch, heads, tokens, head_dim] CUDA tensor with contiguous head_dim."""
    if not t.is_cuda or t.dim() != 4 or t.stride(3) != 1:
        raise ValueError("expected a CUDA tensor [batch, heads, tokens, head_dim] with contiguous head_dim")
    return obc_tensor(t.data_ptr(), _dtype_code(t), t.stride(0), t.stride(1), t.stride(2))


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t) -> int | None:
    return None if t is None else t.data_ptr()


def _workspace(nbytes: int, like: torch.Tensor, ws: torch.Tensor | None) -> torch.Tensor:
    if ws is not None:
        return ws
    return torch.empty(max(nbytes, 256), dtype=torch.uint8, device=like.device)


def variants_mask(variants) -> int:
    m = 0
    for v in variants:
        m |= VARIANTS[v] if isinstance(v, str) else int(v)
    return m


def score_params(q, k, *, seq_lens=None, scale=0.0, causal=True, variants=("VK",), path="auto",
                 mask_lens=None) -> obc_score_params:
    B, Hq, W, d = q.shape
    _, Hkv, Nmax, _ = k.shape
    return obc_score_params(C.sizeof(obc_score_params), B, Hq, Hkv, d, W, Nmax, _ptr(seq_lens), float(scale),
                            int(bool(causal)), variants_mask(variants), PATHS[path] if isinstance(path, str) else path,
                            _ptr(mask_lens))


def obc_score_workspace(p: obc_score_params) -> int:
    n = C.c_size_t(0)
    _check(lib().obc_score_workspace(C.byref(p), C.byref(n)), "obc_score_workspace")
    return n.value


def obc_score(q, k, v, *, seq_lens=None, scale=0.0, causal=True, variants=("VK",), path="auto",
              scores=None, workspace=None):
    """q [B,Hq,W,d], k/v [B,Hkv,Nmax,d] CUDA tensors -> fp32 scores [n_variants,B,Hkv,Nmax]
    (planes in V, K, VK, ATTN, VATP order).  Enqueued on the current stream."""
    p = score_params(q, k, seq_lens=seq_lens, scale=scale, causal=causal, variants=variants, path=path)
    B, Hkv, Nmax = k.shape[0], k.shape[1], k.shape[2]
    n_planes = bin(p.variants).count("1")
    if scores is None:
        scores = torch.empty((n_planes, B, Hkv, Nmax), dtype=torch.float32, device=k.device)
    ws = _workspace(obc_score_workspace(p), k, workspace)
    _check(lib().obc_score(C.byref(p), as_tensor4(q), as_tensor4(k), as_tensor4(v), scores.data_ptr(),
                           ws.data_ptr(), ws.numel(), _stream()), "obc_score")
    return scores


def obc_window_attention(q, k, v, *, seq_lens=None, mask_lens=None, scale=0.0, causal=True, path="auto",
                         o_out=None, lse_out=None, workspace=None):
    """Window attention of one token shard: (o fp32 [B,Hq,W,d], lse fp32 [B,Hq,W]) over the shard's own
    tokens; mask_lens int32 [B] = sequence length minus the position of the shard's first token."""
    p = score_params(q, k, seq_lens=seq_lens, scale=scale, causal=causal, variants=("VK",), path=path, mask_lens=mask_lens)
    B, Hq, W, d = q.shape
    if o_out is None:
        o_out = torch.empty((B, Hq, W, d), dtype=torch.float32, device=k.device)
    if lse_out is None:
        lse_out = torch.empty((B, Hq, W), dtype=torch.float32, device=k.device)
    ws = _workspace(obc_score_workspace(p), k, workspace)
    _check(lib().obc_window_attention(C.byref(p), as_tensor4(q), as_tensor4(k), as_tensor4(v), o_out.data_ptr(),
                                      lse_out.data_ptr(), ws.data_ptr(), ws.numel(), _stream()), "obc_window_attention")
    return o_out, lse_out


def obc_merge_attention(o_parts, lse_parts, *, o_out=None, lse_out=None):
    """Attention over the whole sequence from its shards': o_parts fp32 [P,B,Hq,W,d], lse_parts fp32 [P,B,Hq,W]."""
    if o_parts.dtype != torch.float32 or lse_parts.dtype != torch.float32 or not (o_parts.is_contiguous() and lse_parts.is_contiguous()):
        raise ValueError("o_parts and lse_parts must be contiguous float32 tensors")
    if tuple(o_parts.shape[:-1]) != tuple(lse_parts.shape):
        raise ValueError("lse_parts must be shaped like o_parts without its last axis")
    P, d = o_parts.shape[0], o_parts.shape[-1]
    rows = lse_parts[0].numel()
    if o_out is None:
        o_out = torch.empty(o_parts.shape[1:], dtype=torch.float32, device=o_parts.device)
    if lse_out is None:
        lse_out = torch.empty(lse_parts.shape[1:], dtype=torch.float32, device=o_parts.device)
    _check(lib().obc_merge_attention(P, rows, d, o_parts.data_ptr(), lse_parts.data_ptr(), o_out.data_ptr(),
                                     lse_out.data_ptr(), _stream()), "obc_merge_attention")
    return o_out, lse_out


def obc_shard_indices(idx, token_offset: int, n_local: int, *, idx_local=None, counts=None):
    """A token shard's share of the kept indices idx int32 [B,Hkv,stride]: (idx_local, counts), see include/obcache.h."""
    if idx.dtype != torch.int32 or not idx.is_contiguous():
        raise ValueError("idx must be a contiguous int32 tensor")
    B, Hkv, stride = idx.shape
    if idx_local is None:
        idx_local = torch.empty_like(idx)
    if counts is None:
        counts = torch.empty((B, Hkv), dtype=torch.int32, device=idx.device)
    _check(lib().obc_shard_indices(B, Hkv, stride, idx.data_ptr(), int(token_offset), int(n_local), idx_local.data_ptr(),
                                   counts.data_ptr(), _stream()), "obc_shard_indices")
    return idx_local, counts


def obc_score_given(q, k, v, o, lse, *, seq_lens=None, scale=0.0, causal=True, variants=("VK",), path="auto",
                    scores=None, workspace=None, mask_lens=None):
    """obc_score from attention outputs the caller already has: o [B,Hq,W,d] (f32 or bf16) and lse
    fp32 [B,Hq,W] (natural log, contiguous) of the window rows; no window attention is recomputed."""
    p = score_params(q, k, seq_lens=seq_lens, scale=scale, causal=causal, variants=variants, path=path, mask_lens=mask_lens)
    B, Hkv, Nmax = k.shape[0], k.shape[1], k.shape[2]
    if tuple(o.shape) != tuple(q.shape) or tuple(lse.shape) != tuple(q.shape[:3]):
        raise ValueError("o must be shaped like q and lse like q without its last axis")
    if lse.dtype != torch.float32 or not lse.is_contiguous():
        raise ValueError("lse must be a contiguous float32 tensor")
    n_planes = bin(p.variants).count("1")
    if scores is None:
        scores = torch.empty((n_planes, B, Hkv, Nmax), dtype=torch.float32, device=k.device)
    ws = _workspace(obc_score_workspace(p), k, workspace)
    _check(lib().obc_score_given(C.byref(p), as_tensor4(q), as_tensor4(k), as_tensor4(v), as_tensor4(o),
                                 lse.data_ptr(), scores.data_ptr(), ws.data_ptr(), ws.numel(), _stream()),
           "obc_score_given")
    return scores


def obc_score_status(workspace) -> None:
    """Synchronise and raise ObcError(OBC_ERR_TIMEOUT) if a bounded device-side wait gave up."""
    _check(lib().obc_score_status(workspace.data_ptr(), _stream()), "obc_score_status")


def obc_score_kernel_spans(workspace) -> tuple[float, float]:
    """Synchronise; return the device-side extents (us) of the window-statistics kernel and of the fused
    score kernel since the header words were last zero, and zero them.  (0, 0) on the CUDA-core path."""
    p1, p2 = C.c_double(0), C.c_double(0)
    _check(lib().obc_score_kernel_spans(workspace.data_ptr(), _stream(), C.byref(p1), C.byref(p2)),
           "obc_score_kernel_spans")
    return p1.value, p2.value


def select_params(scores, *, budget=0, budgets=None, idx_stride=None, seq_lens=None, n_sink=0, n_recent=0,
                  pool="none", pool_kernel=1) -> obc_select_params:
    B, Hkv, Nmax = scores.shape
    if idx_stride is None:
        idx_stride = budget
    return obc_select_params(C.sizeof(obc_select_params), B, Hkv, Nmax, _ptr(seq_lens), int(budget), _ptr(budgets),
                             int(idx_stride), n_sink, n_recent, POOLS[pool] if isinstance(pool, str) else pool,
                             pool_kernel)


def obc_select_workspace(p: obc_select_params) -> int:
    n = C.c_size_t(0)
    _check(lib().obc_select_workspace(C.byref(p), C.byref(n)), "obc_select_workspace")
    return n.value


def obc_select(scores, *, budget=0, budgets=None, idx_stride=None, seq_lens=None, n_sink=0, n_recent=0,
               pool="none", pool_kernel=1, idx=None, workspace=None):
    """scores fp32 [B,Hkv,Nmax] -> int32 idx [B,Hkv,idx_stride] (ascending, padded with -1)."""
    p = select_params(scores, budget=budget, budgets=budgets, idx_stride=idx_stride, seq_lens=seq_lens,
                      n_sink=n_sink, n_recent=n_recent, pool=pool, pool_kernel=pool_kernel)
    if idx is None:
        idx = torch.empty((p.batch, p.n_kv_heads, p.idx_stride), dtype=torch.int32, device=scores.device)
    ws = _workspace(obc_select_workspace(p), scores, workspace)
    _check(lib().obc_select(C.byref(p), scores.data_ptr(), idx.data_ptr(), ws.data_ptr(), ws.numel(), _stream()),
           "obc_select")
    return idx


def obc_select_adaptive(scores, *, budget, safeguard=0.2, idx_stride=None, seq_lens=None, n_sink=0, n_recent=0,
                        pool="none", pool_kernel=1, idx=None, counts=None, workspace=None):
    """Head-adaptive budgets: scores fp32 [B,Hkv,Nmax] -> (idx int32 [B,Hkv,idx_stride] padded with -1,
    counts int32 [B,Hkv]).  Every head keeps floor(safeguard * n_hh) tokens by its own ranking; the rest of the
    layer's Hkv * n_hh slots go to the best remaining tokens of all heads together."""
    p = select_params(scores, budget=budget, idx_stride=idx_stride, seq_lens=seq_lens, n_sink=n_sink,
                      n_recent=n_recent, pool=pool, pool_kernel=pool_kernel)
    if idx is None:
        idx = torch.empty((p.batch, p.n_kv_heads, p.idx_stride), dtype=torch.int32, device=scores.device)
    if counts is None:
        counts = torch.empty((p.batch, p.n_kv_heads), dtype=torch.int32, device=scores.device)
    n = C.c_size_t(0)
    _check(lib().obc_select_adaptive_workspace(C.byref(p), float(safeguard), C.byref(n)), "obc_select_adaptive_workspace")
    ws = _workspace(n.value, scores, workspace)
    _check(lib().obc_select_adaptive(C.byref(p), float(safeguard), scores.data_ptr(), idx.data_ptr(), counts.data_ptr(),
                                     ws.data_ptr(), ws.numel(), _stream()), "obc_select_adaptive")
    return idx, counts


SELECT_NOALLOC_MAX_KEYS = 1 << 20


def obc_select_noalloc(scores, idx, *, budget=0, budgets=None, seq_lens=None, n_sink=0, n_recent=0,
                       pool="none", pool_kernel=1):
    """obc_select without a workspace, for callers that may not allocate device memory (an engine
    plug-in without an allocator, a serving loop with a fixed memory budget): the key scratch is a
    fixed 4 MiB array inside the library.  `idx` [B,Hkv,idx_stride] int32 is the caller's buffer;
    this wrapper allocates nothing either.  Raises ObcError(OBC_ERR_CAPACITY) when
    B*Hkv*Nmax > SELECT_NOALLOC_MAX_KEYS.  Calls on one device share the scratch: do not let two
    of them overlap on the GPU; make the first call on a device outside stream capture."""
    p = select_params(scores, budget=budget, budgets=budgets, idx_stride=idx.shape[2], seq_lens=seq_lens,
                      n_sink=n_sink, n_recent=n_recent, pool=pool, pool_kernel=pool_kernel)
    _check(lib().obc_select_noalloc(C.byref(p), scores.data_ptr(), idx.data_ptr(), _stream()), "obc_select_noalloc")
    return idx


def obc_compact(k, v, idx, *, k_out=None, v_out=None, scores_in=None, scores_out=None):
    """Gather kept rows: k/v [B,Hkv,Nmax,d], idx [B,Hkv,S] -> k_out/v_out [B,Hkv,S,d]."""
    B, Hkv, Nmax, d = k.shape
    S = idx.shape[2]
    if k_out is None:
        k_out = torch.zeros((B, Hkv, S, d), dtype=k.dtype, device=k.device)
    if v_out is None:
        v_out = torch.zeros((B, Hkv, S, d), dtype=v.dtype, device=v.device)
    if scores_in is not None and scores_out is None:
        scores_out = torch.zeros((B, Hkv, S), dtype=torch.float32, device=k.device)
    _check(lib().obc_compact(B, Hkv, d, S, Nmax, as_tensor4(k), as_tensor4(v), idx.data_ptr(), as_tensor4(k_out),
                             as_tensor4(v_out), _ptr(scores_in), _ptr(scores_out), _stream()), "obc_compact")
    return (k_out, v_out) if scores_in is None else (k_out, v_out, scores_out)


def decode_params(q_t, k_cache, *, budget, n_sink, n_recent, variant="VK", scale=0.0, acc_window=0,
                  s_hist=None) -> obc_decode_params:
    B, Hq, _, d = q_t.shape
    _, Hkv, cap, _ = k_cache.shape
    if acc_window > 0 and s_hist is not None:
        assert s_hist.dtype == torch.float32 and s_hist.is_contiguous() and tuple(s_hist.shape) == (B, Hkv, acc_window, cap)
    return obc_decode_params(C.sizeof(obc_decode_params), B, Hq, Hkv, d, cap, budget, n_sink, n_recent,
                             VARIANTS[variant] if isinstance(variant, str) else variant, float(scale),
                             int(acc_window), _ptr(s_hist))


def obc_decode_workspace(p: obc_decode_params) -> int:
    n = C.c_size_t(0)
    _check(lib().obc_decode_workspace(C.byref(p), C.byref(n)), "obc_decode_workspace")
    return n.value


def obc_decode_step(q_t, k_t, v_t, k_cache, v_cache, s_acc, pos, state, step_pos, *, budget, n_sink, n_recent,
                    variant="VK", scale=0.0, workspace=None, acc_window=0, s_hist=None):
    """One in-place decode rescoring + eviction step (see include/obcache.h).  With acc_window = w > 0 the
    accumulator is the sum of the last w steps' scores and s_hist is the zero-initialised fp32 ring
    [B,Hkv,w,capacity] that holds them."""
    p = decode_params(q_t, k_cache, budget=budget, n_sink=n_sink, n_recent=n_recent, variant=variant, scale=scale,
                      acc_window=acc_window, s_hist=s_hist)
    ws = _workspace(obc_decode_workspace(p), k_cache, workspace)
    _check(lib().obc_decode_step(C.byref(p), as_tensor4(q_t), as_tensor4(k_t), as_tensor4(v_t), as_tensor4(k_cache),
                                 as_tensor4(v_cache), s_acc.data_ptr(), pos.data_ptr(), state.data_ptr(),
                                 int(step_pos), ws.data_ptr(), ws.numel(), _stream()), "obc_decode_step")
    return ws


def obc_profile_begin():
    """Start bracketing every library kernel with CUDA events (benchmark use)."""
    _check(lib().obc_profile_begin(), "obc_profile_begin")


def obc_profile_end() -> dict:
    """Stop recording; returns {kernel name: (launches, total ms)}."""
    buf = (obc_kernel_time * 64)()
    n = C.c_int32(0)
    _check(lib().obc_profile_end(buf, 64, C.byref(n)), "obc_profile_end")
    return {buf[i].name.decode(): (buf[i].launches, buf[i].ms_total) for i in range(n.value)}


def evict_prefill(q, k, v, *, budget=0, budgets=None, seq_lens=None, variant="VK", n_sink=0, n_recent=None,
                  pool="none", pool_kernel=1, causal=True, path="auto"):
    """The whole prefill hot path: score -> pool/select -> compact.  Returns (k_out, v_out, idx, scores)."""
    n_recent = q.shape[2] if n_recent is None else n_recent
    scores = obc_score(q, k, v, seq_lens=seq_lens, causal=causal, variants=(variant,), path=path)
    stride = int(budget) if budgets is None else int(budgets.max().item())
    idx = obc_select(scores[0], budget=budget, budgets=budgets, idx_stride=stride, seq_lens=seq_lens,
                     n_sink=n_sink, n_recent=n_recent, pool=pool, pool_kernel=pool_kernel)
    k_out, v_out = obc_compact(k, v, idx)
    return k_out, v_out, idx, scores
