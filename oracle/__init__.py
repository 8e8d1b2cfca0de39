"""CPU oracle of the Orthrus generation-step hot path: TEST INFRASTRUCTURE ONLY.

A thin ctypes loader around `orthrus_oracle.c` (plain C, fp64 accumulation).
Only the test suite, the smoke check and the benchmark's CPU-baseline leg may
import this package; the CUDA library and its Python binding never do.

All tensors are torch CPU tensors (bf16, fp32 or fp64, contiguous).  Attention
results come back as float64 tensors.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "orthrus_oracle.c")
_LIB = os.path.join(_HERE, "liborthrus_oracle.so")

VIEW_DIFFUSION = 0
VIEW_AR = 1

_DTYPE_CODE = {torch.bfloat16: 0, torch.float32: 1, torch.float64: 2}


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP) next to its source."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    subprocess.run(["gcc", "-O2", "-fopenmp", "-std=c11", "-shared", "-fPIC",
                    "-o", tmp, _SRC, "-lm"], check=True)
    os.replace(tmp, _LIB)
    return _LIB


class _AttnDesc(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("block", ctypes.c_int32),
                ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("capacity", ctypes.c_int64),
                ("q", ctypes.c_void_p), ("k_blk", ctypes.c_void_p),
                ("v_blk", ctypes.c_void_p), ("k_cache", ctypes.c_void_p),
                ("v_cache", ctypes.c_void_p), ("cache_len", ctypes.c_void_p),
                ("scale", ctypes.c_double)]


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_block_attend.restype = ctypes.c_int
        _lib.oracle_block_attend.argtypes = [ctypes.POINTER(_AttnDesc), ctypes.c_int,
                                             ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64]
        _lib.oracle_block_attend_rows.restype = ctypes.c_int
        _lib.oracle_block_attend_rows.argtypes = [ctypes.POINTER(_AttnDesc), ctypes.c_int,
                                                  ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p]
        _lib.oracle_consensus_accept.restype = ctypes.c_int
        _lib.oracle_consensus_accept.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p,
                                                 ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                                 ctypes.c_void_p, ctypes.c_void_p,
                                                 ctypes.c_void_p, ctypes.c_void_p]
        _lib.oracle_consensus_sample.restype = ctypes.c_int
        _lib.oracle_consensus_sample.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
                                                 ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                                 ctypes.c_double, ctypes.c_int32, ctypes.c_int32,
                                                 ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p,
                                                 ctypes.c_void_p, ctypes.c_void_p]
        _lib.oracle_kv_append.restype = ctypes.c_int
        _lib.oracle_lm_head_argmax.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
                                               ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32,
                                               ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p]
        _lib.oracle_accept_rule.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32,
                                            ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p,
                                            ctypes.c_void_p]
        _lib.oracle_kv_append.argtypes = [ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                          ctypes.c_int32, ctypes.c_int64, ctypes.c_int,
                                          ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                          ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                          ctypes.c_int]
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def _check(t: torch.Tensor, name: str) -> torch.Tensor:
    if t.device.type != "cpu" or not t.is_contiguous():
        raise ValueError(f"{name}: the oracle takes contiguous CPU tensors")
    return t


def _desc(q, k_blk, v_blk, k_cache, v_cache, cache_len, scale) -> _AttnDesc:
    """k_blk = v_blk = None: the block's K/V rows are the cache rows [P_b, P_b + K)."""
    B, K, Hq, d = q.shape
    Hkv, cap = k_cache.shape[1], k_cache.shape[2]
    dt = q.dtype
    in_cache = k_blk is None and v_blk is None
    for n, t in (("q", q), ("k_cache", k_cache), ("v_cache", v_cache)) + \
            (() if in_cache else (("k_blk", k_blk), ("v_blk", v_blk))):
        _check(t, n)
        if t.dtype != dt:
            raise ValueError("all attention tensors must share one dtype")
    if not in_cache and (tuple(k_blk.shape) != (B, K, Hkv, d) or tuple(v_blk.shape) != (B, K, Hkv, d)):
        raise ValueError("block KV must be [B][K][Hkv][d]")
    if tuple(k_cache.shape) != (B, Hkv, cap, d) or tuple(v_cache.shape) != (B, Hkv, cap, d):
        raise ValueError("cache must be [B][Hkv][capacity][d]")
    _check(cache_len, "cache_len")
    if cache_len.dtype != torch.int32 or cache_len.numel() != B:
        raise ValueError("cache_len must be int32 [B]")
    return _AttnDesc(B, K, Hq, Hkv, d, _DTYPE_CODE[dt], cap,
                     q.data_ptr(), None if in_cache else k_blk.data_ptr(),
                     None if in_cache else v_blk.data_ptr(),
                     k_cache.data_ptr(), v_cache.data_ptr(), cache_len.data_ptr(),
                     float(scale) if scale else 0.0)


def block_attend(view: int, q, k_blk, v_blk, k_cache, v_cache, cache_len,
                 scale: Optional[float] = None, return_weights: bool = False):
    """Dual-view block attention (Eq. 4 for VIEW_DIFFUSION; the causal verify pass
    of Section 3.3 for VIEW_AR).  Returns out [B][K][Hq][d] float64, and with
    `return_weights` also the softmax weights [B][K][Hq][max P_b + K]."""
    a = _desc(q, k_blk, v_blk, k_cache, v_cache, cache_len, scale)
    B, K, Hq, d = q.shape
    out = torch.empty((B, K, Hq, d), dtype=torch.float64)
    w = None
    stride = 0
    if return_weights:
        stride = int(cache_len.max()) + K if B else K
        w = torch.zeros((B, K, Hq, stride), dtype=torch.float64)
    rc = lib().oracle_block_attend(ctypes.byref(a), view, out.data_ptr(),
                                   w.data_ptr() if w is not None else None, stride)
    if rc != 0:
        raise RuntimeError(f"oracle_block_attend failed ({rc})")
    return (out, w) if return_weights else out


def block_attend_rows(view: int, rows: torch.Tensor, q, k_blk, v_blk, k_cache, v_cache,
                      cache_len, scale: Optional[float] = None) -> torch.Tensor:
    """Same attention for sampled rows only; rows int32 [n][3] = (b, i, hq).
    Returns [n][d] float64."""
    a = _desc(q, k_blk, v_blk, k_cache, v_cache, cache_len, scale)
    rows = _check(rows.to(torch.int32).contiguous(), "rows")
    out = torch.empty((rows.shape[0], q.shape[3]), dtype=torch.float64)
    rc = lib().oracle_block_attend_rows(ctypes.byref(a), view, rows.data_ptr(),
                                        rows.shape[0], out.data_ptr())
    if rc != 0:
        raise RuntimeError(f"oracle_block_attend_rows failed ({rc})")
    return out


def consensus_accept(logits: torch.Tensor, draft: torch.Tensor
                     ) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor, torch.Tensor]:
    """Greedy consensus (Eq. 8).  Returns (n_commit [B], committed [B][K],
    ar_argmax [B][K], next_anchor [B]), all int32."""
    _check(logits, "logits")
    _check(draft, "draft")
    B, K, V = logits.shape
    if draft.dtype != torch.int32 or tuple(draft.shape) != (B, K):
        raise ValueError("draft must be int32 [B][K]")
    n = torch.empty(B, dtype=torch.int32)
    com = torch.empty((B, K), dtype=torch.int32)
    arg = torch.empty((B, K), dtype=torch.int32)
    nxt = torch.empty(B, dtype=torch.int32)
    rc = lib().oracle_consensus_accept(logits.data_ptr(), _DTYPE_CODE[logits.dtype],
                                       draft.data_ptr(), B, K, V, n.data_ptr(),
                                       com.data_ptr(), arg.data_ptr(), nxt.data_ptr())
    if rc != 0:
        raise RuntimeError(f"oracle_consensus_accept failed ({rc})")
    return n, com, arg, nxt


def consensus_sample(ar_logits: torch.Tensor, diff_logits: torch.Tensor, draft: torch.Tensor,
                     u_accept: torch.Tensor, u_resample: torch.Tensor, temperature: float):
    """Sampled consensus for T > 0 (the rejection-sampling rule of Section 3.3).
    u_accept, u_resample: [B][K] in [0, 1).  Returns (n_commit [B], committed [B][K],
    next_anchor [B]) int32 and margin [B][2] float64: [:, 0] the relative distance of the
    nearest accept test from flipping, [:, 1] the distance of the resampling point from
    the edges of the chosen token's residual mass, as a fraction of that mass (inf if no
    token was resampled)."""
    _check(ar_logits, "ar_logits")
    _check(diff_logits, "diff_logits")
    _check(draft, "draft")
    B, K, V = ar_logits.shape
    if diff_logits.shape != ar_logits.shape or diff_logits.dtype != ar_logits.dtype:
        raise ValueError("the two logit tensors must agree in shape and dtype")
    if draft.dtype != torch.int32 or tuple(draft.shape) != (B, K):
        raise ValueError("draft must be int32 [B][K]")
    ua = u_accept.to(torch.float64).contiguous()
    ur = u_resample.to(torch.float64).contiguous()
    n = torch.empty(B, dtype=torch.int32)
    com = torch.empty((B, K), dtype=torch.int32)
    nxt = torch.empty(B, dtype=torch.int32)
    margin = torch.empty((B, 2), dtype=torch.float64)
    rc = lib().oracle_consensus_sample(ar_logits.data_ptr(), diff_logits.data_ptr(),
                                       _DTYPE_CODE[ar_logits.dtype], draft.data_ptr(),
                                       ua.data_ptr(), ur.data_ptr(), float(temperature), B, K, V,
                                       n.data_ptr(), com.data_ptr(), nxt.data_ptr(), margin.data_ptr())
    if rc != 0:
        raise RuntimeError(f"oracle_consensus_sample failed ({rc})")
    return n, com, nxt, margin


def lm_head_argmax(hidden: torch.Tensor, lm_head: torch.Tensor, rows: Optional[torch.Tensor] = None
                   ) -> Tuple[torch.Tensor, torch.Tensor]:
    """Greedy token of rows of hidden [R][H] under the LM head [V][H] (logit = dot product in
    fp64).  rows: optional int32 list of row numbers (default: all).  Returns (arg [n] int32,
    top2 [n][2] float64 = the largest logit and the largest among the other ids)."""
    _check(hidden, "hidden")
    _check(lm_head, "lm_head")
    R, H = hidden.shape
    V, H2 = lm_head.shape
    if H2 != H or hidden.dtype != lm_head.dtype:
        raise ValueError("hidden [R][H] and lm_head [V][H] must agree in H and dtype")
    if rows is not None:
        rows = _check(rows.to(torch.int32).contiguous(), "rows")
        if rows.numel() and (int(rows.min()) < 0 or int(rows.max()) >= R):
            raise ValueError("row out of range")
    n = R if rows is None else rows.numel()
    arg = torch.empty(n, dtype=torch.int32)
    top2 = torch.empty((n, 2), dtype=torch.float64)
    rc = lib().oracle_lm_head_argmax(hidden.data_ptr(), lm_head.data_ptr(), _DTYPE_CODE[hidden.dtype],
                                     None if rows is None else rows.data_ptr(), n, V, H,
                                     arg.data_ptr(), top2.data_ptr())
    if rc != 0:
        raise RuntimeError(f"oracle_lm_head_argmax failed ({rc})")
    return arg, top2


def accept_rule(g: torch.Tensor, draft: torch.Tensor) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """The halt/commit rule of Section 3.3 on given greedy tokens g [B][K] int32.
    Returns (n_commit [B], committed [B][K], next_anchor [B])."""
    _check(g, "g")
    _check(draft, "draft")
    B, K = g.shape
    if g.dtype != torch.int32 or draft.dtype != torch.int32 or tuple(draft.shape) != (B, K):
        raise ValueError("g and draft must be int32 [B][K]")
    n = torch.empty(B, dtype=torch.int32)
    com = torch.empty((B, K), dtype=torch.int32)
    nxt = torch.empty(B, dtype=torch.int32)
    rc = lib().oracle_accept_rule(g.data_ptr(), draft.data_ptr(), B, K, n.data_ptr(), com.data_ptr(),
                                  nxt.data_ptr())
    if rc != 0:
        raise RuntimeError(f"oracle_accept_rule failed ({rc})")
    return n, com, nxt


def lm_head_consensus(hidden: torch.Tensor, lm_head: torch.Tensor, draft: torch.Tensor):
    """Greedy consensus from the AR view's last hidden states [B][K][H] and the LM head [V][H].
    Returns (n_commit, committed, ar_argmax [B][K], next_anchor) int32 and top2 [B][K][2]."""
    B, K, H = hidden.shape
    arg, top2 = lm_head_argmax(hidden.reshape(B * K, H), lm_head)
    g = arg.reshape(B, K).contiguous()
    n, com, nxt = accept_rule(g, draft)
    return n, com, g, nxt, top2.reshape(B, K, 2)


def kv_append(k_cache, v_cache, cache_len, k_blk, v_blk, n_commit, update_len: bool = True) -> int:
    """KV commit, in place on k_cache / v_cache / cache_len.  Returns the C status
    (0, or -3 if some sequence would overflow its capacity and was skipped)."""
    for n_, t in (("k_cache", k_cache), ("v_cache", v_cache), ("cache_len", cache_len),
                  ("k_blk", k_blk), ("v_blk", v_blk), ("n_commit", n_commit)):
        _check(t, n_)
    B, Hkv, cap, d = k_cache.shape
    K = k_blk.shape[1]
    return int(lib().oracle_kv_append(B, K, Hkv, d, cap, _DTYPE_CODE[k_cache.dtype],
                                      k_cache.data_ptr(), v_cache.data_ptr(),
                                      cache_len.data_ptr(), k_blk.data_ptr(),
                                      v_blk.data_ptr(), n_commit.data_ptr(),
                                      1 if update_len else 0))


def block_kv_write(k_cache, v_cache, cache_len, k_blk, v_blk) -> int:
    """Step 1 of the write-then-truncate commit: all K block rows go behind the prefix, the
    length stays.  In place; returns the C status (0, or -3 if a sequence lacked room)."""
    for n_, t in (("k_cache", k_cache), ("v_cache", v_cache), ("cache_len", cache_len),
                  ("k_blk", k_blk), ("v_blk", v_blk)):
        _check(t, n_)
    B, Hkv, cap, d = k_cache.shape
    K = k_blk.shape[1]
    f = lib().oracle_block_kv_write
    f.argtypes = [ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int64,
                  ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                  ctypes.c_void_p]
    return int(f(B, K, Hkv, d, cap, _DTYPE_CODE[k_cache.dtype], k_cache.data_ptr(), v_cache.data_ptr(),
                 cache_len.data_ptr(), k_blk.data_ptr(), v_blk.data_ptr()))


def commit_len(cache_len, n_commit, block: int, capacity: int) -> int:
    """Step 2: cache_len += n_commit, in place.  Returns the C status."""
    _check(cache_len, "cache_len")
    _check(n_commit, "n_commit")
    f = lib().oracle_commit_len
    f.argtypes = [ctypes.c_int32, ctypes.c_int32, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p]
    return int(f(cache_len.numel(), block, capacity, cache_len.data_ptr(), n_commit.data_ptr()))


def rope_block(x: torch.Tensor, cache_len: torch.Tensor, theta: float = 10000.0) -> torch.Tensor:
    """Rotary embedding of block tensor x [B][K][H][d] at positions cache_len[b] + i (half-split
    pairing).  Returns float64 of the same shape."""
    _check(x, "x")
    _check(cache_len, "cache_len")
    B, K, H, d = x.shape
    y = torch.empty((B, K, H, d), dtype=torch.float64)
    f = lib().oracle_rope_block
    f.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                  ctypes.c_int32, ctypes.c_void_p, ctypes.c_double, ctypes.c_void_p]
    rc = f(x.data_ptr(), _DTYPE_CODE[x.dtype], B, K, H, d, cache_len.data_ptr(), float(theta), y.data_ptr())
    if rc != 0:
        raise RuntimeError(f"oracle_rope_block failed ({rc})")
    return y


def multi_block_attend(q, k_blk, v_blk, k_cache, v_cache, cache_len, anchors,
                       scale: Optional[float] = None) -> torch.Tensor:
    """Diffusion-view attention under the multi-block mask of Eq. 6.  q [S][NB][K][Hq][d];
    k_blk, v_blk [S][NB][K][Hkv][d]; cache [S][Hkv][capacity][d] holding cache_len[s] clean
    positions; anchors int32 [S][NB].  Returns [S][NB][K][Hq][d] float64."""
    S, NB, K, Hq, d = q.shape
    Hkv = k_cache.shape[1]
    for n_, t in (("q", q), ("k_blk", k_blk), ("v_blk", v_blk), ("k_cache", k_cache), ("v_cache", v_cache),
                  ("cache_len", cache_len), ("anchors", anchors)):
        _check(t, n_)
    if tuple(k_blk.shape) != (S, NB, K, Hkv, d) or tuple(v_blk.shape) != (S, NB, K, Hkv, d):
        raise ValueError("block KV must be [S][NB][K][Hkv][d]")
    if anchors.dtype != torch.int32 or tuple(anchors.shape) != (S, NB):
        raise ValueError("anchors must be int32 [S][NB]")
    if int((anchors.long() > cache_len.long().view(S, 1)).sum()) or int((anchors < 0).sum()):
        raise ValueError("anchors must lie in [0, cache_len]")
    a = _AttnDesc(S, K, Hq, Hkv, d, _DTYPE_CODE[q.dtype], k_cache.shape[2], q.data_ptr(), k_blk.data_ptr(),
                  v_blk.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(), cache_len.data_ptr(),
                  float(scale) if scale else 0.0)
    out = torch.empty((S, NB, K, Hq, d), dtype=torch.float64)
    f = lib().oracle_multi_block_attend
    f.argtypes = [ctypes.POINTER(_AttnDesc), ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p]
    rc = f(ctypes.byref(a), NB, anchors.data_ptr(), out.data_ptr())
    if rc != 0:
        raise RuntimeError(f"oracle_multi_block_attend failed ({rc})")
    return out
