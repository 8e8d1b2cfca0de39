"""Thin ctypes binding of liborthrus.so (argument marshalling only).

Every function has the name of the C entry point it calls; tensors are torch CUDA
tensors whose device pointers are handed over unchanged.  torch is used for device
memory and streams, nothing else.  There is no fallback: if the library has not
been built, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liborthrus.so")

OK = 0
ERR_TIMEOUT = 6
BF16, FP32 = 0, 1
DEV_BAD_CACHE_LEN, DEV_APPEND_OVERFLOW, DEV_WAIT_TIMEOUT = 1, 2, 4

EXPORTS = [
    "orthrus_attend_workspace_bytes", "orthrus_workspace_init",
    "orthrus_diffusion_block_attend", "orthrus_ar_verify_attend",
    "orthrus_multi_block_workspace_bytes", "orthrus_multi_block_attend",
    "orthrus_consensus_workspace_bytes", "orthrus_consensus_accept",
    "orthrus_consensus_accept_static", "orthrus_consensus_sample_workspace_bytes",
    "orthrus_consensus_sample",
    "orthrus_lm_head_consensus_workspace_bytes", "orthrus_lm_head_consensus",
    "orthrus_kv_append", "orthrus_kv_append_layers", "orthrus_block_kv_write", "orthrus_commit_len",
    "orthrus_rope_block_kv_write", "orthrus_read_status", "orthrus_set_path", "orthrus_last_path",
    "orthrus_launch_count", "orthrus_status_string", "orthrus_version",
]


class OrthrusError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = _lib.orthrus_status_string(code).decode() if _lib is not None else str(code)
        super().__init__(f"{where}: {msg} (status {code})")


class Layer(ctypes.Structure):
    """Mirror of orthrus_layer_t."""
    _fields_ = [("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
                ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("block", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("capacity", ctypes.c_int64), ("k_cache", ctypes.c_void_p),
                ("v_cache", ctypes.c_void_p), ("cache_len", ctypes.c_void_p),
                ("max_len_hint", ctypes.c_int32), ("softmax_scale", ctypes.c_float),
                ("flags", ctypes.c_uint32)]


LAYER_CACHE_QUIESCENT, LAYER_NO_EARLY_LAUNCH, LAYER_BLOCK_IN_CACHE = 1, 2, 4


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2605_12825_b200.build` "
            "(there is no CPU or PyTorch fallback for the Orthrus kernels)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    LP = ctypes.POINTER(Layer)
    lib.orthrus_attend_workspace_bytes.restype = sz
    lib.orthrus_attend_workspace_bytes.argtypes = [LP]
    lib.orthrus_workspace_init.restype = ctypes.c_int
    lib.orthrus_workspace_init.argtypes = [vp, sz, vp]
    for name in ("orthrus_diffusion_block_attend", "orthrus_ar_verify_attend"):
        f = getattr(lib, name)
        f.restype = ctypes.c_int
        f.argtypes = [LP, vp, vp, vp, vp, vp, sz, vp]
    lib.orthrus_multi_block_workspace_bytes.restype = sz
    lib.orthrus_multi_block_workspace_bytes.argtypes = [LP, i32]
    lib.orthrus_multi_block_attend.restype = ctypes.c_int
    lib.orthrus_multi_block_attend.argtypes = [LP, i32, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.orthrus_consensus_workspace_bytes.restype = sz
    lib.orthrus_consensus_workspace_bytes.argtypes = [i32, i32, i32]
    lib.orthrus_consensus_accept.restype = ctypes.c_int
    lib.orthrus_consensus_accept.argtypes = [vp, i32, vp, i32, i32, i32, vp, vp, vp, vp, vp, sz, vp]
    lib.orthrus_consensus_accept_static.restype = ctypes.c_int
    lib.orthrus_consensus_accept_static.argtypes = [vp, i32, vp, i32, i32, i32, vp, vp, vp, vp, vp]
    lib.orthrus_consensus_sample_workspace_bytes.restype = sz
    lib.orthrus_consensus_sample_workspace_bytes.argtypes = [i32, i32, i32]
    lib.orthrus_consensus_sample.restype = ctypes.c_int
    lib.orthrus_consensus_sample.argtypes = [vp, vp, i32, vp, vp, vp, ctypes.c_float, i32, i32, i32,
                                             vp, vp, vp, vp, sz, vp]
    lib.orthrus_lm_head_consensus_workspace_bytes.restype = sz
    lib.orthrus_lm_head_consensus_workspace_bytes.argtypes = [i32, i32, i32]
    lib.orthrus_lm_head_consensus.restype = ctypes.c_int
    lib.orthrus_lm_head_consensus.argtypes = [vp, vp, i32, i32, vp, i32, i32, i32, vp, vp, vp, vp, vp, sz, vp]
    lib.orthrus_kv_append.restype = ctypes.c_int
    lib.orthrus_kv_append.argtypes = [LP, vp, vp, vp, i32, vp, sz, vp]
    lib.orthrus_kv_append_layers.restype = ctypes.c_int
    lib.orthrus_kv_append_layers.argtypes = [LP, i32, ctypes.POINTER(vp), ctypes.POINTER(vp), vp, i32,
                                             vp, sz, vp]
    lib.orthrus_block_kv_write.restype = ctypes.c_int
    lib.orthrus_block_kv_write.argtypes = [LP, vp, vp, vp, sz, vp]
    lib.orthrus_commit_len.restype = ctypes.c_int
    lib.orthrus_commit_len.argtypes = [LP, vp, vp, sz, vp]
    lib.orthrus_rope_block_kv_write.restype = ctypes.c_int
    lib.orthrus_rope_block_kv_write.argtypes = [LP, vp, vp, vp, ctypes.c_float, vp, vp, sz, vp]
    lib.orthrus_read_status.restype = ctypes.c_int
    lib.orthrus_read_status.argtypes = [vp, vp, ctypes.POINTER(i32)]
    lib.orthrus_set_path.restype = ctypes.c_int
    lib.orthrus_set_path.argtypes = [ctypes.c_char_p]
    lib.orthrus_last_path.restype = ctypes.c_char_p
    lib.orthrus_launch_count.restype = i64
    lib.orthrus_status_string.restype = ctypes.c_char_p
    lib.orthrus_status_string.argtypes = [ctypes.c_int]
    lib.orthrus_version.restype = i32
    return lib


_lib = None
_lib = _load()


def lib() -> ctypes.CDLL:
    return _lib


def dtype_code(dt: torch.dtype) -> int:
    if dt == torch.bfloat16:
        return BF16
    if dt == torch.float32:
        return FP32
    raise TypeError(f"unsupported dtype {dt}")


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def _check(code: int, where: str) -> None:
    if code != OK:
        raise OrthrusError(code, where)


def make_layer(k_cache: torch.Tensor, v_cache: torch.Tensor, cache_len: torch.Tensor,
               n_q_heads: int, block: int, max_len_hint: int = 0,
               softmax_scale: float = 0.0, flags: int = 0) -> Layer:
    """Describe one layer's shared cache ([B][Hkv][capacity][d]) and block shape."""
    B, Hkv, cap, d = k_cache.shape
    return Layer(B, n_q_heads, Hkv, d, block, dtype_code(k_cache.dtype), cap,
                 k_cache.data_ptr(), v_cache.data_ptr(), cache_len.data_ptr(),
                 max_len_hint, softmax_scale, flags)


def orthrus_attend_workspace_bytes(layer: Layer) -> int:
    return int(_lib.orthrus_attend_workspace_bytes(ctypes.byref(layer)))


def orthrus_workspace_init(workspace: torch.Tensor, stream=None) -> None:
    _check(_lib.orthrus_workspace_init(workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                       _stream(stream)), "orthrus_workspace_init")


def new_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    ws = torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)
    orthrus_workspace_init(ws)
    return ws


def orthrus_diffusion_block_attend(layer: Layer, q_diff, k_diff_blk, v_diff_blk, out, workspace,
                                   stream=None) -> None:
    _check(_lib.orthrus_diffusion_block_attend(
        ctypes.byref(layer), _ptr(q_diff), _ptr(k_diff_blk), _ptr(v_diff_blk), _ptr(out),
        _ptr(workspace), workspace.numel(), _stream(stream)), "orthrus_diffusion_block_attend")


def orthrus_ar_verify_attend(layer: Layer, q_ar, k_ar_blk, v_ar_blk, out, workspace,
                             stream=None) -> None:
    _check(_lib.orthrus_ar_verify_attend(
        ctypes.byref(layer), _ptr(q_ar), _ptr(k_ar_blk), _ptr(v_ar_blk), _ptr(out),
        _ptr(workspace), workspace.numel(), _stream(stream)), "orthrus_ar_verify_attend")


def orthrus_multi_block_workspace_bytes(layer: Layer, n_blocks: int) -> int:
    return int(_lib.orthrus_multi_block_workspace_bytes(ctypes.byref(layer), n_blocks))


def orthrus_multi_block_attend(layer: Layer, anchors, q_diff, k_diff_blk, v_diff_blk, out, workspace,
                               stream=None) -> None:
    """Diffusion-view attention under the multi-block mask of Eq. 6; anchors int32 [S][n_blocks],
    q_diff / out [S][n_blocks][K][Hq][d], block K/V [S][n_blocks][K][Hkv][d]."""
    _check(_lib.orthrus_multi_block_attend(
        ctypes.byref(layer), anchors.shape[1], _ptr(anchors), _ptr(q_diff), _ptr(k_diff_blk), _ptr(v_diff_blk),
        _ptr(out), _ptr(workspace), workspace.numel(), _stream(stream)), "orthrus_multi_block_attend")


def orthrus_consensus_workspace_bytes(batch: int, block: int, vocab: int) -> int:
    return int(_lib.orthrus_consensus_workspace_bytes(batch, block, vocab))


def orthrus_consensus_accept(ar_logits, draft, n_commit, committed, ar_argmax, next_anchor,
                             workspace, stream=None) -> None:
    B, K, V = ar_logits.shape
    _check(_lib.orthrus_consensus_accept(
        _ptr(ar_logits), dtype_code(ar_logits.dtype), _ptr(draft), B, K, V, _ptr(n_commit),
        _ptr(committed), _ptr(ar_argmax), _ptr(next_anchor), _ptr(workspace), workspace.numel(),
        _stream(stream)), "orthrus_consensus_accept")


def orthrus_consensus_sample_workspace_bytes(batch: int, block: int, vocab: int) -> int:
    return int(_lib.orthrus_consensus_sample_workspace_bytes(batch, block, vocab))


def orthrus_consensus_sample(ar_logits, diff_logits, draft, u_accept, u_resample, temperature: float,
                             n_commit, committed, next_anchor, workspace, stream=None) -> None:
    """Sampled consensus for T > 0; u_accept / u_resample are float32 [B][K] device tensors."""
    B, K, V = ar_logits.shape
    if diff_logits.shape != ar_logits.shape or diff_logits.dtype != ar_logits.dtype:
        raise TypeError("the two logit tensors must agree in shape and dtype")
    if u_accept.dtype != torch.float32 or u_resample.dtype != torch.float32:
        raise TypeError("the uniforms must be float32")
    _check(_lib.orthrus_consensus_sample(
        _ptr(ar_logits), _ptr(diff_logits), dtype_code(ar_logits.dtype), _ptr(draft), _ptr(u_accept),
        _ptr(u_resample), float(temperature), B, K, V, _ptr(n_commit), _ptr(committed), _ptr(next_anchor),
        _ptr(workspace), workspace.numel(), _stream(stream)), "orthrus_consensus_sample")


STATIC_CONSENSUS_SCRATCH_BYTES = 65536


def orthrus_consensus_accept_static(ar_logits, draft, n_commit, committed, ar_argmax, next_anchor,
                                    stream=None) -> None:
    """Consensus without a caller-provided workspace: for callers that may not allocate
    device memory.  The scratch is a fixed array inside the library, shared by all calls
    on a device (calls that overlap on the GPU race on it).  Problems that need more than
    STATIC_CONSENSUS_SCRATCH_BYTES of scratch raise OrthrusError (workspace too small)."""
    B, K, V = ar_logits.shape
    _check(_lib.orthrus_consensus_accept_static(
        _ptr(ar_logits), dtype_code(ar_logits.dtype), _ptr(draft), B, K, V, _ptr(n_commit),
        _ptr(committed), _ptr(ar_argmax), _ptr(next_anchor), _stream(stream)),
        "orthrus_consensus_accept_static")


def orthrus_lm_head_consensus_workspace_bytes(batch: int, block: int, vocab: int) -> int:
    return int(_lib.orthrus_lm_head_consensus_workspace_bytes(batch, block, vocab))


def orthrus_lm_head_consensus(hidden, lm_head, draft, n_commit, committed, ar_argmax, next_anchor,
                              workspace, stream=None) -> None:
    """Greedy consensus from the last hidden states [B][K][H] and the LM head [V][H] (bf16);
    the logits are never materialised."""
    B, K, H = hidden.shape
    V = lm_head.shape[0]
    _check(_lib.orthrus_lm_head_consensus(
        _ptr(hidden), _ptr(lm_head), dtype_code(hidden.dtype), H, _ptr(draft), B, K, V, _ptr(n_commit),
        _ptr(committed), _ptr(ar_argmax), _ptr(next_anchor), _ptr(workspace), workspace.numel(),
        _stream(stream)), "orthrus_lm_head_consensus")


def orthrus_kv_append(layer: Layer, k_ar_blk, v_ar_blk, n_commit, update_len: bool = True,
                      workspace=None, stream=None) -> None:
    _check(_lib.orthrus_kv_append(
        ctypes.byref(layer), _ptr(k_ar_blk), _ptr(v_ar_blk), _ptr(n_commit),
        1 if update_len else 0, _ptr(workspace), 0 if workspace is None else workspace.numel(),
        _stream(stream)), "orthrus_kv_append")


def orthrus_kv_append_layers(layers, k_ar_blks, v_ar_blks, n_commit, update_len: bool = True,
                             workspace=None, stream=None) -> None:
    """`layers`: sequence of Layer; `k_ar_blks` / `v_ar_blks`: one tensor per layer."""
    n = len(layers)
    arr = (Layer * n)(*layers)
    kp = (ctypes.c_void_p * n)(*[t.data_ptr() for t in k_ar_blks])
    vp = (ctypes.c_void_p * n)(*[t.data_ptr() for t in v_ar_blks])
    _check(_lib.orthrus_kv_append_layers(
        arr, n, kp, vp, _ptr(n_commit), 1 if update_len else 0, _ptr(workspace),
        0 if workspace is None else workspace.numel(), _stream(stream)), "orthrus_kv_append_layers")


def _ws_args(workspace):
    return _ptr(workspace), 0 if workspace is None else workspace.numel()


def orthrus_block_kv_write(layer: Layer, k_blk, v_blk, workspace=None, stream=None) -> None:
    """All K block rows go behind the prefix (cache rows [P_b, P_b + K)); lengths unchanged."""
    _check(_lib.orthrus_block_kv_write(ctypes.byref(layer), _ptr(k_blk), _ptr(v_blk), *_ws_args(workspace),
                                       _stream(stream)), "orthrus_block_kv_write")


def orthrus_commit_len(layer: Layer, n_commit, workspace=None, stream=None) -> None:
    """cache_len += n_commit for the layer's length array."""
    _check(_lib.orthrus_commit_len(ctypes.byref(layer), _ptr(n_commit), *_ws_args(workspace), _stream(stream)),
           "orthrus_commit_len")


def orthrus_rope_block_kv_write(layer: Layer, q, k_blk, v_blk, rope_theta: float, q_out, workspace=None,
                                stream=None) -> None:
    """Rotary embedding of the block's queries (to q_out) and keys, keys and values written to
    cache rows [P_b, P_b + K)."""
    _check(_lib.orthrus_rope_block_kv_write(ctypes.byref(layer), _ptr(q), _ptr(k_blk), _ptr(v_blk),
                                            float(rope_theta), _ptr(q_out), *_ws_args(workspace), _stream(stream)),
           "orthrus_rope_block_kv_write")


def orthrus_read_status(workspace, stream=None) -> int:
    out = ctypes.c_int32(-1)
    code = _lib.orthrus_read_status(workspace.data_ptr(), _stream(stream), ctypes.byref(out))
    if code != ERR_TIMEOUT:                 # a timeout is reported through the word it returns
        _check(code, "orthrus_read_status")
    return int(out.value)


def orthrus_set_path(name: str) -> None:
    _check(_lib.orthrus_set_path(name.encode()), "orthrus_set_path")


def orthrus_last_path() -> str:
    return _lib.orthrus_last_path().decode()


def orthrus_launch_count() -> int:
    return int(_lib.orthrus_launch_count())


def orthrus_version() -> int:
    return int(_lib.orthrus_version())
