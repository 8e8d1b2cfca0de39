"""CPU-side checks of the C-ABI library: it loads, exports every symbol the header
declares, and rejects host-detectable misuse before launching anything."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2605_12825_b200 import build
    build.build()
    from paper_2605_12825_b200 import binding
    return binding


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "orthrus.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(orthrus_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert "orthrus_diffusion_block_attend" in names and "orthrus_kv_append" in names
    for n in names:
        assert hasattr(lib.lib(), n), n
    assert set(names) == set(lib.EXPORTS)
    assert lib.orthrus_version() >= 100


def test_status_strings(lib):
    s = {lib.lib().orthrus_status_string(c).decode() for c in range(7)}
    assert len(s) == 7


def _layer(lib, **kw):
    d = dict(batch=1, n_q_heads=8, n_kv_heads=2, head_dim=64, block=8, dtype=0, capacity=1024,
             k_cache=0x1000, v_cache=0x2000, cache_len=0x3000, max_len_hint=512, softmax_scale=0.0,
             flags=0)
    d.update(kw)
    return lib.Layer(*[d[f[0]] for f in lib.Layer._fields_])


def test_workspace_query_and_plan(lib):
    assert lib.orthrus_attend_workspace_bytes(_layer(lib)) >= 256
    assert lib.orthrus_attend_workspace_bytes(_layer(lib, n_q_heads=7)) == 0      # Hq % Hkv
    assert lib.orthrus_attend_workspace_bytes(_layer(lib, head_dim=48)) == 0
    assert lib.orthrus_attend_workspace_bytes(_layer(lib, max_len_hint=1020)) == 0  # + K > cap
    big = lib.orthrus_attend_workspace_bytes(
        _layer(lib, n_q_heads=32, n_kv_heads=8, head_dim=128, block=16, capacity=4160,
               max_len_hint=4096))
    assert big > 256      # long prefix, few units: split-KV partials are needed
    assert lib.orthrus_consensus_workspace_bytes(1, 16, 151936) > 256
    assert lib.orthrus_consensus_workspace_bytes(0, 16, 10) == 0


@pytest.mark.parametrize("bad,code", [
    (dict(n_q_heads=7), 1), (dict(head_dim=48), 2), (dict(block=65), 2), (dict(dtype=5), 2),
    (dict(max_len_hint=1020), 3), (dict(k_cache=0), 1), (dict(k_cache=0x1008), 1),
    (dict(softmax_scale=-1.0), 1), (dict(flags=8), 1), (dict(flags=16), 1),
])
def test_attend_rejects_bad_descriptors_before_launch(lib, bad, code):
    L = _layer(lib, **bad)
    n0 = lib.orthrus_launch_count()
    for fn in (lib.lib().orthrus_diffusion_block_attend, lib.lib().orthrus_ar_verify_attend):
        rc = fn(ctypes.byref(L), 0x4000, 0x5000, 0x6000, 0x7000, 0x8000, 1 << 30, None)
        assert rc == code
    assert lib.orthrus_launch_count() == n0


def test_null_and_small_workspace(lib):
    # head_dim 64 takes a path that keeps its split-KV partials in the workspace
    L = _layer(lib, n_q_heads=32, n_kv_heads=8, head_dim=64, block=16, capacity=4160,
               max_len_hint=4096)
    f = lib.lib().orthrus_ar_verify_attend
    assert f(ctypes.byref(L), None, 0x5000, 0x6000, 0x7000, 0x8000, 1 << 30, None) == 1
    assert f(ctypes.byref(L), 0x4000, 0x5000, 0x6000, 0x7000, 0x8000, 256, None) == 4
    assert f(None, 0x4000, 0x5000, 0x6000, 0x7000, 0x8000, 256, None) == 1
    g = lib.lib().orthrus_consensus_accept
    assert g(0x1000, 0, 0x2000, 1, 8, 1000, 0x3000, 0x4000, 0x5000, 0x6000, 0x7000, 8, None) == 4
    assert g(0x1000, 3, 0x2000, 1, 8, 1000, 0x3000, 0x4000, 0x5000, 0x6000, 0x7000, 1 << 20, None) == 2
    assert g(None, 0, 0x2000, 1, 8, 1000, 0x3000, 0x4000, 0x5000, 0x6000, 0x7000, 1 << 20, None) == 1
    a = lib.lib().orthrus_kv_append
    assert a(ctypes.byref(L), None, 0x2000, 0x3000, 1, None, 0, None) == 1
    assert lib.lib().orthrus_set_path(b"bogus") == 1
    assert lib.lib().orthrus_set_path(b"auto") == 0


def test_lm_head_consensus_rejects_misuse_before_launch(lib):
    h = lib.lib().orthrus_lm_head_consensus
    wsb = lib.lib().orthrus_lm_head_consensus_workspace_bytes
    # one (value, id) pair per row and vocabulary tile (at least 128 entries wide), after the header
    assert wsb(2, 16, 1000) == 256 + 2 * 16 * 8 * 8
    assert wsb(0, 16, 1000) == 0
    ok = dict(hidden=0x1000, lm_head=0x2000, dtype=0, H=4096, draft=0x3000, B=1, K=16, V=151936,
              n=0x4000, com=0x5000, arg=0x6000, nxt=0x7000, ws=0x8000, wsb=1 << 30)

    def call(**kw):
        a = dict(ok, **kw)
        return h(a["hidden"], a["lm_head"], a["dtype"], a["H"], a["draft"], a["B"], a["K"], a["V"],
                 a["n"], a["com"], a["arg"], a["nxt"], a["ws"], a["wsb"], None)

    assert call(hidden=None) == 1 and call(lm_head=None) == 1 and call(ws=None) == 1
    assert call(B=0) == 1 and call(H=0) == 1
    assert call(dtype=1) == 2                      # fp32 operands are not supported
    assert call(H=4100) == 2                       # rows must be a multiple of 16 bytes
    assert call(hidden=0x1008) == 1                # 16-byte alignment of the operands
    assert call(draft=0x3002) == 1
    assert call(wsb=1024) == 4


def test_block_write_calls_reject_misuse_before_launch(lib):
    L = _layer(lib)
    n0 = lib.orthrus_launch_count()
    w = lib.lib().orthrus_block_kv_write
    assert w(ctypes.byref(L), None, 0x2000, None, 0, None) == 1
    assert w(ctypes.byref(L), 0x1008, 0x2000, None, 0, None) == 1          # misaligned block tensor
    assert w(ctypes.byref(L), 0x1000, 0x2000, 0x3000, 8, None) == 4        # workspace smaller than its header
    assert w(None, 0x1000, 0x2000, None, 0, None) == 1
    c = lib.lib().orthrus_commit_len
    assert c(ctypes.byref(L), None, None, 0, None) == 1
    assert c(ctypes.byref(L), 0x1002, None, 0, None) == 1
    r = lib.lib().orthrus_rope_block_kv_write
    assert r(ctypes.byref(L), 0x1000, 0x2000, 0x3000, 0.0, 0x4000, None, 0, None) == 1    # theta must be > 0
    assert r(ctypes.byref(L), 0x1000, 0x2000, 0x3000, 1e4, None, None, 0, None) == 1
    assert r(ctypes.byref(_layer(lib, head_dim=48)), 0x1000, 0x2000, 0x3000, 1e4, 0x4000, None, 0, None) == 2
    # with the block in the cache the attention calls take no block tensors
    A = _layer(lib, flags=4)
    f = lib.lib().orthrus_ar_verify_attend
    assert f(ctypes.byref(A), 0x4000, None, None, 0x7000, 0x8000, 16, None) == 4           # only the workspace is short
    assert f(ctypes.byref(_layer(lib)), 0x4000, None, None, 0x7000, 0x8000, 1 << 30, None) == 1
    assert lib.orthrus_launch_count() == n0
