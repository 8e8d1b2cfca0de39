"""Edge cases of Eq. 4's two masks on the tcgen05 kernel itself (head_dim 128, the kernel every
benchmark configuration runs): empty and tile-aligned prefixes, CTAs of a cluster that get no
tile, the CTA that owns nothing but the block tile, a planted key behind the causal mask,
position-coded values, and the clamp of an impossible cache length.  Every case asserts that
the tcgen05 path was the one taken."""
import pytest
import torch

import oracle
from paper_2605_12825_b200 import workloads as W
from _gpu_util import Guarded, assert_close, binding, oracle_attend, run_attend, small_workload

pytestmark = pytest.mark.gpu
VIEWS = [oracle.VIEW_DIFFUSION, oracle.VIEW_AR]
NAN = float("nan")
# (Hq, Hkv, K): group x block = 64 rows (half an MMA tile) and 128 rows (a full one)
TILE_SHAPES = [(8, 2, 16), (16, 2, 16)]
QUIESCENT = 1


def fixed_prefix_inputs(wl, lens, **kw):
    """Inputs of `wl` with the given per-sequence prefix lengths and NaN behind every prefix."""
    t = W.attention_inputs(wl, **kw)
    t["cache_len"][:] = torch.tensor(lens, dtype=torch.int32)
    for b, p in enumerate(lens):
        t["k_cache"][b, :, p:, :] = NAN
        t["v_cache"][b, :, p:, :] = NAN
    return t


@pytest.mark.parametrize("view", VIEWS)
@pytest.mark.parametrize("P", [0, 1, 3, 17, 63, 64, 65, 127, 128, 129, 257])
@pytest.mark.parametrize("shape", TILE_SHAPES)
@pytest.mark.parametrize("splits", [1, 2, 16])
def test_tiny_prefixes_on_the_tcgen05_kernel(view, P, shape, splits):
    """The grid is sized for 1024 positions (16 tiles), the prefixes are far shorter: with 16
    splits most CTAs of a cluster have no tile at all and the last one holds only the block
    tile; with one split the lone CTA walks every tile including a ragged last one."""
    Hq, Hkv, K = shape
    wl = small_workload(2, K, Hq, Hkv, 128, 1024, 1024, std=0.5, name=f"tc_edge_{Hq}_{K}")
    t = fixed_prefix_inputs(wl, [P, max(P - 1, 0)])
    got, status, used = run_attend(view, t, wl, max_len_hint=1024, path="tcgen05", splits=splits)
    assert used == "tcgen05" and status == 0
    assert_close(got, oracle_attend(view, t), torch.bfloat16, f"P={P} splits={splits}")


@pytest.mark.parametrize("view", VIEWS)
@pytest.mark.parametrize("P", [0, 64, 130])
@pytest.mark.parametrize("shape", TILE_SHAPES)
def test_tiny_prefixes_with_early_prefetch(view, P, shape):
    """The same with the cache-quiescent promise: prefix tiles are requested before the wait for
    the preceding kernel, which must not change what is computed (empty prefix included)."""
    Hq, Hkv, K = shape
    wl = small_workload(2, K, Hq, Hkv, 128, 1024, 1024, std=0.5, name=f"tc_edge_q_{Hq}_{K}")
    t = fixed_prefix_inputs(wl, [P, 700])
    got, status, used = run_attend(view, t, wl, max_len_hint=1024, path="tcgen05", splits=16,
                                   flags=QUIESCENT)
    assert used == "tcgen05" and status == 0
    assert_close(got, oracle_attend(view, t), torch.bfloat16, f"P={P}")


@pytest.mark.parametrize("shape", TILE_SHAPES)
@pytest.mark.parametrize("splits", [1, 2, 16])
def test_planted_key_hidden_by_the_causal_rule_tcgen05(shape, splits):
    """A block key with an overwhelming score: every diffusion row collapses onto its value row,
    AR rows before it must not see it at all."""
    Hq, Hkv, K = shape
    wl = small_workload(1, K, Hq, Hkv, 128, 1024, 1024, std=0.3, name=f"tc_plant_{Hq}_{K}")
    t = fixed_prefix_inputs(wl, [150])
    i_star = 11
    for name in ("q_diff", "q_ar"):
        t[name][..., 0] = 1.0
    for name in ("k_diff_blk", "k_ar_blk"):
        t[name][0, i_star, 0, :] = 0
        t[name][0, i_star, 0, 0] = 400.0
    for view in VIEWS:
        got, status, used = run_attend(view, t, wl, max_len_hint=1024, path="tcgen05", splits=splits)
        assert used == "tcgen05" and status == 0
        assert_close(got, oracle_attend(view, t), torch.bfloat16)
        vb = t["v_diff_blk"] if view == oracle.VIEW_DIFFUSION else t["v_ar_blk"]
        target = vb[0, i_star, 0].double()
        for i in range(K):
            d_i = float((got[0, i, 0].double() - target).abs().max())
            if view == oracle.VIEW_DIFFUSION or i >= i_star:
                assert d_i < 1e-2, (view, i, d_i)
            else:
                assert d_i > 5e-2, (view, i, d_i)


@pytest.mark.parametrize("view", VIEWS)
@pytest.mark.parametrize("shape", TILE_SHAPES)
@pytest.mark.parametrize("P", [40, 64, 100])
def test_position_coded_values_tcgen05(view, shape, P):
    """Zero queries give uniform weights; with V[:, 0] holding the key's position, O[0] is the
    mean visible position, which moves by 0.5 for every key wrongly shown or hidden.  Positions
    up to 255 and their half-integer means are exact in bf16."""
    Hq, Hkv, K = shape
    wl = small_workload(1, K, Hq, Hkv, 128, 1024, 1024, std=0.2, name=f"tc_pos_{Hq}_{K}")
    t = fixed_prefix_inputs(wl, [P])
    t["q_diff"].zero_(); t["q_ar"].zero_()
    t["v_cache"][0, :, :P, 0] = torch.arange(P, dtype=torch.float32).to(torch.bfloat16)
    for n in ("v_diff_blk", "v_ar_blk"):
        t[n][0, :, :, 0] = torch.arange(P, P + K, dtype=torch.float32).view(K, 1).to(torch.bfloat16)
    got, status, used = run_attend(view, t, wl, max_len_hint=1024, path="tcgen05", splits=2)
    assert used == "tcgen05" and status == 0
    for i in range(K):
        last = P + K - 1 if view == oracle.VIEW_DIFFUSION else P + i
        for hq in (0, Hq - 1):
            assert abs(float(got[0, i, hq, 0]) - last / 2.0) <= 0.13, (i, hq, float(got[0, i, hq, 0]))


@pytest.mark.parametrize("shape", TILE_SHAPES)
@pytest.mark.parametrize("splits", [1, 16])
@pytest.mark.parametrize("bad", ["too_long", "negative"])
def test_bad_cache_len_is_clamped_and_flagged_tcgen05(shape, splits, bad):
    Hq, Hkv, K = shape
    wl = small_workload(2, K, Hq, Hkv, 128, 300, 300, std=0.5, name=f"tc_clamp_{Hq}_{K}")
    t = W.attention_inputs(wl)
    hi = wl.capacity - wl.block
    t["cache_len"][1] = wl.capacity + 5 if bad == "too_long" else -3
    got, status, used = run_attend(oracle.VIEW_AR, t, wl, max_len_hint=hi, path="tcgen05", splits=splits)
    assert used == "tcgen05" and status & 1
    t["cache_len"][1] = hi if bad == "too_long" else 0
    assert_close(got, oracle_attend(oracle.VIEW_AR, t), torch.bfloat16)


@pytest.mark.parametrize("path,d", [("simt", 32), ("mma", 64), ("simt", 128)])
def test_length_above_the_hint_is_clamped_and_flagged_on_the_split_paths(path, d):
    """The split-KV grids of the SIMT and mma paths are sized from max_len_hint.  A device-side
    length above a stale hint (but within the capacity) is clamped to what the grid covers and
    flagged; nothing is read or written outside the output and the workspace."""
    b = binding()
    wl = small_workload(2, 8, 8, 2, d, 2000, 2000, std=0.5, name=f"stale_{path}_{d}")
    t = W.attention_inputs(wl)
    hint = 500
    dev = {k: v.cuda() for k, v in t.items()}
    layer = b.make_layer(dev["k_cache"], dev["v_cache"], dev["cache_len"], wl.n_q_heads, wl.block, hint)
    b.orthrus_set_path(path)
    try:
        nbytes = b.orthrus_attend_workspace_bytes(layer)
        pad = 4096
        buf = torch.full((nbytes + 2 * pad,), 0x5A, dtype=torch.uint8, device="cuda")
        ws = buf[pad:pad + nbytes]
        ws.zero_()
        out = Guarded(tuple(t["q_ar"].shape), t["q_ar"].dtype)
        b.orthrus_ar_verify_attend(layer, dev["q_ar"], dev["k_ar_blk"], dev["v_ar_blk"], out.t, ws)
        assert b.orthrus_last_path() == path
        status = b.orthrus_read_status(ws)
    finally:
        b.orthrus_set_path("auto")
    assert status & 1
    assert out.intact()
    assert bool((buf[:pad] == 0x5A).all()) and bool((buf[pad + nbytes:] == 0x5A).all())
    got = out.t.cpu()
    assert torch.isfinite(got.float()).all()
    # the clamped length is what the planned splits cover: at least the hint, a whole number of
    # 128-position granules, never more than the true length
    ok = False
    for P in range(512, 2000 + 1, 128):
        t2 = dict(t); t2["cache_len"] = torch.full((2,), P, dtype=torch.int32)
        ref = oracle_attend(oracle.VIEW_AR, t2)
        err = float((got.double() - ref).abs().max())
        if err <= 1e-2 * float(ref.abs().max()):
            ok = True
            break
    assert ok, "output matches no clamped prefix length"


def test_timeout_bit_is_reported_as_a_status():
    """orthrus_read_status turns the wait-timeout bit of the status word into its own return
    code (the bit is planted from the host here; no wait is made to run out)."""
    import ctypes
    b = binding()
    ws = b.new_workspace(256)
    ws[:4].view(torch.int32).fill_(b.DEV_WAIT_TIMEOUT | b.DEV_BAD_CACHE_LEN)
    out = ctypes.c_int32(-1)
    rc = b.lib().orthrus_read_status(ws.data_ptr(), torch.cuda.current_stream().cuda_stream, ctypes.byref(out))
    assert rc == b.ERR_TIMEOUT and out.value == 5
    assert b.orthrus_read_status(ws) == 5
    ws[:4].view(torch.int32).fill_(b.DEV_BAD_CACHE_LEN)
    rc = b.lib().orthrus_read_status(ws.data_ptr(), torch.cuda.current_stream().cuda_stream, ctypes.byref(out))
    assert rc == 0 and out.value == 1
