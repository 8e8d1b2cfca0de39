"""Parity of the persistent (tile-scheduled) form of the tcgen05 kernel, forced with
ORTHRUS_TC_SCHEDULE=stream on shapes small enough for the oracle: CTAs whose range covers several
whole units, units cut between two and many CTAs, empty prefixes (units of one tile), fewer tiles
than CTAs, both views, the block read from the cache, repeated calls on one workspace (the arrival
counters must return to zero)."""
import os

import pytest
import torch

import oracle
from paper_2605_12825_b200 import workloads as W
from _gpu_util import Guarded, assert_close, binding, oracle_attend, small_workload

pytestmark = pytest.mark.gpu
VIEWS = [oracle.VIEW_DIFFUSION, oracle.VIEW_AR]
NAN = float("nan")


@pytest.fixture(autouse=True)
def stream_schedule():
    old = os.environ.get("ORTHRUS_TC_SCHEDULE")
    os.environ["ORTHRUS_TC_SCHEDULE"] = "stream"
    yield
    if old is None:
        os.environ.pop("ORTHRUS_TC_SCHEDULE", None)
    else:
        os.environ["ORTHRUS_TC_SCHEDULE"] = old


def run(view, t, wl, flags=0, calls=1):
    b = binding()
    d = {k: v.cuda() for k, v in t.items()}
    layer = b.make_layer(d["k_cache"], d["v_cache"], d["cache_len"], wl.n_q_heads, wl.block,
                         int(t["cache_len"].max()), 0.0, flags)
    ws = b.new_workspace(b.orthrus_attend_workspace_bytes(layer))
    q, kb, vb = ("q_diff", "k_diff_blk", "v_diff_blk") if view == oracle.VIEW_DIFFUSION else ("q_ar", "k_ar_blk", "v_ar_blk")
    fn = b.orthrus_diffusion_block_attend if view == oracle.VIEW_DIFFUSION else b.orthrus_ar_verify_attend
    out = Guarded(tuple(t[q].shape), t[q].dtype)
    b.orthrus_set_path("tcgen05")
    try:
        for _ in range(calls):
            out.t.fill_(7.0)
            if flags & b.LAYER_BLOCK_IN_CACHE:
                fn(layer, d[q], None, None, out.t, ws)
            else:
                fn(layer, d[q], d[kb], d[vb], out.t, ws)
        assert b.orthrus_last_path() == "tcgen05"
        assert b.orthrus_read_status(ws) == 0
    finally:
        b.orthrus_set_path("auto")
    assert out.intact()
    # behind the header: partial tiles, then the arrival counters, which must all be back at zero
    tail = ws[-(((wl.batch * wl.n_kv_heads * 4 + 255) // 256) * 256):].view(torch.int32)
    assert int(tail.abs().sum()) == 0
    return out.t.cpu()


@pytest.mark.parametrize("view", VIEWS)
@pytest.mark.parametrize("shape", [
    # B, K, Hq, Hkv, d, pmin, pmax
    (40, 16, 32, 8, 128, 0, 600),       # 320 units, about 2 tiles per CTA: CTAs span several whole units
    (32, 32, 32, 8, 128, 1024, 8192),   # the ragged serving shape
    (3, 16, 8, 2, 128, 3000, 9000),     # 6 units over 296 CTAs: every unit cut into many pieces
    (2, 8, 4, 4, 128, 0, 0),            # empty prefixes: 8 tiles in all, most CTAs idle
    (5, 1, 4, 4, 128, 1, 700),          # block of one, M = 1
    (7, 16, 16, 2, 128, 63, 65),        # M = 128, prefixes around a tile edge
    (128, 4, 8, 2, 128, 10, 300),       # the most batch entries the ranking holds
])
def test_stream_schedule_matches_the_oracle(view, shape):
    wl = small_workload(*shape, std=0.7, name=f"sk_{shape}")
    t = W.attention_inputs(wl, fill_tail=NAN)
    got = run(view, t, wl, calls=2)
    if shape[0] * shape[6] > 100000:     # the large case: sampled rows
        g = torch.Generator().manual_seed(1)
        B, K, Hq = wl.batch, wl.block, wl.n_q_heads
        flat = torch.randperm(B * K * Hq, generator=g)[:128]
        rows = torch.stack([flat // (K * Hq), (flat // Hq) % K, flat % Hq], dim=1).to(torch.int32)
        q, kb, vb = ("q_diff", "k_diff_blk", "v_diff_blk") if view == oracle.VIEW_DIFFUSION else ("q_ar", "k_ar_blk", "v_ar_blk")
        ref = oracle.block_attend_rows(view, rows, t[q], t[kb], t[vb], t["k_cache"], t["v_cache"], t["cache_len"])
        assert torch.isfinite(got.float()).all()
        assert_close(got[rows[:, 0].long(), rows[:, 1].long(), rows[:, 2].long()], ref, torch.bfloat16, str(shape))
    else:
        assert_close(got, oracle_attend(view, t), torch.bfloat16, str(shape))


@pytest.mark.parametrize("view", VIEWS)
def test_stream_schedule_with_the_block_in_the_cache_and_early_launch(view):
    b = binding()
    wl = small_workload(24, 16, 16, 4, 128, 0, 900, std=0.7, name="sk_incache")
    t = W.attention_inputs(wl, fill_tail=NAN)
    kb, vb = ("k_diff_blk", "v_diff_blk") if view == oracle.VIEW_DIFFUSION else ("k_ar_blk", "v_ar_blk")
    q = "q_diff" if view == oracle.VIEW_DIFFUSION else "q_ar"
    oracle.block_kv_write(t["k_cache"], t["v_cache"], t["cache_len"], t[kb], t[vb])
    ref = oracle.block_attend(view, t[q], None, None, t["k_cache"], t["v_cache"], t["cache_len"])
    got = run(view, t, wl, flags=b.LAYER_BLOCK_IN_CACHE | b.LAYER_CACHE_QUIESCENT, calls=3)
    assert_close(got, ref, torch.bfloat16)


def test_stream_schedule_multi_block():
    b = binding()
    S, NB, K, Hq, Hkv, d = 6, 8, 8, 8, 2, 128
    g = torch.Generator().manual_seed(3)
    mk = lambda *s: (torch.randn(*s, generator=g) * 0.7).to(torch.bfloat16)
    lens = torch.randint(200, 1500, (S,), generator=g).to(torch.int32)
    cap = 1536
    anchors = torch.stack([torch.randint(0, int(lens[s]) + 1, (NB,), generator=g) for s in range(S)]).to(torch.int32)
    c = dict(q=mk(S, NB, K, Hq, d), k_blk=mk(S, NB, K, Hkv, d), v_blk=mk(S, NB, K, Hkv, d),
             k_cache=mk(S, Hkv, cap, d), v_cache=mk(S, Hkv, cap, d), cache_len=lens, anchors=anchors)
    ref = oracle.multi_block_attend(c["q"], c["k_blk"], c["v_blk"], c["k_cache"], c["v_cache"], lens, anchors)
    dev = {k: v.cuda() for k, v in c.items()}
    layer = b.make_layer(dev["k_cache"], dev["v_cache"], dev["cache_len"], Hq, K, int(anchors.max()))
    ws = b.new_workspace(b.orthrus_multi_block_workspace_bytes(layer, NB))
    out = torch.empty_like(dev["q"])
    b.orthrus_multi_block_attend(layer, dev["anchors"], dev["q"], dev["k_blk"], dev["v_blk"], out, ws)
    assert b.orthrus_read_status(ws) == 0 and b.orthrus_last_path() == "tcgen05"
    assert_close(out.cpu(), ref, torch.bfloat16)
