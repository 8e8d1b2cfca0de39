"""GPU parity of the multi-block diffusion-view attention (the mask of Eq. 6) against the oracle, on
all three kernel paths: several anchors per sequence over one shared clean cache, anchors at 0 and
at the end, NaN planted where no row may look."""
import os

import pytest
import torch

import oracle
from _gpu_util import Guarded, assert_close, binding

pytestmark = pytest.mark.gpu
NAN = float("nan")


def make_case(S, NB, K, Hq, Hkv, d, L_max, dtype, seed, std=0.7):
    g = torch.Generator().manual_seed(seed)
    mk = lambda *s: (torch.randn(*s, generator=g) * std).to(dtype)
    cap = (L_max + K + 63) // 64 * 64
    lens = torch.randint(max(1, L_max // 2), L_max + 1, (S,), generator=g, dtype=torch.int64).to(torch.int32)
    anchors = torch.stack([torch.randint(0, int(lens[s]) + 1, (NB,), generator=g) for s in range(S)]).to(torch.int32)
    anchors[0, 0] = 0                       # a block that sees only itself
    anchors[-1, -1] = int(lens[-1])         # a block behind the whole context (the inference case)
    c = dict(q=mk(S, NB, K, Hq, d), k_blk=mk(S, NB, K, Hkv, d), v_blk=mk(S, NB, K, Hkv, d),
             k_cache=mk(S, Hkv, cap, d), v_cache=mk(S, Hkv, cap, d), cache_len=lens, anchors=anchors)
    for s in range(S):                      # nothing at or beyond the clean length is ever visible
        c["k_cache"][s, :, int(lens[s]):] = NAN
        c["v_cache"][s, :, int(lens[s]):] = NAN
    return c


@pytest.mark.parametrize("path,shape", [
    ("simt", (2, 3, 4, 4, 2, 32, 90)), ("simt", (1, 5, 8, 8, 2, 128, 200)),
    ("mma", (2, 3, 8, 8, 2, 64, 300)), ("mma", (2, 4, 16, 8, 2, 128, 500)),
    ("tcgen05", (2, 4, 16, 8, 2, 128, 700)),        # M = 64
    ("tcgen05", (1, 6, 32, 16, 4, 128, 1000)),      # M = 128
    ("tcgen05", (3, 2, 8, 32, 8, 128, 4096)),       # the 8B head layout, block 8
])
@pytest.mark.parametrize("splits", [0, 4])
def test_multi_block_attention_matches_the_oracle(path, shape, splits):
    b = binding()
    S, NB, K, Hq, Hkv, d, L_max = shape
    dtype = torch.bfloat16
    c = make_case(S, NB, K, Hq, Hkv, d, L_max, dtype, seed=sum(shape))
    ref = oracle.multi_block_attend(c["q"], c["k_blk"], c["v_blk"], c["k_cache"], c["v_cache"], c["cache_len"],
                                    c["anchors"])
    dev = {k: v.cuda() for k, v in c.items()}
    layer = b.make_layer(dev["k_cache"], dev["v_cache"], dev["cache_len"], Hq, K, int(c["anchors"].max()))
    old = os.environ.pop("ORTHRUS_SPLITS", None)
    if splits:
        os.environ["ORTHRUS_SPLITS"] = str(splits)
    try:
        b.orthrus_set_path(path)
        ws = b.new_workspace(b.orthrus_multi_block_workspace_bytes(layer, NB))
        out = Guarded(tuple(c["q"].shape), dtype)
        b.orthrus_multi_block_attend(layer, dev["anchors"], dev["q"], dev["k_blk"], dev["v_blk"], out.t, ws)
        assert b.orthrus_last_path() == path
        assert b.orthrus_read_status(ws) == 0
    finally:
        b.orthrus_set_path("auto")
        os.environ.pop("ORTHRUS_SPLITS", None)
        if old is not None:
            os.environ["ORTHRUS_SPLITS"] = old
    assert out.intact()
    assert_close(out.t.cpu(), ref, dtype, str(shape))


# Shapes of the tcgen05 path whose blocks share query tiles: (S, NB, K, Hq, Hkv, d, L_max)
PACKED_SHAPES = [
    (2, 12, 8, 8, 2, 128, 900),     # 3 query tiles of 4 blocks; the third reads tile 1 of the block axis
    (1, 5, 24, 4, 2, 128, 700),     # blocks straddle query tiles and 64-key tiles of the block axis
    (2, 7, 16, 2, 2, 128, 500),     # one head per group: 128 positions per query tile, ragged last tile
    (1, 16, 4, 16, 2, 128, 2500),   # 4-wide blocks, 8 heads per group: 4 blocks per tile
    (3, 2, 32, 2, 1, 128, 300),     # two blocks fill a tile exactly
]


@pytest.mark.parametrize("shape", PACKED_SHAPES)
@pytest.mark.parametrize("splits", [0, 1, 4])
@pytest.mark.parametrize("anchor_mode", ["random", "sorted", "zero"])
def test_multi_block_packed_query_tiles(shape, splits, anchor_mode):
    """Blocks that share a 128-row query tile: per-row prefix limits, block-diagonal block keys, block
    keys spread over several 64-key tiles, clusters with more CTAs than tiles (all anchors 0)."""
    b = binding()
    S, NB, K, Hq, Hkv, d, L_max = shape
    dtype = torch.bfloat16
    c = make_case(S, NB, K, Hq, Hkv, d, L_max, dtype, seed=sum(shape) + 1)
    if anchor_mode == "sorted":
        c["anchors"] = c["anchors"].sort(dim=1).values.contiguous()
    elif anchor_mode == "zero":
        c["anchors"].zero_()
    ref = oracle.multi_block_attend(c["q"], c["k_blk"], c["v_blk"], c["k_cache"], c["v_cache"], c["cache_len"],
                                    c["anchors"])
    dev = {k: v.cuda() for k, v in c.items()}
    # (with every anchor at 0 the bound stays at L_max: clusters larger than the tile count)
    hint = L_max if anchor_mode == "zero" else int(c["anchors"].max())
    layer = b.make_layer(dev["k_cache"], dev["v_cache"], dev["cache_len"], Hq, K, hint)
    outs = {}
    saved = {k: os.environ.pop(k, None) for k in ("ORTHRUS_SPLITS", "ORTHRUS_MULTI_BLOCK_PACK")}
    try:
        if splits:
            os.environ["ORTHRUS_SPLITS"] = str(splits)
        for pack in ("1", "0"):
            os.environ["ORTHRUS_MULTI_BLOCK_PACK"] = pack
            ws = b.new_workspace(b.orthrus_multi_block_workspace_bytes(layer, NB))
            out = Guarded(tuple(c["q"].shape), dtype)
            b.orthrus_multi_block_attend(layer, dev["anchors"], dev["q"], dev["k_blk"], dev["v_blk"], out.t, ws)
            assert b.orthrus_last_path() == "tcgen05"
            assert b.orthrus_read_status(ws) == 0
            assert out.intact()
            outs[pack] = out.t.cpu()
    finally:
        for k, v in saved.items():
            os.environ.pop(k, None)
            if v is not None:
                os.environ[k] = v
    assert_close(outs["1"], ref, dtype, f"packed {shape}")
    assert_close(outs["0"], ref, dtype, f"one unit per block {shape}")


def test_multi_block_fp32_mode_and_single_block_case():
    """fp32 test mode at 1e-5; and one block per sequence anchored at the clean length gives the very
    bytes orthrus_diffusion_block_attend gives (the same launch on the same data)."""
    b = binding()
    c = make_case(2, 3, 8, 8, 2, 64, 150, torch.float32, seed=5)
    ref = oracle.multi_block_attend(c["q"], c["k_blk"], c["v_blk"], c["k_cache"], c["v_cache"], c["cache_len"],
                                    c["anchors"])
    dev = {k: v.cuda() for k, v in c.items()}
    layer = b.make_layer(dev["k_cache"], dev["v_cache"], dev["cache_len"], 8, 8, int(c["anchors"].max()))
    ws = b.new_workspace(b.orthrus_multi_block_workspace_bytes(layer, 3))
    out = torch.empty_like(dev["q"])
    b.orthrus_multi_block_attend(layer, dev["anchors"], dev["q"], dev["k_blk"], dev["v_blk"], out, ws)
    assert_close(out.cpu(), ref, torch.float32)

    c1 = make_case(2, 1, 16, 8, 2, 128, 400, torch.bfloat16, seed=6)
    c1["anchors"] = c1["cache_len"].view(2, 1).clone()
    d1 = {k: v.cuda() for k, v in c1.items()}
    layer = b.make_layer(d1["k_cache"], d1["v_cache"], d1["cache_len"], 8, 16, int(c1["cache_len"].max()))
    ws = b.new_workspace(b.orthrus_multi_block_workspace_bytes(layer, 1))
    multi = torch.empty_like(d1["q"])
    b.orthrus_multi_block_attend(layer, d1["anchors"], d1["q"], d1["k_blk"], d1["v_blk"], multi, ws)
    single = torch.empty_like(d1["q"][:, 0])
    b.orthrus_diffusion_block_attend(layer, d1["q"][:, 0].contiguous(), d1["k_blk"][:, 0].contiguous(),
                                     d1["v_blk"][:, 0].contiguous(), single, ws)
    assert torch.equal(multi[:, 0].view(torch.int16), single.view(torch.int16))


def test_multi_block_bad_anchor_is_clamped_and_flagged():
    b = binding()
    c = make_case(1, 2, 8, 8, 2, 128, 100, torch.bfloat16, seed=8)
    cap = c["k_cache"].shape[2]
    c["k_cache"].nan_to_num_(0.0); c["v_cache"].nan_to_num_(0.0)
    c["anchors"][0, 1] = cap + 7
    dev = {k: v.cuda() for k, v in c.items()}
    layer = b.make_layer(dev["k_cache"], dev["v_cache"], dev["cache_len"], 8, 8)
    ws = b.new_workspace(b.orthrus_multi_block_workspace_bytes(layer, 2))
    out = torch.empty_like(dev["q"])
    b.orthrus_multi_block_attend(layer, dev["anchors"], dev["q"], dev["k_blk"], dev["v_blk"], out, ws)
    assert b.orthrus_read_status(ws) & b.DEV_BAD_CACHE_LEN
    assert torch.isfinite(out.float()).all()
