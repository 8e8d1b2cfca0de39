"""GPU parity of the two block-attention calls against the CPU oracle, element by
element on small and adversarial shapes (several tiles, ragged tails, tiny prefixes,
peaked scores, planted keys at masked positions, NaN beyond the prefix)."""
import math

import pytest
import torch

import oracle
from paper_2605_12825_b200 import workloads as W
from _gpu_util import (assert_close, oracle_attend, run_attend, small_workload)

pytestmark = pytest.mark.gpu
VIEWS = [oracle.VIEW_DIFFUSION, oracle.VIEW_AR]
NAN = float("nan")
PATHS = ["simt", "mma", "tcgen05"]


def taken(path, wl):
    """The path a request resolves to: tcgen05 needs head_dim 128, mma needs 64 or 128."""
    if path == "tcgen05" and wl.head_dim != 128:
        path = "mma"
    if path == "mma" and wl.head_dim not in (64, 128):
        path = "simt"
    return path


@pytest.mark.parametrize("view", VIEWS)
@pytest.mark.parametrize("P", [0, 1, 3, 17, 63, 64, 65, 130, 257])
@pytest.mark.parametrize("path", PATHS)
def test_tiny_prefixes_bf16(view, P, path):
    wl = small_workload(2, 8, 8, 2, 64, P, P, std=0.5)
    t = W.attention_inputs(wl, fill_tail=NAN)
    got, status, used = run_attend(view, t, wl, path=path)
    assert status == 0 and used == taken(path, wl)
    assert_close(got, oracle_attend(view, t), torch.bfloat16, f"P={P}")


@pytest.mark.parametrize("view", VIEWS)
@pytest.mark.parametrize("shape", [
    # B, K, Hq, Hkv, d, pmin, pmax
    (1, 1, 4, 4, 128, 100, 100),       # block of one, no grouping
    (3, 3, 8, 1, 128, 5, 300),         # odd block, one KV head, ragged
    (2, 16, 32, 8, 128, 200, 700),     # M = 64
    (2, 32, 16, 4, 128, 64, 1000),     # M = 128
    (1, 32, 16, 2, 64, 333, 333),      # M = 256: two row tiles
    (2, 64, 2, 2, 128, 10, 90),        # widest block
    (1, 5, 6, 2, 64, 77, 77),          # M = 15, not a multiple of anything
    (1, 64, 8, 2, 128, 150, 150),      # head_dim 128, M = 256: two row tiles of 32 positions
    (2, 32, 16, 2, 128, 40, 500),      # G = 8, K = 32: M = 256, ragged
    (1, 50, 6, 2, 128, 333, 333),      # G = 3: row tiles of 42 positions (126 rows), last one short
    (1, 7, 20, 2, 128, 90, 90),        # G = 10: row tiles of 12 positions, K = 7 fits one
    (2, 64, 64, 1, 128, 20, 200),      # G = 64: two positions per row tile, 32 row tiles
])
@pytest.mark.parametrize("path", PATHS)
def test_shapes_bf16(view, shape, path):
    wl = small_workload(*shape, std=0.7)
    t = W.attention_inputs(wl, fill_tail=NAN)
    got, status, used = run_attend(view, t, wl, path=path)
    assert status == 0 and used == taken(path, wl)
    assert_close(got, oracle_attend(view, t), torch.bfloat16, str(shape))


@pytest.mark.parametrize("view", VIEWS)
@pytest.mark.parametrize("d", [32, 256])
def test_other_head_dims_take_the_simt_path(view, d):
    wl = small_workload(2, 4, 4, 2, d, 20, 150, std=0.5)
    t = W.attention_inputs(wl, fill_tail=NAN)
    got, status, used = run_attend(view, t, wl)
    assert status == 0 and used == "simt"
    assert_close(got, oracle_attend(view, t), torch.bfloat16)


@pytest.mark.parametrize("view", VIEWS)
@pytest.mark.parametrize("shape", [(2, 8, 8, 2, 64, 0, 300), (1, 16, 32, 8, 128, 515, 515),
                                   (2, 3, 4, 2, 32, 40, 41)])
def test_fp32_mode(view, shape):
    wl = small_workload(*shape, dtype="fp32", std=0.6)
    t = W.attention_inputs(wl, fill_tail=NAN)
    got, status, used = run_attend(view, t, wl)
    assert status == 0 and used == "simt"
    assert_close(got, oracle_attend(view, t), torch.float32, str(shape))


@pytest.mark.parametrize("view", VIEWS)
@pytest.mark.parametrize("splits", [1, 2, 3, 7, 12, 16])
@pytest.mark.parametrize("path", PATHS)
def test_forced_splits_agree(view, splits, path):
    """Split-KV with empty, partial and full splits (ragged batch) gives the same result."""
    wl = small_workload(3, 16, 8, 2, 128, 1, 900, std=0.7)
    t = W.attention_inputs(wl, fill_tail=NAN)
    got, status, _ = run_attend(view, t, wl, path=path, splits=splits)
    assert status == 0
    assert_close(got, oracle_attend(view, t), torch.bfloat16, f"splits={splits}")


@pytest.mark.parametrize("view", VIEWS)
@pytest.mark.parametrize("path", PATHS)
def test_peaked_scores(view, path):
    """Queries scaled x16: the softmax is dominated by a few keys, so wrong masks or
    a wrong running max show up at full magnitude."""
    wl = small_workload(2, 16, 8, 2, 128, 100, 600, std=1.0 / math.sqrt(128) * 4)
    t = W.attention_inputs(wl, q_gain=16.0, fill_tail=NAN)
    got, status, _ = run_attend(view, t, wl, path=path, splits=3)
    assert status == 0
    assert_close(got, oracle_attend(view, t), torch.bfloat16)


@pytest.mark.parametrize("path", PATHS)
def test_planted_key_hidden_by_the_causal_rule(path):
    """A block key with an overwhelming score: every diffusion row collapses onto its
    value row, AR rows before it must not see it at all."""
    wl = small_workload(1, 8, 4, 1, 64, 50, 50, std=0.3)
    t = W.attention_inputs(wl, fill_tail=NAN)
    i_star = 5
    for name in ("q_diff", "q_ar"):
        t[name][..., 0] = 1.0
    for name in ("k_diff_blk", "k_ar_blk"):
        t[name][0, i_star, 0, :] = 0
        t[name][0, i_star, 0, 0] = 400.0
    for view in VIEWS:
        got, status, _ = run_attend(view, t, wl, path=path)
        ref = oracle_attend(view, t)
        assert_close(got, ref, torch.bfloat16)
        vb = t["v_diff_blk"] if view == oracle.VIEW_DIFFUSION else t["v_ar_blk"]
        target = vb[0, i_star, 0].double()
        for i in range(8):
            d_i = float((got[0, i, 0].double() - target).abs().max())
            if view == oracle.VIEW_DIFFUSION or i >= i_star:
                assert d_i < 1e-2
            else:
                assert d_i > 5e-2


@pytest.mark.parametrize("view", VIEWS)
def test_position_coded_values(view):
    """V[:, 0] holds the key's position: O[0] is the expected attended position, which
    exposes any off-by-one in which keys are visible."""
    wl = small_workload(1, 8, 4, 2, 64, 40, 40, dtype="fp32", std=0.2)
    t = W.attention_inputs(wl)
    P, K = 40, 8
    t["q_diff"].zero_(); t["q_ar"].zero_()
    t["v_cache"][0, :, :, 0] = torch.arange(wl.capacity, dtype=torch.float32)
    for n in ("v_diff_blk", "v_ar_blk"):
        t[n][0, :, :, 0] = torch.arange(P, P + K, dtype=torch.float32).view(K, 1)
    got, _, _ = run_attend(view, t, wl)
    for i in range(K):
        last = P + K - 1 if view == oracle.VIEW_DIFFUSION else P + i
        assert abs(float(got[0, i, 0, 0]) - last / 2.0) < 1e-4


def test_bad_cache_len_is_clamped_and_flagged():
    wl = small_workload(2, 4, 4, 2, 64, 30, 30, std=0.5)
    t = W.attention_inputs(wl)
    t["cache_len"][1] = wl.capacity            # beyond capacity - K
    got, status, _ = run_attend(oracle.VIEW_AR, t, wl, max_len_hint=wl.capacity - wl.block)
    assert status & 1
    t["cache_len"][1] = wl.capacity - wl.block
    assert_close(got, oracle_attend(oracle.VIEW_AR, t), torch.bfloat16)
    assert torch.isfinite(got.float()).all()
