"""Pins of the oracle's write-then-truncate commit, of block attention with the block's K/V
rows taken from the cache, and of the rotary embedding of a block.  None of them retypes
the oracle's formula: the attention is checked against the library attention over one
concatenated key sequence with an explicit mask, the two-step commit against the append byte
for byte, the rotation against the transformers library's rotary embedding and against the
properties that define it."""
import math

import pytest
import torch
import torch.nn.functional as F

import oracle

VIEWS = [oracle.VIEW_DIFFUSION, oracle.VIEW_AR]


def make_case(B=2, K=5, Hq=4, Hkv=2, d=16, cap=40, lens=(7, 19), seed=0, dtype=torch.float64):
    g = torch.Generator().manual_seed(seed)
    mk = lambda *s: torch.randn(*s, generator=g, dtype=torch.float64).to(dtype)
    return dict(q=mk(B, K, Hq, d), k_blk=mk(B, K, Hkv, d), v_blk=mk(B, K, Hkv, d),
                k_cache=mk(B, Hkv, cap, d), v_cache=mk(B, Hkv, cap, d),
                cache_len=torch.tensor(lens, dtype=torch.int32))


@pytest.mark.parametrize("view", VIEWS)
def test_in_cache_block_equals_library_attention_over_one_key_sequence(view):
    """With the block rows at cache positions [P, P+K), both views are ordinary attention of
    query position P+i over keys 0..P+K-1 under a mask: everything (diffusion view) or j <= P+i
    (AR view).  Rows beyond P+K hold NaN and must never be read."""
    c = make_case()
    B, K, Hq, d = c["q"].shape
    Hkv = c["k_cache"].shape[1]
    G = Hq // Hkv
    oracle.block_kv_write(c["k_cache"], c["v_cache"], c["cache_len"], c["k_blk"], c["v_blk"])
    for b in range(B):
        P = int(c["cache_len"][b])
        c["k_cache"][b, :, P + K:] = float("nan")
        c["v_cache"][b, :, P + K:] = float("nan")
    got = oracle.block_attend(view, c["q"], None, None, c["k_cache"], c["v_cache"], c["cache_len"])
    assert torch.isfinite(got).all()
    for b in range(B):
        P = int(c["cache_len"][b])
        n = P + K
        j = torch.arange(n).view(1, n)
        i = torch.arange(K).view(K, 1)
        mask = (j <= P + i) if view == oracle.VIEW_AR else torch.ones(K, n, dtype=torch.bool)
        for hq in range(Hq):
            h = hq // G
            ref = F.scaled_dot_product_attention(c["q"][b, :, hq].unsqueeze(0), c["k_cache"][b, h, :n].unsqueeze(0),
                                                 c["v_cache"][b, h, :n].unsqueeze(0), attn_mask=mask.unsqueeze(0))
            assert torch.allclose(got[b, :, hq], ref[0], atol=1e-12, rtol=1e-12)


@pytest.mark.parametrize("view", VIEWS)
def test_in_cache_block_equals_block_tensors_holding_the_same_rows(view):
    c = make_case(seed=3)
    with_blk = oracle.block_attend(view, c["q"], c["k_blk"], c["v_blk"], c["k_cache"], c["v_cache"], c["cache_len"])
    oracle.block_kv_write(c["k_cache"], c["v_cache"], c["cache_len"], c["k_blk"], c["v_blk"])
    in_cache = oracle.block_attend(view, c["q"], None, None, c["k_cache"], c["v_cache"], c["cache_len"])
    assert torch.equal(with_blk, in_cache)
    rows = torch.tensor([[0, 0, 0], [1, 4, 3], [1, 2, 1]], dtype=torch.int32)
    some = oracle.block_attend_rows(view, rows, c["q"], None, None, c["k_cache"], c["v_cache"], c["cache_len"])
    assert torch.equal(some, in_cache[rows[:, 0].long(), rows[:, 1].long(), rows[:, 2].long()])


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_write_then_length_bump_leaves_what_the_append_leaves(dtype):
    """Write all K rows (the diffusion view's first, then the AR view's over them), then grow
    the length by n: rows below the new length and the length itself are those of the append;
    the rows between the new length and P+K hold the unconfirmed AR rows; nothing beyond."""
    c = make_case(dtype=dtype, seed=5)
    diff = make_case(dtype=dtype, seed=6)
    n = torch.tensor([2, 5], dtype=torch.int32)
    a = {k: v.clone() for k, v in c.items()}
    assert oracle.kv_append(a["k_cache"], a["v_cache"], a["cache_len"], a["k_blk"], a["v_blk"], n) == 0
    w = {k: v.clone() for k, v in c.items()}
    assert oracle.block_kv_write(w["k_cache"], w["v_cache"], w["cache_len"], diff["k_blk"], diff["v_blk"]) == 0
    assert torch.equal(w["cache_len"], c["cache_len"])
    assert oracle.block_kv_write(w["k_cache"], w["v_cache"], w["cache_len"], w["k_blk"], w["v_blk"]) == 0
    assert oracle.commit_len(w["cache_len"], n, 5, 40) == 0
    assert torch.equal(w["cache_len"], a["cache_len"])
    bits = lambda x: x.view(torch.int16 if dtype == torch.bfloat16 else torch.int32)
    for b in range(2):
        P, new = int(c["cache_len"][b]), int(a["cache_len"][b])
        for name, blk in (("k_cache", "k_blk"), ("v_cache", "v_blk")):
            assert torch.equal(bits(w[name][b, :, :new]), bits(a[name][b, :, :new]))
            assert torch.equal(bits(w[name][b, :, new:P + 5]), bits(c[blk][b, new - P:].transpose(0, 1).contiguous()))
            assert torch.equal(bits(w[name][b, :, P + 5:]), bits(c[name][b, :, P + 5:]))


def test_write_and_bump_refuse_what_does_not_fit():
    c = make_case(lens=(7, 36))                  # 36 + 5 > 40
    before = c["k_cache"].clone()
    assert oracle.block_kv_write(c["k_cache"], c["v_cache"], c["cache_len"], c["k_blk"], c["v_blk"]) == -3
    assert torch.equal(c["k_cache"][1], before[1]) and not torch.equal(c["k_cache"][0], before[0])
    lens = torch.tensor([7, 36], dtype=torch.int32)
    assert oracle.commit_len(lens, torch.tensor([6, 4], dtype=torch.int32), 5, 40) == -3   # 6 > K
    assert lens.tolist() == [7, 40]
    assert oracle.commit_len(lens, torch.tensor([1, 1], dtype=torch.int32), 5, 40) == -3   # 40 + 1 > 40
    assert lens.tolist() == [8, 40]


# ------------------------------------------------------------------------------ rotary embedding

def test_rotation_matches_the_transformers_library():
    from transformers import LlamaConfig
    from transformers.models.llama import modeling_llama as m
    B, K, H, d, theta = 2, 6, 3, 32, 50000.0
    g = torch.Generator().manual_seed(2)
    x = torch.randn(B, K, H, d, generator=g, dtype=torch.float64)
    lens = torch.tensor([3, 41], dtype=torch.int32)
    got = oracle.rope_block(x, lens, theta)
    cfg = LlamaConfig(hidden_size=H * d, num_attention_heads=H, num_key_value_heads=H, head_dim=d, rope_theta=theta)
    rot = m.LlamaRotaryEmbedding(cfg)
    pos = lens.long().view(B, 1) + torch.arange(K).view(1, K)
    cos, sin = rot(x, pos)                                        # [B][K][d], fp32 angles
    ref, _ = m.apply_rotary_pos_emb(x, x, cos.double(), sin.double(), unsqueeze_dim=2)
    assert float((got - ref).abs().max()) < 2e-5                  # the library's angles are fp32


def test_rotation_properties():
    B, K, H, d = 1, 9, 2, 16
    g = torch.Generator().manual_seed(4)
    q = torch.randn(B, K, H, d, generator=g, dtype=torch.float64)
    k = torch.randn(B, K, H, d, generator=g, dtype=torch.float64)
    zero = torch.zeros(1, dtype=torch.int32)
    rq = oracle.rope_block(q, zero)
    assert torch.allclose(rq[:, 0], q[:, 0], atol=1e-15)          # position 0 is the identity
    half = d // 2
    n_in = q[..., :half] ** 2 + q[..., half:] ** 2                # every (c, c + d/2) pair keeps its norm
    n_out = rq[..., :half] ** 2 + rq[..., half:] ** 2
    assert torch.allclose(n_in, n_out, atol=1e-12)
    # scores depend on the distance of the two positions only: the same vectors 100 positions on
    a = oracle.rope_block(q, torch.tensor([0], dtype=torch.int32))
    b_ = oracle.rope_block(k, torch.tensor([0], dtype=torch.int32))
    a2 = oracle.rope_block(q, torch.tensor([100], dtype=torch.int32))
    b2 = oracle.rope_block(k, torch.tensor([100], dtype=torch.int32))
    s1 = torch.einsum("bihd,bjhd->bhij", a, b_)
    s2 = torch.einsum("bihd,bjhd->bhij", a2, b2)
    assert torch.allclose(s1, s2, atol=1e-9)
    # the slowest pair turns by pos * theta^(-(d-2)/d): one closed-form angle
    x = torch.zeros(1, 1, 1, d, dtype=torch.float64); x[..., half - 1] = 1.0
    y = oracle.rope_block(x, torch.tensor([7], dtype=torch.int32), theta=10000.0)
    ang = 7 * 10000.0 ** (-(d - 2) / d)
    assert abs(float(y[0, 0, 0, half - 1]) - math.cos(ang)) < 1e-12
    assert abs(float(y[0, 0, 0, d - 1]) - math.sin(ang)) < 1e-12


def test_rotation_of_bf16_input_widens_exactly():
    x = torch.randn(1, 2, 1, 8, generator=torch.Generator().manual_seed(1)).to(torch.bfloat16)
    lens = torch.tensor([5], dtype=torch.int32)
    assert torch.equal(oracle.rope_block(x, lens), oracle.rope_block(x.double(), lens))
