"""Pins of the oracle's multi-block diffusion-view attention (the mask of Eq. 6): against the
library attention over the concatenated keys with the mask built from the two viewing rules, its
single-block case against the inference-time diffusion view, and the isolation properties the
paper states (no block sees another block; no row sees the context at or after its anchor)."""
import torch
import torch.nn.functional as F

import oracle


def make_case(S=2, NB=3, K=4, Hq=4, Hkv=2, d=8, cap=24, lens=(20, 13), anchors=((5, 0, 20), (13, 7, 1)), seed=0):
    g = torch.Generator().manual_seed(seed)
    mk = lambda *s: torch.randn(*s, generator=g, dtype=torch.float64)
    return dict(q=mk(S, NB, K, Hq, d), k_blk=mk(S, NB, K, Hkv, d), v_blk=mk(S, NB, K, Hkv, d),
                k_cache=mk(S, Hkv, cap, d), v_cache=mk(S, Hkv, cap, d),
                cache_len=torch.tensor(lens, dtype=torch.int32),
                anchors=torch.tensor(anchors, dtype=torch.int32))


def run(c):
    return oracle.multi_block_attend(c["q"], c["k_blk"], c["v_blk"], c["k_cache"], c["v_cache"],
                                     c["cache_len"], c["anchors"])


def test_against_library_attention_with_the_two_viewing_rules():
    """Rule (i): a diffusion row attends to the clean positions before its block's anchor.  Rule (ii):
    it attends to every row of its own block and to no other block.  The mask is built from these
    two sentences, not from the formula, and handed to the library attention."""
    c = make_case()
    got = run(c)
    S, NB, K, Hq, d = c["q"].shape
    G = Hq // c["k_cache"].shape[1]
    for s in range(S):
        L = int(c["cache_len"][s])
        mask = torch.zeros(NB * K, L + NB * K, dtype=torch.bool)
        for j in range(NB):
            rows = slice(j * K, (j + 1) * K)
            mask[rows, :int(c["anchors"][s, j])] = True                   # rule (i)
            mask[rows, L + j * K:L + (j + 1) * K] = True                  # rule (ii)
        for hq in range(Hq):
            h = hq // G
            keys = torch.cat([c["k_cache"][s, h, :L], c["k_blk"][s, :, :, h].reshape(NB * K, d)])
            vals = torch.cat([c["v_cache"][s, h, :L], c["v_blk"][s, :, :, h].reshape(NB * K, d)])
            ref = F.scaled_dot_product_attention(c["q"][s, :, :, hq].reshape(1, NB * K, d), keys.unsqueeze(0),
                                                 vals.unsqueeze(0), attn_mask=mask.unsqueeze(0))
            assert torch.allclose(got[s, :, :, hq].reshape(NB * K, d), ref[0], atol=1e-12, rtol=1e-12)


def test_one_block_at_the_end_is_the_inference_time_diffusion_view():
    """Inference is the single-block case with the anchor at the end of the context: the prefix fully
    visible, the block bidirectional (Eq. 4)."""
    c = make_case(NB=1, anchors=((20,), (13,)))
    got = run(c)
    ref = oracle.block_attend(oracle.VIEW_DIFFUSION, c["q"][:, 0].contiguous(), c["k_blk"][:, 0].contiguous(),
                              c["v_blk"][:, 0].contiguous(), c["k_cache"], c["v_cache"], c["cache_len"])
    assert torch.allclose(got[:, 0], ref, atol=1e-13, rtol=1e-13)


def test_every_block_is_the_single_block_view_of_its_own_anchor():
    c = make_case()
    got = run(c)
    for j in range(3):
        ref = oracle.block_attend(oracle.VIEW_DIFFUSION, c["q"][:, j].contiguous(), c["k_blk"][:, j].contiguous(),
                                  c["v_blk"][:, j].contiguous(), c["k_cache"], c["v_cache"],
                                  c["anchors"][:, j].contiguous())
        assert torch.allclose(got[:, j], ref, atol=1e-13, rtol=1e-13)


def test_blocks_are_isolated_and_the_future_is_hidden():
    c = make_case()
    base = run(c)
    # another block's keys and values are invisible: overwrite block 1 with huge values
    d2 = {k: v.clone() for k, v in c.items()}
    d2["k_blk"][:, 1] = 50.0; d2["v_blk"][:, 1] = 1e6
    alt = run(d2)
    assert torch.equal(alt[:, 0], base[:, 0]) and torch.equal(alt[:, 2], base[:, 2])
    assert not torch.allclose(alt[:, 1], base[:, 1])
    # clean positions at or after a block's anchor are invisible to it (sequence 0, block 0: anchor 5)
    d3 = {k: v.clone() for k, v in c.items()}
    d3["k_cache"][0, :, 5:] = float("nan"); d3["v_cache"][0, :, 5:] = float("nan")
    alt = run(d3)
    assert torch.equal(alt[0, 0], base[0, 0])
    assert torch.isnan(alt[0, 2]).any()                 # block 2 of that sequence (anchor 20) does see them
    # an anchor at 0 leaves only the block itself: with zero queries the output is the block's mean value
    d4 = {k: v.clone() for k, v in c.items()}
    d4["q"].zero_()
    alt = run(d4)
    G = 2
    for hq in range(4):
        assert torch.allclose(alt[0, 1, :, hq], c["v_blk"][0, 1, :, hq // G].mean(0).expand(4, 8), atol=1e-13)
