"""GPU parity of the write-then-truncate commit (Section 3.3, last paragraph) against the oracle:
the block write and the length bump byte for byte, block attention with the block's K/V rows
read from the cache on all three kernel paths, the rotary embedding fused with the write, and
the generation loop run end to end on these calls."""
import pytest
import torch

import oracle
from paper_2605_12825_b200 import workloads as W
from _gpu_util import Guarded, assert_close, binding, small_workload

pytestmark = pytest.mark.gpu
VIEWS = [oracle.VIEW_DIFFUSION, oracle.VIEW_AR]
NAN = float("nan")


def bits(x):
    return x.view(torch.int16 if x.dtype == torch.bfloat16 else torch.int32)


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_block_write_and_length_bump_bit_exact(dtype):
    b = binding()
    wl = small_workload(3, 8, 8, 2, 64, 5, 40, dtype=dtype, name=f"bw_{dtype}")
    t = W.attention_inputs(wl)
    n = torch.tensor([1, 8, 4], dtype=torch.int32)
    ref = {k: v.clone() for k, v in t.items()}
    assert oracle.block_kv_write(ref["k_cache"], ref["v_cache"], ref["cache_len"], ref["k_diff_blk"], ref["v_diff_blk"]) == 0
    assert oracle.block_kv_write(ref["k_cache"], ref["v_cache"], ref["cache_len"], ref["k_ar_blk"], ref["v_ar_blk"]) == 0
    d = {k: v.cuda() for k, v in t.items()}
    layer = b.make_layer(d["k_cache"], d["v_cache"], d["cache_len"], wl.n_q_heads, wl.block)
    ws = b.new_workspace(256)
    b.orthrus_block_kv_write(layer, d["k_diff_blk"], d["v_diff_blk"], ws)
    b.orthrus_block_kv_write(layer, d["k_ar_blk"], d["v_ar_blk"], ws)
    assert torch.equal(d["cache_len"].cpu(), t["cache_len"])              # the write moves no length
    assert torch.equal(bits(d["k_cache"].cpu()), bits(ref["k_cache"]))
    assert torch.equal(bits(d["v_cache"].cpu()), bits(ref["v_cache"]))
    assert oracle.commit_len(ref["cache_len"], n, wl.block, wl.capacity) == 0
    b.orthrus_commit_len(layer, n.cuda(), ws)
    assert torch.equal(d["cache_len"].cpu(), ref["cache_len"])
    assert b.orthrus_read_status(ws) == 0
    # the append of the same rows leaves the same live rows and the same lengths
    app = {k: v.clone() for k, v in t.items()}
    oracle.kv_append(app["k_cache"], app["v_cache"], app["cache_len"], app["k_ar_blk"], app["v_ar_blk"], n)
    assert torch.equal(app["cache_len"], ref["cache_len"])
    for s in range(3):
        L = int(app["cache_len"][s])
        assert torch.equal(bits(d["k_cache"].cpu()[s, :, :L]), bits(app["k_cache"][s, :, :L]))


def test_write_and_bump_skip_and_flag_what_does_not_fit():
    b = binding()
    wl = small_workload(2, 8, 4, 2, 64, 20, 20, name="bw_over")
    t = W.attention_inputs(wl)
    cap = wl.capacity
    t["cache_len"][1] = cap - 3                                          # no room for 8 rows
    d = {k: v.cuda() for k, v in t.items()}
    before = d["k_cache"].clone()
    layer = b.make_layer(d["k_cache"], d["v_cache"], d["cache_len"], wl.n_q_heads, wl.block)
    ws = b.new_workspace(256)
    b.orthrus_block_kv_write(layer, d["k_ar_blk"], d["v_ar_blk"], ws)
    assert b.orthrus_read_status(ws) & b.DEV_APPEND_OVERFLOW
    assert torch.equal(d["k_cache"][1], before[1]) and not torch.equal(d["k_cache"][0], before[0])
    b.orthrus_workspace_init(ws)
    b.orthrus_commit_len(layer, torch.tensor([9, 2], dtype=torch.int32).cuda(), ws)   # 9 > K
    assert b.orthrus_read_status(ws) & b.DEV_APPEND_OVERFLOW
    assert d["cache_len"].cpu().tolist() == [20, cap - 1]


@pytest.mark.parametrize("view", VIEWS)
@pytest.mark.parametrize("path,shape", [
    ("simt", (2, 8, 8, 2, 32, 0, 130)), ("simt", (2, 5, 4, 2, 128, 3, 70)),
    ("mma", (2, 8, 8, 2, 64, 0, 300)), ("mma", (3, 16, 8, 2, 128, 1, 500)),
    ("tcgen05", (3, 16, 8, 2, 128, 0, 700)),       # M = 64, ragged, one empty prefix
    ("tcgen05", (2, 32, 16, 4, 128, 64, 1000)),    # M = 128
    ("tcgen05", (1, 64, 8, 2, 128, 150, 150)),     # two row tiles
    ("tcgen05", (2, 3, 4, 4, 128, 63, 65)),        # tiny block straddling a tile edge
])
@pytest.mark.parametrize("splits", [0, 3])
def test_attention_with_the_block_in_the_cache(view, path, shape, splits):
    """The block's rows sit at cache rows [P, P+K); everything behind them is NaN.  The result must
    equal the oracle's (which reads the same cache) under the parity tolerance."""
    import os
    b = binding()
    wl = small_workload(*shape, std=0.7, name=f"incache_{path}_{shape}")
    t = W.attention_inputs(wl, fill_tail=NAN)
    kb, vb = ("k_diff_blk", "v_diff_blk") if view == oracle.VIEW_DIFFUSION else ("k_ar_blk", "v_ar_blk")
    q = t["q_diff"] if view == oracle.VIEW_DIFFUSION else t["q_ar"]
    oracle.block_kv_write(t["k_cache"], t["v_cache"], t["cache_len"], t[kb], t[vb])
    ref = oracle.block_attend(view, q, None, None, t["k_cache"], t["v_cache"], t["cache_len"])
    d = {k: v.cuda() for k, v in t.items()}
    layer = b.make_layer(d["k_cache"], d["v_cache"], d["cache_len"], wl.n_q_heads, wl.block,
                         int(t["cache_len"].max()), 0.0, b.LAYER_BLOCK_IN_CACHE | b.LAYER_CACHE_QUIESCENT)
    old = os.environ.pop("ORTHRUS_SPLITS", None)
    if splits:
        os.environ["ORTHRUS_SPLITS"] = str(splits)
    try:
        b.orthrus_set_path(path)
        ws = b.new_workspace(b.orthrus_attend_workspace_bytes(layer))
        out = Guarded(tuple(q.shape), q.dtype)
        fn = b.orthrus_diffusion_block_attend if view == oracle.VIEW_DIFFUSION else b.orthrus_ar_verify_attend
        fn(layer, q.cuda(), None, None, out.t, ws)
        assert b.orthrus_last_path() == path
        assert b.orthrus_read_status(ws) == 0
    finally:
        b.orthrus_set_path("auto")
        os.environ.pop("ORTHRUS_SPLITS", None)
        if old is not None:
            os.environ["ORTHRUS_SPLITS"] = old
    assert out.intact()
    assert_close(out.t.cpu(), ref, torch.bfloat16, str(shape))


@pytest.mark.parametrize("dtype,theta", [("bf16", 10000.0), ("bf16", 1000000.0), ("fp32", 10000.0)])
@pytest.mark.parametrize("lens", [(0, 77), (4000, 32000)])
def test_rotary_embedding_fused_with_the_block_write(dtype, theta, lens):
    """Rotated queries, rotated keys in the cache and copied values against the oracle's fp64
    rotation rounded once: at most one unit in the last place of the output type apart (the kernel
    rounds a double through float); values bit-exact; nothing else in the cache touched."""
    b = binding()
    wl = small_workload(2, 16, 8, 2, 128, 1, 1, dtype=dtype, std=1.0, name=f"rope_{dtype}_{lens}")
    t = W.attention_inputs(wl)
    cap = lens[1] + 64
    dt = t["q_ar"].dtype
    g = torch.Generator().manual_seed(9)
    kc = torch.randn(2, 2, cap, 128, generator=g).to(dt)
    vc = torch.randn(2, 2, cap, 128, generator=g).to(dt)
    cl = torch.tensor(lens, dtype=torch.int32)
    d_kc, d_vc, d_cl = kc.cuda(), vc.cuda(), cl.cuda()
    layer = b.make_layer(d_kc, d_vc, d_cl, wl.n_q_heads, wl.block)
    q_out = Guarded(tuple(t["q_ar"].shape), dt)
    ws = b.new_workspace(256)
    b.orthrus_rope_block_kv_write(layer, t["q_ar"].cuda(), t["k_ar_blk"].cuda(), t["v_ar_blk"].cuda(), theta,
                                  q_out.t, ws)
    assert b.orthrus_read_status(ws) == 0 and q_out.intact()
    rq = oracle.rope_block(t["q_ar"], cl, theta)
    rk = oracle.rope_block(t["k_ar_blk"], cl, theta)
    ulp = 2.0 ** -8 if dtype == "bf16" else 2.0 ** -23          # relative spacing of the type

    def close(got, ref):
        return bool(((got.double() - ref).abs() <= ulp * ref.abs().clamp(min=2.0 ** -20)).all())

    assert close(q_out.t.cpu(), rq)
    got_k, got_v = d_kc.cpu(), d_vc.cpu()
    for s in range(2):
        P = lens[s]
        assert close(got_k[s, :, P:P + 16].transpose(0, 1), rk[s])
        assert torch.equal(bits(got_v[s, :, P:P + 16].transpose(0, 1).contiguous()), bits(t["v_ar_blk"][s]))
        for got, orig in ((got_k, kc), (got_v, vc)):
            assert torch.equal(bits(got[s, :, :P]), bits(orig[s, :, :P]))
            assert torch.equal(bits(got[s, :, P + 16:]), bits(orig[s, :, P + 16:]))
    assert torch.equal(d_cl.cpu(), cl)
    # in place on the queries
    q2 = t["q_ar"].cuda().clone()
    b.orthrus_rope_block_kv_write(layer, q2, t["k_ar_blk"].cuda(), t["v_ar_blk"].cuda(), theta, q2, ws)
    assert torch.equal(bits(q2.cpu()), bits(q_out.t.cpu()))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_generation_loop_on_the_truncate_commit(dtype):
    """The loop of Section 3.3 with every block written behind the prefix by the fused rotary write,
    attention reading the block from the cache, and the commit a length bump: lossless against
    width-1 greedy decoding through the same calls (re-synchronised every cycle), consensus bit-exact
    against the oracle on the GPU's logits, cache length grows by n."""
    from harness.decoder import Decoder, ForcedDraftLoop
    b = binding()
    b.orthrus_set_path("auto")
    if dtype == torch.float32:
        layers, hidden, n_q, n_kv, d, ffn, vocab, B, T, K, n_new, eps = 2, 128, 4, 2, 32, 256, 500, 3, 40, 8, 40, 1e-4
    else:
        layers, hidden, n_q, n_kv, d, ffn, vocab, B, T, K, n_new, eps = 3, 512, 8, 2, 128, 1024, 2000, 4, 300, 16, 48, 0.25
    cap = T + 2 * n_new + 4 * K + 8
    g = torch.Generator().manual_seed(11)
    prompt = torch.randint(0, vocab, (B, T), generator=g).cuda()
    dec = Decoder(b, layers, hidden, n_q, n_kv, d, ffn, vocab, dtype, B, cap, K, seed=3,
                  flags=b.LAYER_CACHE_QUIESCENT, commit_mode="truncate")
    anchor = dec.prefill(prompt)
    loop = ForcedDraftLoop(dec, anchor, 0.65, seed=5, fused=False)
    cycles, total, ties = 0, 0, 0
    while int(loop.done.min()) < n_new:
        loop.lookahead(want_gap=True)
        loop.force_drafts()
        len_before = dec.cache_len.cpu().clone()
        loop.cycle()
        rn, rcom, rarg, rnxt = oracle.consensus_accept(loop.logits.cpu(), loop.draft.cpu())
        assert torch.equal(dec.n_commit.cpu(), rn) and torch.equal(dec.committed.cpu(), rcom)
        assert torch.equal(dec.next_anchor.cpu(), rnxt)
        assert torch.equal(dec.cache_len.cpu(), len_before + rn)
        look, gaps = loop.look.cpu(), loop.gaps.cpu()
        for s in range(B):
            for i in range(int(rn[s])):
                if int(rcom[s, i]) != int(look[s, i]):
                    assert float(gaps[s, i]) < eps, (s, i, float(gaps[s, i]))
                    ties += 1
                    break
        total += int(rn.sum()); cycles += 1
        assert cycles <= 4 * n_new
    assert loop.status() == 0
    if dtype == torch.float32:
        assert ties == 0
    assert 1.5 < total / (cycles * B) < 4.5
    if dtype == torch.bfloat16:
        assert b.orthrus_last_path() == "tcgen05"
