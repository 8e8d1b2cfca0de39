"""Parity at the benchmark's full sizes, in the launch configuration bench.py times
(kernel path "auto", layers marked cache-quiescent, max_len_hint = longest prefix):
attention on sampled query rows the oracle computes one by one, plus finiteness of
every output; consensus and commit in full (they are cheap for the oracle)."""
import pytest
import torch

import oracle
from paper_2605_12825_b200 import workloads as W
from _gpu_util import TOL, binding, oracle_attend_rows

pytestmark = pytest.mark.gpu
N_SAMPLES = 96


def sample_rows(wl, lens, seed):
    g = torch.Generator().manual_seed(seed)
    B, K, Hq = wl.batch, wl.block, wl.n_q_heads
    flat = torch.randperm(B * K * Hq, generator=g)[:N_SAMPLES]
    rows = torch.stack([flat // (K * Hq), (flat // Hq) % K, flat % Hq], dim=1).to(torch.int32)
    # always include the first and last block position of the longest and shortest sequence
    lo, hi = int(lens.argmin()), int(lens.argmax())
    extra = torch.tensor([[lo, 0, 0], [lo, K - 1, Hq - 1], [hi, 0, Hq - 1], [hi, K - 1, 0]],
                         dtype=torch.int32)
    return torch.cat([rows, extra])


@pytest.mark.parametrize("name,layer", [("cfg1_tiny", 0), ("cfg2_8b_b1", 0), ("cfg2_8b_b1", 35),
                                        ("cfg3_ragged", 0), ("cfg4_long", 0), ("cfg5_loop", 3)])
def test_attention_at_bench_size(name, layer):
    b = binding()
    wl = W.CONFIGS[name]
    t = W.attention_inputs(wl, layer=layer)
    d = {k: v.cuda() for k, v in t.items()}
    lyr = b.make_layer(d["k_cache"], d["v_cache"], d["cache_len"], wl.n_q_heads, wl.block,
                       int(t["cache_len"].max()), 0.0, b.LAYER_CACHE_QUIESCENT)
    ws = b.new_workspace(b.orthrus_attend_workspace_bytes(lyr))
    out_d = torch.empty_like(d["q_diff"])
    out_a = torch.empty_like(d["q_ar"])
    b.orthrus_set_path("auto")
    # back to back, as in the benchmark's step
    b.orthrus_diffusion_block_attend(lyr, d["q_diff"], d["k_diff_blk"], d["v_diff_blk"], out_d, ws)
    b.orthrus_ar_verify_attend(lyr, d["q_ar"], d["k_ar_blk"], d["v_ar_blk"], out_a, ws)
    assert b.orthrus_read_status(ws) == 0
    if wl.head_dim == 128:
        assert b.orthrus_last_path() == "tcgen05"
    rows = sample_rows(wl, t["cache_len"], seed=layer + 1)
    atol, rtol = TOL[torch.bfloat16]
    for view, out in ((oracle.VIEW_DIFFUSION, out_d), (oracle.VIEW_AR, out_a)):
        o = out.cpu().double()
        assert torch.isfinite(o).all()
        ref = oracle_attend_rows(view, rows, t)
        got = o[rows[:, 0].long(), rows[:, 1].long(), rows[:, 2].long()]
        err = float((got - ref).abs().max())
        scale = float(ref.abs().max())
        assert err <= atol and err <= rtol * scale, (name, view, err, scale)
        # every row is a convex combination of value rows: bounded by the largest |V|
        vmax = max(float(t["v_cache"].float().abs().max()), 1.0)
        assert float(o.abs().max()) <= vmax


@pytest.mark.parametrize("name", ["cfg2_8b_b1", "cfg3_ragged", "cfg4_long", "cfg5_loop"])
def test_consensus_and_commit_at_bench_size(name):
    b = binding()
    wl = W.CONFIGS[name]
    lg = W.logits(wl)
    greedy = oracle.consensus_accept(lg, torch.zeros(wl.batch, wl.block, dtype=torch.int32))[2]
    draft = W.drafts(wl, greedy)
    ref = oracle.consensus_accept(lg, draft)
    B, K, V = lg.shape
    i32 = dict(dtype=torch.int32, device="cuda")
    outs = [torch.zeros(B, **i32), torch.zeros(B, K, **i32), torch.zeros(B, K, **i32), torch.zeros(B, **i32)]
    ws = b.new_workspace(b.orthrus_consensus_workspace_bytes(B, K, V))
    b.orthrus_consensus_accept(lg.cuda(), draft.cuda(), *outs, ws)
    for g, r, what in zip(outs, ref, ("n_commit", "committed", "ar_argmax", "next_anchor")):
        assert torch.equal(g.cpu(), r), what
    # commit of two layers' AR-view block KV into small stand-in caches of the same geometry
    # per position (capacity cut down to keep the host copy small; the rows touched are the same)
    lens = W.prefix_lengths(wl)
    cap = 64 + wl.block
    small = torch.clamp(lens, max=64)
    g = torch.Generator().manual_seed(5)
    mk = lambda *s: torch.randn(*s, generator=g).to(torch.bfloat16)
    layers, refs, dev = [], [], []
    dl = small.cuda()
    for l in range(2):
        c = dict(k_cache=mk(B, wl.n_kv_heads, cap, wl.head_dim), v_cache=mk(B, wl.n_kv_heads, cap, wl.head_dim),
                 k_blk=mk(B, K, wl.n_kv_heads, wl.head_dim), v_blk=mk(B, K, wl.n_kv_heads, wl.head_dim))
        r = {k: v.clone() for k, v in c.items()}
        rl = small.clone()
        oracle.kv_append(r["k_cache"], r["v_cache"], rl, r["k_blk"], r["v_blk"], ref[0])
        refs.append((r, rl))
        dd = {k: v.cuda() for k, v in c.items()}
        dev.append(dd)
        layers.append(b.make_layer(dd["k_cache"], dd["v_cache"], dl, wl.n_q_heads, K))
    aws = b.new_workspace(256)
    b.orthrus_kv_append_layers(layers, [x["k_blk"] for x in dev], [x["v_blk"] for x in dev], outs[0], True, aws)
    assert b.orthrus_read_status(aws) == 0
    for dd, (r, rl) in zip(dev, refs):
        assert torch.equal(dd["k_cache"].cpu().view(torch.int16), r["k_cache"].view(torch.int16))
        assert torch.equal(dd["v_cache"].cpu().view(torch.int16), r["v_cache"].view(torch.int16))
        assert torch.equal(dl.cpu(), rl)
