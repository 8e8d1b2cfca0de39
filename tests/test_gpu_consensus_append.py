"""GPU parity (bit-exact) of the consensus and KV-commit calls against the oracle."""
import pytest
import torch

import oracle
from paper_2605_12825_b200 import workloads as W
from _gpu_util import Guarded, binding, small_workload

pytestmark = pytest.mark.gpu


def run_consensus(logits, draft):
    b = binding()
    B, K, V = logits.shape
    ws = b.new_workspace(b.orthrus_consensus_workspace_bytes(B, K, V))
    outs = [Guarded((B,), torch.int32), Guarded((B, K), torch.int32),
            Guarded((B, K), torch.int32), Guarded((B,), torch.int32)]
    b.orthrus_consensus_accept(logits.cuda(), draft.cuda(), outs[0].t, outs[1].t, outs[2].t,
                               outs[3].t, ws)
    torch.cuda.synchronize()
    assert all(o.intact() for o in outs)
    return [o.t.cpu() for o in outs]


def check_consensus(logits, draft):
    got = run_consensus(logits, draft)
    ref = oracle.consensus_accept(logits, draft)
    for g, r, name in zip(got, ref, ("n_commit", "committed", "ar_argmax", "next_anchor")):
        assert torch.equal(g, r), name
    return ref


@pytest.mark.parametrize("B,K,V", [(1, 8, 1000), (2, 16, 32000), (3, 5, 1001), (2, 3, 33),
                                   (1, 1, 7), (4, 32, 4099), (1, 16, 151936)])
@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_consensus_matches_oracle(B, K, V, dtype):
    wl = small_workload(B, K, 1, 1, 32, 1, 1, dtype=dtype, V=V).with_(match_min=0.3, match_max=0.9)
    lg = W.logits(wl)
    g = oracle.consensus_accept(lg, torch.zeros(B, K, dtype=torch.int32))[2]
    draft = W.drafts(wl, g)
    n, *_ = check_consensus(lg, draft)
    assert int(n.min()) >= 1 and int(n.max()) <= K


def test_consensus_ties_and_special_values():
    V = 5000
    lg = torch.randn(2, 4, V, generator=torch.Generator().manual_seed(3)).to(torch.bfloat16)
    lg[0, 0, 4097] = 9.0; lg[0, 0, 13] = 9.0; lg[0, 0, 4999] = 9.0      # three-way tie
    lg[0, 1, :] = -float("inf")                                         # nothing finite
    lg[0, 2, :] = 1.5                                                   # everything ties
    lg[0, 3, V - 1] = 50.0                                              # last element wins
    lg[1, 0, 0] = 50.0                                                  # first element wins
    lg[1, 1, 7] = float("inf")
    lg[1, 2, 100] = float("nan"); lg[1, 2, 200] = 30.0                  # NaN never wins
    draft = torch.tensor([[13, 0, 0, V - 1], [0, 7, 200, 1]], dtype=torch.int32)
    n, com, arg, nxt = check_consensus(lg, draft)
    assert arg[0].tolist()[:4] == [13, 0, 0, V - 1]
    assert arg[1].tolist()[:3] == [0, 7, 200]
    assert n.tolist() == [4, 4]


@pytest.mark.parametrize("V,dtype", [(1001, torch.float32), (4099, torch.bfloat16), (7, torch.bfloat16)])
def test_consensus_rows_without_a_finite_value_on_ragged_vocabularies(V, dtype):
    """Rows whose start or end is not 16-byte aligned have scalar head and tail elements:
    a row of -inf (with or without a few NaN) must still resolve to token 0 there, and an
    ordinary row next to it must not be disturbed by the odd alignment."""
    lg = torch.randn(2, 3, V, generator=torch.Generator().manual_seed(4)).to(dtype)
    lg[0, 0, :] = -float("inf")
    lg[0, 1, :] = -float("inf"); lg[0, 1, 0] = float("nan"); lg[0, 1, V - 1] = float("nan")
    lg[0, 2, :] = -float("inf"); lg[0, 2, V - 1] = -1e30                 # the only finite value, in the tail
    lg[1, 0, :] = float("nan")
    lg[1, 1, :] = -float("inf"); lg[1, 1, 1] = -float("inf"); lg[1, 1, 0] = -3.0   # head element wins
    draft = torch.zeros(2, 3, dtype=torch.int32)
    n, com, arg, nxt = check_consensus(lg, draft)
    assert arg[0].tolist() == [0, 0, V - 1] and arg[1].tolist()[:2] == [0, 0]


def test_consensus_all_agree_and_none_agree():
    wl = small_workload(4, 8, 1, 1, 32, 1, 1, V=2000)
    lg = W.logits(wl)
    g = oracle.consensus_accept(lg, torch.zeros(4, 8, dtype=torch.int32))[2]
    n, com, _, nxt = check_consensus(lg, g.clone())
    assert n.tolist() == [8] * 4 and torch.equal(nxt, g[:, -1])
    wrong = (g + 1) % 2000
    n, com, _, nxt = check_consensus(lg, wrong.to(torch.int32))
    assert n.tolist() == [1] * 4 and torch.equal(nxt, g[:, 0])


def make_append_case(dtype, B=3, K=8, Hkv=2, d=64, cap=64, seed=0):
    g = torch.Generator().manual_seed(seed)
    mk = lambda *s: torch.randn(*s, generator=g).to(dtype)
    return dict(k_cache=mk(B, Hkv, cap, d), v_cache=mk(B, Hkv, cap, d),
                k_blk=mk(B, K, Hkv, d), v_blk=mk(B, K, Hkv, d))


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("update_len", [True, False])
def test_append_bit_exact(dtype, update_len):
    b = binding()
    c = make_append_case(dtype)
    lens = torch.tensor([0, 17, 56], dtype=torch.int32)
    n = torch.tensor([1, 8, 5], dtype=torch.int32)
    ref = {k: v.clone() for k, v in c.items()}
    ref_len = lens.clone()
    assert oracle.kv_append(ref["k_cache"], ref["v_cache"], ref_len, ref["k_blk"], ref["v_blk"], n,
                            update_len) == 0
    d = {k: v.cuda() for k, v in c.items()}
    dl = lens.cuda()
    layer = b.make_layer(d["k_cache"], d["v_cache"], dl, 4, 8)
    ws = b.new_workspace(256)
    b.orthrus_kv_append(layer, d["k_blk"], d["v_blk"], n.cuda(), update_len, ws)
    assert b.orthrus_read_status(ws) == 0
    bits = lambda x: x.view(torch.int16 if dtype == torch.bfloat16 else torch.int32)
    assert torch.equal(bits(d["k_cache"].cpu()), bits(ref["k_cache"]))
    assert torch.equal(bits(d["v_cache"].cpu()), bits(ref["v_cache"]))
    assert torch.equal(dl.cpu(), ref_len)


def test_append_overflow_is_skipped_and_flagged():
    b = binding()
    c = make_append_case(torch.bfloat16)
    lens = torch.tensor([0, 60, 10], dtype=torch.int32)      # 60 + 8 > 64
    n = torch.tensor([2, 8, 9], dtype=torch.int32)           # 9 > K
    d = {k: v.cuda() for k, v in c.items()}
    dl = lens.cuda()
    layer = b.make_layer(d["k_cache"], d["v_cache"], dl, 4, 8)
    ws = b.new_workspace(256)
    b.orthrus_kv_append(layer, d["k_blk"], d["v_blk"], n.cuda(), True, ws)
    assert b.orthrus_read_status(ws) == b.DEV_APPEND_OVERFLOW
    assert dl.cpu().tolist() == [2, 60, 10]
    assert torch.equal(d["k_cache"][1:].cpu().view(torch.int16), c["k_cache"][1:].view(torch.int16))
    b.orthrus_workspace_init(ws)
    assert b.orthrus_read_status(ws) == 0


def test_one_full_cycle_tiny_config():
    """Diffusion attend, AR verify attend, consensus and commit chained on the device
    for the tiny configuration, each result compared with the oracle's."""
    from _gpu_util import assert_close, oracle_attend, run_attend
    wl = W.CONFIGS["cfg1_tiny"]
    t = W.attention_inputs(wl)
    for view in (oracle.VIEW_DIFFUSION, oracle.VIEW_AR):
        got, status, _ = run_attend(view, t, wl)
        assert status == 0
        assert_close(got, oracle_attend(view, t), torch.bfloat16)
    lg = W.logits(wl)
    g = oracle.consensus_accept(lg, torch.zeros(1, 8, dtype=torch.int32))[2]
    draft = W.drafts(wl, g)
    n_ref, com_ref, arg_ref, nxt_ref = check_consensus(lg, draft)
    b = binding()
    d = {k: v.cuda() for k, v in t.items()}
    layer = b.make_layer(d["k_cache"], d["v_cache"], d["cache_len"], wl.n_q_heads, wl.block)
    b.orthrus_kv_append(layer, d["k_ar_blk"], d["v_ar_blk"], n_ref.cuda(), True)
    ref = {k: v.clone() for k, v in t.items()}
    oracle.kv_append(ref["k_cache"], ref["v_cache"], ref["cache_len"], ref["k_ar_blk"],
                     ref["v_ar_blk"], n_ref)
    assert torch.equal(d["cache_len"].cpu(), ref["cache_len"])
    assert torch.equal(d["k_cache"].cpu().view(torch.int16), ref["k_cache"].view(torch.int16))
    assert torch.equal(d["v_cache"].cpu().view(torch.int16), ref["v_cache"].view(torch.int16))


@pytest.mark.parametrize("update_len", [True, False])
@pytest.mark.parametrize("shared_len", [True, False])
def test_append_layers_bit_exact(update_len, shared_len):
    """The multi-layer commit equals the oracle's commit applied layer by layer; a length
    array shared by several layers grows once."""
    b = binding()
    L = 5
    cases = [make_append_case(torch.bfloat16, seed=10 + l) for l in range(L)]
    lens0 = torch.tensor([0, 17, 56], dtype=torch.int32)
    n = torch.tensor([1, 8, 5], dtype=torch.int32)
    ref = [{k: v.clone() for k, v in c.items()} for c in cases]
    ref_lens = [lens0.clone() for _ in range(L)]
    for l in range(L):
        oracle.kv_append(ref[l]["k_cache"], ref[l]["v_cache"], ref_lens[l], ref[l]["k_blk"],
                         ref[l]["v_blk"], n, update_len)
    dev = [{k: v.cuda() for k, v in c.items()} for c in cases]
    dl = [lens0.cuda()] * L if shared_len else [lens0.cuda() for _ in range(L)]
    layers = [b.make_layer(d["k_cache"], d["v_cache"], dl[l], 4, 8) for l, d in enumerate(dev)]
    ws = b.new_workspace(256)
    b.orthrus_kv_append_layers(layers, [d["k_blk"] for d in dev], [d["v_blk"] for d in dev],
                               n.cuda(), update_len, ws)
    assert b.orthrus_read_status(ws) == 0
    for l in range(L):
        assert torch.equal(dev[l]["k_cache"].cpu().view(torch.int16), ref[l]["k_cache"].view(torch.int16))
        assert torch.equal(dev[l]["v_cache"].cpu().view(torch.int16), ref[l]["v_cache"].view(torch.int16))
        assert torch.equal(dl[l].cpu(), ref_lens[l])


def test_append_layers_overflow_is_skipped_and_flagged():
    b = binding()
    cases = [make_append_case(torch.bfloat16, seed=20 + l) for l in range(2)]
    lens = torch.tensor([0, 60, 10], dtype=torch.int32).cuda()      # 60 + 8 > 64
    n = torch.tensor([2, 8, 9], dtype=torch.int32)                  # 9 > K
    dev = [{k: v.cuda() for k, v in c.items()} for c in cases]
    layers = [b.make_layer(d["k_cache"], d["v_cache"], lens, 4, 8) for d in dev]
    ws = b.new_workspace(256)
    b.orthrus_kv_append_layers(layers, [d["k_blk"] for d in dev], [d["v_blk"] for d in dev],
                               n.cuda(), True, ws)
    assert b.orthrus_read_status(ws) == b.DEV_APPEND_OVERFLOW
    assert lens.cpu().tolist() == [2, 60, 10]
    for d, c in zip(dev, cases):
        assert torch.equal(d["k_cache"][1:].cpu().view(torch.int16), c["k_cache"][1:].view(torch.int16))
