"""GPU parity of the fused LM-head consensus (tensor-core product with the argmax of Eq. 8 in
its read-out) against the oracle's fp64 logits.

The greedy token is an integer decided by floating point: the kernel compares fp32 sums of
exact bf16 products, the oracle fp64 sums.  Where the oracle's two largest logits are further
apart than the fp32 accumulation error allows (TOL, relative to the largest logit's size) the
tokens must be identical; in a closer call the kernel's token must be one whose fp64 logit is
within TOL of the largest.  Everything downstream of the tokens (n_commit, committed,
next_anchor) is integer work and must equal the oracle's accept rule on the kernel's tokens
bit for bit.  Operands with small integer values make every logit exact in both precisions;
there the tokens must agree everywhere, ties included."""
import pytest
import torch

import oracle
from _gpu_util import Guarded, binding

pytestmark = pytest.mark.gpu

TOL = 1e-4          # fp32 accumulation of <= 8192 bf16 products of unit scale stays below 1e-5


def run_fused(hidden, lm_head, draft):
    b = binding()
    B, K, H = hidden.shape
    V = lm_head.shape[0]
    ws = b.new_workspace(b.orthrus_lm_head_consensus_workspace_bytes(B, K, V))
    outs = [Guarded((B,), torch.int32), Guarded((B, K), torch.int32),
            Guarded((B, K), torch.int32), Guarded((B,), torch.int32)]
    b.orthrus_lm_head_consensus(hidden.cuda(), lm_head.cuda(), draft.cuda(), outs[0].t, outs[1].t,
                                outs[2].t, outs[3].t, ws)
    torch.cuda.synchronize()
    assert b.orthrus_read_status(ws) == 0
    assert all(o.intact() for o in outs)
    return [o.t.cpu() for o in outs]


def drafts_from(arg, V, rate, gen):
    draft = arg.clone()
    flip = torch.rand(arg.shape, generator=gen) >= rate
    draft[flip] = (draft[flip] + 1 + torch.randint(0, V - 1, (int(flip.sum()),), generator=gen).int()) % V
    return draft.to(torch.int32)


def check(hidden, lm_head, rate=0.6, seed=0, exact=False, max_unclear=None):
    B, K, H = hidden.shape
    V = lm_head.shape[0]
    ref_arg, top2 = oracle.lm_head_argmax(hidden.reshape(B * K, H), lm_head)
    ref_arg = ref_arg.reshape(B, K)
    draft = drafts_from(ref_arg, V, rate, torch.Generator().manual_seed(seed))
    n, com, arg, nxt = run_fused(hidden, lm_head, draft)
    if exact:
        assert torch.equal(arg, ref_arg)
    else:
        scale = top2[:, 0].abs().clamp(min=1.0)
        clear = ((top2[:, 0] - top2[:, 1]) > TOL * scale).reshape(B, K)
        assert torch.equal(arg[clear], ref_arg[clear]), "decided rows differ"
        limit = max(1, B * K // 20) if max_unclear is None else max_unclear
        assert int((~clear).sum()) <= limit, "the inputs should rarely be near-ties"
        for bi, ki in (~clear).nonzero().tolist():
            r = bi * K + ki
            v = int(arg[bi, ki])
            assert 0 <= v < V
            got = float(hidden[bi, ki].double() @ lm_head[v].double())
            assert got >= float(top2[r, 0]) - TOL * float(scale[r])
    assert bool(((arg >= 0) & (arg < V)).all())
    rn, rcom, rnxt = oracle.accept_rule(arg.contiguous(), draft)
    assert torch.equal(n, rn) and torch.equal(com, rcom) and torch.equal(nxt, rnxt)
    return n, arg, ref_arg


def rand_case(B, K, V, H, seed):
    g = torch.Generator().manual_seed(seed)
    hidden = torch.randn(B, K, H, generator=g).to(torch.bfloat16)
    lm_head = (torch.randn(V, H, generator=g) / H ** 0.5).to(torch.bfloat16)
    return hidden, lm_head


@pytest.mark.parametrize("B,K,V,H", [
    (1, 8, 1000, 64),        # one stage, ragged vocabulary tile
    (2, 16, 5000, 256),      # the stage ring wraps once per item
    (3, 5, 257, 72),         # ragged last stage (72 = 64 + 8), one entry in the second tile
    (9, 32, 3001, 512),      # three row tiles, the last ragged (288 rows)
    (1, 16, 60000, 128),     # more items than SMs: every CTA loops, accumulators alternate
    (1, 1, 7, 8),            # the smallest everything
    (4, 32, 2048, 1024),     # exact tiles, 16 stages per item
    (1, 16, 4099, 4096),     # the hidden size of the 8B-class configurations
    (64, 64, 1000, 128),     # 4096 rows: sixteen 256-row tiles
    (2, 100, 777, 200),      # 200 rows (one 256-row tile, ragged), hidden 200 = 3 stages + 8 columns
    (5, 26, 300, 64),        # 130 rows: two rows past the 128-row shape
])
def test_fused_matches_oracle(B, K, V, H):
    hidden, lm_head = rand_case(B, K, V, H, seed=B * 1000 + K + V + H)
    n, *_ = check(hidden, lm_head, seed=V)
    assert int(n.min()) >= 1 and int(n.max()) <= K


def test_integer_operands_agree_everywhere_ties_included():
    g = torch.Generator().manual_seed(4)
    B, K, V, H = 3, 16, 1500, 192
    hidden = torch.randint(-3, 4, (B, K, H), generator=g).to(torch.bfloat16)
    lm_head = torch.randint(-3, 4, (V, H), generator=g).to(torch.bfloat16)
    check(hidden, lm_head, exact=True)


def test_duplicated_rows_tie_across_tiles_and_the_lowest_id_wins():
    hidden, lm_head = rand_case(2, 8, 2000, 128, seed=21)
    # rows 300, 1301 (another vocabulary tile) and 1999 (the ragged tile) all equal a strong
    # copy of one hidden row: a three-way exact tie on that row
    lm_head[300] = hidden[1, 3] * 4
    lm_head[1301] = lm_head[300]
    lm_head[1999] = lm_head[300]
    # (the strong row also wins, and so ties with its copies, on other hidden rows; identical
    # operand rows give identical fp32 sums, so the lowest id must win wherever that happens)
    n, arg, ref_arg = check(hidden, lm_head, max_unclear=16)
    assert int(arg[1, 3]) == 300 and int(ref_arg[1, 3]) == 300
    assert torch.equal(arg, ref_arg)


def test_special_values():
    hidden, lm_head = rand_case(1, 4, 600, 64, seed=8)
    hidden[0, 0] = 0                                    # every logit 0: everything ties -> id 0
    lm_head[500, 0] = float("inf"); hidden[0, 1, 0] = 1.0   # a +inf logit on row 1
    lm_head[78, 5] = float("nan"); hidden[0, 1, 5] = 0.5    # a NaN logit on every row: never wins
    n, com, arg, nxt = run_fused(hidden, lm_head, torch.zeros(1, 4, dtype=torch.int32))
    ref_arg, _ = oracle.lm_head_argmax(hidden.reshape(4, 64), lm_head)
    assert int(arg[0, 0]) == 0 == int(ref_arg[0])
    assert int(arg[0, 1]) == 500 == int(ref_arg[1])
    assert int(arg[0, 2]) != 78 and int(arg[0, 3]) != 78


def test_repeated_calls_and_unfused_path_agree_on_clear_rows():
    # the two-step path (library matrix product rounded to bf16, then orthrus_consensus_accept)
    # decides on rounded logits; wherever those have a unique maximum that is also clear in
    # fp64, both paths must name the same token
    b = binding()
    B, K, V, H = 4, 16, 8000, 512
    hidden, lm_head = rand_case(B, K, V, H, seed=99)
    ref_arg, top2 = oracle.lm_head_argmax(hidden.reshape(B * K, H), lm_head)
    draft = drafts_from(ref_arg.reshape(B, K), V, 0.7, torch.Generator().manual_seed(1))
    first = run_fused(hidden, lm_head, draft)
    second = run_fused(hidden, lm_head, draft)
    for x, y in zip(first, second):
        assert torch.equal(x, y)
    logits = (hidden.cuda().reshape(B * K, H) @ lm_head.cuda().T).reshape(B, K, V).contiguous()
    ws = b.new_workspace(b.orthrus_consensus_workspace_bytes(B, K, V))
    i32 = dict(dtype=torch.int32, device="cuda")
    outs = [torch.zeros(B, **i32), torch.zeros(B, K, **i32), torch.zeros(B, K, **i32), torch.zeros(B, **i32)]
    b.orthrus_consensus_accept(logits, draft.cuda(), *outs, ws)
    torch.cuda.synchronize()
    clear = ((top2[:, 0] - top2[:, 1]) > 2.0 ** -7 * top2[:, 0].abs().clamp(min=1.0)).reshape(B, K)
    assert int(clear.sum()) > B * K // 2
    assert torch.equal(outs[2].cpu()[clear], first[2][clear])


def test_full_size_serving_shape_on_sampled_rows():
    """The ragged serving configuration at full size (32 sequences x 32 positions, hidden
    4096, vocabulary 128256: eight row tiles, 501 vocabulary tiles, 4008 items on the
    persistent grid).  The oracle computes sampled rows one by one; integer outputs are
    checked against the accept rule on the kernel's own tokens for every sequence."""
    B, K, V, H = 32, 32, 128256, 4096
    hidden, lm_head = rand_case(B, K, V, H, seed=12825)
    rows = torch.tensor([0, 127, 128, 500, 1023, 777], dtype=torch.int32)   # tile edges and interiors
    ref_arg, top2 = oracle.lm_head_argmax(hidden.reshape(B * K, H), lm_head, rows)
    g = torch.Generator().manual_seed(2)
    draft = torch.randint(0, V, (B, K), generator=g, dtype=torch.int32)
    for j, r in enumerate(rows.tolist()):
        draft[r // K, r % K] = ref_arg[j]
    n, com, arg, nxt = run_fused(hidden, lm_head, draft)
    flat = arg.reshape(-1)
    for j, r in enumerate(rows.tolist()):
        scale = max(1.0, abs(float(top2[j, 0])))
        if float(top2[j, 0] - top2[j, 1]) > TOL * scale:
            assert int(flat[r]) == int(ref_arg[j]), r
        else:
            got = float(hidden.reshape(B * K, H)[r].double() @ lm_head[int(flat[r])].double())
            assert got >= float(top2[j, 0]) - TOL * scale
    assert bool(((arg >= 0) & (arg < V)).all())
    rn, rcom, rnxt = oracle.accept_rule(arg.contiguous(), draft)
    assert torch.equal(n, rn) and torch.equal(com, rcom) and torch.equal(nxt, rnxt)
    # every row's token must at least beat a random sample of other ids on the device
    hd, wd = hidden.cuda().reshape(B * K, H).float(), lm_head.cuda()
    cand = torch.randint(0, V, (64,), generator=g)
    lg_c = hd @ wd[cand.cuda()].float().T
    lg_a = (hd * wd[flat.cuda().long()].float()).sum(-1)
    assert bool((lg_a.unsqueeze(1) >= lg_c - 1e-3).all())


def test_replay_from_a_cuda_graph_follows_new_inputs():
    """The call allocates nothing and never synchronises, so (after one eager call has set the
    kernel attributes) it can be captured; a replay must see the buffers' current contents."""
    b = binding()
    B, K, V, H = 2, 16, 3000, 256
    hidden, lm_head = rand_case(B, K, V, H, seed=5)
    hd, wd = hidden.cuda(), lm_head.cuda()
    ws = b.new_workspace(b.orthrus_lm_head_consensus_workspace_bytes(B, K, V))
    i32 = dict(dtype=torch.int32, device="cuda")
    draft = torch.zeros(B, K, **i32)
    outs = [torch.zeros(B, **i32), torch.zeros(B, K, **i32), torch.zeros(B, K, **i32), torch.zeros(B, **i32)]
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        b.orthrus_lm_head_consensus(hd, wd, draft, *outs, ws, stream=stream)
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            b.orthrus_lm_head_consensus(hd, wd, draft, *outs, ws, stream=stream)
        for seed in (6, 7):
            h2, _ = rand_case(B, K, V, H, seed=seed)
            ref_arg, top2 = oracle.lm_head_argmax(h2.reshape(B * K, H), lm_head)
            d2 = drafts_from(ref_arg.reshape(B, K), V, 0.7, torch.Generator().manual_seed(seed))
            hd.copy_(h2.cuda()); draft.copy_(d2.cuda())
            g.replay()
            stream.synchronize()
            arg = outs[2].cpu()
            clear = ((top2[:, 0] - top2[:, 1]) > TOL * top2[:, 0].abs().clamp(min=1.0)).reshape(B, K)
            assert torch.equal(arg[clear], ref_arg.reshape(B, K)[clear])
            rn, rcom, rnxt = oracle.accept_rule(arg.contiguous(), d2)
            assert torch.equal(outs[0].cpu(), rn) and torch.equal(outs[1].cpu(), rcom)
            assert torch.equal(outs[3].cpu(), rnxt)
    assert b.orthrus_read_status(ws) == 0
