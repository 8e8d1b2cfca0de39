"""End-to-end generation loop on a random-initialised decoder (the shape of the fifth
benchmark configuration, scaled down): prefill, then repeated block-K draft / verify /
consensus / commit through the C ABI, with drafts forced to agree with the AR greedy
trajectory at a set rate so that acceptance is controlled.

Checks: (1) the lossless guarantee of Section 3.3 - the committed stream equals plain
greedy decoding (the same library path at block width 1) token for token in the fp32
test mode; in bf16, block-K verification and width-1 decoding round differently, so
equality is required up to the first position whose top-2 logit gap in the width-1 run
is below a stated epsilon; (2) every cycle's consensus equals the oracle's on the GPU's
own logits, bit for bit; (3) 1 <= n <= K and the cache length grows by n."""
import pytest
import torch

import oracle
from harness.decoder import Decoder
from _gpu_util import binding

pytestmark = pytest.mark.gpu


def greedy_trajectory(dec, anchor, n_new, fused=False):
    """Width-1 decoding with the AR view: returns tokens [B][n_new] and top-2 gaps.  fused:
    the greedy token comes from orthrus_lm_head_consensus on the hidden states."""
    b = dec.b
    B = anchor.shape[0]
    i32 = dict(dtype=torch.int32, device="cuda")
    outs = [torch.zeros(B, **i32), torch.zeros(B, 1, **i32), torch.zeros(B, 1, **i32), torch.zeros(B, **i32)]
    cws = b.new_workspace(b.orthrus_consensus_workspace_bytes(B, 1, dec.V))
    toks, gaps = [], []
    draft = torch.zeros(B, 1, **i32)
    if fused:
        cws = b.new_workspace(b.orthrus_lm_head_consensus_workspace_bytes(B, 1, dec.V))
    for _ in range(n_new):
        logits, ks, vs, hn = dec.forward_block(anchor.view(B, 1), "ar", 1, return_hidden=True)
        if fused:
            b.orthrus_lm_head_consensus(hn, dec.lm_head_rows(), draft, *outs, cws)
        else:
            b.orthrus_consensus_accept(logits, draft, *outs, cws)
        top2 = logits.float().topk(2, dim=-1).values[:, 0]
        gaps.append((top2[:, 0] - top2[:, 1]).cpu())
        dec.commit(ks, vs, outs[0], 1)
        anchor = outs[3].clone()
        toks.append(anchor.cpu())
    return torch.stack(toks, 1), torch.stack(gaps, 1)


def run_loop(dtype, layers, hidden, n_q, n_kv, d, ffn, vocab, B, T, K, n_new, rate, eps, fused=False):
    b = binding()
    b.orthrus_set_path("auto")
    cap = T + n_new + 2 * K + 8
    g = torch.Generator().manual_seed(11)
    prompt = torch.randint(0, vocab, (B, T), generator=g).cuda()

    ref = Decoder(b, layers, hidden, n_q, n_kv, d, ffn, vocab, dtype, B, cap, K, seed=3)
    anchor0 = ref.prefill(prompt)
    traj, gaps = greedy_trajectory(ref, anchor0, n_new + K, fused)

    dec = Decoder(b, layers, hidden, n_q, n_kv, d, ffn, vocab, dtype, B, cap, K, seed=3,
                  flags=b.LAYER_CACHE_QUIESCENT)
    anchor = dec.prefill(prompt)
    assert torch.equal(anchor.cpu(), anchor0.cpu())
    streams = [[] for _ in range(B)]
    cycles, total = 0, 0
    fws = b.new_workspace(b.orthrus_lm_head_consensus_workspace_bytes(B, K, vocab)) if fused else None
    while min(len(s) for s in streams) < n_new:
        done = torch.tensor([len(s) for s in streams])
        # forced drafts: the trajectory token with probability `rate`, else a uniform token
        idx = (done.view(B, 1) + torch.arange(K)).clamp(max=traj.shape[1] - 1)
        want = torch.gather(traj, 1, idx)
        coin = torch.rand(B, K, generator=g) < rate
        draft = torch.where(coin, want, torch.randint(0, vocab, (B, K), generator=g, dtype=torch.int32))
        draft = draft.to(torch.int32).cuda()
        len_before = dec.cache_len.cpu().clone()
        # forward pass 1: the diffusion view over [anchor, mask x (K-1)]
        blk = torch.full((B, K), vocab, dtype=torch.int32, device="cuda")
        blk[:, 0] = anchor
        d_logits, _, _ = dec.forward_block(blk, "diff", K)
        assert torch.isfinite(d_logits.float()).all()
        # forward pass 2: the AR view over [anchor, draft_1 .. draft_{K-1}]
        ar_in = torch.cat([anchor.view(B, 1), draft[:, :K - 1]], dim=1)
        logits, ks, vs, hn = dec.forward_block(ar_in, "ar", K, return_hidden=True)
        if fused:
            # the greedy tokens straight from the hidden states; the oracle's fp64 logits decide
            # wherever its two largest are clearly apart, and the accept rule is exact
            b.orthrus_lm_head_consensus(hn, dec.lm_head_rows(), draft, dec.n_commit, dec.committed,
                                        dec.ar_argmax, dec.next_anchor, fws)
            assert b.orthrus_read_status(fws) == 0
            oarg, top2 = oracle.lm_head_argmax(hn.cpu().reshape(B * K, -1), dec.lm_head_rows().cpu())
            clear = ((top2[:, 0] - top2[:, 1]) > 1e-4 * top2[:, 0].abs().clamp(min=1.0)).reshape(B, K)
            garg = dec.ar_argmax.cpu()
            assert torch.equal(garg[clear], oarg.reshape(B, K)[clear])
            rn, rcom, rnxt = oracle.accept_rule(garg.contiguous(), draft.cpu())
            rarg = garg
        else:
            b.orthrus_consensus_accept(logits, draft, dec.n_commit, dec.committed, dec.ar_argmax,
                                       dec.next_anchor, dec.cws)
            rn, rcom, rarg, rnxt = oracle.consensus_accept(logits.cpu(), draft.cpu())
        assert torch.equal(dec.n_commit.cpu(), rn) and torch.equal(dec.committed.cpu(), rcom)
        assert torch.equal(dec.ar_argmax.cpu(), rarg) and torch.equal(dec.next_anchor.cpu(), rnxt)
        assert int(rn.min()) >= 1 and int(rn.max()) <= K
        dec.commit(ks, vs, dec.n_commit, K)
        assert torch.equal(dec.cache_len.cpu(), len_before + rn)
        assert b.orthrus_read_status(dec.ws) == 0
        for s in range(B):
            streams[s].extend(rcom[s, :int(rn[s])].tolist())
        anchor = dec.next_anchor.clone()
        cycles += 1
        total += int(rn.sum())
    # lossless: equal to greedy decoding, up to a near tie of the width-1 run (bf16 only)
    near_ties = 0
    for s in range(B):
        got = streams[s][:n_new]
        exp = traj[s, :n_new].tolist()
        for i, (x, y) in enumerate(zip(got, exp)):
            if x != y:
                assert float(gaps[s, i]) < eps, (s, i, x, y, float(gaps[s, i]))
                near_ties += 1
                break
    return total / (cycles * B), near_ties


def test_lossless_generation_fp32_reduced_model():
    mean_n, ties = run_loop(torch.float32, layers=2, hidden=128, n_q=4, n_kv=2, d=32, ffn=256,
                            vocab=500, B=3, T=40, K=8, n_new=40, rate=0.65, eps=1e-4)
    assert ties == 0
    assert 1.5 < mean_n < 4.5          # E[n] = (1 - p^K) / (1 - p) = 2.77 for p = 0.65, K = 8


def test_generation_bf16_tcgen05_shapes():
    """head_dim 128, G = 4, K = 16 (M = 64): the shapes of the benchmark's decoder configuration."""
    mean_n, ties = run_loop(torch.bfloat16, layers=3, hidden=512, n_q=8, n_kv=2, d=128, ffn=1024,
                            vocab=2000, B=4, T=300, K=16, n_new=48, rate=0.65, eps=0.25)
    assert ties <= 2
    assert 1.5 < mean_n < 4.5
    assert binding().orthrus_last_path() == "tcgen05"


def test_generation_bf16_consensus_fused_with_the_lm_head():
    """The same loop with the greedy tokens taken straight from the last hidden states
    (orthrus_lm_head_consensus): no logits tensor is handed to the consensus, in the loop or in
    the width-1 reference run."""
    mean_n, ties = run_loop(torch.bfloat16, layers=3, hidden=512, n_q=8, n_kv=2, d=128, ffn=1024,
                            vocab=2000, B=4, T=300, K=16, n_new=48, rate=0.65, eps=0.25, fused=True)
    assert ties <= 2
    assert 1.5 < mean_n < 4.5


def test_sampled_generation_loop_fp32():
    """Temperature 1: drafts are SAMPLED from the diffusion view's own logits, verified by
    the AR view and reconciled by rejection sampling.  Every cycle's outcome equals the
    oracle's on the GPU's own logits (up to near ties), and the cache grows by n."""
    b = binding()
    b.orthrus_set_path("auto")
    layers, hidden, n_q, n_kv, d, ffn, vocab = 2, 128, 4, 2, 32, 256, 400
    B, T_prompt, K, cycles, temp = 3, 30, 6, 10, 1.0
    cap = T_prompt + cycles * K + 8
    g = torch.Generator().manual_seed(23)
    prompt = torch.randint(0, vocab, (B, T_prompt), generator=g).cuda()
    dec = Decoder(b, layers, hidden, n_q, n_kv, d, ffn, vocab, torch.float32, B, cap, K, seed=4)
    anchor = dec.prefill(prompt)
    sws = b.new_workspace(b.orthrus_consensus_sample_workspace_bytes(B, K, vocab))
    i32 = dict(dtype=torch.int32, device="cuda")
    n_c, com, nxt = torch.zeros(B, **i32), torch.zeros(B, K, **i32), torch.zeros(B, **i32)
    total, undecided = 0, 0
    for _ in range(cycles):
        blk = torch.full((B, K), vocab, dtype=torch.int32, device="cuda")
        blk[:, 0] = anchor
        d_logits, _, _ = dec.forward_block(blk, "diff", K)
        # row i of the diffusion pass proposes the token after block position i
        q = torch.softmax(d_logits.float().cpu() / temp, -1)
        draft = torch.multinomial(q.view(-1, vocab), 1, generator=g).view(B, K).to(torch.int32)
        ar_in = torch.cat([anchor.view(B, 1), draft[:, :K - 1].cuda()], dim=1)
        logits, ks, vs = dec.forward_block(ar_in, "ar", K)
        ua, ur = torch.rand(B, K, generator=g), torch.rand(B, K, generator=g)
        len_before = dec.cache_len.cpu().clone()
        b.orthrus_consensus_sample(logits, d_logits, draft.cuda(), ua.cuda(), ur.cuda(), temp, n_c, com, nxt, sws)
        rn, rcom, rnxt, margin = oracle.consensus_sample(logits.cpu(), d_logits.cpu(), draft, ua.double(),
                                                         ur.double(), temp)
        ok = (margin[:, 0] > 1e-4) & (margin[:, 1] > 1e-2)
        undecided += int((~ok).sum())
        assert torch.equal(n_c.cpu()[ok], rn[ok]) and torch.equal(com.cpu()[ok], rcom[ok])
        assert torch.equal(nxt.cpu()[ok], rnxt[ok])
        assert int(n_c.min()) >= 1 and int(n_c.max()) <= K
        dec.commit(ks, vs, n_c, K)
        assert torch.equal(dec.cache_len.cpu(), len_before + n_c.cpu())
        anchor = nxt.clone()
        total += int(n_c.sum())
    assert undecided <= 2 and total >= cycles * B
