"""Pins of the oracle's sampled consensus (temperature T > 0, Section 3.3), none of which
retypes its formula:
  * the committed token of a one-position block follows the AR distribution whatever the
    draft distribution is (the losslessness the paper claims for its rejection sampling);
  * drafts drawn from q are kept at rate sum_v min(p, q) = 1 - TV(p, q), the textbook
    acceptance rate of speculative sampling;
  * equal distributions keep everything; disjoint ones reject and the correction token is
    numpy's inverse CDF of p;
  * at low temperature the rule collapses onto the greedy consensus of Eq. 8;
  * structure: 1 <= n <= K, committed prefix = kept drafts, padding -1, next anchor.
"""
import numpy as np
import torch

import oracle


def softmax(x):
    x = x - x.max(-1, keepdim=True).values
    e = x.exp()
    return e / e.sum(-1, keepdim=True)


def test_single_position_output_follows_the_ar_distribution():
    g = torch.Generator().manual_seed(1)
    V, N = 7, 120000
    la = torch.randn(V, generator=g, dtype=torch.float64) * 1.5
    ld = torch.randn(V, generator=g, dtype=torch.float64) * 1.5
    T = 0.8
    p, q = softmax(la / T), softmax(ld / T)
    draft = torch.multinomial(q, N, replacement=True, generator=g).to(torch.int32).view(N, 1)
    ua = torch.rand(N, 1, generator=g, dtype=torch.float64)
    ur = torch.rand(N, 1, generator=g, dtype=torch.float64)
    n, com, nxt, _ = oracle.consensus_sample(la.expand(N, 1, V).contiguous(), ld.expand(N, 1, V).contiguous(),
                                             draft, ua, ur, T)
    assert n.tolist() == [1] * N and torch.equal(com[:, 0], nxt)
    freq = torch.bincount(com[:, 0].long(), minlength=V).double() / N
    sigma = (p * (1 - p) / N).sqrt()
    assert ((freq - p).abs() <= 4.5 * sigma + 1e-9).all(), (freq, p)
    # and it is not simply echoing the drafts: their distribution is visibly different
    assert (torch.bincount(draft[:, 0].long(), minlength=V).double() / N - p).abs().max() > 10 * sigma.max()


def test_acceptance_rate_is_one_minus_total_variation():
    g = torch.Generator().manual_seed(2)
    V, N, K = 11, 60000, 1
    la = torch.randn(V, generator=g, dtype=torch.float64)
    ld = torch.randn(V, generator=g, dtype=torch.float64)
    p, q = softmax(la), softmax(ld)
    draft = torch.multinomial(q, N, replacement=True, generator=g).to(torch.int32).view(N, K)
    ua = torch.rand(N, K, generator=g, dtype=torch.float64)
    ur = torch.rand(N, K, generator=g, dtype=torch.float64)
    n, com, _, _ = oracle.consensus_sample(la.expand(N, K, V).contiguous(), ld.expand(N, K, V).contiguous(),
                                           draft, ua, ur, 1.0)
    kept = (com[:, 0] == draft[:, 0]) & (ua[:, 0] * q[draft[:, 0].long()] <= p[draft[:, 0].long()])
    rate = float(kept.double().mean())
    expect = float(torch.minimum(p, q).sum())
    assert abs(rate - expect) < 4.5 * (expect * (1 - expect) / N) ** 0.5


def test_two_positions_first_token_marginal_and_structure():
    g = torch.Generator().manual_seed(3)
    V, N, K = 5, 80000, 3
    la = torch.randn(K, V, generator=g, dtype=torch.float64)
    ld = torch.randn(K, V, generator=g, dtype=torch.float64)
    q = softmax(ld)
    draft = torch.stack([torch.multinomial(q[k], N, replacement=True, generator=g) for k in range(K)], 1).to(torch.int32)
    ua = torch.rand(N, K, generator=g, dtype=torch.float64)
    ur = torch.rand(N, K, generator=g, dtype=torch.float64)
    n, com, nxt, _ = oracle.consensus_sample(la.expand(N, K, V).contiguous(), ld.expand(N, K, V).contiguous(),
                                             draft.contiguous(), ua, ur, 1.0)
    assert int(n.min()) >= 1 and int(n.max()) == K
    p0 = softmax(la[0])
    freq = torch.bincount(com[:, 0].long(), minlength=V).double() / N
    assert ((freq - p0).abs() <= 4.5 * (p0 * (1 - p0) / N).sqrt()).all()
    for b in range(0, N, 997):
        nb = int(n[b])
        assert com[b, nb:].tolist() == [-1] * (K - nb) and int(nxt[b]) == int(com[b, nb - 1])
        assert com[b, :nb - 1].tolist() == draft[b, :nb - 1].tolist()       # kept drafts come first
        if nb == K and int(com[b, K - 1]) == int(draft[b, K - 1]):
            continue
    # P(n = K and all kept) = prod_k sum_v min(p_k, q_k) for independent positions
    all_kept = ((n == K) & (com == draft).all(1)).double().mean()
    expect = float(torch.prod(torch.minimum(softmax(la), q).sum(-1)))
    # (a correction token equal to the rejected draft cannot occur: its residual mass is 0)
    assert abs(float(all_kept) - expect) < 4.5 * (expect * (1 - expect) / N) ** 0.5


def test_equal_distributions_keep_every_draft():
    g = torch.Generator().manual_seed(4)
    B, K, V = 4, 6, 50
    lg = torch.randn(B, K, V, generator=g).to(torch.bfloat16)
    draft = torch.randint(0, V, (B, K), generator=g, dtype=torch.int32)
    ua = torch.rand(B, K, generator=g, dtype=torch.float64)
    n, com, nxt, _ = oracle.consensus_sample(lg, lg.clone(), draft, ua, ua, 0.7)
    assert n.tolist() == [K] * B and torch.equal(com, draft) and torch.equal(nxt, draft[:, -1])


def test_disjoint_support_rejects_and_inverts_the_ar_cdf():
    V, N = 9, 500
    la = torch.full((V,), -1e4, dtype=torch.float64)
    la[[1, 4, 6]] = torch.tensor([0.3, 1.2, -0.5], dtype=torch.float64)      # p lives on {1, 4, 6}
    ld = torch.full((V,), -1e4, dtype=torch.float64)
    ld[2] = 0.0                                                             # q is a point mass on 2
    p = softmax(la)
    u = (torch.arange(N, dtype=torch.float64) + 0.5) / N
    draft = torch.full((N, 1), 2, dtype=torch.int32)
    n, com, _, _ = oracle.consensus_sample(la.expand(N, 1, V).contiguous(), ld.expand(N, 1, V).contiguous(),
                                           draft, torch.full((N, 1), 0.5, dtype=torch.float64), u.view(N, 1), 1.0)
    expect = np.searchsorted(np.cumsum(p.numpy()), u.numpy(), side="right")
    assert n.tolist() == [1] * N and com[:, 0].tolist() == expect.tolist()


def test_low_temperature_collapses_onto_the_greedy_rule():
    g = torch.Generator().manual_seed(5)
    B, K, V = 6, 8, 300
    la = torch.randn(B, K, V, generator=g).to(torch.float32)
    ld = torch.randn(B, K, V, generator=g).to(torch.float32)
    greedy = la.argmax(-1).to(torch.int32)
    coin = torch.rand(B, K, generator=g) < 0.7
    draft = torch.where(coin, greedy, torch.randint(0, V, (B, K), generator=g, dtype=torch.int32)).contiguous()
    ua = torch.rand(B, K, generator=g, dtype=torch.float64) * 0.98 + 0.01
    ur = torch.rand(B, K, generator=g, dtype=torch.float64)
    # the diffusion logits only need to leave the drafts a non-vanishing probability
    n, com, nxt, _ = oracle.consensus_sample(la, ld * 1e-3, draft, ua, ur, 1e-3)
    rn, rcom, _, rnxt = oracle.consensus_accept(la, draft)
    assert torch.equal(n, rn) and torch.equal(com, rcom) and torch.equal(nxt, rnxt)
