"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests re-types the oracle's loop: each compares it with an
independent statement (an explicit mask matrix with a naive softmax, a library
attention routine, a closed form, an invariance, a sequential decode of a toy
model, a byte comparison).
"""
import math
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from paper_2605_12825_b200 import workloads as W

TOL = 1e-12


def tiny(B=2, K=4, Hq=4, Hkv=2, d=8, P=(5, 3), cap=16, seed=0, dtype=torch.float64):
    g = torch.Generator().manual_seed(seed)
    r = lambda *s: torch.randn(*s, generator=g, dtype=torch.float64).to(dtype)
    t = dict(q_diff=r(B, K, Hq, d), q_ar=r(B, K, Hq, d),
             k_diff_blk=r(B, K, Hkv, d), v_diff_blk=r(B, K, Hkv, d),
             k_ar_blk=r(B, K, Hkv, d), v_ar_blk=r(B, K, Hkv, d),
             k_cache=r(B, Hkv, cap, d), v_cache=r(B, Hkv, cap, d),
             cache_len=torch.tensor(list(P), dtype=torch.int32))
    return t


def brute_force(view, q, k_blk, v_blk, k_cache, v_cache, cache_len):
    """Second formulation: per sequence build the (P+K)-long key/value sequence,
    an explicit (P+K)x(P+K) boolean mask for the whole sequence as the paper's
    two viewing rules state them, a naive softmax (no max subtraction), and keep
    the K block rows."""
    q, k_blk, v_blk, k_cache, v_cache = [x.double().numpy() for x in
                                         (q, k_blk, v_blk, k_cache, v_cache)]
    B, K, Hq, d = q.shape
    Hkv = k_blk.shape[2]
    G = Hq // Hkv
    out = np.zeros((B, K, Hq, d))
    for b in range(B):
        P = int(cache_len[b])
        n = P + K
        mask = np.zeros((n, n), dtype=bool)
        for qi in range(n):
            for kj in range(n):
                if view == oracle.VIEW_AR:
                    mask[qi, kj] = kj <= qi                       # ordinary causal model
                else:
                    in_ctx = kj < P                               # context before the anchor
                    same_blk = kj >= P and qi >= P                # bidirectional inside block
                    mask[qi, kj] = in_ctx or same_blk
        # GQA expansion: each KV head serves G consecutive query heads
        keys = np.concatenate([k_cache[b, :, :P, :], k_blk[b].transpose(1, 0, 2)], axis=1)
        vals = np.concatenate([v_cache[b, :, :P, :], v_blk[b].transpose(1, 0, 2)], axis=1)
        keys = np.repeat(keys, G, axis=0)        # [Hq][n][d]
        vals = np.repeat(vals, G, axis=0)
        for hq in range(Hq):
            qs = np.zeros((n, d))
            qs[P:] = q[b, :, hq, :]
            S = qs @ keys[hq].T / np.sqrt(d)
            E = np.where(mask, np.exp(S), 0.0)
            Wt = E / E.sum(axis=1, keepdims=True)
            out[b, :, hq, :] = (Wt @ vals[hq])[P:]
    return out


def run(view, t, **kw):
    if view == oracle.VIEW_DIFFUSION:
        return oracle.block_attend(view, t["q_diff"], t["k_diff_blk"], t["v_diff_blk"],
                                   t["k_cache"], t["v_cache"], t["cache_len"], **kw)
    return oracle.block_attend(view, t["q_ar"], t["k_ar_blk"], t["v_ar_blk"],
                               t["k_cache"], t["v_cache"], t["cache_len"], **kw)


def args_of(view, t):
    if view == oracle.VIEW_DIFFUSION:
        return (t["q_diff"], t["k_diff_blk"], t["v_diff_blk"], t["k_cache"], t["v_cache"],
                t["cache_len"])
    return (t["q_ar"], t["k_ar_blk"], t["v_ar_blk"], t["k_cache"], t["v_cache"], t["cache_len"])


VIEWS = [oracle.VIEW_DIFFUSION, oracle.VIEW_AR]


@pytest.mark.parametrize("view", VIEWS)
@pytest.mark.parametrize("shape", [
    dict(B=2, K=4, Hq=4, Hkv=2, d=8, P=(5, 3)),
    dict(B=1, K=3, Hq=2, Hkv=2, d=4, P=(0,)),           # no prefix at all
    dict(B=2, K=1, Hq=3, Hkv=1, d=5, P=(1, 4)),         # block of one, odd sizes
    dict(B=3, K=2, Hq=6, Hkv=3, d=8, P=(17, 0, 2), cap=24),
])
def test_brute_force_mask_matrix(view, shape):
    t = tiny(seed=11, **shape)
    got = run(view, t).numpy()
    ref = brute_force(view, *args_of(view, t))
    np.testing.assert_allclose(got, ref, rtol=0, atol=TOL)


@pytest.mark.parametrize("view", VIEWS)
def test_rows_sum_to_one_and_masked_weights_are_zero(view):
    t = tiny(seed=3)
    out, w = run(view, t, return_weights=True)
    B, K, Hq, _ = t["q_diff"].shape
    for b in range(B):
        P = int(t["cache_len"][b])
        for i in range(K):
            for hq in range(Hq):
                row = w[b, i, hq]
                assert abs(float(row.sum()) - 1.0) < TOL
                assert (row[: P + (K if view == oracle.VIEW_DIFFUSION else i + 1)] > 0).all()
                if view == oracle.VIEW_AR:
                    assert (row[P + i + 1:] == 0).all()       # future block keys: exactly 0
                else:
                    assert (row[P + K:] == 0).all()


def sdpa(q, k, v, mask=None):
    """Library attention (torch SDPA, fp64): q [H][Lq][d], k/v [H][Lk][d]."""
    return F.scaled_dot_product_attention(q.double(), k.double(), v.double(), attn_mask=mask)


def test_block_of_one_is_plain_decode_attention():
    """With K=1 both views are the base model's decode step over P+1 keys."""
    t = tiny(B=2, K=1, Hq=4, Hkv=2, d=8, P=(6, 2), seed=5)
    t["q_ar"] = t["q_diff"].clone()
    t["k_ar_blk"] = t["k_diff_blk"].clone()
    t["v_ar_blk"] = t["v_diff_blk"].clone()
    o_d = run(oracle.VIEW_DIFFUSION, t)
    o_a = run(oracle.VIEW_AR, t)
    assert torch.equal(o_d, o_a)
    G = 2
    for b in range(2):
        P = int(t["cache_len"][b])
        k = torch.cat([t["k_cache"][b, :, :P], t["k_diff_blk"][b].transpose(0, 1)], dim=1)
        v = torch.cat([t["v_cache"][b, :, :P], t["v_diff_blk"][b].transpose(0, 1)], dim=1)
        k = k.repeat_interleave(G, dim=0)
        v = v.repeat_interleave(G, dim=0)
        ref = sdpa(t["q_diff"][b].transpose(0, 1), k, v)      # [Hq][1][d]
        torch.testing.assert_close(o_d[b].transpose(0, 1), ref, rtol=0, atol=TOL)


def test_ar_view_is_the_causal_model_on_the_full_sequence():
    """Library pin at K>1: run torch's causal SDPA over the whole (P+K)-long
    sequence and keep the last K rows."""
    t = tiny(B=1, K=4, Hq=4, Hkv=2, d=8, P=(7,), seed=8)
    o = run(oracle.VIEW_AR, t)
    P, K, G = 7, 4, 2
    k = torch.cat([t["k_cache"][0, :, :P], t["k_ar_blk"][0].transpose(0, 1)], dim=1)
    v = torch.cat([t["v_cache"][0, :, :P], t["v_ar_blk"][0].transpose(0, 1)], dim=1)
    k = k.repeat_interleave(G, dim=0)
    v = v.repeat_interleave(G, dim=0)
    qfull = torch.zeros(4, P + K, 8, dtype=torch.float64)
    qfull[:, P:] = t["q_ar"][0].transpose(0, 1)
    ref = F.scaled_dot_product_attention(qfull, k, v, is_causal=True)[:, P:]
    torch.testing.assert_close(o[0].transpose(0, 1), ref, rtol=0, atol=TOL)


def test_cross_view_last_row_and_first_row():
    t = tiny(seed=9)
    for n in ("q", "k", "v"):
        pass
    t["q_ar"] = t["q_diff"].clone()
    t["k_ar_blk"] = t["k_diff_blk"].clone()
    t["v_ar_blk"] = t["v_diff_blk"].clone()
    o_d = run(oracle.VIEW_DIFFUSION, t)
    o_a = run(oracle.VIEW_AR, t)
    K = t["q_diff"].shape[1]
    # the last causal row sees every block key, like a diffusion row
    torch.testing.assert_close(o_a[:, K - 1], o_d[:, K - 1], rtol=0, atol=TOL)
    # the other rows differ (the views are not the same function)
    assert (o_a[:, 0] - o_d[:, 0]).abs().max() > 1e-3


@pytest.mark.parametrize("view", VIEWS)
def test_zero_query_gives_mean_of_visible_values(view):
    t = tiny(seed=13)
    t["q_diff"].zero_()
    t["q_ar"].zero_()
    o = run(view, t)
    B, K, Hq, d = t["q_diff"].shape
    G = Hq // t["k_cache"].shape[1]
    vb = t["v_diff_blk"] if view == oracle.VIEW_DIFFUSION else t["v_ar_blk"]
    for b in range(B):
        P = int(t["cache_len"][b])
        for i in range(K):
            nb = K if view == oracle.VIEW_DIFFUSION else i + 1
            for hq in range(Hq):
                h = hq // G
                mean = (t["v_cache"][b, h, :P].sum(0) + vb[b, :nb, h].sum(0)) / (P + nb)
                torch.testing.assert_close(o[b, i, hq], mean, rtol=0, atol=TOL)


def test_planted_key_allowed_vs_masked():
    """A key with an overwhelming score pulls the output to its value row when it
    is visible, and has no effect at all when the causal rule hides it."""
    B, K, Hq, Hkv, d = 1, 4, 2, 1, 8
    t = tiny(B=B, K=K, Hq=Hq, Hkv=Hkv, d=d, P=(5,), seed=21)
    base = run(oracle.VIEW_AR, t)
    i_star = 2
    # make block key i_star align with every query, with a huge norm
    t2 = {k: v.clone() for k, v in t.items()}
    t2["k_ar_blk"][0, i_star, 0] = 0
    t2["q_ar"][0, :, :, :] = 0
    t2["q_ar"][0, :, :, 0] = 1.0
    t2["k_ar_blk"][0, i_star, 0, 0] = 200.0 * math.sqrt(d)
    # remove other keys' component along the query so the planted score dominates
    t2["k_cache"][..., 0] = 0
    for ip in range(K):
        if ip != i_star:
            t2["k_ar_blk"][0, ip, 0, 0] = 0
    o = run(oracle.VIEW_AR, t2)
    for i in range(K):
        for hq in range(Hq):
            if i >= i_star:      # visible: output collapses onto that value row
                torch.testing.assert_close(o[0, i, hq], t2["v_ar_blk"][0, i_star, 0],
                                           rtol=0, atol=1e-9)
            else:                # hidden: uniform over the P+i+1 visible keys
                mean = (t2["v_cache"][0, 0, :5].sum(0) + t2["v_ar_blk"][0, :i + 1, 0].sum(0)) / (5 + i + 1)
                torch.testing.assert_close(o[0, i, hq], mean, rtol=0, atol=TOL)
    # same plant in the diffusion view is visible to every row
    t3 = {k: v.clone() for k, v in t2.items()}
    t3["q_diff"] = t2["q_ar"].clone()
    t3["k_diff_blk"] = t2["k_ar_blk"].clone()
    t3["v_diff_blk"] = t2["v_ar_blk"].clone()
    od = run(oracle.VIEW_DIFFUSION, t3)
    for i in range(K):
        torch.testing.assert_close(od[0, i, 0], t3["v_diff_blk"][0, i_star, 0], rtol=0, atol=1e-9)
    assert base.shape == o.shape


@pytest.mark.parametrize("view", VIEWS)
def test_position_coded_values_give_expected_position(view):
    """V_j[0] = j (prefix) / P+i' (block) makes O[0] the expected attended position;
    with zero queries that is the midpoint of the visible range."""
    t = tiny(B=1, K=4, Hq=2, Hkv=1, d=4, P=(9,), cap=16, seed=2)
    P, K = 9, 4
    t["q_diff"].zero_(); t["q_ar"].zero_()
    t["v_cache"][0, 0, :, 0] = torch.arange(16, dtype=torch.float64)
    for n in ("v_diff_blk", "v_ar_blk"):
        t[n][0, :, 0, 0] = torch.arange(P, P + K, dtype=torch.float64)
    o = run(view, t)
    for i in range(K):
        last = P + K - 1 if view == oracle.VIEW_DIFFUSION else P + i
        assert abs(float(o[0, i, 0, 0]) - last / 2.0) < TOL


@pytest.mark.parametrize("view", VIEWS)
def test_prefix_permutation_invariance(view):
    t = tiny(seed=31)
    o = run(view, t)
    t2 = {k: v.clone() for k, v in t.items()}
    for b in range(2):
        P = int(t["cache_len"][b])
        perm = torch.randperm(P, generator=torch.Generator().manual_seed(b))
        t2["k_cache"][b, :, :P] = t["k_cache"][b, :, :P][:, perm]
        t2["v_cache"][b, :, :P] = t["v_cache"][b, :, :P][:, perm]
    torch.testing.assert_close(run(view, t2), o, rtol=0, atol=TOL)


def test_block_permutation_invariance_diffusion_only():
    t = tiny(seed=32)
    perm = torch.tensor([2, 0, 3, 1])
    t2 = {k: v.clone() for k, v in t.items()}
    for n in ("k_diff_blk", "v_diff_blk", "k_ar_blk", "v_ar_blk"):
        t2[n] = t[n][:, perm].contiguous()
    torch.testing.assert_close(run(oracle.VIEW_DIFFUSION, t2), run(oracle.VIEW_DIFFUSION, t),
                               rtol=0, atol=TOL)
    # the causal view is order-sensitive
    assert (run(oracle.VIEW_AR, t2) - run(oracle.VIEW_AR, t)).abs().max() > 1e-3


@pytest.mark.parametrize("view", VIEWS)
def test_rows_past_the_prefix_are_never_read(view):
    t = tiny(seed=33)
    o = run(view, t)
    t2 = {k: v.clone() for k, v in t.items()}
    for b in range(2):
        P = int(t["cache_len"][b])
        t2["k_cache"][b, :, P:] = 1e30
        t2["v_cache"][b, :, P:] = float("nan")
    assert torch.equal(run(view, t2), o)


@pytest.mark.parametrize("view", VIEWS)
def test_explicit_scale_and_default_scale(view):
    t = tiny(seed=34)
    d = t["q_diff"].shape[-1]
    o = run(view, t)
    o2 = run(view, t, scale=1.0 / math.sqrt(d))
    torch.testing.assert_close(o, o2, rtol=0, atol=TOL)
    # doubling q equals doubling the scale
    t2 = {k: v.clone() for k, v in t.items()}
    t2["q_diff"] *= 2; t2["q_ar"] *= 2
    torch.testing.assert_close(run(view, t2), run(view, t, scale=2.0 / math.sqrt(d)),
                               rtol=0, atol=TOL)


@pytest.mark.parametrize("view", VIEWS)
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_narrow_inputs_are_widened_exactly(view, dtype):
    t = tiny(seed=35, dtype=dtype)
    o = run(view, t)
    t64 = {k: (v.double() if v.is_floating_point() else v) for k, v in t.items()}
    assert torch.equal(run(view, t64), o)


@pytest.mark.parametrize("view", VIEWS)
def test_sampled_rows_equal_full_tensor(view):
    t = tiny(seed=36)
    o = run(view, t)
    rows = torch.tensor([[0, 0, 0], [1, 3, 2], [0, 2, 3], [1, 1, 1]], dtype=torch.int32)
    got = oracle.block_attend_rows(view, rows, *args_of(view, t))
    for s, (b, i, hq) in enumerate(rows.tolist()):
        assert torch.equal(got[s], o[b, i, hq])


@pytest.mark.parametrize("view", VIEWS)
def test_split_merge_formula_reproduces_single_pass(view):
    """Partial (max, sum, unnormalised output) triples over two disjoint key sets,
    merged as m = max m_s, l = sum e^{m_s-m} l_s, O = sum e^{m_s-m} O_s / l, equal the
    one-pass oracle result (independent check of the split-KV merge rule)."""
    t = tiny(B=1, K=3, Hq=2, Hkv=1, d=4, P=(11,), cap=16, seed=37)
    o = run(view, t).numpy()
    q, kb, vb, kc, vc, cl = [x.numpy() if x.is_floating_point() else x for x in args_of(view, t)]
    P, K, d = 11, 3, 4
    for i in range(K):
        nb = K if view == oracle.VIEW_DIFFUSION else i + 1
        keys = np.concatenate([kc[0, 0, :P], kb[0, :nb, 0]])
        vals = np.concatenate([vc[0, 0, :P], vb[0, :nb, 0]])
        for hq in range(2):
            s = keys @ q[0, i, hq] / math.sqrt(d)
            parts = []
            for sl in (slice(0, 4), slice(4, None)):
                m = s[sl].max(); e = np.exp(s[sl] - m)
                parts.append((m, e.sum(), e @ vals[sl]))
            m = max(p[0] for p in parts)
            l = sum(math.exp(p[0] - m) * p[1] for p in parts)
            O = sum(math.exp(p[0] - m) * p[2] for p in parts) / l
            np.testing.assert_allclose(O, o[0, i, hq], rtol=0, atol=TOL)


# --------------------------------------------------------------------------- consensus

def _load_cases():
    path = os.path.join(os.path.dirname(__file__), "golden", "consensus_cases.txt")
    cases = []
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        g, y, n, com, nxt = [list(map(int, part.split())) for part in line.split("|")]
        cases.append((g, y, n[0], com, nxt[0]))
    return cases


def _logits_with_argmax(g, V=12, seed=0):
    gen = torch.Generator().manual_seed(seed)
    lg = torch.randn(1, len(g), V, generator=gen, dtype=torch.float32)
    for i, tok in enumerate(g):
        lg[0, i, tok] = 10.0
    return lg


@pytest.mark.parametrize("case", _load_cases())
def test_consensus_hand_worked(case):
    g, y, n, com, nxt = case
    lg = _logits_with_argmax(g)
    n_c, committed, arg, anchor = oracle.consensus_accept(
        lg, torch.tensor([y], dtype=torch.int32))
    assert arg[0].tolist() == g
    assert int(n_c[0]) == n
    assert committed[0].tolist() == com
    assert int(anchor[0]) == nxt


class ToyARModel:
    """A deterministic stand-in for a causal language model: the logits after a
    context are a fixed pseudo-random function of that context."""

    def __init__(self, V, seed):
        self.V, self.seed = V, seed

    def logits(self, context):
        h = hash((self.seed,) + tuple(context)) & 0x7FFFFFFF
        return np.random.RandomState(h).standard_normal(self.V).astype(np.float32)

    def greedy(self, context):
        return int(np.argmax(self.logits(context)))


@pytest.mark.parametrize("seed", range(6))
def test_lossless_equals_sequential_greedy_decoding(seed):
    """Section 3.3's guarantee: cycle after cycle, the committed stream equals
    token-by-token greedy decoding of the same causal model."""
    V, K, total = 50, 5, 40
    model = ToyARModel(V, seed)
    rng = np.random.RandomState(seed)
    prompt = [1, 2, 3]
    # plain AR greedy decode
    ar = list(prompt)
    for _ in range(total + K):
        ar.append(model.greedy(ar))
    # draft/verify cycles; drafts agree with the greedy continuation at a random rate
    seq = list(prompt)
    anchor_ctx = list(prompt)            # context up to and including the anchor x_t
    n_hist = []
    while len(seq) < len(prompt) + total:
        truth = []
        ctx = list(anchor_ctx)
        for _ in range(K):
            tok = model.greedy(ctx); truth.append(tok); ctx.append(tok)
        draft = [tk if rng.rand() < 0.7 else int(rng.randint(V)) for tk in truth]
        # verify rows: row k conditioned on the anchor context and drafts 0..k-1
        rows = np.stack([model.logits(anchor_ctx + draft[:k]) for k in range(K)])
        n_c, committed, _, anchor = oracle.consensus_accept(
            torch.from_numpy(rows).view(1, K, V), torch.tensor([draft], dtype=torch.int32))
        n = int(n_c[0]); n_hist.append(n)
        assert 1 <= n <= K
        toks = committed[0, :n].tolist()
        assert (committed[0, n:] == -1).all()
        seq += toks
        anchor_ctx = anchor_ctx + toks
        assert int(anchor[0]) == toks[-1]
    assert seq == ar[:len(seq)]
    assert max(n_hist) > 1               # the drafts did speed things up


def test_consensus_ties_take_the_lowest_id_and_bounds():
    lg = torch.zeros(2, 3, 9, dtype=torch.bfloat16)
    lg[0, 0, 4] = 1.0; lg[0, 0, 7] = 1.0          # tie between 4 and 7
    lg[0, 1, 8] = 2.0
    lg[0, 2, :] = -float("inf")                    # all -inf: id 0
    lg[1, 0, 0] = -1.0; lg[1, 0, 1:] = -2.0
    lg[1, 1, 3] = 0.5; lg[1, 1, 2] = 0.5
    draft = torch.tensor([[4, 8, 0], [0, 3, 5]], dtype=torch.int32)
    n, com, arg, nxt = oracle.consensus_accept(lg, draft)
    assert arg.tolist() == [[4, 8, 0], [0, 2, 0]]
    assert n.tolist() == [3, 2]
    assert com.tolist() == [[4, 8, 0], [0, 2, -1]]
    assert nxt.tolist() == [0, 2]


@pytest.mark.parametrize("p,K,expect", [(0.7, 8, 3.141), (0.6, 16, 2.499), (0.5, 16, 2.000),
                                        (0.65, 16, 2.854)])
def test_expected_commit_length_statistical(p, K, expect):
    """With independent agreement rate p the committed length is min(Geom, K):
    E[n] = (1 - p^K) / (1 - p); tokens per forward pass = E[n] / 2 (Eq. 9)."""
    assert abs((1 - p ** K) / (1 - p) - expect) < 2e-3
    V, B = 64, 4000
    gen = torch.Generator().manual_seed(1)
    lg = torch.randn(B, K, V, generator=gen)
    g = lg.argmax(-1)
    wl = W.Workload("stat", B, 1, 1, 8, K, V, 1, 1, match_min=p, match_max=p)
    draft = W.drafts(wl, g, seed=7)
    n, *_ = oracle.consensus_accept(lg, draft)
    pe = p + (1 - p) / V                       # chance coincidence of a random draft
    want = (1 - pe ** K) / (1 - pe)
    assert abs(float(n.double().mean()) - want) < 0.08
    assert int(n.min()) >= 1 and int(n.max()) <= K


# --------------------------------------------------------------------------- append

@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_append_bytes(dtype):
    B, K, Hkv, d, cap = 3, 4, 2, 8, 12
    g = torch.Generator().manual_seed(4)
    kc = torch.randn(B, Hkv, cap, d, generator=g).to(dtype)
    vc = torch.randn(B, Hkv, cap, d, generator=g).to(dtype)
    kb = torch.randn(B, K, Hkv, d, generator=g).to(dtype)
    vb = torch.randn(B, K, Hkv, d, generator=g).to(dtype)
    lens = torch.tensor([0, 5, 8], dtype=torch.int32)
    n = torch.tensor([1, 4, 3], dtype=torch.int32)
    kc0, vc0, lens0 = kc.clone(), vc.clone(), lens.clone()
    assert oracle.kv_append(kc, vc, lens, kb, vb, n) == 0
    assert lens.tolist() == [1, 9, 11]
    bits = lambda x: x.view(torch.int16 if dtype == torch.bfloat16 else torch.int32)
    for b in range(B):
        p, nb = int(lens0[b]), int(n[b])
        for cache, cache0, blk in ((kc, kc0, kb), (vc, vc0, vb)):
            assert torch.equal(bits(cache[b, :, :p]), bits(cache0[b, :, :p]))
            assert torch.equal(bits(cache[b, :, p + nb:]), bits(cache0[b, :, p + nb:]))
            for i in range(nb):
                assert torch.equal(bits(cache[b, :, p + i]), bits(blk[b, i]))
    # update_len = False leaves the lengths alone; overflow is refused per sequence
    lens2 = torch.tensor([0, 5, 10], dtype=torch.int32)
    kc2 = kc0.clone(); vc2 = vc0.clone()
    rc = oracle.kv_append(kc2, vc2, lens2, kb, vb, n, update_len=False)
    assert rc == -3 and lens2.tolist() == [0, 5, 10]
    assert torch.equal(bits(kc2[2]), bits(kc0[2]))


def test_append_then_attend_equals_longer_prefix():
    """After committing n AR-view rows, the next cycle's prefix holds exactly
    those rows: attention over the grown cache equals attention computed with
    the rows placed there by hand."""
    t = tiny(B=1, K=4, Hq=2, Hkv=1, d=8, P=(5,), cap=16, seed=40)
    n = torch.tensor([3], dtype=torch.int32)
    kc, vc, cl = t["k_cache"].clone(), t["v_cache"].clone(), t["cache_len"].clone()
    oracle.kv_append(kc, vc, cl, t["k_ar_blk"], t["v_ar_blk"], n)
    t2 = dict(t, k_cache=kc, v_cache=vc, cache_len=cl)
    t3 = {k: v.clone() for k, v in t.items()}
    t3["k_cache"][0, 0, 5:8] = t["k_ar_blk"][0, :3, 0]
    t3["v_cache"][0, 0, 5:8] = t["v_ar_blk"][0, :3, 0]
    t3["cache_len"] = torch.tensor([8], dtype=torch.int32)
    assert torch.equal(run(oracle.VIEW_DIFFUSION, t2), run(oracle.VIEW_DIFFUSION, t3))


# --------------------------------------------------------------------------- workloads

def test_transient_block_kv_is_4p5_mib_on_the_8b_shape():
    """Appendix B: the only extra KV of the diffusion view is the K-position block;
    on the 8B shape (36 layers, 8 KV heads, head_dim 128) at K=32 in bf16 that is
    4.5 MiB."""
    wl = W.CONFIGS["cfg2_8b_b1"].with_(block=32, prefix_min=8, prefix_max=8)
    t = W.attention_inputs(wl)
    per_layer = t["k_diff_blk"].numel() * 2 + t["v_diff_blk"].numel() * 2
    assert per_layer * 36 == int(4.5 * 2 ** 20)


def test_workload_seeding_is_reproducible_and_distinct():
    wl = W.CONFIGS["cfg1_tiny"]
    a = W.attention_inputs(wl)
    b = W.attention_inputs(wl)
    c = W.attention_inputs(wl, layer=1)
    assert all(torch.equal(a[k], b[k]) for k in a)
    assert not torch.equal(a["q_diff"], c["q_diff"])
    assert not torch.equal(a["q_diff"], a["q_ar"])
    assert a["k_cache"].dtype == torch.bfloat16
    assert abs(float(a["k_cache"].float().std()) - 1 / 8) < 5e-3
    r = W.prefix_lengths(W.CONFIGS["cfg3_ragged"])
    assert int(r.min()) >= 1024 and int(r.max()) <= 8192 and len(set(r.tolist())) > 16
