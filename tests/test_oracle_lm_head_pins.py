"""Pins of the oracle's greedy consensus taken straight from the last hidden states
(logit = hidden row . LM-head row, then Eq. 8 and the halt/commit rule of Section 3.3),
none of which retypes its loops:
  * planted maxima: one-hot hidden rows select a column of the LM head, whose largest
    entry is known by construction (a transposed or mis-strided operand fails this);
  * small-integer operands make every logit an exact integer, so the logits-based rule
    (pinned elsewhere) on the library matrix product must give identical outputs, ties
    and all;
  * the library matrix product in float64 agrees on random bf16 operands wherever the
    reported margin is not a rounding-level tie, and the reported top-2 values are the
    two largest entries of that product;
  * duplicated LM-head rows tie and the smallest id wins; a NaN never wins;
  * row subsets give the rows of the full result;
  * the accept rule on given greedy tokens against a sequential walk written as data.
"""
import numpy as np
import pytest
import torch

import oracle


def test_one_hot_hidden_rows_select_planted_maxima():
    g = torch.Generator().manual_seed(3)
    V, H, R = 37, 12, 12
    W = torch.rand(V, H, generator=g, dtype=torch.float64)          # in [0, 1)
    planted = torch.randint(0, V, (H,), generator=g)
    for c in range(H):
        W[planted[c], c] = 2.0 + c                                    # the largest entry of column c
    cols = torch.randperm(H, generator=g)[:R]
    hidden = torch.zeros(R, H, dtype=torch.float64)
    hidden[torch.arange(R), cols] = 3.0
    arg, top2 = oracle.lm_head_argmax(hidden, W)
    assert arg.tolist() == planted[cols].tolist()
    assert torch.allclose(top2[:, 0], 3.0 * (2.0 + cols.double()))
    # a negative one-hot flips the order: the smallest entry of the column wins
    arg_neg, _ = oracle.lm_head_argmax(-hidden, W)
    assert arg_neg.tolist() == W[:, cols].argmin(0).tolist()


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32, torch.float64])
def test_integer_operands_agree_with_the_logits_rule_exactly(dtype):
    g = torch.Generator().manual_seed(11)
    B, K, V, H = 5, 6, 23, 9
    hidden = torch.randint(-3, 4, (B, K, H), generator=g).to(dtype)
    W = torch.randint(-3, 4, (V, H), generator=g).to(dtype)           # many exact ties
    logits = (hidden.double().reshape(B * K, H) @ W.double().T).reshape(B, K, V).float()
    ref_arg = torch.from_numpy(np.argmax(logits.numpy(), axis=-1).astype(np.int32))   # first maximum
    draft = ref_arg.clone()
    flip = torch.rand(B, K, generator=g) < 0.35
    draft[flip] = (draft[flip] + 1) % V
    n0, com0, arg0, nxt0 = oracle.consensus_accept(logits.contiguous(), draft)
    n1, com1, arg1, nxt1, top2 = oracle.lm_head_consensus(hidden, W, draft)
    assert torch.equal(arg1, ref_arg) and torch.equal(arg0, arg1)
    assert torch.equal(n0, n1) and torch.equal(com0, com1) and torch.equal(nxt0, nxt1)
    assert torch.equal(top2[..., 0], logits.double().max(-1).values)
    assert (top2[..., 1] <= top2[..., 0]).all()


def test_library_matrix_product_on_random_bf16_operands():
    g = torch.Generator().manual_seed(5)
    R, V, H = 9, 301, 96                                              # V != H: a transposed read fails
    hidden = torch.randn(R, H, generator=g).to(torch.bfloat16)
    W = (torch.randn(V, H, generator=g) / H ** 0.5).to(torch.bfloat16)
    arg, top2 = oracle.lm_head_argmax(hidden, W)
    ref = hidden.double().numpy() @ W.double().numpy().T
    srt = np.sort(ref, axis=1)
    assert np.allclose(top2[:, 0].numpy(), srt[:, -1], rtol=1e-13, atol=1e-13)
    assert np.allclose(top2[:, 1].numpy(), srt[:, -2], rtol=1e-13, atol=1e-13)
    clear = (srt[:, -1] - srt[:, -2]) > 1e-9
    assert clear.all()
    assert arg.tolist() == np.argmax(ref, axis=1).tolist()


def test_ties_take_the_smallest_id_and_nan_never_wins():
    H = 4
    W = torch.tensor([[0.5, 0, 0, 0], [1, 0, 0, 0], [1, 0, 0, 0], [float("nan"), 0, 0, 0], [1, 0, 0, 0]],
                     dtype=torch.float32)
    hidden = torch.tensor([[2.0, 0, 0, 0]], dtype=torch.float32)
    arg, top2 = oracle.lm_head_argmax(hidden, W)
    assert arg.tolist() == [1]
    assert top2[0].tolist() == [2.0, 2.0]                             # the runner-up is the tied id 2
    # a single vocabulary entry: no runner-up
    arg, top2 = oracle.lm_head_argmax(hidden, W[:1].contiguous())
    assert arg.tolist() == [0] and top2[0, 0] == 1.0 and top2[0, 1] == -float("inf")


def test_row_subsets_are_rows_of_the_full_result():
    g = torch.Generator().manual_seed(9)
    R, V, H = 20, 57, 16
    hidden = torch.randn(R, H, generator=g).to(torch.bfloat16)
    W = torch.randn(V, H, generator=g).to(torch.bfloat16)
    arg, top2 = oracle.lm_head_argmax(hidden, W)
    rows = torch.tensor([19, 0, 7, 7, 3], dtype=torch.int32)
    a2, t2 = oracle.lm_head_argmax(hidden, W, rows)
    assert torch.equal(a2, arg[rows.long()]) and torch.equal(t2, top2[rows.long()])
    with pytest.raises(ValueError):
        oracle.lm_head_argmax(hidden, W, torch.tensor([R], dtype=torch.int32))


def test_accept_rule_cases_written_out():
    # (greedy tokens, drafts) -> (n, committed, next anchor), from the rule of Section 3.3:
    # drafts are kept while they equal the greedy token, the first mismatch contributes the
    # correction token, a fully agreeing block commits K tokens.
    cases = [
        ([5, 6, 7, 8], [5, 6, 7, 8], 4, [5, 6, 7, 8], 8),
        ([5, 6, 7, 8], [9, 6, 7, 8], 1, [5, -1, -1, -1], 5),
        ([5, 6, 7, 8], [5, 6, 0, 8], 3, [5, 6, 7, -1], 7),
        ([5, 6, 7, 8], [5, 6, 7, 0], 4, [5, 6, 7, 8], 8),
        ([5, 6, 7, 8], [5, 0, 7, 8], 2, [5, 6, -1, -1], 6),
    ]
    g = torch.tensor([c[0] for c in cases], dtype=torch.int32)
    d = torch.tensor([c[1] for c in cases], dtype=torch.int32)
    n, com, nxt = oracle.accept_rule(g, d)
    assert n.tolist() == [c[2] for c in cases]
    assert com.tolist() == [c[3] for c in cases]
    assert nxt.tolist() == [c[4] for c in cases]
