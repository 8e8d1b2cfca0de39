"""The consensus entry point that allocates nothing.

Some users of this library run where device memory cannot be allocated: a plugin inside
a host runtime that owns all allocations, or a server whose memory budget is frozen
before the first request.  They can pass inputs and outputs but no workspace, so
orthrus_consensus_accept_static keeps its scratch in an array built into the library.
This file checks, through the C ABI, that it returns exactly what the workspace variant
returns (every output is an integer, so "within tolerance" means identical), on two
calls in a row with different inputs - the second call finds the first call's leftovers
in the shared array - and that an oversized problem is refused before anything runs.

It is collected last on purpose: a run that stops at the first failure has then already
exercised every other test.
"""
import ctypes

import pytest
import torch

pytestmark = pytest.mark.gpu


def _both(b, logits, draft):
    B, K, V = logits.shape
    lg, dr = logits.cuda(), draft.cuda()
    i32 = dict(dtype=torch.int32, device="cuda")
    ref = [torch.full((B,), -7, **i32), torch.full((B, K), -7, **i32),
           torch.full((B, K), -7, **i32), torch.full((B,), -7, **i32)]
    got = [torch.full_like(t, -9) for t in ref]
    ws = b.new_workspace(b.orthrus_consensus_workspace_bytes(B, K, V))
    b.orthrus_consensus_accept(lg, dr, *ref, ws)
    b.orthrus_consensus_accept_static(lg, dr, *got)
    torch.cuda.synchronize()
    return [t.cpu() for t in ref], [t.cpu() for t in got]


def test_static_consensus_matches_workspace_variant_twice_in_a_row():
    from paper_2605_12825_b200 import binding as b
    g = torch.Generator().manual_seed(77)
    # second problem is smaller and differently shaped: stale pairs of the first call stay
    # in the array beyond what the second call writes
    for (B, K, V, dt) in [(3, 16, 40000, torch.bfloat16), (2, 5, 1001, torch.float32)]:
        logits = torch.randn(B, K, V, generator=g).to(dt)
        top = logits.float().argmax(-1).to(torch.int32)         # only to plant agreeing drafts
        coin = torch.rand(B, K, generator=g) < 0.7
        draft = torch.where(coin, top, torch.randint(0, V, (B, K), generator=g, dtype=torch.int32))
        ref, got = _both(b, logits, draft.contiguous())
        for r, o, name in zip(ref, got, ("n_commit", "committed", "ar_argmax", "next_anchor")):
            assert torch.equal(r, o), name
        assert int(ref[0].min()) >= 1


def test_static_consensus_refuses_what_does_not_fit():
    from paper_2605_12825_b200 import binding as b
    f = b.lib().orthrus_consensus_accept_static
    n0 = b.orthrus_launch_count()
    # 9000 rows need 9000 * 8 bytes of scratch at the very least: more than the array holds
    rc = f(0x1000, 0, 0x2000, 9000, 1, 64, 0x3000, 0x4000, 0x5000, 0x6000, None)
    assert rc == 4 and b.orthrus_launch_count() == n0
    assert b.STATIC_CONSENSUS_SCRATCH_BYTES < 9000 * 8
