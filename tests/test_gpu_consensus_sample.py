"""GPU parity of the sampled consensus (temperature > 0) against the oracle.

Every decision the rule takes compares two floating-point quantities (u*q(y) with p(y);
u*total with a running sum).  The kernel evaluates the exponentials in fp32 (sums in
double, fixed order), the oracle everything in fp64, so a comparison that is within
rounding of a tie may legitimately fall either way.  The oracle reports, per sequence,
how far its decisions were from flipping: the nearest accept test relative to the
quantities compared, and the resampling point relative to the width of the chosen
token's residual mass.  Sequences whose accept margin exceeds 1e-4 and whose resampling
point is more than 1 % of the token's width away from its edges (nearly all) must agree
bit for bit; the rest are only checked for validity."""
import pytest
import torch

import oracle
from _gpu_util import Guarded, binding

pytestmark = pytest.mark.gpu
MARGIN_ACCEPT, MARGIN_PICK = 1e-4, 1e-2


def run_gpu(la, ld, draft, ua, ur, T):
    b = binding()
    B, K, V = la.shape
    ws = b.new_workspace(b.orthrus_consensus_sample_workspace_bytes(B, K, V))
    outs = [Guarded((B,), torch.int32), Guarded((B, K), torch.int32), Guarded((B,), torch.int32)]
    b.orthrus_consensus_sample(la.cuda(), ld.cuda(), draft.cuda(), ua.float().cuda(), ur.float().cuda(), T,
                               outs[0].t, outs[1].t, outs[2].t, ws)
    torch.cuda.synchronize()
    assert all(o.intact() for o in outs)
    return [o.t.cpu() for o in outs]


def make_case(B, K, V, dtype, seed, keep=0.7, spread=1.0):
    g = torch.Generator().manual_seed(seed)
    la = (torch.randn(B, K, V, generator=g) * spread).to(dtype)
    ld = (la.float() + 0.7 * torch.randn(B, K, V, generator=g)).to(dtype)     # a related draft model
    q = torch.softmax(ld.float(), -1)
    draft = torch.multinomial(q.view(-1, V), 1, generator=g).view(B, K).to(torch.int32)
    ua = torch.rand(B, K, generator=g).float()
    ur = torch.rand(B, K, generator=g).float()
    return la, ld, draft.contiguous(), ua, ur


def check(la, ld, draft, ua, ur, T, min_decided=0.9):
    n, com, nxt = run_gpu(la, ld, draft, ua, ur, T)
    rn, rcom, rnxt, margin = oracle.consensus_sample(la, ld, draft, ua.double(), ur.double(), T)
    B, K, V = la.shape
    decided = (margin[:, 0] > MARGIN_ACCEPT) & (margin[:, 1] > MARGIN_PICK)
    assert int((~decided).sum()) <= max(1, int((1 - min_decided) * B)), margin      # near ties are rare
    assert torch.equal(n[decided], rn[decided])
    assert torch.equal(com[decided], rcom[decided])
    assert torch.equal(nxt[decided], rnxt[decided])
    # validity everywhere: 1 <= n <= K, kept drafts first, padding, anchor, token ids in range
    for s in range(B):
        k = int(n[s])
        assert 1 <= k <= K
        assert com[s, :k - 1].tolist() == draft[s, :k - 1].tolist()
        assert com[s, k:].tolist() == [-1] * (K - k)
        assert 0 <= int(com[s, k - 1]) < V and int(nxt[s]) == int(com[s, k - 1])
    return rn


@pytest.mark.parametrize("B,K,V", [(1, 8, 1000), (3, 5, 1001), (2, 16, 32000), (4, 3, 33), (1, 1, 7),
                                   (2, 32, 4099), (1, 16, 151936), (16, 4, 8192)])
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_sampled_consensus_matches_oracle(B, K, V, dtype):
    la, ld, draft, ua, ur = make_case(B, K, V, dtype, seed=B * 1000 + K)
    rn = check(la, ld, draft, ua, ur, 0.9)
    assert int(rn.min()) >= 1


def test_at_the_ragged_serving_size():
    """Batch 32, block 32, vocabulary 128256 (the largest logits tensor of the benchmark
    configurations), bf16."""
    la, ld, draft, ua, ur = make_case(32, 32, 128256, torch.bfloat16, seed=5)
    rn = check(la, ld, draft, ua, ur, 1.0)
    assert 1.0 < float(rn.double().mean()) < 32.0


@pytest.mark.parametrize("T", [0.3, 1.0, 2.5])
def test_temperatures(T):
    la, ld, draft, ua, ur = make_case(6, 8, 5000, torch.bfloat16, seed=17, spread=2.0)
    check(la, ld, draft, ua, ur, T)


def test_every_draft_kept_and_immediate_rejection():
    g = torch.Generator().manual_seed(9)
    B, K, V = 3, 6, 2000
    la = torch.randn(B, K, V, generator=g).to(torch.bfloat16)
    draft = torch.randint(0, V, (B, K), generator=g, dtype=torch.int32)
    ua = torch.rand(B, K, generator=g)
    ur = torch.rand(B, K, generator=g)
    n, com, nxt = run_gpu(la, la.clone(), draft, ua, ur, 1.0)          # p == q: nothing can be rejected
    assert n.tolist() == [K] * B and torch.equal(com, draft) and torch.equal(nxt, draft[:, -1])
    # a draft model that puts all its mass where the AR model has none: rejected at once
    ld = torch.full((B, K, V), -30.0)
    la2 = la.float().clone()
    for s in range(B):
        for k in range(K):
            ld[s, k, draft[s, k]] = 30.0
            la2[s, k, draft[s, k]] = -60.0
    check(la2.to(torch.bfloat16), ld.to(torch.bfloat16), draft, ua, ur, 1.0)
    n, com, _ = run_gpu(la2.to(torch.bfloat16), ld.to(torch.bfloat16), draft, ua, ur, 1.0)
    assert n.tolist() == [1] * B and (com[:, 0] != draft[:, 0]).all()


def test_distribution_of_the_committed_token_on_the_gpu():
    """One position, many sequences: the committed tokens follow the AR distribution."""
    g = torch.Generator().manual_seed(21)
    V, N = 16, 4000
    la = (torch.randn(V, generator=g) * 1.5).to(torch.float32)
    ld = (torch.randn(V, generator=g) * 1.5).to(torch.float32)
    p, q = torch.softmax(la.double(), -1), torch.softmax(ld.double(), -1)
    draft = torch.multinomial(q, N, replacement=True, generator=g).to(torch.int32).view(N, 1)
    ua, ur = torch.rand(N, 1, generator=g), torch.rand(N, 1, generator=g)
    n, com, _ = run_gpu(la.expand(N, 1, V).contiguous(), ld.expand(N, 1, V).contiguous(), draft, ua, ur, 1.0)
    freq = torch.bincount(com[:, 0].long(), minlength=V).double() / N
    assert ((freq - p).abs() <= 4.5 * (p * (1 - p) / N).sqrt() + 1e-9).all()


def test_rejects_bad_arguments_on_the_host():
    b = binding()
    f = b.lib().orthrus_consensus_sample
    import ctypes
    args = [0x1000, 0x2000, 0, 0x3000, 0x4000, 0x5000, ctypes.c_float(1.0), 2, 4, 100,
            0x6000, 0x7000, 0x8000, 0x9000, 1 << 20, None]
    n0 = b.orthrus_launch_count()
    bad_T = list(args); bad_T[6] = ctypes.c_float(0.0)
    assert f(*bad_T) == 1
    small = list(args); small[14] = 64
    assert f(*small) == 4
    null = list(args); null[1] = None
    assert f(*null) == 1
    assert b.orthrus_launch_count() == n0


def test_staged_verification_in_a_child_process():
    """Large problems verify the block in two stages (the second only for sequences without a
    rejection so far).  The stage boundary is chosen when the library is first used, so the
    small cases above are repeated in a child process with the boundary forced to 2 positions:
    rejections before, at and after the boundary, and blocks kept whole."""
    import os
    import subprocess
    import sys
    env = dict(os.environ, ORTHRUS_SAMPLE_FIRST_STAGE="2")
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.abspath(__file__), "-x", "-q",
                        "-k", "matches_oracle or temperatures or every_draft_kept or distribution"],
                       env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout
