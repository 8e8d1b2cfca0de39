"""The oracle's C code under AddressSanitizer and UndefinedBehaviorSanitizer: a small
run of every entry point (ragged batch, empty prefix, both views, weights requested,
consensus with ties and specials, the LM-head argmax, append with an overflowing sequence) in a child
process, which must finish without a sanitizer report."""
import os
import subprocess
import sys
import tempfile

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r'''
import ctypes, sys, torch
sys.path.insert(0, {root!r})
import oracle
oracle._LIB = {lib!r}
oracle.build = lambda force=False: {lib!r}
g = torch.Generator().manual_seed(0)
B, K, Hq, Hkv, d, cap = 3, 5, 6, 2, 16, 40
mk = lambda *s: (torch.randn(*s, generator=g) * 0.5).to(torch.bfloat16)
q, kb, vb = mk(B, K, Hq, d), mk(B, K, Hkv, d), mk(B, K, Hkv, d)
kc, vc = mk(B, Hkv, cap, d), mk(B, Hkv, cap, d)
lens = torch.tensor([0, 17, 35], dtype=torch.int32)
for view in (oracle.VIEW_DIFFUSION, oracle.VIEW_AR):
    out, w = oracle.block_attend(view, q, kb, vb, kc, vc, lens, return_weights=True)
    assert torch.isfinite(out).all() and abs(float(w.sum(-1).mean()) - 1.0) < 1e-9
    rows = torch.tensor([[0, 0, 0], [2, 4, 5], [1, 2, 3]], dtype=torch.int32)
    r = oracle.block_attend_rows(view, rows, q, kb, vb, kc, vc, lens)
    assert torch.allclose(r[1], out[2, 4, 5])
lg = torch.randn(B, K, 1001, generator=g).to(torch.bfloat16)
lg[0, 0, 7] = 9.0; lg[0, 0, 900] = 9.0; lg[1, 1, :] = float("-inf"); lg[2, 2, 3] = float("nan")
draft = torch.randint(0, 1001, (B, K), generator=g, dtype=torch.int32)
n, com, arg, nxt = oracle.consensus_accept(lg, draft)
assert arg[0, 0] == 7 and 1 <= int(n.min()) and int(n.max()) <= K
rc = oracle.kv_append(kc, vc, lens, kb, vb, torch.tensor([1, 5, 5], dtype=torch.int32))
assert rc == 0 and lens.tolist() == [1, 22, 40]
rc = oracle.kv_append(kc, vc, lens, kb, vb, torch.tensor([1, 1, 1], dtype=torch.int32))
assert rc != 0 and lens.tolist() == [2, 23, 40]
hid, W = mk(B, K, 24), mk(77, 24)
n2, com2, g2, nxt2, top2 = oracle.lm_head_consensus(hid, W, draft % 77)
assert 1 <= int(n2.min()) and int(n2.max()) <= K and bool((top2[..., 0] >= top2[..., 1]).all())
a3, _ = oracle.lm_head_argmax(hid.reshape(B * K, 24), W, torch.tensor([14, 0], dtype=torch.int32))
assert a3.tolist() == [int(g2[2, 4]), int(g2[0, 0])]
print("sanitized run ok")
'''


def test_oracle_under_asan_ubsan():
    asan = subprocess.run(["gcc", "-print-file-name=libasan.so"], capture_output=True, text=True).stdout.strip()
    if not os.path.isabs(asan) or not os.path.exists(asan):
        pytest.skip("no libasan in this toolchain")
    with tempfile.TemporaryDirectory() as tmp:
        lib = os.path.join(tmp, "liborthrus_oracle_san.so")
        subprocess.run(["gcc", "-O1", "-g", "-fopenmp", "-std=c11", "-shared", "-fPIC",
                        "-fsanitize=address,undefined", "-fno-sanitize-recover=undefined",
                        "-o", lib, os.path.join(ROOT, "oracle", "orthrus_oracle.c"), "-lm"], check=True)
        env = dict(os.environ, LD_PRELOAD=asan, OMP_NUM_THREADS="2",
                   ASAN_OPTIONS="detect_leaks=0:abort_on_error=1", UBSAN_OPTIONS="halt_on_error=1")
        r = subprocess.run([sys.executable, "-c", CHILD.format(root=ROOT, lib=lib)], env=env,
                           capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "sanitized run ok" in r.stdout, (r.stdout[-2000:], r.stderr[-4000:])
    assert "ERROR: AddressSanitizer" not in r.stderr and "runtime error" not in r.stderr
