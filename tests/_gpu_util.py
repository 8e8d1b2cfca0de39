"""Helpers of the GPU parity tests: move a seeded workload to the device, run the
C-ABI calls, and compare with the CPU oracle under the stated tolerances."""
import os

import torch

import oracle
from paper_2605_12825_b200 import workloads as W

# bf16 inputs against the fp64 oracle: max-abs 2e-2 and max-abs / max|ref| 1e-2
# (both gates); fp32 test mode: 1e-5 on both.
TOL = {torch.bfloat16: (2e-2, 1e-2), torch.float32: (1e-5, 1e-5)}

SENTINEL = 12345.0


def binding():
    from paper_2605_12825_b200 import binding as b
    return b


def to_dev(t):
    return {k: v.cuda() for k, v in t.items()}


class Guarded:
    """A device tensor embedded in a larger sentinel-filled buffer."""

    def __init__(self, shape, dtype, pad=1024):
        n = 1
        for s in shape:
            n *= s
        self.buf = torch.full((n + 2 * pad,), SENTINEL, dtype=dtype, device="cuda")
        self.pad, self.n = pad, n
        self.t = self.buf[pad:pad + n].view(*shape)

    def intact(self):
        return bool((self.buf[:self.pad] == SENTINEL).all()) and \
            bool((self.buf[self.pad + self.n:] == SENTINEL).all())


def run_attend(view, t, wl, max_len_hint=None, path=None, splits=None, flags=0):
    """Runs one attention call on device copies of `t`; returns (out_cpu, status, path)."""
    b = binding()
    d = to_dev(t)
    hint = int(t["cache_len"].max()) if max_len_hint is None else max_len_hint
    layer = b.make_layer(d["k_cache"], d["v_cache"], d["cache_len"], wl.n_q_heads, wl.block, hint,
                         0.0, flags)
    old = os.environ.pop("ORTHRUS_SPLITS", None)
    if splits:
        os.environ["ORTHRUS_SPLITS"] = str(splits)
    try:
        ws = b.new_workspace(b.orthrus_attend_workspace_bytes(layer))
        out = Guarded(tuple(t["q_diff"].shape), t["q_diff"].dtype)
        b.orthrus_set_path(path or "auto")
        if view == oracle.VIEW_DIFFUSION:
            b.orthrus_diffusion_block_attend(layer, d["q_diff"], d["k_diff_blk"], d["v_diff_blk"],
                                             out.t, ws)
        else:
            b.orthrus_ar_verify_attend(layer, d["q_ar"], d["k_ar_blk"], d["v_ar_blk"], out.t, ws)
        used = b.orthrus_last_path()
        status = b.orthrus_read_status(ws)
    finally:
        b.orthrus_set_path("auto")
        os.environ.pop("ORTHRUS_SPLITS", None)
        if old is not None:
            os.environ["ORTHRUS_SPLITS"] = old
    assert out.intact(), "attention wrote outside its output tensor"
    return out.t.cpu(), status, used


def oracle_attend(view, t):
    if view == oracle.VIEW_DIFFUSION:
        return oracle.block_attend(view, t["q_diff"], t["k_diff_blk"], t["v_diff_blk"],
                                   t["k_cache"], t["v_cache"], t["cache_len"])
    return oracle.block_attend(view, t["q_ar"], t["k_ar_blk"], t["v_ar_blk"],
                               t["k_cache"], t["v_cache"], t["cache_len"])


def oracle_attend_rows(view, rows, t):
    if view == oracle.VIEW_DIFFUSION:
        return oracle.block_attend_rows(view, rows, t["q_diff"], t["k_diff_blk"], t["v_diff_blk"],
                                        t["k_cache"], t["v_cache"], t["cache_len"])
    return oracle.block_attend_rows(view, rows, t["q_ar"], t["k_ar_blk"], t["v_ar_blk"],
                                    t["k_cache"], t["v_cache"], t["cache_len"])


# element-wise criterion next to the two tensor-level gates: |gpu - ref| <= r * rms(ref) + r * |ref|
# with r the relative tolerance of the dtype, on at least this share of the elements (an error
# confined to small elements or to a few rows passes the tensor-level gates but not this one)
ELEMENTWISE_FLOOR = 0.999


def assert_close(got, ref, dtype, what=""):
    atol, rtol = TOL[dtype]
    got = got.double()
    assert torch.isfinite(got).all(), f"{what}: non-finite output"
    diff = (got - ref).abs()
    err = float(diff.max())
    scale = float(ref.abs().max())
    assert err <= atol, f"{what}: max-abs {err:.3e} > {atol}"
    assert err <= rtol * scale, f"{what}: max-abs {err:.3e} > {rtol} * max|ref| {scale:.3e}"
    rms = float(ref.pow(2).mean().sqrt())
    share = float((diff <= rtol * rms + rtol * ref.abs()).double().mean())
    assert share >= ELEMENTWISE_FLOOR, f"{what}: only {share:.5f} of the elements within {rtol} (rms + |ref|)"
    return err, scale


def small_workload(B, K, Hq, Hkv, d, pmin, pmax, dtype="bf16", V=64, std=1.0, name=None):
    return W.Workload(name or f"t_{B}_{K}_{Hq}_{Hkv}_{d}_{pmin}_{pmax}_{dtype}", B, Hq, Hkv, d, K,
                      V, pmin, pmax, value_std=std, dtype=dtype)
