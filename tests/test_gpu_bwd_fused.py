"""GPU: the single-pass backward (one key-tile-stationary kernel forms dK, dV and adds its share of dQ into a fixed-point
accumulator) against the fp64 oracle, element by element.  The library does not pick it by itself (it measured slower
than the two-kernel path); VT_ATTN_BWD_PATH=fused selects it.  Also: bit-identity from run to run, agreement with the
two-kernel path."""
import os

import numpy as np
import pytest

from helpers import check_fwd, check_grad, dev, host
from oracle import attn_oracle as orc
from paper_2601_16238_b200.inputs import AttnConfig, make_inputs

pytestmark = pytest.mark.gpu


class forced_path:
    def __init__(self, which):
        self.which = which

    def __enter__(self):
        self.old = os.environ.get("VT_ATTN_BWD_PATH")
        os.environ["VT_ATTN_BWD_PATH"] = self.which

    def __exit__(self, *exc):
        if self.old is None:
            os.environ.pop("VT_ATTN_BWD_PATH", None)
        else:
            os.environ["VT_ATTN_BWD_PATH"] = self.old


SHAPES = [
    # B, Hq, Hkv, Sq, Sk, D, causal
    (1, 1, 1, 128, 128, 128, 0),
    (1, 2, 2, 256, 256, 128, 1),
    (1, 4, 2, 640, 640, 128, 1),          # GQA 2:1, five tiles
    (2, 4, 1, 333, 450, 128, 0),          # ragged ends, cross-attention lengths, four heads per KV head
    (1, 2, 1, 300, 700, 128, 2),          # bottom-right aligned mask
    (1, 2, 2, 700, 300, 128, 2),          # fewer keys than queries: leading rows see nothing
    (1, 2, 2, 257, 129, 128, 1),          # top-left aligned mask, Sq > Sk
    (1, 2, 2, 384, 384, 96, 1),           # a head dimension that runs in the 128-column kernel with zero columns
    (1, 3, 3, 200, 520, 72, 0),
    (1, 1, 1, 1, 1, 128, 1),
    (1, 2, 1, 1, 300, 128, 0),
]


@pytest.mark.parametrize("B,Hq,Hkv,Sq,Sk,D,causal", SHAPES)
def test_single_pass_backward_matches_the_oracle(vt, B, Hq, Hkv, Sq, Sk, D, causal):
    import torch
    cfg = AttnConfig("fused", 21, B, Hq, Hkv, Sq, Sk, D, causal, True)
    q, k, v, d_o = make_inputs(cfg)
    tq, tk, tv, tdo = dev(q), dev(k), dev(v), dev(d_o)
    o, lse = vt.vt_attn_fwd(tq, tk, tv, causal, cfg.scale)
    with forced_path("fused"):
        assert vt.vt_attn_bwd_kernel_kind(B, Hq, Hkv, Sq, Sk, D) == 1
        runs = [vt.vt_attn_bwd(tq, tk, tv, o, tdo, lse, causal, cfg.scale) for _ in range(3)]
    with forced_path("split"):
        assert vt.vt_attn_bwd_kernel_kind(B, Hq, Hkv, Sq, Sk, D) == 0
        split = vt.vt_attn_bwd(tq, tk, tv, o, tdo, lse, causal, cfg.scale)
    torch.cuda.synchronize()
    rc, detail = vt.vt_attn_device_status()
    assert rc == 0, f"device status {rc} detail {detail:#x}"
    for other in runs[1:]:
        for a, b in zip(runs[0], other):
            assert torch.equal(a, b), "the single-pass backward must give the same bits on every run"
    refs = orc.attn_bwd(q, k, v, d_o, causal, cfg.scale)
    for name, a, ref in zip(("dQ", "dK", "dV"), runs[0], refs):
        check_grad(host(a), ref, name, f"single-pass {cfg}")
    # the two paths round differently (fp32 sums in tensor memory against fixed-point sums of per-tile products) but
    # compute the same thing: they agree far inside the tolerance against the oracle
    for name, a, b, ref in zip(("dQ", "dK", "dV"), runs[0], split, refs):
        assert np.abs(host(a) - host(b)).max() <= 1e-2 * np.abs(ref).max() + 1e-5, name


def test_single_pass_backward_fp16(vt):
    import torch
    from paper_2601_16238_b200.inputs import normal_f16
    B, Hq, Hkv, Sq, Sk, D, causal = 1, 4, 2, 400, 530, 128, 2
    scale = float(np.float32(1.0) / np.sqrt(np.float32(D)))
    bits = [normal_f16(s, 9370 + i) for i, s in enumerate(((B, Hq, Sq, D), (B, Hkv, Sk, D), (B, Hkv, Sk, D), (B, Hq, Sq, D)))]
    q, k, v, d_o = (torch.from_numpy(np.ascontiguousarray(x).view(np.int16)).view(torch.float16).cuda() for x in bits)
    o, lse = vt.vt_attn_fwd_f16(q, k, v, causal, scale)
    with forced_path("fused"):
        got = vt.vt_attn_bwd_f16(q, k, v, o, d_o, lse, causal, scale)
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0
    refs = orc.attn_bwd(*(orc.f16_bits_to_f64(x) for x in bits), causal, scale)
    for name, a, ref in zip(("dQ", "dK", "dV"), got, refs):
        check_grad(host(a), ref, name, "single-pass fp16")


def test_single_pass_backward_on_a_long_sequence_with_a_poisoned_workspace(vt):
    """(1, 16, 4, 2048, 2048, 128) causal, 16 tiles per head and more blocks than SMs: all of dQ, dK, dV against the
    oracle, a poisoned workspace, the same bits twice; and a workspace that only holds Delta gets the two-kernel path."""
    import torch
    cfg = AttnConfig("fused_long", 22, 1, 16, 4, 2048, 2048, 128, True, True)
    dims = (cfg.B, cfg.Hq, cfg.Hkv, cfg.Sq, cfg.Sk, cfg.D)
    assert vt.vt_attn_bwd_kernel_kind(*dims) == 0            # the library's own choice is the two-kernel path
    q, k, v, d_o = make_inputs(cfg)
    tq, tk, tv, tdo = dev(q), dev(k), dev(v), dev(d_o)
    o, lse = vt.vt_attn_fwd(tq, tk, tv, True, cfg.scale)
    refs = orc.attn_bwd(q, k, v, d_o, True, cfg.scale)
    with forced_path("fused"):
        assert vt.vt_attn_bwd_kernel_kind(*dims) == 1
        ws = torch.full((vt.vt_attn_bwd_workspace_bytes(*dims) // 4,), float("nan"), device="cuda").view(torch.uint8)
        a = vt.vt_attn_bwd(tq, tk, tv, o, tdo, lse, True, cfg.scale, workspace=ws)
        b = vt.vt_attn_bwd(tq, tk, tv, o, tdo, lse, True, cfg.scale, workspace=ws)      # finds the first call's sums in the workspace
        small = torch.empty(cfg.B * cfg.Hq * cfg.Sq * 4, dtype=torch.uint8, device="cuda")
        c = vt.vt_attn_bwd(tq, tk, tv, o, tdo, lse, True, cfg.scale, workspace=small)
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0
    for x, y in zip(a, b):
        assert torch.equal(x, y)
    for name, x, ref in zip(("dQ", "dK", "dV"), a, refs):
        check_grad(host(x), ref, name, "single-pass, long sequence")
    for name, x, ref in zip(("dQ", "dK", "dV"), c, refs):
        check_grad(host(x), ref, name, "two-kernel path with the small workspace")


def test_fixed_point_scale_follows_the_size_of_the_gradients(vt):
    """dO scaled by 2^-20 and by 2^12: the accumulator's unit follows max |dO| (a bound on the sums, not a fixed unit), so
    tiny and huge upstream gradients keep the same relative accuracy."""
    import torch
    cfg = AttnConfig("fused_scale", 23, 1, 2, 2, 512, 512, 128, True, True)
    q, k, v, d_o = make_inputs(cfg)
    tq, tk, tv = dev(q), dev(k), dev(v)
    o, lse = vt.vt_attn_fwd(tq, tk, tv, True, cfg.scale)
    refs = orc.attn_bwd(q, k, v, d_o, True, cfg.scale)
    for mult in (2.0 ** -20, 2.0 ** 12):
        tdo = (dev(d_o).float() * mult).to(torch.bfloat16)         # exact: a power of two
        with forced_path("fused"):
            got = vt.vt_attn_bwd(tq, tk, tv, o, tdo, lse, True, cfg.scale)
        torch.cuda.synchronize()
        for name, a, ref in zip(("dQ", "dK", "dV"), got, refs):
            check_grad(host(a) / mult, ref, name, f"dO x {mult}")
    assert vt.vt_attn_device_status()[0] == 0
