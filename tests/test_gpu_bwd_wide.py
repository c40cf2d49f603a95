"""GPU: the backward for head dimensions above 128 (up to 256): Delta, a dK/dV kernel that keeps 128 keys x 256 columns
stationary and walks the queries 64 at a time (in two blocks: one accumulates dK, the other dV), and a dQ kernel that
keeps 128 queries stationary and walks the keys 64 at a time - against the fp64 oracle, element by element."""
import numpy as np
import pytest

from helpers import check_fwd, check_grad, dev, host
from oracle import attn_oracle as orc
from paper_2601_16238_b200.inputs import AttnConfig, make_inputs

pytestmark = pytest.mark.gpu

SHAPES = [
    # B, Hq, Hkv, Sq, Sk, D, causal
    (1, 1, 1, 128, 128, 256, 0),
    (1, 2, 2, 64, 64, 256, 1),
    (1, 2, 1, 200, 333, 256, 0),          # ragged ends, two heads per KV head
    (2, 4, 2, 300, 300, 192, 1),          # the other common size: 192 = 3 boxes of 64 columns
    (1, 2, 2, 257, 129, 136, 1),          # eight columns in the second half; top-left mask with Sq > Sk
    (1, 2, 1, 190, 450, 256, 2),          # bottom-right aligned mask
    (1, 2, 2, 450, 190, 200, 2),          # fewer keys than queries: leading rows see nothing
    (1, 3, 3, 1, 1, 256, 1),
    (1, 2, 2, 640, 640, 256, 1),
    (1, 2, 1, 4096, 4096, 256, 0),        # two full-length heads of the benchmark's d256_s4096_nc workload (one KV head)
    (1, 2, 2, 2048, 2048, 256, 1),
]


@pytest.mark.parametrize("B,Hq,Hkv,Sq,Sk,D,causal", SHAPES)
def test_backward_above_128_columns_matches_the_oracle(vt, B, Hq, Hkv, Sq, Sk, D, causal):
    import torch
    cfg = AttnConfig("wide", 24, B, Hq, Hkv, Sq, Sk, D, causal, True)
    q, k, v, d_o = make_inputs(cfg)
    tq, tk, tv, tdo = dev(q), dev(k), dev(v), dev(d_o)
    assert vt.vt_attn_bwd_kernel_kind(B, Hq, Hkv, Sq, Sk, D) == 2
    o, lse = vt.vt_attn_fwd(tq, tk, tv, causal, cfg.scale)
    dq, dk, dv = (torch.full_like(t, float("nan")) for t in (tq, tk, tv))
    ws = torch.full((max(64, vt.vt_attn_bwd_workspace_bytes(B, Hq, Hkv, Sq, Sk, D) // 4),), float("nan"), device="cuda").view(torch.uint8)
    vt.vt_attn_bwd(tq, tk, tv, o, tdo, lse, causal, cfg.scale, dq, dk, dv, ws)
    again = vt.vt_attn_bwd(tq, tk, tv, o, tdo, lse, causal, cfg.scale)
    torch.cuda.synchronize()
    rc, detail = vt.vt_attn_device_status()
    assert rc == 0, f"device status {rc} detail {detail:#x}"
    for a, b in zip((dq, dk, dv), again):
        assert torch.equal(a, b)
    o_ref, lse_ref = orc.attn_fwd(q, k, v, causal, cfg.scale)
    finite = np.isfinite(lse_ref)
    assert np.abs(host(o) - o_ref).max() <= max(1e-2, 2.0 ** -8 * np.abs(o_ref).max())
    assert (np.abs(host(lse)[finite] - lse_ref[finite]) <= 1e-3 * np.maximum(1.0, np.abs(lse_ref[finite]))).all()
    refs = orc.attn_bwd(q, k, v, d_o, causal, cfg.scale)
    for name, a, ref in zip(("dQ", "dK", "dV"), (dq, dk, dv), refs):
        check_grad(host(a), ref, name, f"wide {cfg}")


def test_backward_above_128_columns_fp16(vt):
    import torch
    from paper_2601_16238_b200.inputs import normal_f16
    B, Hq, Hkv, Sq, Sk, D, causal = 1, 4, 2, 260, 390, 256, 1
    scale = float(np.float32(1.0) / np.sqrt(np.float32(D)))
    bits = [normal_f16(s, 9470 + i) for i, s in enumerate(((B, Hq, Sq, D), (B, Hkv, Sk, D), (B, Hkv, Sk, D), (B, Hq, Sq, D)))]
    q, k, v, d_o = (torch.from_numpy(np.ascontiguousarray(x).view(np.int16)).view(torch.float16).cuda() for x in bits)
    o, lse = vt.vt_attn_fwd_f16(q, k, v, causal, scale)
    got = vt.vt_attn_bwd_f16(q, k, v, o, d_o, lse, causal, scale)
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0
    refs = orc.attn_bwd(*(orc.f16_bits_to_f64(x) for x in bits), causal, scale)
    for name, a, ref in zip(("dQ", "dK", "dV"), got, refs):
        check_grad(host(a), ref, name, "wide fp16")


@pytest.mark.parametrize("B,Hq,Hkv,Sq,Sk,D,Dv,causal", [
    (1, 4, 2, 300, 300, 192, 128, 1),      # the 192 / 128 pair
    (2, 2, 2, 200, 333, 128, 256, 0),      # V wider than Q / K
    (1, 2, 1, 129, 257, 64, 128, 2),       # both within 128 columns: still the kernels that take two widths
    (1, 2, 2, 260, 260, 256, 72, 1),
])
def test_backward_with_v_of_its_own_width(vt, B, Hq, Hkv, Sq, Sk, D, Dv, causal):
    """vt_attn_bwd_dv against the oracle on tensors padded with zero columns to a common width: zero columns of Q and K
    add nothing to the scores and get zero gradients, zero columns of V and dO give zero columns of dV."""
    import torch
    from paper_2601_16238_b200.inputs import normal_bf16
    scale = float(np.float32(1.0) / np.sqrt(np.float32(D)))
    q, k, v, d_o = (normal_bf16(s, 9500 + i) for i, s in enumerate(((B, Hq, Sq, D), (B, Hkv, Sk, D), (B, Hkv, Sk, Dv), (B, Hq, Sq, Dv))))
    tq, tk, tv, tdo = dev(q), dev(k), dev(v), dev(d_o)
    o, lse = vt.vt_attn_fwd_dv(tq, tk, tv, causal, scale)
    dq, dk, dv = vt.vt_attn_bwd_dv(tq, tk, tv, o, tdo, lse, causal, scale)
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0
    assert dq.shape == tq.shape and dk.shape == tk.shape and dv.shape == tv.shape
    W = max(D, Dv)
    pad = lambda bits, w: np.concatenate([orc.bf16_bits_to_f64(bits), np.zeros(bits.shape[:3] + (W - w,))], axis=-1)      # noqa: E731
    gq, gk, gv = orc.attn_bwd(pad(q, D), pad(k, D), pad(v, Dv), pad(d_o, Dv), causal, scale)
    assert (gq[..., D:] == 0).all() and (gk[..., D:] == 0).all() and (gv[..., Dv:] == 0).all()
    for name, a, ref in (("dQ", dq, gq[..., :D]), ("dK", dk, gk[..., :D]), ("dV", dv, gv[..., :Dv])):
        check_grad(host(a), ref, name, f"D={D} Dv={Dv}")
