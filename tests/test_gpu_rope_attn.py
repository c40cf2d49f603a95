"""GPU: vt_attn_fwd_rope - attention whose queries are turned by the rotary position embedding inside the kernel -
against the oracle: rotary oracle on Q (and K), then the attention oracle.  The keys handed to the kernel are the
oracle's rotated keys rounded once to bf16 (the entry point's contract is "keys already rotated"), and the attention
oracle gets the same bits; the rotated queries are rounded to bf16 on both sides (that rounding is part of the entry
point's definition), so what is compared is the in-kernel rotation of Q plus the attention."""
import numpy as np
import pytest

from helpers import TOL_LSE, TOL_O, dev, host
from oracle import attn_oracle as orc
from oracle import suite_oracle as so
from paper_2601_16238_b200.inputs import AttnConfig, f32_to_bf16_bits, make_inputs

pytestmark = pytest.mark.gpu

CASES = [
    # B, Hq, Hkv, Sq, Sk, D, causal, q_pos0
    (1, 2, 2, 128, 128, 128, 0, 0),
    (2, 4, 2, 300, 300, 128, 1, 0),            # several tiles, ragged end, GQA
    (1, 2, 2, 200, 456, 64, 2, 256),           # the queries are the last 200 positions of 456 (chunked prefill): offset positions
    (1, 3, 3, 65, 65, 64, 0, 0),
    (1, 10, 10, 2048, 2048, 128, 1, 0),        # one batch entry of the paper's benchmark shape
]


@pytest.mark.parametrize("B,Hq,Hkv,Sq,Sk,D,causal,q_pos0", CASES)
def test_attention_with_in_kernel_query_rotation(vt, B, Hq, Hkv, Sq, Sk, D, causal, q_pos0):
    import torch
    from paper_2601_16238_b200 import suite
    cfg = AttnConfig("rope", 41, B, Hq, Hkv, Sq, Sk, D, causal, False)
    q, k, v = make_inputs(cfg, with_do=False)
    n_pos = max(Sk, q_pos0 + Sq)
    cos64, sin64 = so.rope_tables(n_pos, D)
    qf, kf = orc.bf16_bits_to_f64(q), orc.bf16_bits_to_f64(k)
    k_rot_bits = f32_to_bf16_bits(so.rope_apply(kf, cos64[:Sk], sin64[:Sk]).astype(np.float32))     # keys at positions 0 .. Sk-1
    # the entry point's definition: the rotated queries are rounded to bf16 before the products (as they would be had a
    # separate rotary kernel written them to memory), so the reference rounds them too
    q_rot_bits = f32_to_bf16_bits(so.rope_apply(qf, cos64[q_pos0:q_pos0 + Sq], sin64[q_pos0:q_pos0 + Sq]).astype(np.float32))
    o_ref, lse_ref = orc.attn_fwd(q_rot_bits, k_rot_bits, v, causal, cfg.scale)

    cos, sin = suite.vt_suite_rope_tables(n_pos, D)
    assert np.abs(host(cos) - cos64).max() <= 1e-6            # the device tables are the oracle's, rounded to fp32
    o, lse = vt.vt_attn_fwd_rope(dev(q), dev(k_rot_bits), dev(v), cos, sin, causal, cfg.scale, q_pos0)
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0
    assert np.abs(host(o) - o_ref).max() <= max(TOL_O, 2.0 ** -8 * np.abs(o_ref).max())
    assert (np.abs(host(lse) - lse_ref) <= TOL_LSE * np.maximum(1.0, np.abs(lse_ref))).all()
    # the same thing in two steps: rotate Q with the suite's kernel, then plain attention (the rotated Q is rounded to
    # bf16 either way; the two kernels may contract their multiply-adds differently, so allow a bf16 step on Q's effect)
    q_rot_dev = suite.vt_suite_rope_apply(dev(q), cos[q_pos0:q_pos0 + Sq].contiguous(), sin[q_pos0:q_pos0 + Sq].contiguous())
    o2, lse2 = vt.vt_attn_fwd(q_rot_dev, dev(k_rot_bits), dev(v), causal, cfg.scale)
    torch.cuda.synchronize()
    assert np.abs(host(o) - host(o2)).max() <= 2.0 ** -6 * max(1.0, np.abs(o_ref).max())


def test_rope_entry_point_argument_checks(vt):
    import torch
    from paper_2601_16238_b200 import suite
    q = torch.zeros(1, 2, 64, 128, dtype=torch.bfloat16, device="cuda")
    cos, sin = suite.vt_suite_rope_tables(64, 128)
    with pytest.raises(vt.VtAttnError) as e:
        vt.vt_attn_fwd_rope(q, q, q, cos, sin, 0, 0.1, q_pos0=1)             # positions 1 .. 64 exceed the 64 table rows
    assert e.value.status == vt.ERR_INVALID_ARGUMENT
    q96 = torch.zeros(1, 2, 64, 96, dtype=torch.bfloat16, device="cuda")
    cos96, sin96 = suite.vt_suite_rope_tables(64, 96)
    with pytest.raises(vt.VtAttnError) as e:
        vt.vt_attn_fwd_rope(q96, q96, q96, cos96, sin96, 0, 0.1)
    assert e.value.status == vt.ERR_UNSUPPORTED
    with pytest.raises(ValueError):
        vt.vt_attn_fwd_rope(q, q, q, cos[:, :32].contiguous(), sin[:, :32].contiguous(), 0, 0.1)
