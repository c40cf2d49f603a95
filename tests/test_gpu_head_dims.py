"""GPU parity for head dimensions other than 64 and 128 (any multiple of 8 up to 128; the kernels run them in the next
larger built size, reading the missing columns as zero): forward and backward against the fp64 oracle through every
family of entry points, with the outputs poisoned first so that a column written past a row's end, or one left
unwritten, shows."""
import numpy as np
import pytest

from helpers import TOL_GRAD, TOL_LSE, TOL_O, check_fwd, check_grad, dev, host
from oracle import attn_oracle as orc
from paper_2601_16238_b200.inputs import AttnConfig, make_inputs, normal_bf16, normal_f16

pytestmark = pytest.mark.gpu

SHAPES = [
    # B, Hq, Hkv, Sq, Sk, D, causal
    (2, 4, 4, 200, 200, 96, 1),
    (1, 4, 2, 300, 260, 96, 0),
    (2, 6, 2, 129, 400, 80, 2),
    (1, 2, 2, 257, 257, 72, 1),
    (1, 3, 3, 130, 130, 120, 0),
    (1, 2, 1, 140, 140, 104, 1),
    (2, 4, 4, 150, 150, 32, 1),
    (1, 8, 8, 65, 65, 40, 0),
    (1, 2, 2, 260, 100, 8, 2),           # the smallest dimension; fewer keys than queries (rows without a key)
    (1, 2, 2, 128, 128, 16, 0),
    (1, 4, 4, 384, 384, 56, 1),
    (1, 40, 40, 1024, 1024, 96, 1),      # the causal two-tiles-in-sequence forward kernel
]


@pytest.mark.parametrize("B,Hq,Hkv,Sq,Sk,D,causal", SHAPES)
def test_other_head_dims_match_the_oracle(vt, B, Hq, Hkv, Sq, Sk, D, causal):
    import torch
    cfg = AttnConfig("hd", 21, B, Hq, Hkv, Sq, Sk, D, causal, True)
    q, k, v, d_o = make_inputs(cfg)
    tq, tk, tv, tdo = dev(q), dev(k), dev(v), dev(d_o)
    # the tensors sit inside larger poisoned buffers: anything written past their ends is seen
    def guarded(like):
        buf = torch.full((like.numel() + 256,), float("nan"), dtype=like.dtype, device="cuda")
        return buf, buf[128:128 + like.numel()].view(like.shape)
    o_buf, o = guarded(tq)
    lse = torch.full((B, Hq, Sq), float("nan"), device="cuda")
    vt.vt_attn_fwd(tq, tk, tv, causal, cfg.scale, o, lse)
    bufs, grads = zip(*(guarded(t) for t in (tq, tk, tv)))
    vt.vt_attn_bwd(tq, tk, tv, o, tdo, lse, causal, cfg.scale, *grads)
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0
    for buf in (o_buf,) + bufs:
        assert torch.isnan(buf[:128].float()).all() and torch.isnan(buf[-128:].float()).all(), "wrote outside the tensor"
    if B * Hq * Sq * Sk > 3e7:           # the long case: the oracle on three heads
        heads = [(0, 0), (0, Hq // 2), (B - 1, Hq - 1)]
    else:
        heads = [(b, h) for b in range(B) for h in range(Hq)]
    G = Hq // Hkv
    full = len(heads) == B * Hq
    if full:
        o_ref, lse_ref = orc.attn_fwd(q, k, v, causal, cfg.scale)
        o_h, lse_h = host(o), host(lse)
        assert not np.isnan(o_h).any() and not np.isnan(lse_h).any()
        finite = np.isfinite(lse_ref)
        assert (np.isneginf(lse_h) == ~finite).all() and (o_h[~finite] == 0.0).all()
        assert np.abs(o_h - o_ref).max() <= max(TOL_O, 2.0 ** -8 * np.abs(o_ref).max())
        assert (np.abs(lse_h[finite] - lse_ref[finite]) <= TOL_LSE * np.maximum(1.0, np.abs(lse_ref[finite]))).all()
        refs = orc.attn_bwd(q, k, v, d_o, causal, cfg.scale)
        for nm, a, b in zip(("dQ", "dK", "dV"), grads, refs):
            check_grad(host(a), b, nm, f"D={D}")
    else:
        assert not torch.isnan(o.float()).any() and not torch.isnan(lse).any()
        for g in grads:
            assert not torch.isnan(g.float()).any()
        for b, h in heads:
            o_ref, lse_ref = orc.attn_fwd(q[b:b + 1, h:h + 1], k[b:b + 1, h // G:h // G + 1], v[b:b + 1, h // G:h // G + 1], causal, cfg.scale)
            check_fwd(host(o[b:b + 1, h:h + 1]), host(lse[b:b + 1, h:h + 1]), o_ref, lse_ref, f"D={D} head ({b},{h})")
            if G == 1:
                refs = orc.attn_bwd(q[b:b + 1, h:h + 1], k[b:b + 1, h:h + 1], v[b:b + 1, h:h + 1], d_o[b:b + 1, h:h + 1], causal, cfg.scale)
                for nm, a, r in zip(("dQ", "dK", "dV"), grads, refs):
                    check_grad(host(a[b:b + 1, h:h + 1]), r, nm, f"D={D} head ({b},{h})")


@pytest.mark.parametrize("D", [96, 48])
def test_other_head_dims_fp16(vt, D):
    import torch
    B, Hq, Hkv, Sq, Sk, causal = 1, 4, 2, 200, 230, 2
    scale = float(np.float32(1.0) / np.sqrt(np.float32(D)))
    q, k, v, d_o = (normal_f16(s, 9500 + i) for i, s in enumerate(((B, Hq, Sq, D), (B, Hkv, Sk, D), (B, Hkv, Sk, D), (B, Hq, Sq, D))))
    t = [torch.from_numpy(x.view(np.int16)).view(torch.float16).cuda() for x in (q, k, v, d_o)]
    o = torch.full_like(t[0], float("nan"))
    lse = torch.full((B, Hq, Sq), float("nan"), device="cuda")
    vt.vt_attn_fwd_f16(t[0], t[1], t[2], causal, scale, o, lse)
    grads = [torch.full_like(x, float("nan")) for x in t[:3]]
    vt.vt_attn_bwd_f16(t[0], t[1], t[2], o, t[3], lse, causal, scale, *grads)
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0
    fq, fk, fv, fdo = (orc.f16_bits_to_f64(x) for x in (q, k, v, d_o))
    o_ref, lse_ref = orc.attn_fwd(fq, fk, fv, causal, scale)
    assert np.abs(host(o) - o_ref).max() <= max(TOL_O, 2.0 ** -10 * np.abs(o_ref).max())
    assert (np.abs(host(lse) - lse_ref) <= TOL_LSE * np.maximum(1.0, np.abs(lse_ref))).all()
    for nm, a, b in zip(("dQ", "dK", "dV"), grads, orc.attn_bwd(fq, fk, fv, fdo, causal, scale)):
        check_grad(host(a), b, nm, f"fp16 D={D}")


@pytest.mark.parametrize("D,causal", [(96, True), (24, 2), (112, False)])
def test_other_head_dims_packed(vt, D, causal):
    import torch
    Hq, Hkv = 4, 2
    lens_q, lens_k = [130, 1, 64, 0, 200], [130, 70, 64, 33, 300]
    cu_q = np.concatenate([[0], np.cumsum(lens_q)]).astype(np.int32)
    cu_k = np.concatenate([[0], np.cumsum(lens_k)]).astype(np.int32)
    tq_, tk_ = int(cu_q[-1]), int(cu_k[-1])
    q, k, v, d_o = (normal_bf16(s, 9600 + i) for i, s in enumerate(((tq_, Hq, D), (tk_, Hkv, D), (tk_, Hkv, D), (tq_, Hq, D))))
    scale = float(np.float32(1.0) / np.sqrt(np.float32(D)))
    tq, tk, tv, tdo = dev(q), dev(k), dev(v), dev(d_o)
    cq, ck = torch.from_numpy(cu_q).cuda(), torch.from_numpy(cu_k).cuda()
    o = torch.full_like(tq, float("nan")); lse = torch.full((Hq, tq_), float("nan"), device="cuda")
    vt.vt_attn_fwd_varlen(tq, tk, tv, cq, ck, max(lens_q), max(lens_k), causal, scale, o, lse)
    grads = [torch.full_like(x, float("nan")) for x in (tq, tk, tv)]
    vt.vt_attn_bwd_varlen(tq, tk, tv, o, tdo, lse, cq, ck, max(lens_q), max(lens_k), causal, scale, *grads)
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0
    o_ref, lse_ref = orc.attn_fwd_varlen(q, k, v, cu_q, cu_k, causal, scale)
    o_h, lse_h = host(o), host(lse)
    assert not np.isnan(o_h).any() and not np.isnan(lse_h).any()
    assert np.abs(o_h - o_ref).max() <= max(TOL_O, 2.0 ** -8 * np.abs(o_ref).max())
    finite = np.isfinite(lse_ref)
    assert (np.isneginf(lse_h) == ~finite).all()
    assert (np.abs(lse_h[finite] - lse_ref[finite]) <= TOL_LSE * np.maximum(1.0, np.abs(lse_ref[finite]))).all()
    for nm, a, b in zip(("dQ", "dK", "dV"), grads, orc.attn_bwd_varlen(q, k, v, d_o, cu_q, cu_k, causal, scale)):
        a = host(a)
        assert not np.isnan(a).any(), nm
        assert np.abs(a - b).max() <= TOL_GRAD * np.abs(b).max() + 1e-5, nm


@pytest.mark.parametrize("B,Hq,Hkv,Sq,Sk,D,causal,n_splits", [
    (2, 8, 2, 1, 1000, 96, 2, 0),        # decoding, the heads of a group share a tile
    (1, 4, 4, 3, 700, 40, 0, 4),
    (1, 2, 1, 200, 1500, 80, 2, 3),
])
def test_other_head_dims_splitkv(vt, B, Hq, Hkv, Sq, Sk, D, causal, n_splits):
    import torch
    cfg = AttnConfig("hd_split", 22, B, Hq, Hkv, Sq, Sk, D, causal, False)
    q, k, v = make_inputs(cfg, with_do=False)
    tq, tk, tv = dev(q), dev(k), dev(v)
    o = torch.full_like(tq, float("nan"))
    lse = torch.full(tq.shape[:3], float("nan"), device="cuda")
    vt.vt_attn_fwd_splitkv(tq, tk, tv, causal, cfg.scale, n_splits, o, lse)
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0
    o_ref, lse_ref = orc.attn_fwd(q, k, v, causal, cfg.scale)
    check_fwd(host(o), host(lse), o_ref, lse_ref, f"split D={D}")


def test_merge_kernels_other_head_dim(vt):
    """The running merge of partial results and the gradient accumulation at D = 96 against plain fp64 arithmetic
    (the definition: weights exp(LSE_part - LSE_total))."""
    import torch
    n, D = 777, 96
    rng = np.random.default_rng(5)
    parts = [torch.from_numpy(rng.standard_normal((n, D)).astype(np.float32)).bfloat16().cuda() for _ in range(3)]
    lses = [torch.from_numpy(rng.standard_normal(n).astype(np.float32) * 3).cuda() for _ in range(3)]
    o_acc = torch.full((n, D), float("nan"), device="cuda"); lse_acc = torch.full((n,), float("nan"), device="cuda")
    for i, (p_, l_) in enumerate(zip(parts, lses)):
        vt.vt_attn_merge_partial(o_acc, lse_acc, p_, l_, first=(i == 0))
    out = torch.full((n, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    vt.vt_attn_merge_finish(o_acc, out)
    acc = torch.full((n, D), float("nan"), device="cuda")
    for i, p_ in enumerate(parts):
        vt.vt_attn_accumulate_partial(acc, p_, first=(i == 0))
    torch.cuda.synchronize()
    L = np.stack([host(l_) for l_ in lses]); P = np.stack([host(p_) for p_ in parts])
    tot = np.log(np.exp(L).sum(0))
    want = (np.exp(L - tot)[:, :, None] * P).sum(0)
    assert np.abs(host(lse_acc) - tot).max() <= 1e-5 * np.abs(tot).max() + 1e-5
    assert np.abs(host(o_acc) - want).max() <= 1e-5
    assert np.abs(host(out) - want).max() <= 2.0 ** -8 * np.abs(want).max()
    assert np.abs(host(acc) - P.sum(0)).max() <= 1e-5


@pytest.mark.parametrize("B,Hq,Hkv,Sq,Sk,D,causal", [
    (1, 4, 2, 300, 300, 256, 1),
    (2, 2, 2, 129, 400, 192, 2),
    (1, 3, 3, 200, 260, 136, 0),
    (1, 2, 1, 1100, 1100, 256, 1),
    (1, 2, 2, 65, 65, 224, 0),
])
def test_forward_head_dims_up_to_256(vt, B, Hq, Hkv, Sq, Sk, D, causal):
    """Head dimensions above 128 exist in the forward only (one block per SM, O takes 256 tensor-memory columns); the
    backward answers VT_ATTN_ERR_UNSUPPORTED."""
    import torch
    cfg = AttnConfig("hd256", 23, B, Hq, Hkv, Sq, Sk, D, causal, False)
    q, k, v = make_inputs(cfg, with_do=False)
    tq, tk, tv = dev(q), dev(k), dev(v)
    o = torch.full_like(tq, float("nan"))
    lse = torch.full((B, Hq, Sq), float("nan"), device="cuda")
    vt.vt_attn_fwd(tq, tk, tv, causal, cfg.scale, o, lse)
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0
    o_ref, lse_ref = orc.attn_fwd(q, k, v, causal, cfg.scale)
    check_fwd(host(o), host(lse), o_ref, lse_ref, f"D={D}")
    assert vt.vt_attn_bwd_kernel_kind(B, Hq, Hkv, Sq, Sk, D) == 2          # the backward above 128 columns: tests/test_gpu_bwd_wide.py


def test_forward_head_dim_256_fp16_and_splitkv(vt):
    import torch
    B, Hq, Hkv, Sq, Sk, D = 1, 8, 2, 1, 3000, 256
    cfg = AttnConfig("hd256s", 24, B, Hq, Hkv, Sq, Sk, D, 2, False)
    q, k, v = make_inputs(cfg, with_do=False)
    o, lse = vt.vt_attn_fwd_splitkv(dev(q), dev(k), dev(v), 2, cfg.scale, 0)
    torch.cuda.synchronize()
    o_ref, lse_ref = orc.attn_fwd(q, k, v, 2, cfg.scale)
    check_fwd(host(o), host(lse), o_ref, lse_ref, "split D=256")
    scale = float(np.float32(1.0) / np.sqrt(np.float32(192)))
    qh, kh, vh = (normal_f16(s, 9700 + i) for i, s in enumerate(((1, 2, 260, 192), (1, 2, 260, 192), (1, 2, 260, 192))))
    t = [torch.from_numpy(x.view(np.int16)).view(torch.float16).cuda() for x in (qh, kh, vh)]
    o, lse = vt.vt_attn_fwd_f16(t[0], t[1], t[2], 1, scale)
    torch.cuda.synchronize()
    o_ref, lse_ref = orc.attn_fwd(*(orc.f16_bits_to_f64(x) for x in (qh, kh, vh)), 1, scale)
    assert np.abs(host(o) - o_ref).max() <= max(TOL_O, 2.0 ** -10 * np.abs(o_ref).max())
    assert (np.abs(host(lse) - lse_ref) <= TOL_LSE * np.maximum(1.0, np.abs(lse_ref))).all()


@pytest.mark.parametrize("B,Hq,Hkv,Sq,Sk,D,Dv,causal", [
    (1, 4, 2, 300, 300, 192, 128, 1),        # wider Q / K than V
    (2, 2, 2, 129, 400, 128, 64, 2),
    (1, 2, 2, 200, 260, 64, 128, 0),         # narrower Q / K than V
    (1, 3, 1, 140, 140, 72, 40, 1),
    (1, 2, 2, 520, 520, 256, 256, 1),        # equal widths: the same as vt_attn_fwd
])
def test_forward_with_its_own_v_width(vt, B, Hq, Hkv, Sq, Sk, D, Dv, causal):
    import torch
    q, k = (normal_bf16(s, 9800 + i) for i, s in enumerate(((B, Hq, Sq, D), (B, Hkv, Sk, D))))
    v = normal_bf16((B, Hkv, Sk, Dv), 9802)
    scale = float(np.float32(1.0) / np.sqrt(np.float32(D)))
    tq, tk, tv = dev(q), dev(k), dev(v)
    buf = torch.full((B * Hq * Sq * Dv + 256,), float("nan"), dtype=torch.bfloat16, device="cuda")
    o = buf[128:128 + B * Hq * Sq * Dv].view(B, Hq, Sq, Dv)
    lse = torch.full((B, Hq, Sq), float("nan"), device="cuda")
    vt.vt_attn_fwd_dv(tq, tk, tv, causal, scale, o, lse)
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0
    assert torch.isnan(buf[:128].float()).all() and torch.isnan(buf[-128:].float()).all(), "wrote outside the tensor"
    # the oracle on tensors padded with zero columns to a common width: zero columns of Q and K add nothing to the
    # scores, zero columns of V give zero columns of O
    W = max(D, Dv)
    pad = lambda bits, w: np.concatenate([orc.bf16_bits_to_f64(bits), np.zeros(bits.shape[:3] + (W - w,))], axis=-1)      # noqa: E731
    o_ref, lse_ref = orc.attn_fwd(pad(q, D), pad(k, D), pad(v, Dv), causal, scale)
    assert (o_ref[..., Dv:] == 0).all()
    check_fwd(host(o), host(lse), o_ref[..., :Dv], lse_ref, f"D={D} Dv={Dv}")
    if D == Dv:
        o1, lse1 = vt.vt_attn_fwd(tq, tk, tv, causal, scale)
        torch.cuda.synchronize()
        assert torch.equal(o1, o) and torch.equal(lse1, lse)


@pytest.mark.parametrize("D", [96, 192, 256])
def test_host_buffer_entry_points_with_another_head_dim(vt, D):
    """The host-buffer entry points stage rows of the real length (D = 96: 192-byte rows) and give the bits of the device
    path, also above 128 columns (the backward in two column halves)."""
    import torch
    cfg = AttnConfig("hd_host", 25, 3, 4, 2, 300, 300, D, 1, True)
    bits = make_inputs(cfg)
    hq, hk, hv, hdo = (torch.from_numpy(x.view(np.int16)).view(torch.bfloat16).pin_memory() for x in bits)
    ho = torch.empty_like(hq).pin_memory(); hlse = torch.empty(hq.shape[:3], dtype=torch.float32).pin_memory()
    hdq = torch.empty_like(hq).pin_memory(); hdk = torch.empty_like(hk).pin_memory(); hdv = torch.empty_like(hv).pin_memory()
    dims = (cfg.B, cfg.Hq, cfg.Hkv, cfg.Sq, cfg.Sk, cfg.D)
    staging = torch.empty(vt.vt_attn_host_staging_bytes(*dims, True), dtype=torch.uint8, device="cuda")
    vt.vt_attn_fwd_bwd_host(hq, hk, hv, hdo, ho, hlse, hdq, hdk, hdv, cfg.causal, cfg.scale, staging)
    torch.cuda.synchronize()
    q, k, v, d_o = (dev(x) for x in bits)
    o, lse = vt.vt_attn_fwd(q, k, v, cfg.causal, cfg.scale)
    dq, dk, dv = vt.vt_attn_bwd(q, k, v, o, d_o, lse, cfg.causal, cfg.scale)
    torch.cuda.synchronize()
    for a, b in ((ho, o), (hlse, lse), (hdq, dq), (hdk, dk), (hdv, dv)):
        assert torch.equal(a, b.cpu())
