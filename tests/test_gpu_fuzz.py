"""Seeded random shapes through the forward and backward entry points against the fp64 oracle: batch, heads, group size,
both sequence lengths (from a single row up to several tiles with ragged tails), every head dimension the library takes
and all three mask modes, in combinations nobody wrote down by hand."""
import os

import numpy as np
import pytest

from helpers import TOL_GRAD, TOL_LSE, TOL_O, dev, host
from oracle import attn_oracle as orc
from paper_2601_16238_b200.inputs import AttnConfig, make_inputs

pytestmark = pytest.mark.gpu

# VT_FUZZ_SCALE=k multiplies the number of random cases of every test in this file (default 1: what a normal test run
# does; the tolerance floors quoted in the design notes come from a run with 70, about 2 500 batched and 1 100 packed cases)
SCALE = max(1, int(os.environ.get("VT_FUZZ_SCALE", "1")))


def zero_floor(n_terms):
    """Absolute slack for gradients that are exactly zero in exact arithmetic (a single visible key: P = 1, dS = 0, so dQ
    and dK vanish): the kernel's dS is then the fp32 rounding of <dO, v> - <dO, o> (~1e-6 of either for N(0,1) data),
    and a gradient sums n_terms of them with random signs."""
    return max(1e-5, 2e-6 * float(np.sqrt(n_terms)))


def grad_tol(nm, ref, q, k, d_o, o, scale, rows, keys):
    """Tolerance for one gradient: the relative bound on its largest element, the floor for exactly-zero gradients, and,
    for dQ and dK, what the bf16 rounding of O costs.  The backward's row term delta_i = <dO_i, O_i> reads the rounded
    output, so it is off by up to 2^-9 sum_d |dO_id O_id|; with one or two visible keys dP - delta cancels almost
    completely, the gradient itself is small, and that error is no longer small beside it.  It reaches dQ_i through
    scale * sum_j P_ij K_j (weights summing to 1) and dK_j through scale * sum_i P_ij Q_i (random signs over the rows)."""
    tol = TOL_GRAD * np.abs(ref).max() + zero_floor(max(rows, keys))
    if nm != "dV":
        d_delta = 2.0 ** -9 * np.abs(d_o.astype(np.float64) * o.astype(np.float64)).sum(-1).max()
        other = np.abs(k).max() if nm == "dQ" else np.abs(q).max() * np.sqrt(rows)
        tol += scale * d_delta * float(other)
    return tol


def _cases(n, seed, max_d):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        hkv = int(rng.integers(1, 4))
        g = int(rng.choice([1, 1, 2, 4]))
        sq = int(rng.choice([int(rng.integers(1, 16)), int(rng.integers(16, 300)), int(rng.integers(300, 700))]))
        sk = sq if rng.random() < 0.4 else int(rng.choice([int(rng.integers(1, 16)), int(rng.integers(16, 300)), int(rng.integers(300, 900))]))
        d = 8 * int(rng.integers(1, max_d // 8 + 1))
        out.append((int(rng.integers(1, 4)), hkv * g, hkv, sq, sk, d, int(rng.integers(0, 3)), 5000 + i))
    return out


@pytest.mark.parametrize("B,Hq,Hkv,Sq,Sk,D,causal,seed", _cases(36 * SCALE, 1, 128))
def test_random_shapes_forward_and_backward(vt, B, Hq, Hkv, Sq, Sk, D, causal, seed):
    import torch
    cfg = AttnConfig("fuzz", seed, B, Hq, Hkv, Sq, Sk, D, causal, True)
    q, k, v, d_o = make_inputs(cfg)
    tq, tk, tv, tdo = dev(q), dev(k), dev(v), dev(d_o)
    o = torch.full_like(tq, float("nan"))
    lse = torch.full((B, Hq, Sq), float("nan"), device="cuda")
    vt.vt_attn_fwd(tq, tk, tv, causal, cfg.scale, o, lse)
    grads = [torch.full_like(t, float("nan")) for t in (tq, tk, tv)]
    vt.vt_attn_bwd(tq, tk, tv, o, tdo, lse, causal, cfg.scale, *grads)
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0
    o_ref, lse_ref = orc.attn_fwd(q, k, v, causal, cfg.scale)
    o_h, lse_h = host(o), host(lse)
    assert not np.isnan(o_h).any() and not np.isnan(lse_h).any()
    finite = np.isfinite(lse_ref)
    assert (np.isneginf(lse_h) == ~finite).all() and (o_h[~finite] == 0.0).all()
    # rows that see a key or two reproduce V, |O| can exceed 4 there: allow the bf16 rounding of the output
    assert np.abs(o_h - o_ref).max() <= max(TOL_O, 2.0 ** -8 * np.abs(o_ref).max())
    assert (np.abs(lse_h[finite] - lse_ref[finite]) <= TOL_LSE * np.maximum(1.0, np.abs(lse_ref[finite]))).all()
    for nm, a, b in zip(("dQ", "dK", "dV"), grads, orc.attn_bwd(q, k, v, d_o, causal, cfg.scale)):
        a = host(a)
        assert not np.isnan(a).any(), nm
        assert np.abs(a - b).max() <= grad_tol(nm, b, q, k, d_o, o_h, cfg.scale, Sq * (Hq // Hkv), Sk), nm


def _wide_cases(n, seed):
    return [c[:5] + (136 + 8 * (c[7] * 7 % 16),) + c[6:] for c in _cases(n, seed, 128)]      # D in 136 .. 256


@pytest.mark.parametrize("B,Hq,Hkv,Sq,Sk,D,causal,seed", _wide_cases(16 * SCALE, 5))
def test_random_shapes_backward_above_128_columns(vt, B, Hq, Hkv, Sq, Sk, D, causal, seed):
    import torch
    cfg = AttnConfig("fuzz_wide", seed, B, Hq, Hkv, Sq, Sk, D, causal, True)
    q, k, v, d_o = make_inputs(cfg)
    tq, tk, tv, tdo = dev(q), dev(k), dev(v), dev(d_o)
    o, lse = vt.vt_attn_fwd(tq, tk, tv, causal, cfg.scale)
    grads = [torch.full_like(t, float("nan")) for t in (tq, tk, tv)]
    vt.vt_attn_bwd(tq, tk, tv, o, tdo, lse, causal, cfg.scale, *grads)
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0
    o_h = host(o)
    for nm, a, b in zip(("dQ", "dK", "dV"), grads, orc.attn_bwd(q, k, v, d_o, causal, cfg.scale)):
        a = host(a)
        assert not np.isnan(a).any(), nm
        assert np.abs(a - b).max() <= grad_tol(nm, b, q, k, d_o, o_h, cfg.scale, Sq * (Hq // Hkv), Sk), nm


@pytest.mark.parametrize("B,Hq,Hkv,Sq,Sk,D,causal,seed", [c for c in _cases(40 * SCALE, 6, 128) if c[5] > 64][:12 * SCALE])
def test_random_shapes_single_pass_backward(vt, B, Hq, Hkv, Sq, Sk, D, causal, seed):
    """The opt-in single-pass backward (fixed-point dQ accumulation) on random shapes with 64 < D <= 128."""
    import os
    import torch
    cfg = AttnConfig("fuzz_fused", seed, B, Hq, Hkv, Sq, Sk, D, causal, True)
    q, k, v, d_o = make_inputs(cfg)
    tq, tk, tv, tdo = dev(q), dev(k), dev(v), dev(d_o)
    o, lse = vt.vt_attn_fwd(tq, tk, tv, causal, cfg.scale)
    old = os.environ.get("VT_ATTN_BWD_PATH")
    os.environ["VT_ATTN_BWD_PATH"] = "fused"
    try:
        assert vt.vt_attn_bwd_kernel_kind(B, Hq, Hkv, Sq, Sk, D) == 1
        grads = vt.vt_attn_bwd(tq, tk, tv, o, tdo, lse, causal, cfg.scale)
    finally:
        if old is None:
            os.environ.pop("VT_ATTN_BWD_PATH", None)
        else:
            os.environ["VT_ATTN_BWD_PATH"] = old
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0
    o_h = host(o)
    for nm, a, b in zip(("dQ", "dK", "dV"), grads, orc.attn_bwd(q, k, v, d_o, causal, cfg.scale)):
        a = host(a)
        assert not np.isnan(a).any(), nm
        assert np.abs(a - b).max() <= grad_tol(nm, b, q, k, d_o, o_h, cfg.scale, Sq * (Hq // Hkv), Sk), nm


@pytest.mark.parametrize("B,Hq,Hkv,Sq,Sk,D,causal,seed", _cases(16 * SCALE, 2, 256))
def test_random_shapes_forward_wide_heads_and_splitkv(vt, B, Hq, Hkv, Sq, Sk, D, causal, seed):
    import torch
    cfg = AttnConfig("fuzz", seed, B, Hq, Hkv, Sq, Sk, D, causal, False)
    q, k, v = make_inputs(cfg, with_do=False)
    tq, tk, tv = dev(q), dev(k), dev(v)
    o_ref, lse_ref = orc.attn_fwd(q, k, v, causal, cfg.scale)
    finite = np.isfinite(lse_ref)
    for name, call in (("fwd", lambda: vt.vt_attn_fwd(tq, tk, tv, causal, cfg.scale)),
                       ("splitkv", lambda: vt.vt_attn_fwd_splitkv(tq, tk, tv, causal, cfg.scale, int(seed % 5)))):
        o, lse = call()
        torch.cuda.synchronize()
        assert vt.vt_attn_device_status()[0] == 0
        o_h, lse_h = host(o), host(lse)
        assert (np.isneginf(lse_h) == ~finite).all() and (o_h[~finite] == 0.0).all(), name
        assert np.abs(o_h - o_ref).max() <= max(TOL_O, 2.0 ** -7 * np.abs(o_ref).max()), name
        assert (np.abs(lse_h[finite] - lse_ref[finite]) <= TOL_LSE * np.maximum(1.0, np.abs(lse_ref[finite]))).all(), name


def _packed_cases(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        n_seq = int(rng.integers(1, 7))
        lens_q = [int(rng.choice([0, int(rng.integers(1, 40)), int(rng.integers(40, 400))])) for _ in range(n_seq)]
        if sum(lens_q) == 0:
            lens_q[0] = 5
        same = rng.random() < 0.5
        lens_k = list(lens_q) if same else [int(rng.choice([0, int(rng.integers(1, 40)), int(rng.integers(40, 500))])) for _ in range(n_seq)]
        if sum(lens_k) == 0:
            lens_k[-1] = 9
        hkv = int(rng.integers(1, 3))
        out.append((hkv * int(rng.choice([1, 2, 4])), hkv, 8 * int(rng.integers(1, 17)), int(rng.integers(0, 3)), lens_q, lens_k, 6000 + i))
    return out


@pytest.mark.parametrize("Hq,Hkv,D,causal,lens_q,lens_k,seed", _packed_cases(16 * SCALE, 3))
def test_random_packed_batches(vt, Hq, Hkv, D, causal, lens_q, lens_k, seed):
    import torch
    from paper_2601_16238_b200.inputs import normal_bf16
    cu_q = np.concatenate([[0], np.cumsum(lens_q)]).astype(np.int32)
    cu_k = np.concatenate([[0], np.cumsum(lens_k)]).astype(np.int32)
    tq_, tk_ = int(cu_q[-1]), int(cu_k[-1])
    q, k, v, d_o = (normal_bf16(s, seed * 10 + i) for i, s in enumerate(((tq_, Hq, D), (tk_, Hkv, D), (tk_, Hkv, D), (tq_, Hq, D))))
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
    finite = np.isfinite(lse_ref)
    assert (np.isneginf(lse_h) == ~finite).all()
    assert np.abs(o_h - o_ref).max() <= max(TOL_O, 2.0 ** -8 * np.abs(o_ref).max())
    assert (np.abs(lse_h[finite] - lse_ref[finite]) <= TOL_LSE * np.maximum(1.0, np.abs(lse_ref[finite]))).all()
    for nm, a, b in zip(("dQ", "dK", "dV"), grads, orc.attn_bwd_varlen(q, k, v, d_o, cu_q, cu_k, causal, scale)):
        a = host(a)
        assert not np.isnan(a).any(), nm
        assert np.abs(a - b).max() <= grad_tol(nm, b, q, k, d_o, o_h, scale, max(lens_q) * (Hq // Hkv), max(lens_k)), nm


@pytest.mark.parametrize("Hq,Hkv,D,causal,lens_q,lens_k,seed", _packed_cases(12 * SCALE, 4))
def test_random_packed_batches_splitkv(vt, Hq, Hkv, D, causal, lens_q, lens_k, seed):
    import torch
    from paper_2601_16238_b200.inputs import normal_bf16
    cu_q = np.concatenate([[0], np.cumsum(lens_q)]).astype(np.int32)
    cu_k = np.concatenate([[0], np.cumsum(lens_k)]).astype(np.int32)
    tq_, tk_ = int(cu_q[-1]), int(cu_k[-1])
    q, k, v = (normal_bf16(s, seed * 10 + i) for i, s in enumerate(((tq_, Hq, D), (tk_, Hkv, D), (tk_, Hkv, D))))
    scale = float(np.float32(1.0) / np.sqrt(np.float32(D)))
    tq, tk, tv = dev(q), dev(k), dev(v)
    cq, ck = torch.from_numpy(cu_q).cuda(), torch.from_numpy(cu_k).cuda()
    o = torch.full_like(tq, float("nan")); lse = torch.full((Hq, tq_), float("nan"), device="cuda")
    vt.vt_attn_fwd_splitkv_varlen(tq, tk, tv, cq, ck, max(lens_q), max(lens_k), causal, scale, int(seed % 4), o, lse)
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0
    o_ref, lse_ref = orc.attn_fwd_varlen(q, k, v, cu_q, cu_k, causal, scale)
    o_h, lse_h = host(o), host(lse)
    assert not np.isnan(o_h).any() and not np.isnan(lse_h).any()
    finite = np.isfinite(lse_ref)
    assert (np.isneginf(lse_h) == ~finite).all()
    assert np.abs(o_h - o_ref).max() <= max(TOL_O, 2.0 ** -7 * np.abs(o_ref).max())
    assert (np.abs(lse_h[finite] - lse_ref[finite]) <= TOL_LSE * np.maximum(1.0, np.abs(lse_ref[finite]))).all()
