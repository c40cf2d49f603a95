"""GPU parity for packed (variable-length) batches against the oracle's per-sequence results."""
import numpy as np
import pytest

from helpers import TOL_GRAD, TOL_LSE, TOL_O, dev, host
from oracle import attn_oracle as orc
from paper_2601_16238_b200.inputs import normal_bf16

pytestmark = pytest.mark.gpu

CASES = [
    # name, Hq, Hkv, D, causal, query lengths, key lengths (None = same as queries)
    ("self_causal_d128", 4, 2, 128, True, [300, 1, 128, 129, 64, 65, 511], None),
    ("self_noncausal_d64", 6, 6, 64, False, [65, 65, 200, 17, 128, 2], None),
    ("cross_noncausal_d128", 2, 1, 128, False, [10, 257, 128, 1], [300, 5, 128, 77]),
    ("cross_causal_d64_with_empty", 4, 4, 64, True, [130, 0, 40, 7, 260], [100, 50, 0, 300, 260]),
    ("many_short_d64", 2, 2, 64, True, [3, 9, 1, 31, 64, 2, 5, 127, 33, 8, 70, 4], None),
    # causal = 2: bottom-right aligned inside every sequence (decode / chunked prefill against a cache);
    # sequences with fewer keys than queries have leading rows without any visible key (O = 0, LSE = -inf)
    ("bottom_right_d128", 4, 2, 128, 2, [5, 128, 64, 200, 1, 0, 300], [70, 128, 300, 131, 513, 40, 300]),
    ("bottom_right_d64", 2, 2, 64, 2, [1, 1, 130, 40, 257], [1, 700, 129, 400, 100]),
]


def _run(vt, Hq, Hkv, D, causal, lens_q, lens_k, seed):
    import torch
    lens_k = lens_q if lens_k is None else lens_k
    cu_q = np.concatenate([[0], np.cumsum(lens_q)]).astype(np.int32)
    cu_k = np.concatenate([[0], np.cumsum(lens_k)]).astype(np.int32)
    tq, tk = int(cu_q[-1]), int(cu_k[-1])
    q, k, v, d_o = (normal_bf16(s, seed + i) for i, s in enumerate(((tq, Hq, D), (tk, Hkv, D), (tk, Hkv, D), (tq, Hq, D))))
    scale = float(np.float32(1.0) / np.sqrt(np.float32(D)))
    dq_, dk_, dv_, ddo = dev(q), dev(k), dev(v), dev(d_o)
    cq, ck = torch.from_numpy(cu_q).cuda(), torch.from_numpy(cu_k).cuda()
    # poison the outputs: every element must be written
    o = torch.full_like(dq_, float("nan")); lse = torch.full((Hq, tq), float("nan"), device="cuda")
    vt.vt_attn_fwd_varlen(dq_, dk_, dv_, cq, ck, max(lens_q), max(lens_k), causal, scale, o, lse)
    gq, gk, gv = (torch.full_like(t, float("nan")) for t in (dq_, dk_, dv_))
    vt.vt_attn_bwd_varlen(dq_, dk_, dv_, o, ddo, lse, cq, ck, max(lens_q), max(lens_k), causal, scale, gq, gk, gv)
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0
    return (q, k, v, d_o, cu_q, cu_k, scale), (o, lse, gq, gk, gv)


@pytest.mark.parametrize("name,Hq,Hkv,D,causal,lens_q,lens_k", CASES)
def test_packed_batches_match_the_oracle(vt, name, Hq, Hkv, D, causal, lens_q, lens_k):
    (q, k, v, d_o, cu_q, cu_k, scale), (o, lse, gq, gk, gv) = _run(vt, Hq, Hkv, D, causal, lens_q, lens_k, 8100)
    o_ref, lse_ref = orc.attn_fwd_varlen(q, k, v, cu_q, cu_k, causal, scale)
    o_h, lse_h = host(o), host(lse)
    assert not np.isnan(o_h).any() and not np.isnan(lse_h).any()
    # rows that see one or two keys reproduce V itself, |O| can exceed 4 there: allow bf16 rounding of the output
    assert np.abs(o_h - o_ref).max() <= max(TOL_O, 2.0 ** -8 * np.abs(o_ref).max())
    finite = np.isfinite(lse_ref)
    assert (np.isneginf(lse_h) == ~finite).all()                 # sequences without keys: LSE = -inf exactly
    assert (np.abs(lse_h[finite] - lse_ref[finite]) <= TOL_LSE * np.maximum(1.0, np.abs(lse_ref[finite]))).all()
    refs = orc.attn_bwd_varlen(q, k, v, d_o, cu_q, cu_k, causal, scale)
    for nm, a, b in zip(("dQ", "dK", "dV"), (gq, gk, gv), refs):
        a = host(a)
        assert not np.isnan(a).any(), nm
        assert np.abs(a - b).max() <= TOL_GRAD * np.abs(b).max() + 1e-5, nm


def test_packed_equal_lengths_give_the_same_bits_as_the_batched_entry_point(vt):
    import torch
    B, Hq, Hkv, S, D, causal = 3, 4, 2, 200, 128, True
    (q, k, v, d_o, cu_q, cu_k, scale), (o, lse, gq, gk, gv) = _run(vt, Hq, Hkv, D, causal, [S] * B, None, 8200)
    # same numbers in the [B, H, S, D] layout
    def to_bhsd(x, H):
        return np.ascontiguousarray(x.reshape(B, S, H, D).transpose(0, 2, 1, 3))
    qb, kb, vb, dob = to_bhsd(q, Hq), to_bhsd(k, Hkv), to_bhsd(v, Hkv), to_bhsd(d_o, Hq)
    o2, lse2 = vt.vt_attn_fwd(dev(qb), dev(kb), dev(vb), causal, scale)
    g2 = vt.vt_attn_bwd(dev(qb), dev(kb), dev(vb), o2, dev(dob), lse2, causal, scale)
    torch.cuda.synchronize()
    def to_packed(t, H):
        return t.permute(0, 2, 1, 3).reshape(B * S, H, D)
    assert torch.equal(o, to_packed(o2, Hq))
    assert torch.equal(lse, lse2.permute(1, 0, 2).reshape(Hq, B * S))
    assert torch.equal(gq, to_packed(g2[0], Hq)) and torch.equal(gk, to_packed(g2[1], Hkv)) and torch.equal(gv, to_packed(g2[2], Hkv))


def test_packed_argument_checks(vt):
    import torch
    q = torch.zeros(10, 3, 64, dtype=torch.bfloat16, device="cuda"); k = torch.zeros(10, 2, 64, dtype=torch.bfloat16, device="cuda")
    cu = torch.tensor([0, 10], dtype=torch.int32, device="cuda")
    with pytest.raises(ValueError):
        vt.vt_attn_fwd_varlen(q, k, k, cu, cu, 10, 10, False, 0.1)          # Hq % Hkv != 0: refused by the binding ...
    o = torch.empty_like(q); lse = torch.empty(3, 10, device="cuda")
    rc = vt.load_library().vt_attn_fwd_varlen(q.data_ptr(), k.data_ptr(), k.data_ptr(), o.data_ptr(), lse.data_ptr(), cu.data_ptr(),
                                              cu.data_ptr(), 1, 3, 2, 10, 10, 10, 10, 64, 0, 0.1, None)
    assert rc == vt.ERR_INVALID_ARGUMENT                                    # ... and by the library when called directly
    q = torch.zeros(10, 2, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(vt.VtAttnError) as e:
        vt.vt_attn_fwd_varlen(q, k, k, cu, cu, 11, 10, False, 0.1)          # max_sq > total_q
    assert e.value.status == vt.ERR_INVALID_ARGUMENT
    with pytest.raises(ValueError):
        vt.vt_attn_fwd_varlen(q, k, k, cu.long(), cu, 10, 10, False, 0.1)   # cu_seqlens must be int32


def test_packed_documents_workload_small(vt):
    """The benchmark's packed-documents recipe at a small size, element by element."""
    import torch
    from paper_2601_16238_b200.inputs import VARLEN_CONFIGS, make_varlen_inputs
    cfg = VARLEN_CONFIGS["packed_docs_small"]
    q, k, v, d_o, cu = make_varlen_inputs(cfg)
    lens = cfg.lengths()
    assert sum(lens) == cfg.total and cu[-1] == cfg.total
    cq = torch.from_numpy(cu).cuda()
    o, lse = vt.vt_attn_fwd_varlen(dev(q), dev(k), dev(v), cq, cq, max(lens), max(lens), cfg.causal, cfg.scale)
    g = vt.vt_attn_bwd_varlen(dev(q), dev(k), dev(v), o, dev(d_o), lse, cq, cq, max(lens), max(lens), cfg.causal, cfg.scale)
    torch.cuda.synchronize()
    o_ref, lse_ref = orc.attn_fwd_varlen(q, k, v, cu, cu, cfg.causal, cfg.scale)
    assert np.abs(host(o) - o_ref).max() <= max(TOL_O, 2.0 ** -8 * np.abs(o_ref).max())
    assert (np.abs(host(lse) - lse_ref) <= TOL_LSE * np.maximum(1.0, np.abs(lse_ref))).all()
    for a, b in zip(g, orc.attn_bwd_varlen(q, k, v, d_o, cu, cu, cfg.causal, cfg.scale)):
        assert np.abs(host(a) - b).max() <= TOL_GRAD * np.abs(b).max()


def test_packed_documents_workload_full_size_sampled(vt):
    """The packed benchmark workload at full size: whole documents sampled, oracle per document."""
    import torch
    from paper_2601_16238_b200.inputs import VARLEN_CONFIGS, make_varlen_inputs
    cfg = VARLEN_CONFIGS["packed_docs"]
    q, k, v, d_o, cu = make_varlen_inputs(cfg)
    lens = cfg.lengths()
    cq = torch.from_numpy(cu).cuda()
    o, lse = vt.vt_attn_fwd_varlen(dev(q), dev(k), dev(v), cq, cq, max(lens), max(lens), cfg.causal, cfg.scale)
    g = vt.vt_attn_bwd_varlen(dev(q), dev(k), dev(v), o, dev(d_o), lse, cq, cq, max(lens), max(lens), cfg.causal, cfg.scale)
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0
    o_h, lse_h, g_h = host(o), host(lse), [host(t) for t in g]
    order = np.argsort(lens)
    for i in (int(order[0]), int(order[len(order) // 2]), len(lens) - 1):       # shortest, median, last (cut) document
        a, b = int(cu[i]), int(cu[i + 1])
        sub = np.array([0, b - a], dtype=np.int32)
        o_ref, lse_ref = orc.attn_fwd_varlen(q[a:b], k[a:b], v[a:b], sub, sub, cfg.causal, cfg.scale)
        assert np.abs(o_h[a:b] - o_ref).max() <= TOL_O
        assert (np.abs(lse_h[:, a:b] - lse_ref) <= TOL_LSE * np.maximum(1.0, np.abs(lse_ref))).all()
        for got, ref in zip(g_h, orc.attn_bwd_varlen(q[a:b], k[a:b], v[a:b], d_o[a:b], sub, sub, cfg.causal, cfg.scale)):
            assert np.abs(got[a:b] - ref).max() <= TOL_GRAD * np.abs(ref).max()
