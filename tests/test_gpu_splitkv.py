"""GPU parity for the split-KV forward (keys cut into chunks, merged by LSE) against the fp64 oracle
and against the unsplit kernel."""
import numpy as np
import pytest

from helpers import TOL_LSE, TOL_O, dev, host
from oracle import attn_oracle as orc
from paper_2601_16238_b200.inputs import AttnConfig, make_inputs

pytestmark = pytest.mark.gpu

CASES = [
    # B, Hq, Hkv, Sq, Sk, D, causal, n_splits
    (2, 8, 2, 1, 1000, 128, 0, 0),       # decoding, heads of a group share a tile, library's choice of chunks
    (2, 8, 2, 1, 1000, 128, 2, 5),
    (1, 8, 2, 4, 700, 64, 2, 3),         # four new tokens (speculative decoding), bottom-right mask inside the tile
    (1, 16, 2, 16, 2049, 128, 2, 0),     # 8 heads x 16 queries fill the tile exactly; ragged last step
    (1, 4, 4, 1, 513, 64, 0, 4),         # no group: plain tiles, one live row each
    (1, 2, 1, 200, 1500, 128, 2, 4),     # prefill chunk, two query tiles, G * Sq > 128
    (2, 4, 2, 130, 900, 64, 1, 3),       # top-left causal: late chunks are fully masked for every tile (empty partials)
    (1, 2, 2, 65, 65, 64, 0, 8),         # more chunks asked for than steps exist
    (1, 8, 2, 8, 40, 128, 2, 0),         # a single step
    (1, 4, 1, 32, 600, 64, 2, 2),        # tile filled exactly by 4 heads x 32 queries
    (1, 4, 2, 50, 20, 64, 2, 1),         # fewer keys than queries: empty rows through the merge
]


@pytest.mark.parametrize("B,Hq,Hkv,Sq,Sk,D,causal,n_splits", CASES)
def test_splitkv_matches_the_oracle(vt, B, Hq, Hkv, Sq, Sk, D, causal, n_splits):
    import torch
    cfg = AttnConfig("split", 11, B, Hq, Hkv, Sq, Sk, D, causal, False)
    q, k, v = make_inputs(cfg, with_do=False)
    tq, tk, tv = dev(q), dev(k), dev(v)
    o = torch.full_like(tq, float("nan"))
    lse = torch.full(tq.shape[:3], float("nan"), device="cuda")
    vt.vt_attn_fwd_splitkv(tq, tk, tv, causal, cfg.scale, n_splits, o, lse)
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0
    o_ref, lse_ref = orc.attn_fwd(q, k, v, causal, cfg.scale)
    o_h, lse_h = host(o), host(lse)
    assert not np.isnan(o_h).any() and not np.isnan(lse_h).any()
    assert np.abs(o_h - o_ref).max() <= max(TOL_O, 2.0 ** -8 * np.abs(o_ref).max())
    finite = np.isfinite(lse_ref)
    assert (np.isneginf(lse_h) == ~finite).all()
    assert (o_h[~finite] == 0.0).all()
    assert (np.abs(lse_h[finite] - lse_ref[finite]) <= TOL_LSE * np.maximum(1.0, np.abs(lse_ref[finite]))).all()
    # against the unsplit kernel: same bf16 output up to one rounding step of the merge
    o1, lse1 = vt.vt_attn_fwd(tq, tk, tv, causal, cfg.scale)
    torch.cuda.synchronize()
    assert np.abs(o_h - host(o1)).max() <= 2.0 ** -7 * max(1.0, np.abs(o_ref).max())
    both = finite & np.isfinite(host(lse1))
    assert np.abs(lse_h[both] - host(lse1)[both]).max() <= 1e-4 * max(1.0, np.abs(lse_ref[finite]).max())


def test_splitkv_is_deterministic_and_checks_its_arguments(vt):
    import torch
    cfg = AttnConfig("split", 11, 2, 8, 2, 2, 3000, 128, 2, False)
    q, k, v = make_inputs(cfg, with_do=False)
    tq, tk, tv = dev(q), dev(k), dev(v)
    a = vt.vt_attn_fwd_splitkv(tq, tk, tv, 2, cfg.scale, 6)
    b = vt.vt_attn_fwd_splitkv(tq, tk, tv, 2, cfg.scale, 6)
    torch.cuda.synchronize()
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(vt.VtAttnError) as e:
        vt.vt_attn_fwd_splitkv(tq, tk, tv, 2, cfg.scale, 6, workspace=small)
    assert e.value.status == vt.ERR_WORKSPACE_TOO_SMALL
    with pytest.raises(vt.VtAttnError) as e:
        vt.vt_attn_fwd_splitkv(tq, tk, tv, 2, cfg.scale, 200)
    assert e.value.status == vt.ERR_INVALID_ARGUMENT


def test_decode_shape_at_full_size_sampled_heads(vt):
    """The decoding benchmark shape (B=4, 32 query heads on 8 KV heads, one query, 32768 keys): every row against the oracle
    for two of the batch entries (the oracle does these in well under a second)."""
    import torch
    cfg = AttnConfig("decode_32k", 12, 4, 32, 8, 1, 32768, 128, 2, False)
    q, k, v = make_inputs(cfg, with_do=False)
    o, lse = vt.vt_attn_fwd_splitkv(dev(q), dev(k), dev(v), 2, cfg.scale)
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0
    for b in (0, 3):
        o_ref, lse_ref = orc.attn_fwd(q[b:b + 1], k[b:b + 1], v[b:b + 1], 2, cfg.scale)
        assert np.abs(host(o[b:b + 1]) - o_ref).max() <= TOL_O
        assert (np.abs(host(lse[b:b + 1]) - lse_ref) <= TOL_LSE * np.maximum(1.0, np.abs(lse_ref))).all()


def test_prefill_chunk_shape_at_full_size(vt):
    """The prefill benchmark shape (512 new queries at the end of a 16384-token context, 32 query heads on 8 KV heads,
    bottom-right mask) at full size: every row of O and LSE against the oracle, through the split-KV entry point with the
    split count the library picks and through the plain forward."""
    import torch
    cfg = AttnConfig("prefill_chunk", 13, 1, 32, 8, 512, 16384, 128, 2, False)
    q, k, v = make_inputs(cfg, with_do=False)
    tq, tk, tv = dev(q), dev(k), dev(v)
    o_ref, lse_ref = orc.attn_fwd(q, k, v, 2, cfg.scale)
    for call in (lambda: vt.vt_attn_fwd_splitkv(tq, tk, tv, 2, cfg.scale), lambda: vt.vt_attn_fwd(tq, tk, tv, 2, cfg.scale)):
        o, lse = call()
        torch.cuda.synchronize()
        assert vt.vt_attn_device_status()[0] == 0
        assert np.abs(host(o) - o_ref).max() <= TOL_O
        assert (np.abs(host(lse) - lse_ref) <= TOL_LSE * np.maximum(1.0, np.abs(lse_ref))).all()


PACKED_CASES = [
    # Hq, Hkv, D, causal, query lengths, key lengths, n_splits
    (8, 2, 128, 2, [1, 1, 1, 1, 1], [1000, 37, 2049, 513, 1], 0),            # decoding against caches of different lengths; heads share a tile
    (8, 2, 128, 0, [1, 1, 1], [700, 700, 64], 5),
    (16, 2, 64, 2, [4, 1, 3, 4], [300, 900, 3, 1200], 3),                    # a few new tokens each (8 heads x up to 4 queries)
    (4, 4, 128, 2, [200, 64, 1, 130], [1500, 64, 900, 131], 4),              # prefill chunks of different lengths: plain tiles
    (4, 2, 64, 1, [130, 0, 40, 260], [100, 50, 0, 300], 3),                  # top-left mask, sequences without queries or without keys
    (2, 1, 128, 2, [50, 20], [20, 400], 2),                                  # fewer keys than queries in the first sequence: rows without a key
]


@pytest.mark.parametrize("Hq,Hkv,D,causal,lens_q,lens_k,n_splits", PACKED_CASES)
def test_packed_splitkv_matches_the_oracle(vt, Hq, Hkv, D, causal, lens_q, lens_k, n_splits):
    import torch
    from paper_2601_16238_b200.inputs import normal_bf16
    cu_q = np.concatenate([[0], np.cumsum(lens_q)]).astype(np.int32)
    cu_k = np.concatenate([[0], np.cumsum(lens_k)]).astype(np.int32)
    tq_, tk_ = int(cu_q[-1]), int(cu_k[-1])
    q, k, v = (normal_bf16(s, 8800 + i) for i, s in enumerate(((tq_, Hq, D), (tk_, Hkv, D), (tk_, Hkv, D))))
    scale = float(np.float32(1.0) / np.sqrt(np.float32(D)))
    tq, tk, tv = dev(q), dev(k), dev(v)
    cq, ck = torch.from_numpy(cu_q).cuda(), torch.from_numpy(cu_k).cuda()
    o = torch.full_like(tq, float("nan")); lse = torch.full((Hq, tq_), float("nan"), device="cuda")
    vt.vt_attn_fwd_splitkv_varlen(tq, tk, tv, cq, ck, max(lens_q), max(lens_k), causal, scale, n_splits, o, lse)
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0
    o_ref, lse_ref = orc.attn_fwd_varlen(q, k, v, cu_q, cu_k, causal, scale)
    o_h, lse_h = host(o), host(lse)
    assert not np.isnan(o_h).any() and not np.isnan(lse_h).any()
    finite = np.isfinite(lse_ref)
    assert (np.isneginf(lse_h) == ~finite).all()
    assert (o_h.transpose(1, 0, 2)[~finite] == 0.0).all()
    assert np.abs(o_h - o_ref).max() <= max(TOL_O, 2.0 ** -8 * np.abs(o_ref).max())
    assert (np.abs(lse_h[finite] - lse_ref[finite]) <= TOL_LSE * np.maximum(1.0, np.abs(lse_ref[finite]))).all()
    # against the unsplit packed kernel
    o1, lse1 = vt.vt_attn_fwd_varlen(tq, tk, tv, cq, ck, max(lens_q), max(lens_k), causal, scale)
    torch.cuda.synchronize()
    assert np.abs(o_h - host(o1)).max() <= 2.0 ** -7 * max(1.0, np.abs(o_ref).max())


def test_packed_splitkv_with_max_sq_below_the_longest_sequence(vt):
    """A max_sq that does not cover the longest sequence: its first max_sq tokens (rounded up to whole 128-row tiles) are
    attended as usual, the tokens no block owns come out as O = 0, LSE = -inf - never as whatever the scratch held."""
    import torch
    from paper_2601_16238_b200.inputs import normal_bf16
    Hq, Hkv, D, lens_q, lens_k = 4, 2, 64, [300, 40], [600, 500]
    cu_q = np.concatenate([[0], np.cumsum(lens_q)]).astype(np.int32)
    cu_k = np.concatenate([[0], np.cumsum(lens_k)]).astype(np.int32)
    q, k, v = (normal_bf16(s, 8900 + i) for i, s in enumerate(((340, Hq, D), (1100, Hkv, D), (1100, Hkv, D))))
    scale = 0.125
    cq, ck = torch.from_numpy(cu_q).cuda(), torch.from_numpy(cu_k).cuda()
    need = vt.load_library().vt_attn_fwd_splitkv_varlen_workspace_bytes(2, Hq, Hkv, 340, 128, 600, D, 3)
    ws = torch.full((need // 4,), 1e30, dtype=torch.float32, device="cuda").view(torch.uint8)     # poisoned scratch
    o, lse = vt.vt_attn_fwd_splitkv_varlen(dev(q), dev(k), dev(v), cq, ck, 128, 600, 0, scale, 3, workspace=ws)
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0
    o_ref, lse_ref = orc.attn_fwd_varlen(q, k, v, cu_q, cu_k, 0, scale)
    o_h, lse_h = host(o), host(lse)
    done = np.r_[0:128, 300:340]                        # one tile of the long sequence, all of the short one
    left = np.r_[128:300]
    assert np.abs(o_h[done] - o_ref[done]).max() <= TOL_O
    assert (np.abs(lse_h[:, done] - lse_ref[:, done]) <= TOL_LSE * np.maximum(1.0, np.abs(lse_ref[:, done]))).all()
    assert (o_h[left] == 0.0).all() and np.isneginf(lse_h[:, left]).all()
