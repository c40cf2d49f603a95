"""GPU: the partial-result merge kernels, and the ring-attention schedule run for all ranks' shards by one process on one
GPU (the same per-step kernels and merges each rank of a real ring would run, without the communication)."""
import numpy as np
import pytest

from helpers import TOL_LSE, TOL_O, dev, host
from oracle import attn_oracle as orc
from paper_2601_16238_b200.inputs import AttnConfig, make_inputs

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("D", [64, 128])
def test_merge_of_key_blocks_equals_attention_over_all_keys(vt, D):
    import torch
    cfg = AttnConfig("merge", 14, 2, 4, 2, 200, 900, D, False, False)
    q, k, v = make_inputs(cfg, with_do=False)
    tq, tk, tv = dev(q), dev(k), dev(v)
    o_acc = torch.full(tq.shape, float("nan"), dtype=torch.float32, device="cuda")
    lse_acc = torch.full(tq.shape[:3], float("nan"), dtype=torch.float32, device="cuda")
    cuts = [0, 130, 131, 600, 900]                                      # uneven blocks, one of a single key
    for i, (a, b) in enumerate(zip(cuts, cuts[1:])):
        o_p, lse_p = vt.vt_attn_fwd(tq, tk[:, :, a:b].contiguous(), tv[:, :, a:b].contiguous(), False, cfg.scale)
        vt.vt_attn_merge_partial(o_acc, lse_acc, o_p, lse_p, first=(i == 0))
    o = vt.vt_attn_merge_finish(o_acc)
    torch.cuda.synchronize()
    o_ref, lse_ref = orc.attn_fwd(q, k, v, False, cfg.scale)
    assert np.abs(host(o) - o_ref).max() <= TOL_O
    assert (np.abs(host(lse_acc) - lse_ref) <= TOL_LSE * np.maximum(1.0, np.abs(lse_ref))).all()


@pytest.mark.parametrize("D", [96, 192])
def test_merge_of_many_rows_whose_threads_straddle_warps(vt, D):
    """49 152 query rows at head dimensions whose D / 8 threads per row (12, 24) do not divide a warp: more blocks than the
    GPU holds at once, so a thread of a row may run long after the row's first thread.  The merged result must still be
    attention over all keys (every thread of a row has to weigh with the OLD running LSE), and the same bits every run."""
    import torch
    cfg = AttnConfig("merge_many", 18, 1, 3, 3, 16384, 192, D, False, False)
    q, k, v = make_inputs(cfg, with_do=False)
    tq, tk, tv = dev(q), dev(k), dev(v)
    parts = [vt.vt_attn_fwd(tq, tk[:, :, a:a + 64].contiguous(), tv[:, :, a:a + 64].contiguous(), False, cfg.scale)
             for a in (0, 64, 128)]
    runs = []
    for _ in range(3):
        o_acc = torch.full(tq.shape, float("nan"), dtype=torch.float32, device="cuda")
        lse_acc = torch.full(tq.shape[:3], float("nan"), dtype=torch.float32, device="cuda")
        for i, (o_p, lse_p) in enumerate(parts):
            vt.vt_attn_merge_partial(o_acc, lse_acc, o_p, lse_p, first=(i == 0))
        runs.append((o_acc, lse_acc, vt.vt_attn_merge_finish(o_acc)))
    torch.cuda.synchronize()
    for o_acc, lse_acc, o in runs[1:]:
        assert torch.equal(o_acc, runs[0][0]) and torch.equal(lse_acc, runs[0][1]) and torch.equal(o, runs[0][2])
    o_ref, lse_ref = orc.attn_fwd(q, k, v, False, cfg.scale)
    assert np.abs(host(runs[0][2]) - o_ref).max() <= TOL_O
    assert np.abs(host(runs[0][0]) - o_ref).max() <= TOL_O
    assert (np.abs(host(runs[0][1]) - lse_ref) <= TOL_LSE * np.maximum(1.0, np.abs(lse_ref))).all()


def test_merge_with_empty_parts(vt):
    import torch
    n, D = 300, 64
    o_acc = torch.empty(1, 1, n, D, dtype=torch.float32, device="cuda")
    lse_acc = torch.empty(1, 1, n, dtype=torch.float32, device="cuda")
    part = torch.randn(1, 1, n, D, device="cuda").to(torch.bfloat16)
    lse_p = torch.randn(1, 1, n, device="cuda")
    empty_o = torch.zeros_like(part)
    empty_l = torch.full_like(lse_p, float("-inf"))
    vt.vt_attn_merge_partial(o_acc, lse_acc, empty_o, empty_l, first=True)         # nothing seen yet
    torch.cuda.synchronize()
    assert torch.isneginf(lse_acc).all() and (o_acc == 0).all()
    vt.vt_attn_merge_partial(o_acc, lse_acc, part, lse_p, first=False)             # the first real part is taken as it is
    vt.vt_attn_merge_partial(o_acc, lse_acc, empty_o, empty_l, first=False)        # an empty part changes nothing
    torch.cuda.synchronize()
    assert torch.equal(lse_acc, lse_p) and torch.equal(o_acc, part.float())
    assert torch.equal(vt.vt_attn_merge_finish(o_acc), part)


@pytest.mark.parametrize("world,causal,Hq,Hkv,S_local,D", [(4, True, 4, 2, 200, 128), (3, False, 2, 2, 129, 64), (8, True, 2, 1, 128, 128)])
def test_ring_schedule_on_one_gpu_reproduces_full_attention(vt, world, causal, Hq, Hkv, S_local, D):
    import torch
    from paper_2601_16238_b200.ring import ring_attention_fwd_local
    cfg = AttnConfig("ring", 15, 1, Hq, Hkv, world * S_local, world * S_local, D, causal, False)
    q, k, v = make_inputs(cfg, with_do=False)
    tq, tk, tv = dev(q), dev(k), dev(v)
    shard = lambda t, r: t[:, :, r * S_local:(r + 1) * S_local].contiguous()       # noqa: E731
    res = ring_attention_fwd_local([shard(tq, r) for r in range(world)], [shard(tk, r) for r in range(world)],
                                   [shard(tv, r) for r in range(world)], causal, cfg.scale)
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0
    o_ref, lse_ref = orc.attn_fwd(q, k, v, causal, cfg.scale)
    for r, (o, lse) in enumerate(res):
        sl = slice(r * S_local, (r + 1) * S_local)
        assert np.abs(host(o) - o_ref[:, :, sl]).max() <= max(TOL_O, 2.0 ** -8 * np.abs(o_ref[:, :, sl]).max()), r
        assert (np.abs(host(lse) - lse_ref[:, :, sl]) <= TOL_LSE * np.maximum(1.0, np.abs(lse_ref[:, :, sl]))).all(), r


@pytest.mark.parametrize("world,causal,Hq,Hkv,S_local,D", [(4, True, 4, 2, 200, 128), (3, False, 2, 2, 129, 64)])
def test_ring_backward_schedule_on_one_gpu_reproduces_the_full_gradients(vt, world, causal, Hq, Hkv, S_local, D):
    import torch
    from helpers import check_grad
    from paper_2601_16238_b200.ring import ring_attention_bwd_local, ring_attention_fwd_local
    cfg = AttnConfig("ring_bwd", 16, 1, Hq, Hkv, world * S_local, world * S_local, D, causal, True)
    q, k, v, d_o = make_inputs(cfg)
    shards = lambda bits: [dev(bits)[:, :, r * S_local:(r + 1) * S_local].contiguous() for r in range(world)]      # noqa: E731
    qs, ks, vs, dos = shards(q), shards(k), shards(v), shards(d_o)
    fwd = ring_attention_fwd_local(qs, ks, vs, causal, cfg.scale)
    grads = ring_attention_bwd_local(qs, ks, vs, [o for o, _ in fwd], dos, [l for _, l in fwd], causal, cfg.scale)
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0
    gq, gk, gv = orc.attn_bwd(q, k, v, d_o, causal, cfg.scale)
    cat = lambda i: np.concatenate([host(g[i]) for g in grads], axis=2)      # noqa: E731
    for name, a, b in (("dQ", cat(0), gq), ("dK", cat(1), gk), ("dV", cat(2), gv)):
        check_grad(a, b, name, f"ring world={world}")


def test_accumulate_partial(vt):
    import torch
    a = torch.randn(2, 3, 70, 128, device="cuda").to(torch.bfloat16)
    b = torch.randn(2, 3, 70, 128, device="cuda").to(torch.bfloat16)
    acc = torch.full(a.shape, float("nan"), dtype=torch.float32, device="cuda")
    vt.vt_attn_accumulate_partial(acc, a, first=True)
    vt.vt_attn_accumulate_partial(acc, b, first=False)
    torch.cuda.synchronize()
    assert torch.equal(acc, a.float() + b.float())


@pytest.mark.parametrize("world,Hq,Hkv,chunk,D", [(2, 4, 2, 130, 128), (4, 2, 2, 64, 64), (3, 4, 1, 200, 96)])
def test_zigzag_schedule_on_one_gpu_forward_and_backward(vt, world, Hq, Hkv, chunk, D):
    """The zig-zag layout's sub-blocks with the real kernels and merges, all ranks' shards on one GPU, against the oracle
    on the whole causal sequence."""
    import torch
    from helpers import check_grad
    from paper_2601_16238_b200.ring import ring_attention_zigzag_local, zigzag_shard, zigzag_unshard
    S = 2 * world * chunk
    cfg = AttnConfig("zigzag", 17, 1, Hq, Hkv, S, S, D, True, True)
    q, k, v, d_o = make_inputs(cfg)
    sh = lambda bits: [zigzag_shard(dev(bits), r, world) for r in range(world)]      # noqa: E731
    fwd, grads = ring_attention_zigzag_local(sh(q), sh(k), sh(v), cfg.scale, do2s=sh(d_o))
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0
    o_ref, lse_ref = orc.attn_fwd(q, k, v, True, cfg.scale)
    o = host(zigzag_unshard([o2 for o2, _ in fwd]))
    lse = host(zigzag_unshard([l2 for _, l2 in fwd]))
    assert np.abs(o - o_ref).max() <= max(TOL_O, 2.0 ** -8 * np.abs(o_ref).max())
    assert (np.abs(lse - lse_ref) <= TOL_LSE * np.maximum(1.0, np.abs(lse_ref))).all()
    gq, gk, gv = orc.attn_bwd(q, k, v, d_o, True, cfg.scale)
    for i, (name, ref) in enumerate((("dQ", gq), ("dK", gk), ("dV", gv))):
        check_grad(host(zigzag_unshard([g[i] for g in grads])), ref, name, f"zigzag world={world}")
