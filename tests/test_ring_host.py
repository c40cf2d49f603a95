"""The exchange schedule of ring attention on CPU: 2 and 4 gloo ranks pass K/V shards around the ring; the attention of a
block and the merge are stand-ins built from the oracle (nothing in the package computes on the CPU), so what is under
test is the package's own part: who holds which block when, which mask a block gets, and that every block arrives."""
import os
import socket

import numpy as np
import pytest

from paper_2601_16238_b200.ring import block_mode, kv_owner


def test_every_rank_sees_every_shard_exactly_once():
    for world in (1, 2, 3, 4, 8):
        for rank in range(world):
            assert sorted(kv_owner(rank, s, world) for s in range(world)) == list(range(world))
            assert kv_owner(rank, 0, world) == rank                      # a rank starts with its own shard


def test_block_masks_tile_the_causal_triangle():
    world = 4
    for qr in range(world):
        for kr in range(world):
            want = None if kr > qr else (1 if kr == qr else 0)
            assert block_mode(True, qr, kr) == want
            assert block_mode(False, qr, kr) == 0


class _OracleMerge:
    """fp64 running result (the stand-in for the device merge kernel)."""

    def __init__(self, q):
        self.o = np.zeros(q.shape, dtype=np.float64)
        self.lse = np.full(q.shape[:3], -np.inf)

    def add(self, o_part, lse_part):
        new = np.logaddexp(self.lse, lse_part)
        with np.errstate(invalid="ignore"):
            wa = np.where(np.isneginf(new), 0.0, np.exp(self.lse - new))
            wp = np.where(np.isneginf(new), 0.0, np.exp(lse_part - new))
        self.o = wa[..., None] * self.o + wp[..., None] * o_part
        self.lse = new

    def result(self):
        return self.o, self.lse


def _worker(rank, world, port, causal, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import torch
    import torch.distributed as dist
    from oracle import attn_oracle as orc
    from paper_2601_16238_b200.ring import ring_attention_fwd
    dist.init_process_group("gloo", rank=rank, world_size=world)
    B, Hq, Hkv, S_local, D, scale = 1, 4, 2, 24, 8, 0.31
    rng = np.random.Generator(np.random.Philox(key=5))
    q, k, v = (rng.standard_normal((B, h, world * S_local, D)) for h in (Hq, Hkv, Hkv))       # the same on every rank
    sl = slice(rank * S_local, (rank + 1) * S_local)
    tq, tk, tv = (torch.from_numpy(np.ascontiguousarray(x[:, :, sl])) for x in (q, k, v))

    def attend(q_, k_, v_, mode, scale_):
        return orc.attn_fwd(q_.numpy(), k_.numpy(), v_.numpy(), mode, scale_)

    o, lse = ring_attention_fwd(tq, tk, tv, causal, scale, attend=attend, merge_factory=lambda q_: _OracleMerge(q_.numpy()))
    o_ref, lse_ref = orc.attn_fwd(q, k, v, causal, scale)
    out.put((rank, float(np.abs(o - o_ref[:, :, sl]).max()), float(np.abs(lse - lse_ref[:, :, sl]).max())))
    dist.destroy_process_group()


@pytest.mark.parametrize("world,causal", [(2, False), (2, True), (4, True)])
def test_ring_of_gloo_ranks_reproduces_full_attention(world, causal):
    import torch.multiprocessing as mp
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, causal, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[0] for r in results] == list(range(world))
    for _, eo, el in results:
        assert eo < 1e-12 and el < 1e-12


# ------------------------------------------------------------------------------------------------ backward
class _OracleSum:
    def __init__(self, like):
        import torch
        self.acc = torch.zeros(tuple(like.shape), dtype=torch.float64)

    def add(self, part):
        import torch
        self.acc = self.acc + torch.as_tensor(part)

    def result(self):
        return self.acc.numpy()


def _block_grads(q, k, v, o, d_o, lse, mode, scale):
    """Stand-in for the backward kernels on one (queries, key block) pair: the block's contribution given the GLOBAL
    LSE and Delta (dense numpy; the oracle itself only knows whole softmaxes)."""
    q, k, v, o, d_o, lse = (np.asarray(x, dtype=np.float64) for x in (q, k, v, o, d_o, lse))
    G = q.shape[1] // k.shape[1]
    kk, vv = np.repeat(k, G, axis=1), np.repeat(v, G, axis=1)
    s = scale * np.einsum("bhid,bhjd->bhij", q, kk)
    p = np.exp(s - lse[..., None])
    if mode == 1:
        p = p * np.tril(np.ones(s.shape[-2:]))
    delta = (d_o * o).sum(-1)
    ds = p * (np.einsum("bhid,bhjd->bhij", d_o, vv) - delta[..., None])
    dq = scale * np.einsum("bhij,bhjd->bhid", ds, kk)
    dk = scale * np.einsum("bhij,bhid->bhjd", ds, q).reshape(k.shape[0], k.shape[1], G, *k.shape[2:]).sum(2)
    dv = np.einsum("bhij,bhid->bhjd", p, d_o).reshape(k.shape[0], k.shape[1], G, *k.shape[2:]).sum(2)
    return dq, dk, dv


def _worker_bwd(rank, world, port, causal, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import torch
    import torch.distributed as dist
    from oracle import attn_oracle as orc
    from paper_2601_16238_b200.ring import ring_attention_bwd
    dist.init_process_group("gloo", rank=rank, world_size=world)
    B, Hq, Hkv, S_local, D, scale = 1, 4, 2, 16, 8, 0.37
    rng = np.random.Generator(np.random.Philox(key=6))
    q, k, v, d_o = (rng.standard_normal((B, h, world * S_local, D)) for h in (Hq, Hkv, Hkv, Hq))
    o, lse = orc.attn_fwd(q, k, v, causal, scale)                 # what the ring forward leaves on the ranks
    sl = slice(rank * S_local, (rank + 1) * S_local)
    t = lambda x: torch.from_numpy(np.ascontiguousarray(x[:, :, sl]))       # noqa: E731
    dq, dk, dv = ring_attention_bwd(t(q), t(k), t(v), t(o), t(d_o), t(lse), causal, scale,
                                    attend_bwd=_block_grads, sum_factory=_OracleSum)
    gq, gk, gv = orc.attn_bwd(q, k, v, d_o, causal, scale)
    out.put((rank, max(float(np.abs(a - b[:, :, sl]).max()) for a, b in ((dq, gq), (dk, gk), (dv, gv)))))
    dist.destroy_process_group()


@pytest.mark.parametrize("world,causal", [(2, True), (4, False), (3, True)])
def test_ring_backward_of_gloo_ranks_reproduces_the_full_gradients(world, causal):
    import torch.multiprocessing as mp
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker_bwd, args=(r, world, port, causal, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[0] for r in results] == list(range(world))
    assert all(err < 1e-12 for _, err in results)


# ------------------------------------------------------------------------------------------------ zig-zag layout
def test_zigzag_blocks_tile_the_causal_triangle():
    """Brute force over positions: the union of the sub-blocks of every (query rank, key rank) pair, each with its mask,
    is exactly the causal mask of the whole sequence, and every rank does the same amount of work in every step."""
    from paper_2601_16238_b200.ring import zigzag_blocks, zigzag_chunks
    for world in (1, 2, 3, 4, 5):
        c = 3
        S = 2 * world * c
        seen = np.zeros((S, S), dtype=int)
        for a in range(world):
            work = []
            for step in range(world):
                b = kv_owner(a, step, world)
                units = 0.0
                for qi, ki, mode in zigzag_blocks(a, b):
                    q0, k0 = zigzag_chunks(a, world)[qi] * c, zigzag_chunks(b, world)[ki] * c
                    for i in range(c):
                        for j in range(c):
                            if mode == 0 or j <= i:
                                seen[q0 + i, k0 + j] += 1
                    if mode == 1:
                        assert q0 == k0                      # a causal sub-block sits on the diagonal
                    units += 0.5 if mode == 1 else 1.0
                work.append(units)
            assert all(w == 2.0 for w in work)               # two chunk-by-chunk blocks per step, for every rank
        assert (seen == np.tril(np.ones((S, S), dtype=int))).all()
        owned = sorted(x for r in range(world) for x in zigzag_chunks(r, world))
        assert owned == list(range(2 * world))


def _worker_zigzag(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import torch
    import torch.distributed as dist
    from oracle import attn_oracle as orc
    from paper_2601_16238_b200.ring import ring_attention_bwd_zigzag, ring_attention_fwd_zigzag, zigzag_shard
    dist.init_process_group("gloo", rank=rank, world_size=world)
    B, Hq, Hkv, c, D, scale = 1, 4, 2, 10, 8, 0.29
    S = 2 * world * c
    rng = np.random.Generator(np.random.Philox(key=7))
    q, k, v, d_o = (rng.standard_normal((B, h, S, D)) for h in (Hq, Hkv, Hkv, Hq))
    sh = lambda x: zigzag_shard(torch.from_numpy(x), rank, world)       # noqa: E731

    def attend(q_, k_, v_, mode, scale_):
        return orc.attn_fwd(q_.numpy(), k_.numpy(), v_.numpy(), mode, scale_)

    o2, lse2 = ring_attention_fwd_zigzag(sh(q), sh(k), sh(v), scale, attend=attend, merge_factory=lambda q_: _OracleMerge(q_.numpy()))
    o_ref, lse_ref = orc.attn_fwd(q, k, v, True, scale)
    err_f = max(float(np.abs(o2.numpy() - sh(o_ref).numpy()).max()), float(np.abs(lse2.numpy() - sh(lse_ref[..., None]).numpy()[..., 0]).max()))
    grads = ring_attention_bwd_zigzag(sh(q), sh(k), sh(v), sh(o_ref), sh(d_o), sh(lse_ref[..., None])[..., 0].contiguous(), scale,
                                      attend_bwd=_block_grads, sum_factory=_OracleSum)
    refs = orc.attn_bwd(q, k, v, d_o, True, scale)
    err_b = max(float(np.abs(g.numpy() - sh(r).numpy()).max()) for g, r in zip(grads, refs))
    out.put((rank, err_f, err_b))
    dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_zigzag_ring_of_gloo_ranks_forward_and_backward(world):
    import torch.multiprocessing as mp
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker_zigzag, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[0] for r in results] == list(range(world))
    assert all(ef < 1e-12 and eb < 1e-12 for _, ef, eb in results)


# ------------------------------------------------------------------------------------------------ the benchmark's ring workload
def _worker_bench_ring(rank, world, port, out):
    """The benchmark's own step function and input generator (bench.ring_step / bench.ring_shard_bits) on gloo ranks,
    with the oracle-built stand-ins for the kernels."""
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import torch
    import torch.distributed as dist
    import bench
    from oracle import attn_oracle as orc
    from paper_2601_16238_b200.ring import zigzag_shard, zigzag_unshard
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = {"B": 1, "Hq": 4, "Hkv": 2, "S": 96, "D": 8, "pieces": 8, "index": 77}
    scale = 0.3
    wide = lambda bits: torch.from_numpy(orc.bf16_bits_to_f64(bits))       # noqa: E731
    mine = [wide(x) for x in bench.ring_shard_bits(w, rank, world)]
    # every world size must see the same sequence: rebuild it from all ranks' shards and from a one-rank run
    full = [zigzag_unshard([wide(bench.ring_shard_bits(w, r, world)[t]) for r in range(world)]) for t in range(4)]
    alone = [zigzag_unshard([wide(bench.ring_shard_bits(w, 0, 1)[t])]) for t in range(4)]
    same = all(torch.equal(a, b) for a, b in zip(full, alone))

    def attend(q_, k_, v_, mode, scale_):
        return orc.attn_fwd(q_.numpy(), k_.numpy(), v_.numpy(), mode, scale_)

    o2, lse2, dq2, dk2, dv2 = bench.ring_step(*mine, scale, attend=attend, merge_factory=lambda q_: _OracleMerge(q_.numpy()),
                                              attend_bwd=_block_grads, sum_factory=_OracleSum)
    q, k, v, d_o = (x.numpy() for x in full)
    o_ref, lse_ref = orc.attn_fwd(q, k, v, True, scale)
    refs = orc.attn_bwd(q, k, v, d_o, True, scale)
    sh = lambda x: zigzag_shard(torch.from_numpy(x), rank, world).numpy()      # noqa: E731
    err = max(float(np.abs(np.asarray(o2) - sh(o_ref)).max()), float(np.abs(np.asarray(lse2) - sh(lse_ref[..., None])[..., 0]).max()),
              *(float(np.abs(np.asarray(g) - sh(r)).max()) for g, r in zip((dq2, dk2, dv2), refs)))
    out.put((rank, same, err))
    dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 4])
def test_benchmark_ring_workload_on_gloo_ranks(world):
    import torch.multiprocessing as mp
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker_bench_ring, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[0] for r in results] == list(range(world))
    assert all(same for _, same, _ in results), "every world size must be given the same sequence"
    assert all(err < 1e-12 for _, _, err in results)
