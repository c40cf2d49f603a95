"""Context-parallel ("ring") attention, forward and backward, over several GPUs.

The sequence is cut into ``world`` contiguous shards; rank r owns queries and keys/values of the
positions [r * S_local, (r + 1) * S_local).  The K/V shards travel around the ring: at step s rank r
holds the shard that started on rank (r - s) mod world, attends its own queries to it with the
ordinary forward kernel and folds the partial result into an fp32 running result with
``vt_attn_merge_partial`` (the blocks cover disjoint keys, so LSE' = ln(e^LSE + e^LSE_part) and the
outputs combine with the matching weights).  Under a causal mask a block from a later shard is skipped,
the rank's own block gets the causal mask and blocks from earlier shards none.  While a block is being
attended the next one is already in flight (``torch.distributed`` point-to-point operations: NCCL over
NVLink on GPUs; the received block lands in this GPU's own memory and is read from there, no kernel
reads a peer's memory).

Contiguous shards leave the causal case unbalanced (rank 0 attends one block, the last rank all of
them); the time of a step is the slowest rank's.  The zig-zag layout at the end of this module gives every
rank an early and a late chunk of the sequence, which makes all ranks' steps equal under a causal mask.
The paper leaves multi-GPU attention open; this module has no counterpart there.

``attend`` and ``merge`` default to the library's kernels; the CPU tests of the exchange schedule pass
their own stand-ins, since nothing in this package computes on the CPU.
"""
from __future__ import annotations


def kv_owner(rank: int, step: int, world: int) -> int:
    """Rank whose K/V shard rank ``rank`` holds at ring step ``step``."""
    return (rank - step) % world


def block_mode(causal: bool, q_owner: int, kv_owner_: int):
    """How a query shard attends a key shard: None = not at all, 0 = unmasked, 1 = causal (top-left aligned)."""
    if not causal:
        return 0
    if kv_owner_ > q_owner:
        return None
    return 1 if kv_owner_ == q_owner else 0


def _default_attend(q, k, v, mode, scale):
    from . import binding
    return binding.vt_attn_fwd(q, k, v, mode, scale)


class _DeviceMerge:
    """Running fp32 result on the device, folded with vt_attn_merge_partial."""

    def __init__(self, q):
        import torch
        self.o_acc = torch.empty(q.shape, dtype=torch.float32, device=q.device)
        self.lse = torch.empty(q.shape[:3], dtype=torch.float32, device=q.device)
        self.first = True

    def add(self, o_part, lse_part):
        from . import binding
        binding.vt_attn_merge_partial(self.o_acc, self.lse, o_part, lse_part, self.first)
        self.first = False

    def result(self):
        import torch
        from . import binding
        if self.first:                      # nothing was attended (cannot happen: a rank always attends its own shard)
            self.o_acc.zero_()
            self.lse.fill_(float("-inf"))
        return binding.vt_attn_merge_finish(self.o_acc), self.lse


def ring_attention_fwd(q, k, v, causal: bool, scale: float, group=None, attend=None, merge_factory=None):
    """Forward attention of this rank's query shard against the keys of all ranks.

    q [B, Hq, S_local, D], k / v [B, Hkv, S_local, D] are this rank's shards (every rank passes the same shapes).
    Returns (O [B, Hq, S_local, D], LSE [B, Hq, S_local]).  Collective over ``group``: every rank must call it.
    """
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    rank = dist.get_rank(group) if dist.is_initialized() else 0
    attend = attend or _default_attend
    merge = (merge_factory or _DeviceMerge)(q)
    nxt, prv = (rank + 1) % world, (rank - 1) % world
    cur_k, cur_v = k, v
    for step in range(world):
        reqs, recv_k, recv_v = [], None, None
        if step + 1 < world:
            # pass the block on while it is being attended (the send reads cur_k / cur_v, which nothing writes)
            recv_k, recv_v = torch.empty_like(k), torch.empty_like(v)
            ops = [dist.P2POp(dist.isend, cur_k, dist.get_global_rank(group, nxt) if group is not None else nxt, group),
                   dist.P2POp(dist.isend, cur_v, dist.get_global_rank(group, nxt) if group is not None else nxt, group),
                   dist.P2POp(dist.irecv, recv_k, dist.get_global_rank(group, prv) if group is not None else prv, group),
                   dist.P2POp(dist.irecv, recv_v, dist.get_global_rank(group, prv) if group is not None else prv, group)]
            reqs = dist.batch_isend_irecv(ops)
        mode = block_mode(causal, rank, kv_owner(rank, step, world))
        if mode is not None:
            o_part, lse_part = attend(q, cur_k, cur_v, mode, scale)
            merge.add(o_part, lse_part)
        for r in reqs:
            r.wait()
        if step + 1 < world:
            cur_k, cur_v = recv_k, recv_v
    return merge.result()


def ring_attention_fwd_local(q_shards, k_shards, v_shards, causal: bool, scale: float, attend=None, merge_factory=None):
    """The same schedule for all ranks' shards held by ONE process (lists indexed by rank), without communication: what
    each rank of ``ring_attention_fwd`` computes, step by step, on a single GPU.  Returns a list of (O, LSE) per rank."""
    world = len(q_shards)
    attend = attend or _default_attend
    out = []
    for rank in range(world):
        merge = (merge_factory or _DeviceMerge)(q_shards[rank])
        for step in range(world):
            owner = kv_owner(rank, step, world)
            mode = block_mode(causal, rank, owner)
            if mode is not None:
                merge.add(*attend(q_shards[rank], k_shards[owner], v_shards[owner], mode, scale))
        out.append(merge.result())
    return out


# ---------------------------------------------------------------------------------------------------------
# Backward.  Every rank keeps its queries' side (Q, O, dO, LSE of the FULL softmax - the forward's merged
# result - and the running dQ); the K/V shards travel once more, each with the running dK / dV of its own
# keys.  At a step a rank calls the ordinary backward kernels on (its queries, the held shard): with the
# global LSE and Delta = rowsum(dO * O) these give exactly that block's contribution to dQ, dK and dV, which
# is added to the running sums in fp32.  After `world` hand-overs every dK / dV sum is back on its owner.
# ---------------------------------------------------------------------------------------------------------
def _default_attend_bwd(q, k, v, o, d_o, lse, mode, scale):
    from . import binding
    return binding.vt_attn_bwd(q, k, v, o, d_o, lse, mode, scale)


class _DeviceSum:
    """fp32 running sum of bf16 blocks on the device (vt_attn_accumulate_partial)."""

    def __init__(self, like):
        import torch
        self.acc = torch.zeros(like.shape, dtype=torch.float32, device=like.device)

    def add(self, part):
        from . import binding
        binding.vt_attn_accumulate_partial(self.acc, part, False)

    def result(self):
        from . import binding
        return binding.vt_attn_merge_finish(self.acc)


def ring_attention_bwd(q, k, v, o, d_o, lse, causal: bool, scale: float, group=None, attend_bwd=None, sum_factory=None):
    """Gradients of this rank's shards: (dQ, dK, dV), given the outputs (o, lse) of ``ring_attention_fwd`` and d_o.

    The running dK / dV of a shard travel as fp32 tensors (``.acc`` of the sum objects); they are handed on only after
    this rank's contribution has been added, the K / V shards themselves while the block is being processed."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    rank = dist.get_rank(group) if dist.is_initialized() else 0
    attend_bwd = attend_bwd or _default_attend_bwd
    sum_factory = sum_factory or _DeviceSum
    peer = (lambda r: dist.get_global_rank(group, r)) if group is not None else (lambda r: r)
    nxt, prv = peer((rank + 1) % world), peer((rank - 1) % world)
    dq_sum, dk_sum, dv_sum = sum_factory(q), sum_factory(k), sum_factory(v)
    cur_k, cur_v = k, v
    for step in range(world):
        reqs, recv_k, recv_v = [], None, None
        if step + 1 < world:
            recv_k, recv_v = torch.empty_like(k), torch.empty_like(v)
            reqs = dist.batch_isend_irecv([dist.P2POp(dist.isend, cur_k, nxt, group), dist.P2POp(dist.isend, cur_v, nxt, group),
                                           dist.P2POp(dist.irecv, recv_k, prv, group), dist.P2POp(dist.irecv, recv_v, prv, group)])
        mode = block_mode(causal, rank, kv_owner(rank, step, world))
        if mode is not None:
            dq_p, dk_p, dv_p = attend_bwd(q, cur_k, cur_v, o, d_o, lse, mode, scale)
            dq_sum.add(dq_p)
            dk_sum.add(dk_p)
            dv_sum.add(dv_p)
        for r in reqs:
            r.wait()
        if world > 1:
            # hand the shard's running dK / dV on (after the last step they arrive back at their owner)
            recv_dk, recv_dv = torch.empty_like(dk_sum.acc), torch.empty_like(dv_sum.acc)
            for r in dist.batch_isend_irecv([dist.P2POp(dist.isend, dk_sum.acc, nxt, group), dist.P2POp(dist.isend, dv_sum.acc, nxt, group),
                                             dist.P2POp(dist.irecv, recv_dk, prv, group), dist.P2POp(dist.irecv, recv_dv, prv, group)]):
                r.wait()
            dk_sum.acc, dv_sum.acc = recv_dk, recv_dv
        if step + 1 < world:
            cur_k, cur_v = recv_k, recv_v
    return dq_sum.result(), dk_sum.result(), dv_sum.result()


def ring_attention_bwd_local(q_shards, k_shards, v_shards, o_shards, do_shards, lse_shards, causal: bool, scale: float,
                             attend_bwd=None, sum_factory=None):
    """The backward schedule for all ranks' shards held by one process (no communication): per-rank (dQ, dK, dV)."""
    world = len(q_shards)
    attend_bwd = attend_bwd or _default_attend_bwd
    sum_factory = sum_factory or _DeviceSum
    dq = [sum_factory(x) for x in q_shards]
    dk = [sum_factory(x) for x in k_shards]
    dv = [sum_factory(x) for x in v_shards]
    for step in range(world):
        for rank in range(world):
            owner = kv_owner(rank, step, world)
            mode = block_mode(causal, rank, owner)
            if mode is None:
                continue
            dq_p, dk_p, dv_p = attend_bwd(q_shards[rank], k_shards[owner], v_shards[owner], o_shards[rank], do_shards[rank],
                                          lse_shards[rank], mode, scale)
            dq[rank].add(dq_p)
            dk[owner].add(dk_p)
            dv[owner].add(dv_p)
    return [(dq[r].result(), dk[r].result(), dv[r].result()) for r in range(world)]


# ---------------------------------------------------------------------------------------------------------
# Zig-zag layout for causal masks.  The sequence is cut into 2 * world chunks; rank r owns chunks r and
# 2 * world - 1 - r (an early and a late one), so every rank has the same share of the causal triangle and
# every ring step costs every rank the same: two chunk-by-chunk blocks.  A shard is carried as its two
# chunks stacked, [2, B, H, S_chunk, D] (chunk 0 the early one), so that each chunk is contiguous.
# Which (query chunk, key chunk) pairs of a (query rank, key rank) block are attended, and how:
#   own block       (0, 0) causal, (1, 0) unmasked, (1, 1) causal
#   earlier rank b  its early chunk lies before both query chunks, its late chunk after both: (0, 0), (1, 0) unmasked
#   later rank b    both its chunks lie between the two query chunks: (1, 0), (1, 1) unmasked
# ---------------------------------------------------------------------------------------------------------
def zigzag_chunks(rank: int, world: int):
    """The two chunk indices (of 2 * world) that rank ``rank`` owns."""
    return rank, 2 * world - 1 - rank


def zigzag_blocks(q_rank: int, kv_rank: int):
    """[(query chunk, key chunk, mode)] of a (query rank, key rank) block under a causal mask; chunk 0 / 1 = the
    rank's early / late chunk, mode 0 = unmasked, 1 = causal."""
    if kv_rank == q_rank:
        return [(0, 0, 1), (1, 0, 0), (1, 1, 1)]
    if kv_rank < q_rank:
        return [(0, 0, 0), (1, 0, 0)]
    return [(1, 0, 0), (1, 1, 0)]


def zigzag_shard(x, rank: int, world: int):
    """Rank ``rank``'s shard of a full tensor [B, H, S, D] (S a multiple of 2 * world) as stacked chunks [2, B, H, S_chunk, D]."""
    import torch
    c = x.shape[2] // (2 * world)
    lo, hi = zigzag_chunks(rank, world)
    return torch.stack([x[:, :, lo * c:(lo + 1) * c], x[:, :, hi * c:(hi + 1) * c]]).contiguous()


def zigzag_unshard(shards):
    """Inverse of zigzag_shard over all ranks: list of [2, B, H, S_chunk, ...] -> [B, H, S, ...]."""
    import torch
    world = len(shards)
    chunks = [None] * (2 * world)
    for r, s in enumerate(shards):
        lo, hi = zigzag_chunks(r, world)
        chunks[lo], chunks[hi] = s[0], s[1]
    return torch.cat(chunks, dim=2)


class _Transfer:
    """A started exchange.  ``wait()`` orders the caller's later work (on the current stream) behind its completion."""

    def __init__(self, reqs, event=None):
        self.reqs, self.event = reqs, event

    def wait(self):
        if self.event is not None:
            import torch
            torch.cuda.current_stream().wait_event(self.event)
        else:
            for r in self.reqs:
                r.wait()


def _exchange(tensors, nxt, prv, group, comm_stream=None, after_current=True):
    """Start sending ``tensors`` to the next rank and receiving their counterparts from the previous one.

    ``comm_stream`` (a ``torch.cuda.Stream``, GPU runs only): the point-to-point operations are enqueued there instead of
    on the current stream, so a step's exchange does not queue behind the attention kernels enqueued before it;
    ``after_current`` says whether the tensors to send were produced by work on the current stream that the exchange has
    to wait for (False for blocks that arrived through an earlier exchange on ``comm_stream``).  Returns (transfer, list
    of receive buffers); the buffers may be read on the current stream after ``transfer.wait()``."""
    import torch
    import torch.distributed as dist
    recv = [torch.empty_like(t) for t in tensors]
    ops = [dist.P2POp(dist.isend, t, nxt, group) for t in tensors] + [dist.P2POp(dist.irecv, t, prv, group) for t in recv]
    if comm_stream is None:
        return _Transfer(dist.batch_isend_irecv(ops)), recv
    if after_current:
        comm_stream.wait_stream(torch.cuda.current_stream())
    for t in list(tensors) + recv:
        t.record_stream(comm_stream)                 # the allocator must not hand their memory out while the exchange runs
    with torch.cuda.stream(comm_stream):
        for r in dist.batch_isend_irecv(ops):
            r.wait()                                 # orders comm_stream (not the host) behind the library's own stream
        event = torch.cuda.Event()
        event.record(comm_stream)
    return _Transfer([], event), recv


def ring_attention_fwd_zigzag(q2, k2, v2, scale: float, group=None, attend=None, merge_factory=None, comm_stream=None):
    """Causal forward attention in the zig-zag layout.  q2 [2, B, Hq, S_chunk, D], k2 / v2 [2, B, Hkv, S_chunk, D]: this
    rank's two chunks.  Returns (O2 [2, B, Hq, S_chunk, D], LSE2 [2, B, Hq, S_chunk]).  Collective over ``group``.
    ``comm_stream``: see ``_exchange`` (GPU runs: the K/V blocks travel on a stream of their own)."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    rank = dist.get_rank(group) if dist.is_initialized() else 0
    attend = attend or _default_attend
    merges = [(merge_factory or _DeviceMerge)(q2[i]) for i in range(2)]
    peer = (lambda r: dist.get_global_rank(group, r)) if group is not None else (lambda r: r)
    nxt, prv = peer((rank + 1) % world), peer((rank - 1) % world)
    cur_k, cur_v = k2, v2
    for step in range(world):
        transfer, recv = None, None
        if step + 1 < world:
            transfer, recv = _exchange([cur_k, cur_v], nxt, prv, group, comm_stream, after_current=(step == 0))
        for qi, ki, mode in zigzag_blocks(rank, kv_owner(rank, step, world)):
            merges[qi].add(*attend(q2[qi], cur_k[ki], cur_v[ki], mode, scale))
        if transfer is not None:
            transfer.wait()
            cur_k, cur_v = recv
    (o0, l0), (o1, l1) = merges[0].result(), merges[1].result()
    return torch.stack([torch.as_tensor(o0), torch.as_tensor(o1)]), torch.stack([torch.as_tensor(l0), torch.as_tensor(l1)])


def ring_attention_bwd_zigzag(q2, k2, v2, o2, do2, lse2, scale: float, group=None, attend_bwd=None, sum_factory=None, comm_stream=None):
    """Causal backward in the zig-zag layout: (dQ2, dK2, dV2) stacked like the inputs, given the forward's (o2, lse2)."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    rank = dist.get_rank(group) if dist.is_initialized() else 0
    attend_bwd = attend_bwd or _default_attend_bwd
    sum_factory = sum_factory or _DeviceSum
    peer = (lambda r: dist.get_global_rank(group, r)) if group is not None else (lambda r: r)
    nxt, prv = peer((rank + 1) % world), peer((rank - 1) % world)
    dq = [sum_factory(q2[i]) for i in range(2)]
    dk = [sum_factory(k2[i]) for i in range(2)]
    dv = [sum_factory(v2[i]) for i in range(2)]
    cur_k, cur_v = k2, v2
    for step in range(world):
        transfer, recv = None, None
        if step + 1 < world:
            transfer, recv = _exchange([cur_k, cur_v], nxt, prv, group, comm_stream, after_current=(step == 0))
        for qi, ki, mode in zigzag_blocks(rank, kv_owner(rank, step, world)):
            dq_p, dk_p, dv_p = attend_bwd(q2[qi], cur_k[ki], cur_v[ki], o2[qi], do2[qi], lse2[qi], mode, scale)
            dq[qi].add(dq_p)
            dk[ki].add(dk_p)
            dv[ki].add(dv_p)
        if transfer is not None:
            transfer.wait()
        if world > 1:
            # hand the running dK / dV of the held chunks on (after the last step they are back at their owner); they
            # were just updated on the current stream, so this exchange has to wait for it
            accs = [dk[0].acc, dk[1].acc, dv[0].acc, dv[1].acc]
            transfer2, got = _exchange(accs, nxt, prv, group, comm_stream, after_current=True)
            transfer2.wait()
            dk[0].acc, dk[1].acc, dv[0].acc, dv[1].acc = got
        if recv is not None:
            cur_k, cur_v = recv
    stack = lambda sums: torch.stack([torch.as_tensor(s.result()) for s in sums])      # noqa: E731
    return stack(dq), stack(dk), stack(dv)


def ring_attention_zigzag_fwd_bwd(q2, k2, v2, do2, scale: float, group=None, comm_stream=None, attend=None, merge_factory=None,
                                  attend_bwd=None, sum_factory=None):
    """One training step's attention in the zig-zag layout: the causal forward, then the backward for the upstream
    gradient do2.  Returns (O2, LSE2, dQ2, dK2, dV2).  With one rank (or no process group) nothing is exchanged and the
    three blocks of the rank's own shard are all there is.  This is what the benchmark workload ``ring_causal_64k`` times."""
    o2, lse2 = ring_attention_fwd_zigzag(q2, k2, v2, scale, group, attend, merge_factory, comm_stream)
    dq2, dk2, dv2 = ring_attention_bwd_zigzag(q2, k2, v2, o2, do2, lse2, scale, group, attend_bwd, sum_factory, comm_stream)
    return o2, lse2, dq2, dk2, dv2


def ring_attention_zigzag_local(q2s, k2s, v2s, scale: float, do2s=None, attend=None, merge_factory=None, attend_bwd=None, sum_factory=None):
    """Both zig-zag schedules for all ranks' shards held by one process (lists indexed by rank, no communication).
    Returns [(O2, LSE2)] per rank, and with ``do2s`` also [(dQ2, dK2, dV2)] per rank."""
    import torch
    world = len(q2s)
    attend = attend or _default_attend
    fwd = []
    for rank in range(world):
        merges = [(merge_factory or _DeviceMerge)(q2s[rank][i]) for i in range(2)]
        for step in range(world):
            owner = kv_owner(rank, step, world)
            for qi, ki, mode in zigzag_blocks(rank, owner):
                merges[qi].add(*attend(q2s[rank][qi], k2s[owner][ki], v2s[owner][ki], mode, scale))
        (o0, l0), (o1, l1) = merges[0].result(), merges[1].result()
        fwd.append((torch.stack([torch.as_tensor(o0), torch.as_tensor(o1)]), torch.stack([torch.as_tensor(l0), torch.as_tensor(l1)])))
    if do2s is None:
        return fwd
    attend_bwd = attend_bwd or _default_attend_bwd
    sum_factory = sum_factory or _DeviceSum
    dq = [[sum_factory(q2s[r][i]) for i in range(2)] for r in range(world)]
    dk = [[sum_factory(k2s[r][i]) for i in range(2)] for r in range(world)]
    dv = [[sum_factory(v2s[r][i]) for i in range(2)] for r in range(world)]
    for step in range(world):
        for rank in range(world):
            owner = kv_owner(rank, step, world)
            o2, lse2 = fwd[rank]
            for qi, ki, mode in zigzag_blocks(rank, owner):
                dq_p, dk_p, dv_p = attend_bwd(q2s[rank][qi], k2s[owner][ki], v2s[owner][ki], o2[qi], do2s[rank][qi], lse2[qi], mode, scale)
                dq[rank][qi].add(dq_p)
                dk[owner][ki].add(dk_p)
                dv[owner][ki].add(dv_p)
    stack = lambda sums: torch.stack([torch.as_tensor(s.result()) for s in sums])      # noqa: E731
    return fwd, [(stack(dq[r]), stack(dk[r]), stack(dv[r])) for r in range(world)]
