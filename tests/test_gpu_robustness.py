"""GPU behaviour beyond single-shot parity: repeatability on reused buffers, a poisoned workspace,
guard bands around every output, the host-buffer entry points, the bounded-wait path and CUDA-graph
replay.  The paper's debugging table motivates the first two (stale scratch that only shows after
several iterations)."""
import numpy as np
import pytest

from helpers import check_fwd, check_grad, dev, host
from oracle import attn_oracle as orc
from paper_2601_16238_b200.inputs import CONFIGS, AttnConfig, make_inputs

pytestmark = pytest.mark.gpu


def _guarded(shape, dtype, fill):
    """A tensor carved out of a larger buffer whose 4 KiB borders hold a sentinel."""
    import torch
    n = int(np.prod(shape))
    pad = 4096 // torch.empty(0, dtype=dtype).element_size()
    buf = torch.full((n + 2 * pad,), fill, dtype=dtype, device="cuda")
    return buf, buf[pad:pad + n].view(shape), pad


def _guards_intact(buf, pad, fill):
    import torch
    ref = torch.full((pad,), fill, dtype=buf.dtype, device="cuda")
    return torch.equal(buf[:pad], ref) and torch.equal(buf[-pad:], ref)


@pytest.mark.parametrize("name", ["vit_small", "minigpt", "gqa_ragged"])
def test_outputs_stay_inside_their_buffers_and_repeat_bit_exactly(vt, name):
    import torch
    cfg = {"vit_small": CONFIGS["vit"].with_(B=4), "minigpt": CONFIGS["minigpt"],
           "gqa_ragged": AttnConfig("g", 8, 2, 4, 2, 333, 333, 128, True, True)}[name]
    q, k, v, d_o = (dev(x) for x in make_inputs(cfg))
    bo, o, po = _guarded(q.shape, torch.bfloat16, 7.0)
    bl, lse, pl = _guarded(q.shape[:3], torch.float32, 7.0)
    bq, dq, pq = _guarded(q.shape, torch.bfloat16, 7.0)
    bk, dk, pk = _guarded(k.shape, torch.bfloat16, 7.0)
    bv, dv, pv = _guarded(v.shape, torch.bfloat16, 7.0)
    nws = max(256, vt.vt_attn_bwd_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.Sq, cfg.Sk, cfg.D))
    bw, ws, pw = _guarded((nws,), torch.uint8, 0xFF)          # 0xFF bytes: NaN when read as float
    first = None
    for it in range(20):
        ws.fill_(0xFF)
        vt.vt_attn_fwd(q, k, v, cfg.causal, cfg.scale, o, lse)
        vt.vt_attn_bwd(q, k, v, o, d_o, lse, cfg.causal, cfg.scale, dq, dk, dv, ws)
        torch.cuda.synchronize()
        snap = [t.clone() for t in (o, lse, dq, dk, dv)]
        if first is None:
            first = snap
        else:
            for a, b in zip(first, snap):
                assert torch.equal(a, b), f"iteration {it} differs from the first"
    for buf, pad, fill in ((bo, po, 7.0), (bl, pl, 7.0), (bq, pq, 7.0), (bk, pk, 7.0), (bv, pv, 7.0), (bw, pw, 0xFF)):
        assert _guards_intact(buf, pad, fill)
    for t in first:
        assert torch.isfinite(t.float()).all()
    assert vt.vt_attn_device_status()[0] == 0


def test_host_buffer_entry_points_match_device_path(vt):
    import torch
    cfg = CONFIGS["minigpt"]
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
    # forward-only variant
    ho2 = torch.empty_like(hq).pin_memory(); hlse2 = torch.empty_like(hlse).pin_memory()
    st2 = torch.empty(vt.vt_attn_host_staging_bytes(*dims, False), dtype=torch.uint8, device="cuda")
    vt.vt_attn_fwd_host(hq, hk, hv, ho2, hlse2, cfg.causal, cfg.scale, st2)
    torch.cuda.synchronize()
    assert torch.equal(ho2, ho) and torch.equal(hlse2, hlse)
    with pytest.raises(vt.VtAttnError) as e:
        vt.vt_attn_fwd_host(hq, hk, hv, ho2, hlse2, cfg.causal, cfg.scale, st2[:1024])
    assert e.value.status == vt.ERR_WORKSPACE_TOO_SMALL


def test_host_buffer_entry_points_with_several_chunks(vt):
    """A problem large enough for the host entry points to cut it into chunks that alternate between two streams (whole
    batches or KV-head ranges inside each batch, more and smaller ones when the copies outweigh the kernels); GQA so that
    a chunk's query heads are a multiple of its KV heads.  A chunk may get another forward kernel than the whole problem
    (fewer heads per launch), so the results are compared within rounding, not bit for bit."""
    import torch
    B, Hq, Hkv, S, D = 4, 16, 8, 4096, 128
    gen = torch.Generator(device="cuda").manual_seed(99)
    q, d_o = (torch.randn(B, Hq, S, D, device="cuda", dtype=torch.bfloat16, generator=gen) for _ in range(2))
    k, v = (torch.randn(B, Hkv, S, D, device="cuda", dtype=torch.bfloat16, generator=gen) for _ in range(2))
    scale = float(np.float32(1.0) / np.sqrt(np.float32(D)))
    hq, hk, hv, hdo = (t.cpu().pin_memory() for t in (q, k, v, d_o))
    ho = torch.empty_like(hq).pin_memory(); hlse = torch.empty(B, Hq, S, dtype=torch.float32).pin_memory()
    dims = (B, Hq, Hkv, S, S, D)
    st = torch.empty(vt.vt_attn_host_staging_bytes(*dims, False), dtype=torch.uint8, device="cuda")
    vt.vt_attn_fwd_host(hq, hk, hv, ho, hlse, False, scale, st)
    o, lse = vt.vt_attn_fwd(q, k, v, False, scale)
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0
    assert (hlse - lse.cpu()).abs().max() <= 1e-4
    assert (ho.float() - o.cpu().float()).abs().max() <= 2.0 ** -6 * o.float().abs().max().item()
    hdq = torch.empty_like(hq).pin_memory(); hdk = torch.empty_like(hk).pin_memory(); hdv = torch.empty_like(hv).pin_memory()
    st2 = torch.empty(vt.vt_attn_host_staging_bytes(*dims, True), dtype=torch.uint8, device="cuda")
    vt.vt_attn_fwd_bwd_host(hq, hk, hv, hdo, ho, hlse, hdq, hdk, hdv, True, scale, st2)
    o, lse = vt.vt_attn_fwd(q, k, v, True, scale)
    dq, dk, dv = vt.vt_attn_bwd(q, k, v, o, d_o, lse, True, scale)
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0
    assert (hlse - lse.cpu()).abs().max() <= 1e-4
    for a, b in ((ho, o), (hdq, dq), (hdk, dk), (hdv, dv)):
        a, b = a.float(), b.cpu().float()
        assert (a - b).abs().max() <= 2.0 ** -6 * b.abs().max()


@pytest.mark.parametrize("B,Hq,Hkv,Sq,Sk,D,causal", [(2, 16, 16, 2100, 2100, 128, 0), (1, 16, 4, 4100, 4100, 128, 1), (2, 8, 2, 1000, 1300, 128, 2)])
def test_every_kernel_family_is_bit_identical_from_run_to_run(vt, B, Hq, Hkv, Sq, Sk, D, causal):
    """Twelve back-to-back runs of forward (one-tile or two-tile kernel, by shape), backward, split-KV forward and the
    fp16 entry points on the same inputs: no atomics, no order-dependent reduction, so every run must give the same bits."""
    import torch
    gen = torch.Generator(device="cuda").manual_seed(5)
    q, d_o = (torch.randn(B, Hq, Sq, D, device="cuda", dtype=torch.bfloat16, generator=gen) for _ in range(2))
    k, v = (torch.randn(B, Hkv, Sk, D, device="cuda", dtype=torch.bfloat16, generator=gen) for _ in range(2))
    scale = float(np.float32(1.0) / np.sqrt(np.float32(D)))
    qh, kh, vh, doh = (t.to(torch.float16) for t in (q, k, v, d_o))
    ref = None
    for _ in range(12):
        o, lse = vt.vt_attn_fwd(q, k, v, causal, scale)
        grads = vt.vt_attn_bwd(q, k, v, o, d_o, lse, causal, scale)
        o_s, lse_s = vt.vt_attn_fwd_splitkv(q, k, v, causal, scale, 3)
        o_h, lse_h = vt.vt_attn_fwd_f16(qh, kh, vh, causal, scale)
        grads_h = vt.vt_attn_bwd_f16(qh, kh, vh, o_h, doh, lse_h, causal, scale)
        cur = (o, lse) + tuple(grads) + (o_s, lse_s, o_h, lse_h) + tuple(grads_h)
        if ref is None:
            ref = cur
        else:
            assert all(torch.equal(a, b) for a, b in zip(ref, cur))
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0


def test_calls_on_two_streams_at_once_give_the_serial_results(vt):
    """Two problems enqueued on two non-default streams with nothing ordering them: kernels of both may share the GPU (and
    contend for tensor memory on an SM); each must produce the bits it produces alone."""
    import torch
    cfgs = [CONFIGS["minigpt"], CONFIGS["vit"].with_(B=16)]
    data = [[dev(x) for x in make_inputs(c)] for c in cfgs]
    want = []
    for c, (q, k, v, d_o) in zip(cfgs, data):
        o, lse = vt.vt_attn_fwd(q, k, v, c.causal, c.scale)
        want.append((o, lse) + tuple(vt.vt_attn_bwd(q, k, v, o, d_o, lse, c.causal, c.scale)))
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    got = [None, None]
    for rep in range(10):
        for i, (c, (q, k, v, d_o)) in enumerate(zip(cfgs, data)):
            with torch.cuda.stream(streams[i]):
                o, lse = vt.vt_attn_fwd(q, k, v, c.causal, c.scale, stream=streams[i])
                got[i] = (o, lse) + tuple(vt.vt_attn_bwd(q, k, v, o, d_o, lse, c.causal, c.scale, stream=streams[i]))
    torch.cuda.synchronize()
    assert vt.vt_attn_device_status()[0] == 0
    for w, g in zip(want, got):
        for a, b in zip(w, g):
            assert torch.equal(a, b)


def test_bounded_wait_reports_a_timeout_and_the_context_survives(vt):
    """A warp waits on a barrier nothing signals; after the limit the kernel returns, the status word
    says where, and the next real call works."""
    import torch
    assert vt.vt_attn_device_status()[0] == 0
    vt.vt_attn_selftest_timeout(50)
    rc, detail = vt.vt_attn_device_status()
    assert rc == vt.ERR_DEVICE_TIMEOUT
    assert detail & 0xFF == 9 and (detail >> 8) & 0xFF == 3
    assert vt.vt_attn_device_status()[0] == 0           # reading clears it
    cfg = CONFIGS["tiny"]
    q, k, v = make_inputs(cfg, with_do=False)
    o, lse = vt.vt_attn_fwd(dev(q), dev(k), dev(v), cfg.causal, cfg.scale)
    torch.cuda.synchronize()
    o_ref, lse_ref = orc.attn_fwd(q, k, v, cfg.causal, cfg.scale)
    check_fwd(host(o), host(lse), o_ref, lse_ref, "after timeout")


def test_status_word_without_synchronising(vt):
    """The non-blocking pair: the copy of the status word is enqueued into pinned host memory and is valid once the caller
    has synchronised; the reset is enqueued too."""
    import torch
    assert vt.vt_attn_device_status()[0] == 0
    word = torch.full((1,), -1, dtype=torch.int32).pin_memory()
    vt.vt_attn_device_status_async(word)
    torch.cuda.synchronize()
    assert int(word[0]) == 0
    vt.vt_attn_selftest_timeout(20)
    vt.vt_attn_device_status_async(word)
    vt.vt_attn_device_status_clear()
    torch.cuda.synchronize()
    assert int(word[0]) & 0xFF == 9 and (int(word[0]) >> 8) & 0xFF == 3
    assert vt.vt_attn_device_status()[0] == 0           # cleared by the enqueued reset


def test_host_buffer_calls_from_two_threads(vt):
    """Two host threads call the host-buffer forward + backward on their own streams and staging areas at the same
    time; each must get the bits a lone call gives (the library's two side streams and their events are shared)."""
    import threading
    import torch
    cfgs = [CONFIGS["minigpt"], CONFIGS["vit"].with_(B=16)]
    jobs = []
    for c in cfgs:
        bits = make_inputs(c)
        hq, hk, hv, hdo = (torch.from_numpy(np.ascontiguousarray(x).view(np.int16)).view(torch.bfloat16).pin_memory() for x in bits)
        outs = [torch.empty_like(hq).pin_memory(), torch.empty(hq.shape[:3], dtype=torch.float32).pin_memory(),
                torch.empty_like(hq).pin_memory(), torch.empty_like(hk).pin_memory(), torch.empty_like(hv).pin_memory()]
        staging = torch.empty(vt.vt_attn_host_staging_bytes(c.B, c.Hq, c.Hkv, c.Sq, c.Sk, c.D, True), dtype=torch.uint8, device="cuda")
        jobs.append((c, (hq, hk, hv, hdo), outs, staging, torch.cuda.Stream()))

    def run(job, rounds):
        c, (hq, hk, hv, hdo), (o, lse, dq, dk, dv), staging, st = job
        for _ in range(rounds):
            vt.vt_attn_fwd_bwd_host(hq, hk, hv, hdo, o, lse, dq, dk, dv, c.causal, c.scale, staging, stream=st)
        st.synchronize()

    want = []
    for job in jobs:                                     # serial reference
        run(job, 1)
        want.append([t.clone() for t in job[2]])
        for t in job[2]:
            t.zero_()
    errors = []

    def guarded(job):
        try:
            run(job, 25)
        except Exception as e:                           # noqa: BLE001
            errors.append(e)

    threads = [threading.Thread(target=guarded, args=(job,)) for job in jobs]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    torch.cuda.synchronize()
    assert not errors, errors
    assert vt.vt_attn_device_status()[0] == 0
    for job, w in zip(jobs, want):
        for a, b in zip(job[2], w):
            assert torch.equal(a, b)


def test_calls_can_be_captured_in_a_cuda_graph(vt):
    """The entry points neither synchronise nor allocate, so a stream capture around them works and
    replays give the same bits."""
    import torch
    cfg = CONFIGS["minigpt"]
    q, k, v, d_o = (dev(x) for x in make_inputs(cfg))
    o = torch.empty_like(q); lse = torch.empty(q.shape[:3], dtype=torch.float32, device="cuda")
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    ws = torch.empty(max(256, vt.vt_attn_bwd_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.Sq, cfg.Sk, cfg.D)),
                     dtype=torch.uint8, device="cuda")
    vt.vt_attn_fwd(q, k, v, cfg.causal, cfg.scale, o, lse)
    vt.vt_attn_bwd(q, k, v, o, d_o, lse, cfg.causal, cfg.scale, dq, dk, dv, ws)
    torch.cuda.synchronize()
    want = [t.clone() for t in (o, lse, dq, dk, dv)]
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            vt.vt_attn_fwd(q, k, v, cfg.causal, cfg.scale, o, lse, stream=side)
            vt.vt_attn_bwd(q, k, v, o, d_o, lse, cfg.causal, cfg.scale, dq, dk, dv, ws, stream=side)
    for t in (o, lse, dq, dk, dv):
        t.zero_()
    graph.replay()
    torch.cuda.synchronize()
    for a, b in zip(want, (o, lse, dq, dk, dv)):
        assert torch.equal(a, b)


def test_invalid_arguments_on_the_gpu_path(vt):
    import torch
    q = torch.zeros(1, 2, 128, 512, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(vt.VtAttnError) as e:
        vt.vt_attn_fwd(q, q, q, False, 0.1)
    assert e.value.status == vt.ERR_UNSUPPORTED
    q = torch.zeros(1, 3, 128, 64, dtype=torch.bfloat16, device="cuda")
    k = torch.zeros(1, 2, 128, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(ValueError):                      # the binding refuses Hq % Hkv != 0 before the library is entered ...
        vt.vt_attn_fwd(q, k, k, False, 0.1)
    lib = vt.load_library()                              # ... and the library refuses it when called directly
    o = torch.empty_like(q); lse = torch.empty(1, 3, 128, device="cuda")
    rc = lib.vt_attn_fwd(q.data_ptr(), k.data_ptr(), k.data_ptr(), o.data_ptr(), lse.data_ptr(), 1, 3, 2, 128, 128, 64, 0, 0.1, None)
    assert rc == vt.ERR_INVALID_ARGUMENT
    with pytest.raises(vt.VtAttnError) as e:
        vt.vt_attn_fwd(k, k, k, False, float("nan"))
    assert e.value.status == vt.ERR_INVALID_ARGUMENT
    with pytest.raises(ValueError):
        vt.vt_attn_fwd(q.float(), k, k, False, 0.1)


def test_forward_and_backward_can_be_captured_in_a_cuda_graph(vt):
    """The entry points enqueue kernels only (no allocation, no synchronisation, no host-side state that changes between
    calls), so a forward + backward step can be captured once and replayed on new data in the same buffers."""
    import torch
    cfg = CONFIGS["minigpt"]
    bits = make_inputs(cfg)
    q, k, v, d_o = (dev(x) for x in bits)
    o = torch.empty_like(q); lse = torch.empty(q.shape[:3], dtype=torch.float32, device="cuda")
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    ws = torch.empty(vt.vt_attn_bwd_workspace_bytes(cfg.B, cfg.Hq, cfg.Hkv, cfg.Sq, cfg.Sk, cfg.D), dtype=torch.uint8, device="cuda")

    def step():
        vt.vt_attn_fwd(q, k, v, cfg.causal, cfg.scale, o, lse)
        vt.vt_attn_bwd(q, k, v, o, d_o, lse, cfg.causal, cfg.scale, dq, dk, dv, ws)

    step()                                   # first call outside the capture (one-time kernel attribute set-up)
    torch.cuda.synchronize()
    want = [t.clone() for t in (o, lse, dq, dk, dv)]
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for t in (o, lse, dq, dk, dv):
        t.fill_(float("nan"))
    graph.replay()
    torch.cuda.synchronize()
    for a, b in zip(want, (o, lse, dq, dk, dv)):
        assert torch.equal(a, b)
    # new data in the same buffers: the replay computes on what is there now
    bits2 = make_inputs(cfg, seed_offset=50)
    for t, x in zip((q, k, v, d_o), bits2):
        t.copy_(dev(x))
    graph.replay()
    torch.cuda.synchronize()
    o2, lse2 = vt.vt_attn_fwd(q, k, v, cfg.causal, cfg.scale)
    g2 = vt.vt_attn_bwd(q, k, v, o2, d_o, lse2, cfg.causal, cfg.scale)
    torch.cuda.synchronize()
    assert torch.equal(o, o2) and torch.equal(lse, lse2) and all(torch.equal(a, b) for a, b in zip((dq, dk, dv), g2))
    assert vt.vt_attn_device_status()[0] == 0
