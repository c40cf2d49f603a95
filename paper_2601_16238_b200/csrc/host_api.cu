// Entry points that take HOST buffers, and the build-info query.
//
// The problem is cut into chunks of whole (batch, KV head) groups - every group is an independent attention problem and a
// contiguous slice of each tensor - and the chunks alternate between two internal streams: while chunk i computes, chunk
// i + 1 is copied in and chunk i - 1 is copied out (the two copy directions use different DMA engines), so a call takes
// about max(copies in, kernels, copies out) instead of their sum.  The internal streams fork from and join back into the
// caller's stream with events, so the call is still asynchronous and ordered like any other work on that stream.
#include <mutex>

#include "vt_host.h"

namespace vt {

static size_t align256(size_t n) { return (n + 255) & ~static_cast<size_t>(255); }

constexpr int MAX_CHUNKS = 8;

struct Chunk {
    int b0, nb, g0, ng;          // batches [b0, b0 + nb) x KV heads [g0, g0 + ng)  (nb > 1 only with all KV heads)
};

// Chunks of about equal size: whole batches when there are at least as many batches as chunks, else KV-head ranges inside
// each batch.  `min_units` keeps a chunk large enough to fill the GPU (units = (batch, KV head) groups).
static int make_chunks(int B, int Hkv, int min_units, int max_chunks, Chunk (&out)[MAX_CHUNKS * 2])
{
    const int units = B * Hkv;
    int want = units / (min_units > 0 ? min_units : 1);
    if (want > max_chunks) want = max_chunks;
    if (want < 1) want = 1;
    int n = 0;
    if (want <= B) {
        for (int c = 0; c < want; ++c) {
            const int b0 = static_cast<int>(static_cast<long long>(B) * c / want), b1 = static_cast<int>(static_cast<long long>(B) * (c + 1) / want);
            if (b1 > b0) out[n++] = Chunk{b0, b1 - b0, 0, Hkv};
        }
    } else {
        int per_batch = want / B;
        if (per_batch > Hkv) per_batch = Hkv;
        if (per_batch * B > MAX_CHUNKS * 2) per_batch = (MAX_CHUNKS * 2) / B;
        if (per_batch < 1) per_batch = 1;
        for (int b = 0; b < B; ++b)
            for (int c = 0; c < per_batch; ++c) {
                const int g0 = Hkv * c / per_batch, g1 = Hkv * (c + 1) / per_batch;
                if (g1 > g0) out[n++] = Chunk{b, 1, g0, g1 - g0};
            }
    }
    return n;
}

struct Staging {
    size_t q, k, v, o, lse, d_o, dq, dk, dv, ws, total;     // byte offsets
    size_t q_bytes, kv_bytes, lse_bytes, ws_bytes;
};

static Staging plan(int B, int Hq, int Hkv, int Sq, int Sk, int D, bool with_backward)
{
    Staging s{};
    s.q_bytes = static_cast<size_t>(B) * Hq * Sq * D * 2;
    s.kv_bytes = static_cast<size_t>(B) * Hkv * Sk * D * 2;
    s.lse_bytes = static_cast<size_t>(B) * Hq * Sq * 4;
    // one Delta scratch per chunk, each 256-byte aligned
    s.ws_bytes = with_backward ? vt_attn_bwd_workspace_bytes(B, Hq, Hkv, Sq, Sk, D) + 256 * (MAX_CHUNKS * 2) : 0;
    size_t off = 0;
    auto take = [&off](size_t bytes) { size_t at = off; off += align256(bytes); return at; };
    s.q = take(s.q_bytes);
    s.k = take(s.kv_bytes);
    s.v = take(s.kv_bytes);
    s.o = take(s.q_bytes);
    s.lse = take(s.lse_bytes);
    if (with_backward) {
        s.d_o = take(s.q_bytes);
        s.dq = take(s.q_bytes);
        s.dk = take(s.kv_bytes);
        s.dv = take(s.kv_bytes);
        s.ws = take(s.ws_bytes);
    }
    s.total = off;
    return s;
}

static int copy(void *dst, const void *src, size_t bytes, cudaMemcpyKind kind, cudaStream_t st, const char *what)
{
    cudaError_t e = cudaMemcpyAsync(dst, src, bytes, kind, st);
    if (e != cudaSuccess) return cuda_fail(e, what);
    return VT_ATTN_OK;
}

// Two side streams and three events per device, created on first use and kept (the only host-side state besides the
// tensor-map cache).
struct SideStreams {
    cudaStream_t s[2];
    cudaEvent_t start, done[2];
    bool ready;
};
static SideStreams g_side[64];
static std::mutex g_side_mutex;      // creation of the streams and events
static std::mutex g_call_mutex;      // the fork / enqueue / join of one host-buffer call

static int side_streams(SideStreams **out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    std::lock_guard<std::mutex> lock(g_side_mutex);
    SideStreams &ss = g_side[dev & 63];
    if (!ss.ready) {
        for (int i = 0; i < 2; ++i) {
            if ((e = cudaStreamCreateWithFlags(&ss.s[i], cudaStreamNonBlocking)) != cudaSuccess) return cuda_fail(e, "cudaStreamCreateWithFlags");
            if ((e = cudaEventCreateWithFlags(&ss.done[i], cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e, "cudaEventCreateWithFlags");
        }
        if ((e = cudaEventCreateWithFlags(&ss.start, cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(e, "cudaEventCreateWithFlags");
        ss.ready = true;
    }
    *out = &ss;
    return VT_ATTN_OK;
}

struct HostArgs {
    const uint8_t *q, *k, *v, *d_o;                 // host
    uint8_t *o, *lse, *dq, *dk, *dv;                // host
};

static int run_chunked(bool f16, const HostArgs &h, int B, int Hq, int Hkv, int Sq, int Sk, int D, int causal, float scale, uint8_t *base,
                       const Staging &s, bool with_backward, cudaStream_t user)
{
    const auto fwd = f16 ? vt_attn_fwd_f16 : vt_attn_fwd;      // the two element types are both 16 bits wide: same layout, same copies
    const auto bwd = f16 ? vt_attn_bwd_f16 : vt_attn_bwd;
    const int G = Hq / Hkv;
    // a chunk should still fill the GPU: its smallest grid (one block per 128-key tile and KV head in the backward, one block
    // per SM; per query tile or pair of tiles and query head in the forward, two per SM) gets at least one wave
    const long long per_unit = with_backward ? (Sk + TILE - 1) / TILE : static_cast<long long>((Sq + 2 * TILE - 1) / (2 * TILE)) * G;
    int min_units = static_cast<int>(((with_backward ? NUM_SMS : 2 * NUM_SMS) + per_unit - 1) / per_unit);
    // When the copies take much longer than the kernels (a forward over PCIe: ~50 GB/s in against ~800 TFLOP/s), what the
    // call costs beyond its input copies is the LAST chunk's kernel and output copy: smaller chunks (a quarter of a wave is
    // enough, the kernels are not what is waited for) and twice as many of them shorten that tail.
    const double in_bytes = (with_backward ? 2.0 : 1.0) * static_cast<double>(s.q_bytes) + 2.0 * static_cast<double>(s.kv_bytes);
    const double flops = 4.0 * B * Hq * static_cast<double>(Sq) * Sk * D * (causal ? 0.5 : 1.0) * (with_backward ? 3.5 : 1.0);
    const bool copy_bound = 2.0 * flops / 800e12 < in_bytes / 50e9;
    if (copy_bound) min_units = (min_units + 3) / 4;
    Chunk chunks[MAX_CHUNKS * 2];
    const int n = make_chunks(B, Hkv, min_units, copy_bound ? 2 * MAX_CHUNKS : MAX_CHUNKS, chunks);
    SideStreams *ss = nullptr;
    int rc = side_streams(&ss);
    if (rc != VT_ATTN_OK) return rc;
    // One call at a time per process forks onto and joins from the library's streams and events: a second thread's
    // cudaEventRecord(start) between this thread's record and its waits would move this call's fork point.  Everything
    // below only enqueues, so the lock is held for microseconds.
    std::lock_guard<std::mutex> call_lock(g_call_mutex);
    cudaError_t e;
    if ((e = cudaEventRecord(ss->start, user)) != cudaSuccess) return cuda_fail(e, "cudaEventRecord");
    for (int i = 0; i < 2; ++i)
        if ((e = cudaStreamWaitEvent(ss->s[i], ss->start, 0)) != cudaSuccess) return cuda_fail(e, "cudaStreamWaitEvent");
    size_t ws_off = 0;
    for (int c = 0; c < n && rc == VT_ATTN_OK; ++c) {
        const Chunk &ck = chunks[c];
        cudaStream_t st = ss->s[c & 1];
        const int cB = ck.nb, cHkv = ck.ng, cHq = ck.ng * G;
        const size_t q_off = (static_cast<size_t>(ck.b0) * Hq + static_cast<size_t>(ck.g0) * G) * Sq * D * 2;
        const size_t kv_off = (static_cast<size_t>(ck.b0) * Hkv + ck.g0) * Sk * D * 2;
        const size_t lse_off = (static_cast<size_t>(ck.b0) * Hq + static_cast<size_t>(ck.g0) * G) * Sq * 4;
        const size_t q_bytes = static_cast<size_t>(cB) * cHq * Sq * D * 2, kv_bytes = static_cast<size_t>(cB) * cHkv * Sk * D * 2;
        const size_t lse_bytes = static_cast<size_t>(cB) * cHq * Sq * 4;
        if ((rc = copy(base + s.q + q_off, h.q + q_off, q_bytes, cudaMemcpyHostToDevice, st, "copy q")) != VT_ATTN_OK) break;
        if ((rc = copy(base + s.k + kv_off, h.k + kv_off, kv_bytes, cudaMemcpyHostToDevice, st, "copy k")) != VT_ATTN_OK) break;
        if ((rc = copy(base + s.v + kv_off, h.v + kv_off, kv_bytes, cudaMemcpyHostToDevice, st, "copy v")) != VT_ATTN_OK) break;
        if (with_backward && (rc = copy(base + s.d_o + q_off, h.d_o + q_off, q_bytes, cudaMemcpyHostToDevice, st, "copy dO")) != VT_ATTN_OK) break;
        float *lse = reinterpret_cast<float *>(base + s.lse + lse_off);
        rc = fwd(base + s.q + q_off, base + s.k + kv_off, base + s.v + kv_off, base + s.o + q_off, lse, cB, cHq, cHkv, Sq, Sk, D,
                 causal, scale, st);
        if (rc != VT_ATTN_OK) break;
        if (with_backward) {
            const size_t ws_bytes = vt_attn_bwd_workspace_bytes(cB, cHq, cHkv, Sq, Sk, D);
            rc = bwd(base + s.q + q_off, base + s.k + kv_off, base + s.v + kv_off, base + s.o + q_off, base + s.d_o + q_off, lse,
                     base + s.dq + q_off, base + s.dk + kv_off, base + s.dv + kv_off, cB, cHq, cHkv, Sq, Sk, D, causal, scale,
                     base + s.ws + ws_off, ws_bytes, st);
            if (rc != VT_ATTN_OK) break;
            ws_off += align256(ws_bytes);
        }
        if ((rc = copy(h.o + q_off, base + s.o + q_off, q_bytes, cudaMemcpyDeviceToHost, st, "copy o")) != VT_ATTN_OK) break;
        if ((rc = copy(h.lse + lse_off, lse, lse_bytes, cudaMemcpyDeviceToHost, st, "copy lse")) != VT_ATTN_OK) break;
        if (with_backward) {
            if ((rc = copy(h.dq + q_off, base + s.dq + q_off, q_bytes, cudaMemcpyDeviceToHost, st, "copy dq")) != VT_ATTN_OK) break;
            if ((rc = copy(h.dk + kv_off, base + s.dk + kv_off, kv_bytes, cudaMemcpyDeviceToHost, st, "copy dk")) != VT_ATTN_OK) break;
            if ((rc = copy(h.dv + kv_off, base + s.dv + kv_off, kv_bytes, cudaMemcpyDeviceToHost, st, "copy dv")) != VT_ATTN_OK) break;
        }
    }
    // join, also after an error: the caller's stream must not run ahead of what was enqueued
    for (int i = 0; i < 2; ++i) {
        if ((e = cudaEventRecord(ss->done[i], ss->s[i])) != cudaSuccess) return cuda_fail(e, "cudaEventRecord");
        if ((e = cudaStreamWaitEvent(user, ss->done[i], 0)) != cudaSuccess) return cuda_fail(e, "cudaStreamWaitEvent");
    }
    return rc;
}

}  // namespace vt

extern "C" size_t vt_attn_host_staging_bytes(int B, int Hq, int Hkv, int Sq, int Sk, int D, int with_backward)
{
    vt::Shape s{B, Hq, Hkv, Sq, Sk, D};
    if (vt::check_shape(s, 1.0f, vt::MAX_HEAD_DIM_FWD) != VT_ATTN_OK) return 0;
    return vt::plan(B, Hq, Hkv, Sq, Sk, D, with_backward != 0).total;
}

static int fwd_host_entry(bool f16, const void *q_host, const void *k_host, const void *v_host, void *o_host, float *lse_host,
                          int B, int Hq, int Hkv, int Sq, int Sk, int D, int causal, float scale, void *staging,
                          size_t staging_bytes, void *stream)
{
    using namespace vt;
    Shape sh{B, Hq, Hkv, Sq, Sk, D};
    int rc = check_shape(sh, scale, MAX_HEAD_DIM_FWD);
    if (rc != VT_ATTN_OK) return rc;
    if (!q_host || !k_host || !v_host || !o_host || !lse_host || !ptr_ok(staging, 256)) return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (causal < 0 || causal > 2) return VT_ATTN_ERR_INVALID_ARGUMENT;
    const Staging s = plan(B, Hq, Hkv, Sq, Sk, D, false);
    if (staging_bytes < s.total) return VT_ATTN_ERR_WORKSPACE_TOO_SMALL;
    if ((rc = check_device()) != VT_ATTN_OK) return rc;
    HostArgs h{static_cast<const uint8_t *>(q_host), static_cast<const uint8_t *>(k_host), static_cast<const uint8_t *>(v_host), nullptr,
               static_cast<uint8_t *>(o_host), reinterpret_cast<uint8_t *>(lse_host), nullptr, nullptr, nullptr};
    return run_chunked(f16, h, B, Hq, Hkv, Sq, Sk, D, causal, scale, static_cast<uint8_t *>(staging), s, false, static_cast<cudaStream_t>(stream));
}

extern "C" int vt_attn_fwd_host(const void *q_host, const void *k_host, const void *v_host, void *o_host, float *lse_host,
                                int B, int Hq, int Hkv, int Sq, int Sk, int D, int causal, float scale, void *staging,
                                size_t staging_bytes, void *stream)
{
    return fwd_host_entry(false, q_host, k_host, v_host, o_host, lse_host, B, Hq, Hkv, Sq, Sk, D, causal, scale, staging, staging_bytes, stream);
}

extern "C" int vt_attn_fwd_host_f16(const void *q_host, const void *k_host, const void *v_host, void *o_host, float *lse_host,
                                    int B, int Hq, int Hkv, int Sq, int Sk, int D, int causal, float scale, void *staging,
                                    size_t staging_bytes, void *stream)
{
    return fwd_host_entry(true, q_host, k_host, v_host, o_host, lse_host, B, Hq, Hkv, Sq, Sk, D, causal, scale, staging, staging_bytes, stream);
}

static int fwd_bwd_host_entry(bool f16, const void *q_host, const void *k_host, const void *v_host, const void *d_o_host,
                              void *o_host, float *lse_host, void *dq_host, void *dk_host, void *dv_host, int B,
                              int Hq, int Hkv, int Sq, int Sk, int D, int causal, float scale, void *staging,
                              size_t staging_bytes, void *stream)
{
    using namespace vt;
    Shape sh{B, Hq, Hkv, Sq, Sk, D};
    int rc = check_shape(sh, scale, MAX_HEAD_DIM_FWD);
    if (rc != VT_ATTN_OK) return rc;
    if (!q_host || !k_host || !v_host || !d_o_host || !o_host || !lse_host || !dq_host || !dk_host || !dv_host ||
        !ptr_ok(staging, 256))
        return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (causal < 0 || causal > 2) return VT_ATTN_ERR_INVALID_ARGUMENT;
    const Staging s = plan(B, Hq, Hkv, Sq, Sk, D, true);
    if (staging_bytes < s.total) return VT_ATTN_ERR_WORKSPACE_TOO_SMALL;
    if ((rc = check_device()) != VT_ATTN_OK) return rc;
    HostArgs h{static_cast<const uint8_t *>(q_host), static_cast<const uint8_t *>(k_host), static_cast<const uint8_t *>(v_host),
               static_cast<const uint8_t *>(d_o_host), static_cast<uint8_t *>(o_host), reinterpret_cast<uint8_t *>(lse_host),
               static_cast<uint8_t *>(dq_host), static_cast<uint8_t *>(dk_host), static_cast<uint8_t *>(dv_host)};
    return run_chunked(f16, h, B, Hq, Hkv, Sq, Sk, D, causal, scale, static_cast<uint8_t *>(staging), s, true, static_cast<cudaStream_t>(stream));
}

extern "C" int vt_attn_fwd_bwd_host(const void *q_host, const void *k_host, const void *v_host, const void *d_o_host,
                                    void *o_host, float *lse_host, void *dq_host, void *dk_host, void *dv_host, int B,
                                    int Hq, int Hkv, int Sq, int Sk, int D, int causal, float scale, void *staging,
                                    size_t staging_bytes, void *stream)
{
    return fwd_bwd_host_entry(false, q_host, k_host, v_host, d_o_host, o_host, lse_host, dq_host, dk_host, dv_host, B, Hq, Hkv, Sq, Sk, D,
                              causal, scale, staging, staging_bytes, stream);
}

extern "C" int vt_attn_fwd_bwd_host_f16(const void *q_host, const void *k_host, const void *v_host, const void *d_o_host,
                                        void *o_host, float *lse_host, void *dq_host, void *dk_host, void *dv_host, int B,
                                        int Hq, int Hkv, int Sq, int Sk, int D, int causal, float scale, void *staging,
                                        size_t staging_bytes, void *stream)
{
    return fwd_bwd_host_entry(true, q_host, k_host, v_host, d_o_host, o_host, lse_host, dq_host, dk_host, dv_host, B, Hq, Hkv, Sq, Sk, D,
                              causal, scale, staging, staging_bytes, stream);
}

extern "C" int vt_attn_get_info(int *info, int n)
{
    const int vals[8] = {VT_ATTN_ABI_VERSION, vt::TILE, 64, 256, 128 * 128 * 2 * 3 + 256 + 1024, 256, 1, 3};
    int i = 0;
    for (; i < n && i < 8; ++i) info[i] = vals[i];
    return i;
}
