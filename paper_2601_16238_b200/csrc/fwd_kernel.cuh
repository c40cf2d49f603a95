// Forward fused attention kernel for sm_100a (shared by the plain, packed and split-KV entry points).
//
// One block owns one 128-row query tile of one (batch, query head) and walks the keys it can
// see in steps of 64 ("half tiles").  The score tile S is double-buffered in tensor memory, so the
// tensor core computes S of step t+1 (and O += P V of step t-1) while the softmax warps work on
// step t: inside a block the MMAs and the softmax overlap, and two blocks share an SM.
// Roles (256 threads = two warpgroups):
//   warps 0..3  softmax     : one thread per query row; reads its 64 scores from TMEM, keeps the
//                             running row maximum and row sum in exp2 form, writes the bf16 P
//                             back over S, rescales O only when the maximum has moved by more
//                             than 2^8, and at the end normalises O and writes O and LSE.
//                             This warpgroup raises its register allowance (setmaxnreg).
//   warp 4      TMA producer for Q and the K half tiles (ring of 64-row slots, 128-byte swizzle)
//   warp 5      MMA issuer  : S_t = Q K_t^T (tcgen05, smem x smem -> TMEM, N = 64) and
//                             O += P_t V_t (tcgen05, TMEM x smem -> TMEM); owns the TMEM allocation
//   warp 6      TMA producer for the V half tiles
//   warp 7      idle
#pragma once
#include "vt_host.h"

namespace vt {

constexpr int FWD_THREADS = 256;
constexpr int SOFTMAX_REGS = 216;          // 128 threads x 216 + 128 threads x 40 = 256 x 128
constexpr int OTHER_REGS = 40;
constexpr int BN = 64;                      // keys per step
// Tensor-memory columns of a block: S buffers [0,64), [64,128) (P over the first 32 of each), O in [128,128+D); the
// allocation is a power of two (D = 256: one block per SM).
__host__ __device__ constexpr int fwd_tmem_cols(int D) { return D > 128 ? 512 : 256; }
constexpr uint32_t FWD_KERNEL_ID = 1;
constexpr float RESCALE_THRESHOLD = 8.0f;   // log2 units

// P is written as bf16: tcgen05.mma kind::f16 needs A and B in the same 16-bit format (an
// fp16 P against bf16 V raises an illegal-instruction error on sm_100a), and V arrives as bf16.

template <int D>
struct FwdSmem {
    static constexpr int Q_BYTES = TILE * D * 2;
    static constexpr int KV_BYTES = BN * D * 2;                // one 64-row half tile
    static constexpr int KV_SLOTS = (D == 64) ? 4 : 2;
    static constexpr int OFF_Q = 0;
    static constexpr int OFF_K = OFF_Q + Q_BYTES;
    static constexpr int OFF_V = OFF_K + KV_SLOTS * KV_BYTES;
    static constexpr int OFF_BAR = OFF_V + KV_SLOTS * KV_BYTES;
    static constexpr int BAR_BYTES = 256;
    static constexpr int BYTES = OFF_BAR + BAR_BYTES + 1024;   // + slack to align the base to 1024
};

struct FwdParams {
    __nv_bfloat16 *o;
    float *lse;
    int Hq, G, Sq, Sk;     // packed batches: Sq, Sk are the maxima over the sequences
    int d;                 // head dimension of V and O in global memory (<= the kernel's D; the columns between read as zero)
    int d_qk;              // head dimension of Q and K (the contraction width of S = Q K^T); equal to d except in vt_attn_fwd_dv
    int n_qt;              // query tiles per head (of the longest sequence)
    float scale_log2e;     // scale * log2(e)
    const int *cu_q;       // packed batches only: cumulative sequence lengths [n_seqs + 1], device
    const int *cu_k;
    int total_q;           // packed batches only: tokens in q
    int bottom_right;      // causal only: the mask is aligned to the last query / last key (key j visible iff j <= i + Sk - Sq)
    // SPLIT only: the key steps are cut into n_splits chunks of chunk_steps steps; every chunk writes a normalised fp32
    // partial result and its own LSE, which a merge kernel combines
    int n_splits, chunk_steps;
    float *o_part;         // [n_splits, n_rows, D]
    float *lse_part;       // [n_splits, n_rows]
    long long n_rows;      // B * Hq * Sq (packed batches: total_q * Hq, row = token * Hq + head)
    int hp_tokens;         // PACKED + HPACK: tokens per Q box (the longest sequence's queries)
    int head_group;        // causal kernels: heads per scheduling group (see causal_work_item); 0 or 1: one head after the other
    // ROPE only: rotary tables [positions, D / 2] (fp32) and the position of query 0 (query i sits at rope_pos0 + i)
    const float *rope_cos = nullptr;
    const float *rope_sin = nullptr;
    int rope_pos0 = 0;
    Guard guard;
};

// PACKED: q, o are [total_q, Hq, D], k, v are [total_k, Hkv, D], lse is [Hq, total_q]; "batch" b is a sequence that
// owns the token rows [cu[b], cu[b+1]).  Otherwise the tensors are [B, H, S, D] and lse is [B, Hq, Sq].
// SPLIT: the block walks only its chunk of the key steps and writes a partial result (see FwdParams).
// HPACK (needs G * Sq <= 128, one block per (batch, KV head)): the tile's rows are the Sq queries of all G query heads that
// share the KV head, row = head_in_group * Sq + query, so K / V are walked once for the whole group (decoding shapes).
// With PACKED the Q box is [tokens][heads], so the row is query * G + head_in_group, and the rows past the sequence's
// own queries belong to the next sequence (computed, never stored).
// ROPE (batched layout, D = 64 or 128 and equal to the tensors' head dimension): Q arrives unrotated; once the tile is in
// shared memory every softmax thread turns its own query row by its position's angles ("rotate-half": element i pairs
// with element i + D / 2), writes it back in the tensors' 16-bit type and only then lets the first product start.  K
// must come already rotated: a key tile is walked by every query tile of its head, rotating it here would repeat that
// work once per query tile.
template <int D, bool CAUSAL, bool PACKED, bool SPLIT = false, bool HPACK = false, bool F16 = false, bool ROPE = false>
__global__ void __launch_bounds__(FWD_THREADS, 2)
attn_fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_v, const FwdParams p)
{
    using L = FwdSmem<D>;
    constexpr int SL = L::KV_SLOTS;
    constexpr int NBOX = D / BOX_COLS;                  // 64-column boxes per row
    constexpr int QBOX_BYTES = TILE * BOX_COLS * 2;     // 16 KB
    constexpr int KBOX_BYTES = BN * BOX_COLS * 2;       // 8 KB
    // At D = 64 the exponential unit, not the tensor core, bounds the kernel: one eighth of the
    // exponentials is evaluated with a cubic on the FMA pipe instead (measured +14 %; at D = 128
    // any share made the kernel slower).
    constexpr int POLY_EIGHTHS = (D == 64) ? 1 : 0;

    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *sQ = smem + L::OFF_Q;
    uint8_t *sK = smem + L::OFF_K;
    uint8_t *sV = smem + L::OFF_V;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L::OFF_BAR);
    uint64_t *q_full = bars + 0;
    uint64_t *o_final = bars + 1;
    uint64_t *pv_done = bars + 2;
    uint64_t *s_full = bars + 3;             // [2]
    uint64_t *p_ready = bars + 5;            // [2]
    uint64_t *k_full = bars + 7;             // [SL]
    uint64_t *k_empty = bars + 7 + SL;       // [SL]
    uint64_t *v_full = bars + 7 + 2 * SL;    // [SL]
    uint64_t *v_empty = bars + 7 + 3 * SL;   // [SL]
    uint64_t *q_rot = bars + 7 + 4 * SL;     // ROPE: 128 arrivals, the query rows have been rotated in place
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 8 + 4 * SL);
    volatile uint32_t *abort_flag = tmem_slot + 1;
    static_assert(!ROPE || (!PACKED && !SPLIT && !HPACK && (D == 64 || D == 128)), "rotary queries: batched layout, D = 64 or 128");

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    // work item: heads are the slow index so that the blocks resident at one time share K/V in L2;
    // causal heads hand out their long (late) query tiles first
    int blk = blockIdx.x, split = 0;
    if (SPLIT) {
        split = blk % p.n_splits;
        blk /= p.n_splits;
    }
    int bh = blk / p.n_qt;                        // HPACK: (batch, KV head)
    int qt = blk % p.n_qt;
    if (CAUSAL && !SPLIT && !HPACK) bh = causal_work_item(blk, p.n_qt, static_cast<int>(gridDim.x) / p.n_qt, p.head_group, qt);
    if (CAUSAL) qt = p.n_qt - 1 - qt;
    const int Hkv = p.Hq / p.G;
    const int b = HPACK ? bh / Hkv : bh / p.Hq;
    const int h = HPACK ? (bh % Hkv) * p.G : bh % p.Hq;   // HPACK: first query head of the group
    const int hkv = h / p.G;
    const int bh_kv = b * Hkv + hkv;
    const int q0 = qt * TILE;
    int Sq = p.Sq, Sk = p.Sk, q_base = 0, k_base = 0;     // this block's sequence: lengths and first token rows
    if (PACKED) {
        q_base = p.cu_q[b];
        Sq = p.cu_q[b + 1] - q_base;
        k_base = p.cu_k[b];
        Sk = p.cu_k[b + 1] - k_base;
        if (q0 >= Sq) return;                             // this sequence has no such query tile (whole block leaves)
    }
    // causal: query i sees the keys j <= i + off; rows with i + off < 0 (bottom-right alignment with fewer keys than
    // queries) see none: their softmax is empty, O = 0 and LSE = -inf
    const int off = (CAUSAL && p.bottom_right) ? Sk - Sq : 0;
    int n_t = (Sk + BN - 1) / BN;                         // steps of 64 keys (0: no key is visible to this tile)
    const int q_last = (HPACK ? Sq - 1 : q0 + TILE - 1) + off;      // last key any query of this tile can see (causal)
    if (CAUSAL) n_t = (q_last < 0) ? 0 : min(n_t, q_last / BN + 1);
    int t0 = 0;                                           // first step of this block; n_t counts its steps from here on
    if (SPLIT) {
        // packed batches: every sequence's own steps are cut into n_splits chunks, so a short cache costs its blocks
        // little and leaves no chunk empty while it has keys; otherwise the chunk length is the launch's
        const int cs = PACKED ? (n_t + p.n_splits - 1) / p.n_splits : p.chunk_steps;
        t0 = split * cs;
        n_t = max(0, min(n_t, t0 + cs) - t0);
    }
    // TMA coordinates (column, then the two outer ones) of a box of rows starting at `r` of this block's Q / K / V
    const int qc1 = PACKED ? h : q0, qc2 = PACKED ? q_base + q0 : (HPACK ? b * p.Hq + h : bh);
    auto kv_c1 = [&](int r) { return PACKED ? hkv : r; };
    auto kv_c2 = [&](int r) { return PACKED ? k_base + r : bh_kv; };

    constexpr int PRODUCER_THREAD = 4 * 32;                  // lane 0 of the Q / K producer warp
    const int n_pre = min(n_t, SL);                           // K steps whose loads go out before the block-wide sync
    if (threadIdx.x == PRODUCER_THREAD) {
        mbar_init(q_full, 1);
        mbar_init(o_final, 1);
        mbar_init(pv_done, 1);
        if (ROPE) mbar_init(q_rot, 128);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&s_full[s], 1);
            mbar_init(&p_ready[s], 128);
        }
        for (int s = 0; s < SL; ++s) {
            mbar_init(&k_full[s], 1);
            mbar_init(&k_empty[s], 1);
            mbar_init(&v_full[s], 1);
            mbar_init(&v_empty[s], 1);
        }
        *abort_flag = 0u;
        fence_mbar_init();
        // the producer initialised the barriers itself, so its first loads need not wait for the block-wide sync: their
        // latency overlaps the TMEM allocation and the other roles' start-up
        prefetch_tensormap(&tm_q);
        prefetch_tensormap(&tm_k);
        mbar_arrive_expect_tx(q_full, HPACK ? p.G * (PACKED ? p.hp_tokens : Sq) * D * 2 : L::Q_BYTES);     // HPACK: a box of Sq rows x G heads
        for (int kb = 0; kb < NBOX; ++kb) tma_load_3d(sQ + kb * QBOX_BYTES, &tm_q, q_full, kb * BOX_COLS, qc1, qc2);
        for (int t = 0; t < n_pre; ++t) {
            mbar_arrive_expect_tx(&k_full[t], L::KV_BYTES);
            for (int kb = 0; kb < NBOX; ++kb)
                tma_load_3d(sK + t * L::KV_BYTES + kb * KBOX_BYTES, &tm_k, &k_full[t], kb * BOX_COLS, kv_c1((t0 + t) * BN), kv_c2((t0 + t) * BN));
        }
    }
    if (warp == 5) {
        tmem_alloc(tmem_slot, fwd_tmem_cols(D));
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_O = tmem_base + 128;

    if (warp >= 4) {
        setmaxnreg_dec<OTHER_REGS>();
        if (warp == 4) {
            // -------------------------------------------------------------- TMA producer: Q, K
            if (lane == 0) {
                for (int t = n_pre; t < n_t; ++t) {        // (Q and the first K steps were issued before the sync)
                    const int sl = t % SL;
                    const uint32_t ph = (t / SL) & 1;
                    if (!mbar_wait(&k_empty[sl], ph ^ 1, abort_flag, p.guard, status_word(FWD_KERNEL_ID, ROLE_LOAD, t))) break;
                    mbar_arrive_expect_tx(&k_full[sl], L::KV_BYTES);
                    for (int kb = 0; kb < NBOX; ++kb)
                        tma_load_3d(sK + sl * L::KV_BYTES + kb * KBOX_BYTES, &tm_k, &k_full[sl], kb * BOX_COLS, kv_c1((t0 + t) * BN), kv_c2((t0 + t) * BN));
                }
            }
        } else if (warp == 6) {
            // -------------------------------------------------------------- TMA producer: V
            if (lane == 0) {
                prefetch_tensormap(&tm_v);
                for (int t = 0; t < n_t; ++t) {
                    const int sl = t % SL;
                    const uint32_t ph = (t / SL) & 1;
                    if (!mbar_wait(&v_empty[sl], ph ^ 1, abort_flag, p.guard, status_word(FWD_KERNEL_ID, ROLE_LOAD, t))) break;
                    mbar_arrive_expect_tx(&v_full[sl], L::KV_BYTES);
                    for (int kb = 0; kb < NBOX; ++kb)
                        tma_load_3d(sV + sl * L::KV_BYTES + kb * KBOX_BYTES, &tm_v, &v_full[sl], kb * BOX_COLS, kv_c1((t0 + t) * BN), kv_c2((t0 + t) * BN));
                }
            }
        } else if (warp == 5) {
            // -------------------------------------------------------------- MMA issuer
            constexpr uint32_t IDESC_QK = make_idesc(128, BN, fmt16<F16>(), fmt16<F16>(), 0, 0);
            // a head dimension below D (the columns past it are zero): the products skip the 16-column blocks that hold
            // nothing - fewer contraction steps for S, a narrower N for O
            const int kd = (p.d_qk + 15) >> 4;
            const uint32_t IDESC_PV = make_idesc(128, ((p.d + 15) >> 4) * 16, fmt16<F16>(), fmt16<F16>(), 0, 1);
            const uint32_t tmem_u = __shfl_sync(0xFFFFFFFFu, tmem_base, 0);    // provably warp-uniform copy
            const uint64_t dQ0 = smem_desc_sw128(smem_u32(sQ), 16, 1024);
            bool ok = mbar_wait(ROPE ? q_rot : q_full, 0, abort_flag, p.guard, status_word(FWD_KERNEL_ID, ROLE_MMA, 0xFFFF));
            if (n_t == 0) ok = false;                     // no keys: nothing to issue (Q was still waited for, so no copy is in flight at exit)
            // S_t = Q K_t^T into S buffer t & 1
            auto issue_qk = [&](int t) -> bool {
                const int sl = t % SL;
                if (!mbar_wait(&k_full[sl], (t / SL) & 1, abort_flag, p.guard, status_word(FWD_KERNEL_ID, ROLE_MMA, t))) return false;
                tc_fence_after_sync();
                if (elect_one()) {
                    const uint64_t dK0 = smem_desc_sw128(smem_u32(sK + sl * L::KV_BYTES), 16, 1024);
                    const uint32_t tS = tmem_u + (t & 1) * BN;
#pragma unroll
                    for (int k = 0; k < D / 16; ++k)
                        if (k < kd)
                            umma_ss(tS, desc_advance(dQ0, (k / 4) * QBOX_BYTES + (k % 4) * 32),
                                    desc_advance(dK0, (k / 4) * KBOX_BYTES + (k % 4) * 32), IDESC_QK, k > 0 ? 1u : 0u);
                    umma_commit(&k_empty[sl]);
                    umma_commit(&s_full[t & 1]);
                }
                __syncwarp();
                return true;
            };
            if (ok) ok = issue_qk(0);
            if (ok && n_t > 1) ok = issue_qk(1);
            for (int t = 0; t < n_t && ok; ++t) {
                const int sl = t % SL;
                ok = mbar_wait(&v_full[sl], (t / SL) & 1, abort_flag, p.guard, status_word(FWD_KERNEL_ID, ROLE_MMA, t));
                if (!ok) break;
                ok = mbar_wait(&p_ready[t & 1], (t >> 1) & 1, abort_flag, p.guard, status_word(FWD_KERNEL_ID, ROLE_MMA, t));
                if (!ok) break;
                tc_fence_after_sync();
                if (elect_one()) {
                    const uint64_t dV0 = smem_desc_sw128(smem_u32(sV + sl * L::KV_BYTES), KBOX_BYTES, 1024);
                    const uint32_t tP = tmem_u + (t & 1) * BN;
#pragma unroll
                    for (int k = 0; k < BN / 16; ++k) {
                        // 16 key rows per step: 2 KB further down the swizzled V slot; the second
                        // 64-column half of V sits one box (8 KB) further
                        umma_ts(tmem_u + 128, tP + k * 8, desc_advance(dV0, k * 2048), IDESC_PV, (t > 0 || k > 0) ? 1u : 0u);
                    }
                    umma_commit(&v_empty[sl]);
                    umma_commit(pv_done);
                    if (t == n_t - 1) umma_commit(o_final);
                }
                __syncwarp();
                if (t + 2 < n_t) ok = issue_qk(t + 2);      // overwrites P_t's buffer: ordered behind the PV just issued
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax + epilogue
        setmaxnreg_inc<SOFTMAX_REGS>();
        const int r = warp * 32 + lane;            // row inside the tile == TMEM lane (warp w owns lanes 32w..32w+31)
        const int row = HPACK ? (PACKED ? r / p.G : r % Sq) : q0 + r;     // query index
        const int h_out = HPACK ? h + (PACKED ? r % p.G : r / Sq) : h;    // query head of this row
        const bool live = HPACK ? r < p.G * Sq : true;                    // HPACK: the row holds a query of this work item
        const uint32_t lane_addr = static_cast<uint32_t>(warp * 32) << 16;
        const float c = p.scale_log2e;
        float m_used = -INFINITY;                  // maximum (raw scores) the accumulators are scaled by
        float l = 0.0f;
        bool ok = true;
        if (ROPE) {
            // This thread's query row, in place: chunk c (8 elements) of the first half pairs with chunk c of the second
            // half; in the 128-byte-swizzled tile the 16-byte chunk j of row r sits at chunk j ^ (r & 7) of that row.
            // The row's cosines and sines (D / 2 of each) are requested BEFORE the wait for the tile, so their latency
            // overlaps the tile's own load; read-only loads, all in flight at once.
            const bool have_row = q0 + r < Sq;
            float4 cs4[D / 8], sn4[D / 8];
            if (have_row) {
                const size_t pos = static_cast<size_t>(p.rope_pos0 + q0 + r);
                const float4 *ct = reinterpret_cast<const float4 *>(p.rope_cos + pos * (D / 2));
                const float4 *st = reinterpret_cast<const float4 *>(p.rope_sin + pos * (D / 2));
#pragma unroll
                for (int i = 0; i < D / 8; ++i) {
                    cs4[i] = __ldg(ct + i);
                    sn4[i] = __ldg(st + i);
                }
            }
            ok = mbar_wait(q_full, 0, abort_flag, p.guard, status_word(FWD_KERNEL_ID, ROLE_SOFTMAX, 0xFFFF));
            if (ok && have_row) {
                uint8_t *rowp = sQ + r * 128;
#pragma unroll
                for (int ch = 0; ch < D / 16; ++ch) {
                    uint4 *pa = reinterpret_cast<uint4 *>(rowp + ((ch ^ (r & 7)) << 4));
                    uint4 *pb = (D == 128) ? reinterpret_cast<uint4 *>(rowp + QBOX_BYTES + ((ch ^ (r & 7)) << 4))
                                           : reinterpret_cast<uint4 *>(rowp + (((ch + 4) ^ (r & 7)) << 4));
                    const uint4 a = *pa, bq = *pb;
                    const float4 c0 = cs4[2 * ch], c1 = cs4[2 * ch + 1], s0 = sn4[2 * ch], s1 = sn4[2 * ch + 1];
                    const float cs[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
                    const float sn[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
                    const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {bq.x, bq.y, bq.z, bq.w};
                    uint32_t ya[4], yb[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 fa = unpack16<F16>(aw[e]), fb = unpack16<F16>(bw[e]);
                        ya[e] = pack16<F16>(fa.x * cs[2 * e] - fb.x * sn[2 * e], fa.y * cs[2 * e + 1] - fb.y * sn[2 * e + 1]);
                        yb[e] = pack16<F16>(fb.x * cs[2 * e] + fa.x * sn[2 * e], fb.y * cs[2 * e + 1] + fa.y * sn[2 * e + 1]);
                    }
                    *pa = make_uint4(ya[0], ya[1], ya[2], ya[3]);
                    *pb = make_uint4(yb[0], yb[1], yb[2], yb[3]);
                }
            }
            fence_proxy_async_smem();              // the products read the tile through the async proxy
            mbar_arrive(q_rot);
        }
        const int n_loop = (ROPE && !ok) ? 0 : n_t;         // (a wait gave up while the queries were being rotated)
        for (int t = 0; t < n_loop; ++t) {
            const uint32_t tS = tmem_base + lane_addr + (t & 1) * BN;
            ok = mbar_wait(&s_full[t & 1], (t >> 1) & 1, abort_flag, p.guard, status_word(FWD_KERNEL_ID, ROLE_SOFTMAX, t));
            if (!ok) break;
            tc_fence_after_sync();
            uint32_t sr[2][32];
            tmem_ld32(tS, sr[0]);
            tmem_ld32(tS + 32, sr[1]);
            tmem_wait_ld();
            const int c0 = (t0 + t) * BN;
            const bool need_mask = (c0 + BN > Sk) || (CAUSAL && (c0 + BN - 1 > q0 + off));
            if (need_mask) {
                int limit = Sk - c0;                           // columns >= limit are masked
                if (CAUSAL) limit = min(limit, row + off - c0 + 1);
#pragma unroll
                for (int cc = 0; cc < 2; ++cc)
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (cc * 32 + i >= limit) sr[cc][i] = 0xFF800000u;   // -inf
            }
            // row maximum: four independent chains of 3-input max
            float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int cc = 0; cc < 2; ++cc)
#pragma unroll
                for (int i = 0; i < 32; i += 8)
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        mx[u] = fmax3(mx[u], __uint_as_float(sr[cc][i + 2 * u]), __uint_as_float(sr[cc][i + 2 * u + 1]));
            const float m_new = fmax3(m_used, fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
            if (t == 0) {
                m_used = m_new;
            } else {
                // (HPACK: rows past G * Sq hold whatever shared memory held; they must not trigger rescales)
                const bool moved = live && (m_new - m_used) * c > RESCALE_THRESHOLD;
                if (__any_sync(0xFFFFFFFFu, moved)) {
                    // O must hold every product issued so far: wait for P_{t-1} V_{t-1}
                    ok = mbar_wait(pv_done, (t - 1) & 1, abort_flag, p.guard, status_word(FWD_KERNEL_ID, ROLE_SOFTMAX, t));
                    if (!ok) break;
                    tc_fence_after_sync();
                    // (a row that has seen no key yet keeps m = -inf: nothing to rescale)
                    const float alpha = (CAUSAL && m_new == -INFINITY) ? 1.0f : fast_exp2((m_used - m_new) * c);
                    l *= alpha;
                    m_used = m_new;
#pragma unroll
                    for (int cc = 0; cc < D / 32; ++cc) {
                        uint32_t orow[32];
                        tmem_ld32(tmem_O + lane_addr + cc * 32, orow);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) orow[i] = __float_as_uint(__uint_as_float(orow[i]) * alpha);
                        tmem_st32(tmem_O + lane_addr + cc * 32, orow);
                    }
                }
            }
            // P = exp2(s*c - m*c): packed 2-wide FMA, ex2 (MUFU, or the cubic for a share at D = 64), packed sums
            const float2 c2 = make_float2(c, c);
            const float neg_m = (CAUSAL && m_used == -INFINITY) ? 0.0f : -m_used * c;     // empty row: exp2(-inf - 0) = 0
            const float2 nm2 = make_float2(neg_m, neg_m);
            float2 acc[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
            for (int cc = 0; cc < 2; ++cc) {
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const float2 x = __ffma2_rn(make_float2(__uint_as_float(sr[cc][2 * i]), __uint_as_float(sr[cc][2 * i + 1])), c2, nm2);
                    float2 e;
                    if ((i & 7) < POLY_EIGHTHS) {      // this share of the exponentials runs on the FMA pipe
                        e = exp2_poly2(x);
                    } else {
                        e.x = fast_exp2(x.x);
                        e.y = fast_exp2(x.y);
                    }
                    acc[i & 3] = __fadd2_rn(acc[i & 3], e);
                    pk[i] = pack16<F16>(e.x, e.y);
                }
                tmem_st16(tS + cc * 16, pk);
            }
            const float2 s01 = __fadd2_rn(acc[0], acc[1]), s23 = __fadd2_rn(acc[2], acc[3]);
            l += (s01.x + s01.y) + (s23.x + s23.y);
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(&p_ready[t & 1]);
        }
        const bool store = HPACK ? live : row < Sq;
        // row of the [B, Hq, Sq] tensors, or (PACKED, used by SPLIT only) of the [total_q, Hq] token-major ones
        const size_t rid = PACKED ? static_cast<size_t>(q_base + row) * p.Hq + h_out : (static_cast<size_t>(b) * p.Hq + h_out) * p.Sq + row;
        __nv_bfloat16 *orow_g = PACKED ? p.o + (static_cast<size_t>(q_base + row) * p.Hq + h) * p.d : p.o + rid * p.d;
        float *lse_g = PACKED ? p.lse + static_cast<size_t>(h) * p.total_q + q_base + row : p.lse + rid;
        float *opart_g = nullptr;
        if (SPLIT) {
            opart_g = p.o_part + (static_cast<size_t>(split) * p.n_rows + rid) * D;
            lse_g = p.lse_part + static_cast<size_t>(split) * p.n_rows + rid;
        }
        if (n_t == 0) {
            // no key for this tile (a packed sequence without keys, a masked-out chunk): the softmax is empty, O = 0, LSE = -inf
            if (store) {
                if (SPLIT) {
                    for (int i = 0; i < D / 4; ++i) reinterpret_cast<float4 *>(opart_g)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
                } else {
                    for (int i = 0; i < p.d / 8; ++i) reinterpret_cast<uint4 *>(orow_g)[i] = make_uint4(0, 0, 0, 0);
                }
                *lse_g = -INFINITY;
            }
            ok = false;
        }
        if (ok) ok = mbar_wait(o_final, 0, abort_flag, p.guard, status_word(FWD_KERNEL_ID, ROLE_EPILOGUE, 0));
        if (ok) {
            tc_fence_after_sync();
            const float inv_l = (CAUSAL && m_used == -INFINITY) ? 0.0f : 1.0f / l;     // empty row: O = 0 (LSE below comes out as -inf)
#pragma unroll
            for (int cc = 0; cc < D / 32; ++cc) {
                uint32_t orow[32];
                tmem_ld32(tmem_O + lane_addr + cc * 32, orow);
                tmem_wait_ld();
                if (store && SPLIT) {
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        reinterpret_cast<float4 *>(opart_g + cc * 32)[i] =
                            make_float4(__uint_as_float(orow[4 * i + 0]) * inv_l, __uint_as_float(orow[4 * i + 1]) * inv_l,
                                        __uint_as_float(orow[4 * i + 2]) * inv_l, __uint_as_float(orow[4 * i + 3]) * inv_l);
                } else if (!SPLIT) {
                    // every MMA has completed, so the Q tile's shared memory is free: a private patch per warp to transpose
                    // the stores (whole sectors per instruction); the rows of a warp are consecutive rows of O
                    const size_t stride = PACKED ? static_cast<size_t>(p.Hq) * p.d : static_cast<size_t>(p.d);
                    const int rows_valid = min(32, (HPACK ? p.G * Sq : Sq - q0) - warp * 32);
                    store_rows16<F16>(orow_g - static_cast<size_t>(lane) * stride + cc * 32, stride, orow, inv_l, rows_valid,
                                    sQ + warp * STORE_SCRATCH_BYTES, lane, p.d - cc * 32);
                }
            }
            // LSE in natural log: (m * scale * log2e + log2 l) * ln 2
            if (store) *lse_g = (m_used * c + log2f(l)) * 0.6931471805599453f;
        }
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 5) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, fwd_tmem_cols(D));
    }
}

template <int D, bool CAUSAL, bool PACKED, bool SPLIT = false, bool HPACK = false, bool F16 = false, bool ROPE = false>
static int launch_fwd(const CUtensorMap &tq, const CUtensorMap &tk, const CUtensorMap &tv, const FwdParams &prm,
                      int n_blocks, cudaStream_t stream)
{
    using L = FwdSmem<D>;
    static std::atomic<bool> configured[64];     // set-up is idempotent: two threads may both do it, neither may read a torn flag
    int dev = 0;
    cudaGetDevice(&dev);
    if (!configured[dev & 63].load(std::memory_order_acquire)) {
        cudaError_t e = cudaFuncSetAttribute(attn_fwd_kernel<D, CAUSAL, PACKED, SPLIT, HPACK, F16, ROPE>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::BYTES);
        if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(fwd)");
        configured[dev & 63].store(true, std::memory_order_release);
    }
    attn_fwd_kernel<D, CAUSAL, PACKED, SPLIT, HPACK, F16, ROPE><<<n_blocks, FWD_THREADS, L::BYTES, stream>>>(tq, tk, tv, prm);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "attn_fwd_kernel launch");
    return VT_ATTN_OK;
}

}  // namespace vt
