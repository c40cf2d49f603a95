// Forward kernel for long sequences: one block per SM works on TWO adjacent 128-row query tiles of one head at a time.
//
// Both tiles walk the same keys, 128 at a time, so every K / V tile is loaded once for 256 query rows, and S = Q K^T runs
// with N = 128 (the full MMA rate: an smem x smem MMA with N = 64 runs at two thirds of it).  Tensor memory holds S_A, S_B
// (fp32, 128 columns each; the bf16 P is written over the first 64 columns of its S) and the accumulators O_A, O_B.
// Each tile has its own softmax warpgroup (one thread per query row, 128 scores per step).  The MMA warp issues
//     P_A V (as soon as warpgroup A has written P_A), S_A = Q_A K_next^T, P_B V, S_B = Q_B K_next^T, ...
// so while warpgroup A turns its scores into probabilities the tensor core works for tile B and the other way round:
// the two tiles ping-pong between the exponential unit and the tensor core.
//   warps 0..3  softmax + epilogue of tile A      warps 4..7  softmax + epilogue of tile B
//   warp 8      TMA producer (Q_A, Q_B, K)        warp 9      MMA issuer, TMEM owner
//   warp 10     TMA producer (V)                  warp 11     idle
// Handing P over in two halves of 64 keys lets the first half of P V run under the second half of the exponentials
// (measured +3 %).  Used for D = 128 and long sequences; shorter ones, D = 64, packed and split-KV launches use the
// one-tile kernel of fwd_kernel.cuh, whose smaller blocks start and drain faster.
// Included by fwd.cu (uses FwdParams and the constants of fwd_kernel.cuh).
#pragma once
#include "fwd_kernel.cuh"

namespace vt {

constexpr int PAIR_THREADS = 384;
constexpr int PAIR_SOFTMAX_REGS = 208;      // 256 x 208 + 128 x 80 <= 64 K registers
constexpr int PAIR_OTHER_REGS = 80;
constexpr int PAIR_TMEM_COLS = 512;         // S_A [0,128), S_B [128,256), O_A [256,256+D), O_B [384,384+D)
constexpr uint32_t PAIR_KERNEL_ID = 4;
// Share (in eighths) of the exponentials evaluated with the FMA-pipe cubic instead of the MUFU: both warpgroups of a
// tile pair use the same four exponential units.  Measured on S = 8192: 0 -> 1333, 2 -> 1355, 4 -> 1298 TFLOP/s.
constexpr int PAIR_POLY_EIGHTHS = 2;

template <int D>
struct PairSmem {
    static constexpr int TILE_BYTES = TILE * D * 2;           // a 128-row tile of Q, K or V
    static constexpr int K_SLOTS = 2;
    static constexpr int V_SLOTS = 2;
    static constexpr int OFF_Q = 0;                           // [2]: tile A, tile B
    static constexpr int OFF_K = OFF_Q + 2 * TILE_BYTES;
    static constexpr int OFF_V = OFF_K + K_SLOTS * TILE_BYTES;
    static constexpr int OFF_BAR = OFF_V + V_SLOTS * TILE_BYTES;
    static constexpr int BYTES = OFF_BAR + 256 + 1024;
};

// p.n_qt here counts PAIRS of query tiles per head.
template <int D, bool CAUSAL, bool PACKED, bool F16 = false>
__global__ void __launch_bounds__(PAIR_THREADS, 1)
attn_fwd_pair_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                     const __grid_constant__ CUtensorMap tm_v, const FwdParams p)
{
    using L = PairSmem<D>;
    constexpr int KS = L::K_SLOTS, VS = L::V_SLOTS;
    constexpr int NBOX = D / BOX_COLS;
    constexpr int BOX_BYTES = TILE * BOX_COLS * 2;     // 16 KB: a 64-column box of a 128-row tile

    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *sQ = smem + L::OFF_Q;
    uint8_t *sK = smem + L::OFF_K;
    uint8_t *sV = smem + L::OFF_V;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L::OFF_BAR);
    uint64_t *q_full = bars + 0;
    uint64_t *o_final = bars + 1;            // [2 tiles]
    uint64_t *pv_done = bars + 3;            // [2 tiles]: O of the tile holds every product issued so far
    uint64_t *s_full = bars + 5;             // [2 tiles], one phase per step
    uint64_t *p_ready = bars + 7;            // [2 tiles][2 halves of the keys], 128 arrivals each, one phase per step
    uint64_t *k_full = bars + 11;            // [KS]
    uint64_t *k_empty = bars + 11 + KS;      // [KS]
    uint64_t *v_full = bars + 11 + 2 * KS;   // [VS]
    uint64_t *v_empty = bars + 11 + 2 * KS + VS;   // [VS]
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 11 + 2 * KS + 2 * VS);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    // work item: heads are the slow index (co-resident blocks share K / V in L2); causal heads hand out their long pairs first
    int bh = blockIdx.x / p.n_qt;
    int pr = blockIdx.x % p.n_qt;
    if (CAUSAL) {
        bh = causal_work_item(blockIdx.x, p.n_qt, static_cast<int>(gridDim.x) / p.n_qt, p.head_group, pr);
        pr = p.n_qt - 1 - pr;
    }
    const int b = bh / p.Hq;
    const int h = bh % p.Hq;
    const int hkv = h / p.G;
    const int bh_kv = b * (p.Hq / p.G) + hkv;
    const int q0 = pr * 2 * TILE;                         // first query row of tile A; tile B starts at q0 + 128
    int Sq = p.Sq, Sk = p.Sk, q_base = 0, k_base = 0;     // this block's sequence: lengths and first token rows
    if (PACKED) {
        q_base = p.cu_q[b];
        Sq = p.cu_q[b + 1] - q_base;
        k_base = p.cu_k[b];
        Sk = p.cu_k[b + 1] - k_base;
        if (q0 >= Sq) return;                             // this sequence has no such pair (whole block leaves)
    }
    // causal: query i sees the keys j <= i + off (see fwd_kernel.cuh); n_kv[t]: 128-key steps of tile t (0: nothing to do)
    const int off = (CAUSAL && p.bottom_right) ? Sk - Sq : 0;
    const int n_all = (Sk + TILE - 1) / TILE;
    int n_kv[2];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        const int qs = q0 + t * TILE;
        int n = (qs < Sq) ? n_all : 0;                    // tile B may lie past the end of the sequence
        if (CAUSAL) n = (qs + TILE - 1 + off < 0) ? 0 : min(n, (qs + TILE - 1 + off) / TILE + 1);
        n_kv[t] = n;
    }
    const int n_steps = max(n_kv[0], n_kv[1]);
    auto q_c1 = [&](int t) { return PACKED ? h : q0 + t * TILE; };
    auto q_c2 = [&](int t) { return PACKED ? q_base + q0 + t * TILE : bh; };
    auto kv_c1 = [&](int r) { return PACKED ? hkv : r; };
    auto kv_c2 = [&](int r) { return PACKED ? k_base + r : bh_kv; };

    constexpr int PRODUCER_THREAD = 8 * 32;
    if (threadIdx.x == PRODUCER_THREAD) {
        mbar_init(q_full, 1);
        for (int t = 0; t < 2; ++t) {
            mbar_init(&o_final[t], 1);
            mbar_init(&pv_done[t], 1);
            mbar_init(&s_full[t], 1);
            mbar_init(&p_ready[2 * t], 128);
            mbar_init(&p_ready[2 * t + 1], 128);
        }
        for (int s = 0; s < KS; ++s) {
            mbar_init(&k_full[s], 1);
            mbar_init(&k_empty[s], 1);
        }
        for (int s = 0; s < VS; ++s) {
            mbar_init(&v_full[s], 1);
            mbar_init(&v_empty[s], 1);
        }
        *abort_flag = 0u;
        fence_mbar_init();
        // the producer initialised the barriers itself: its first loads go out before the block-wide sync
        prefetch_tensormap(&tm_q);
        prefetch_tensormap(&tm_k);
        mbar_arrive_expect_tx(q_full, 2 * L::TILE_BYTES);
        for (int t = 0; t < 2; ++t)                        // (a tile B past the end of the tensor reads as zeros)
            for (int kb = 0; kb < NBOX; ++kb)
                tma_load_3d(sQ + t * L::TILE_BYTES + kb * BOX_BYTES, &tm_q, q_full, kb * BOX_COLS, q_c1(t), q_c2(t));
        if (n_steps > 0) {
            mbar_arrive_expect_tx(&k_full[0], L::TILE_BYTES);
            for (int kb = 0; kb < NBOX; ++kb) tma_load_3d(sK + kb * BOX_BYTES, &tm_k, &k_full[0], kb * BOX_COLS, kv_c1(0), kv_c2(0));
        }
    }
    if (warp == 9) {
        tmem_alloc(tmem_slot, PAIR_TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp >= 8) {
        setmaxnreg_dec<PAIR_OTHER_REGS>();
        if (warp == 8) {
            // ------------------------------------------------------------------ TMA producer: K (Q and the first K tile are out already)
            if (lane == 0) {
                for (int j = 1; j < n_steps; ++j) {
                    const int sl = j % KS;
                    if (!mbar_wait(&k_empty[sl], ((j / KS) & 1) ^ 1, abort_flag, p.guard, status_word(PAIR_KERNEL_ID, ROLE_LOAD, j))) break;
                    mbar_arrive_expect_tx(&k_full[sl], L::TILE_BYTES);
                    for (int kb = 0; kb < NBOX; ++kb)
                        tma_load_3d(sK + sl * L::TILE_BYTES + kb * BOX_BYTES, &tm_k, &k_full[sl], kb * BOX_COLS, kv_c1(j * TILE), kv_c2(j * TILE));
                }
            }
        } else if (warp == 10) {
            // ------------------------------------------------------------------ TMA producer: V
            if (lane == 0) {
                prefetch_tensormap(&tm_v);
                for (int j = 0; j < n_steps; ++j) {
                    const int sl = j % VS;
                    if (!mbar_wait(&v_empty[sl], ((j / VS) & 1) ^ 1, abort_flag, p.guard, status_word(PAIR_KERNEL_ID, ROLE_LOAD, j))) break;
                    mbar_arrive_expect_tx(&v_full[sl], L::TILE_BYTES);
                    for (int kb = 0; kb < NBOX; ++kb)
                        tma_load_3d(sV + sl * L::TILE_BYTES + kb * BOX_BYTES, &tm_v, &v_full[sl], kb * BOX_COLS, kv_c1(j * TILE), kv_c2(j * TILE));
                }
            }
        } else if (warp == 9) {
            // ------------------------------------------------------------------ MMA issuer
            constexpr uint32_t IDESC_QK = make_idesc(128, 128, fmt16<F16>(), fmt16<F16>(), 0, 0);
            constexpr uint32_t IDESC_PV = make_idesc(128, D, fmt16<F16>(), fmt16<F16>(), 0, 1);
            const uint32_t tmem_u = __shfl_sync(0xFFFFFFFFu, tmem_base, 0);    // provably warp-uniform copy
            bool ok = mbar_wait(q_full, 0, abort_flag, p.guard, status_word(PAIR_KERNEL_ID, ROLE_MMA, 0xFFFF));
            // S_t(j) = Q_t K_j^T.  `last` : no other product reads K_j after this one, so its completion frees the slot.
            auto issue_qk = [&](int t, int j, bool last) {
                const int sl = j % KS;
                if (elect_one()) {
                    const uint64_t dQ0 = smem_desc_sw128(smem_u32(sQ + t * L::TILE_BYTES), 16, 1024);
                    const uint64_t dK0 = smem_desc_sw128(smem_u32(sK + sl * L::TILE_BYTES), 16, 1024);
                    const uint32_t tS = tmem_u + t * TILE;
#pragma unroll
                    for (int k = 0; k < D / 16; ++k) {
                        const uint32_t o = (k / 4) * BOX_BYTES + (k % 4) * 32;
                        umma_ss(tS, desc_advance(dQ0, o), desc_advance(dK0, o), IDESC_QK, k > 0 ? 1u : 0u);
                    }
                    if (last) umma_commit(&k_empty[sl]);
                    umma_commit(&s_full[t]);
                }
                __syncwarp();
            };
            // the tile that takes part in step j last (frees the K / V slots): B when it is active, else A
            auto last_tile = [&](int j) { return (j < n_kv[1]) ? 1 : 0; };
            if (ok && n_steps > 0) {
                ok = mbar_wait(&k_full[0], 0, abort_flag, p.guard, status_word(PAIR_KERNEL_ID, ROLE_MMA, 0));
                if (ok) {
                    tc_fence_after_sync();
                    for (int t = 0; t < 2; ++t)
                        if (n_kv[t] > 0) issue_qk(t, 0, t == last_tile(0));
                }
            }
            for (int j = 0; j < n_steps && ok; ++j) {
                const int vsl = j % VS;
                ok = mbar_wait(&v_full[vsl], (j / VS) & 1, abort_flag, p.guard, status_word(PAIR_KERNEL_ID, ROLE_MMA, j));
                if (!ok) break;
                bool k_next_ready = false;
                for (int t = 0; t < 2 && ok; ++t) {
                    if (j >= n_kv[t]) continue;
                    const uint64_t dV0 = smem_desc_sw128(smem_u32(sV + vsl * L::TILE_BYTES), BOX_BYTES, 1024);
                    const uint32_t tP = tmem_u + t * TILE;
                    // O_t += P_t V_j, in two halves of 64 keys: the first runs while the softmax still works on the second
                    for (int hf = 0; hf < 2; ++hf) {
                        ok = mbar_wait(&p_ready[2 * t + hf], j & 1, abort_flag, p.guard, status_word(PAIR_KERNEL_ID, ROLE_MMA, j));
                        if (!ok) break;
                        tc_fence_after_sync();
                        if (elect_one()) {
#pragma unroll
                            for (int k = 0; k < 4; ++k)
                                umma_ts(tmem_u + 256 + t * 128, tP + (hf * 4 + k) * 8, desc_advance(dV0, (hf * 4 + k) * 2048), IDESC_PV,
                                        (j > 0 || hf > 0 || k > 0) ? 1u : 0u);
                            if (hf == 1) {
                                umma_commit(&pv_done[t]);
                                if (t == last_tile(j)) umma_commit(&v_empty[vsl]);
                                if (j == n_kv[t] - 1) umma_commit(&o_final[t]);
                            }
                        }
                        __syncwarp();
                    }
                    if (!ok) break;
                    if (j + 1 < n_kv[t]) {                 // next scores of this tile: they overwrite P_t(j), ordered behind the product just issued
                        if (!k_next_ready) {
                            ok = mbar_wait(&k_full[(j + 1) % KS], ((j + 1) / KS) & 1, abort_flag, p.guard, status_word(PAIR_KERNEL_ID, ROLE_MMA, j + 1));
                            if (!ok) break;
                            tc_fence_after_sync();
                            k_next_ready = true;
                        }
                        issue_qk(t, j + 1, t == last_tile(j + 1));
                    }
                }
            }
        }
    } else {
        // ---------------------------------------------------------------------- softmax + epilogue (warpgroup t owns tile t)
        setmaxnreg_inc<PAIR_SOFTMAX_REGS>();
        const int t = warp >> 2;
        const int quad = warp & 3;
        const int r = quad * 32 + lane;            // row inside the tile == TMEM lane
        const int qs = q0 + t * TILE;              // first query row of this tile
        const int row = qs + r;
        const int n_mine = n_kv[t];
        const uint32_t lane_addr = static_cast<uint32_t>(quad * 32) << 16;
        const uint32_t tS = tmem_base + lane_addr + t * TILE;
        const uint32_t tO = tmem_base + lane_addr + 256 + t * 128;
        const float c = p.scale_log2e;
        const float2 c2 = make_float2(c, c);
        float m_used = -INFINITY;                  // maximum (raw scores) the accumulators are scaled by
        float l = 0.0f;
        bool ok = true;
        for (int j = 0; j < n_mine; ++j) {
            ok = mbar_wait(&s_full[t], j & 1, abort_flag, p.guard, status_word(PAIR_KERNEL_ID, ROLE_SOFTMAX, j));
            if (!ok) break;
            tc_fence_after_sync();
            uint32_t sr[4][32];
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) tmem_ld32(tS + cc * 32, sr[cc]);
            tmem_wait_ld();
            const int c0 = j * TILE;
            const bool need_mask = (c0 + TILE > Sk) || (CAUSAL && (c0 + TILE - 1 > qs + off));
            if (need_mask) {
                int limit = Sk - c0;                               // columns >= limit are masked
                if (CAUSAL) limit = min(limit, row + off - c0 + 1);
#pragma unroll
                for (int cc = 0; cc < 4; ++cc)
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (cc * 32 + i >= limit) sr[cc][i] = 0xFF800000u;   // -inf
            }
            // row maximum: eight independent chains of 3-input max
            float mx[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) mx[u] = -INFINITY;
#pragma unroll
            for (int cc = 0; cc < 4; ++cc)
#pragma unroll
                for (int i = 0; i < 32; i += 16)
#pragma unroll
                    for (int u = 0; u < 8; ++u)
                        mx[u] = fmax3(mx[u], __uint_as_float(sr[cc][i + 2 * u]), __uint_as_float(sr[cc][i + 2 * u + 1]));
            const float m_new = fmax3(m_used, fmax3(mx[0], mx[1], mx[2]), fmax3(fmax3(mx[3], mx[4], mx[5]), mx[6], mx[7]));
            if (j == 0) {
                m_used = m_new;
            } else {
                const bool moved = (m_new - m_used) * c > RESCALE_THRESHOLD;
                if (__any_sync(0xFFFFFFFFu, moved)) {
                    // O must hold every product issued so far: wait for P(j-1) V(j-1) of this tile
                    ok = mbar_wait(&pv_done[t], (j - 1) & 1, abort_flag, p.guard, status_word(PAIR_KERNEL_ID, ROLE_SOFTMAX, j));
                    if (!ok) break;
                    tc_fence_after_sync();
                    // (a row that has seen no key yet keeps m = -inf: nothing to rescale)
                    const float alpha = (CAUSAL && m_new == -INFINITY) ? 1.0f : fast_exp2((m_used - m_new) * c);
                    l *= alpha;
                    m_used = m_new;
#pragma unroll
                    for (int cc = 0; cc < D / 32; ++cc) {
                        uint32_t orow[32];
                        tmem_ld32(tO + cc * 32, orow);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) orow[i] = __float_as_uint(__uint_as_float(orow[i]) * alpha);
                        tmem_st32(tO + cc * 32, orow);
                    }
                }
            }
            const float neg_m = (CAUSAL && m_used == -INFINITY) ? 0.0f : -m_used * c;     // empty row: exp2(-inf - 0) = 0
            const float2 nm2 = make_float2(neg_m, neg_m);
            float2 acc[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const float2 x = __ffma2_rn(make_float2(__uint_as_float(sr[cc][2 * i]), __uint_as_float(sr[cc][2 * i + 1])), c2, nm2);
                    float2 e;
                    if ((i & 7) < PAIR_POLY_EIGHTHS) {
                        e = exp2_poly2(x);
                    } else {
                        e.x = fast_exp2(x.x);
                        e.y = fast_exp2(x.y);
                    }
                    acc[i & 3] = __fadd2_rn(acc[i & 3], e);
                    pk[i] = pack16<F16>(e.x, e.y);
                }
                tmem_st16(tS + cc * 16, pk);       // over this thread's own, already read S columns
                if (cc == 1 || cc == 3) {          // a half of the keys is done: the MMA warp may issue its part of P V
                    tmem_wait_st();
                    tc_fence_before_sync();
                    mbar_arrive(&p_ready[2 * t + (cc >> 1)]);
                }
            }
            const float2 s01 = __fadd2_rn(acc[0], acc[1]), s23 = __fadd2_rn(acc[2], acc[3]);
            l += (s01.x + s01.y) + (s23.x + s23.y);
        }
        const bool store = row < Sq;
        __nv_bfloat16 *orow_g = PACKED ? p.o + (static_cast<size_t>(q_base + row) * p.Hq + h) * D
                                       : p.o + (static_cast<size_t>(bh) * p.Sq + row) * D;
        float *lse_g = PACKED ? p.lse + static_cast<size_t>(h) * p.total_q + q_base + row
                              : p.lse + static_cast<size_t>(bh) * p.Sq + row;
        if (n_mine == 0) {
            // no key is visible to this tile (or the tile lies past the end): O = 0 and LSE = -inf for the rows that exist
            if (store) {
                for (int i = 0; i < D / 8; ++i) reinterpret_cast<uint4 *>(orow_g)[i] = make_uint4(0, 0, 0, 0);
                *lse_g = -INFINITY;
            }
            ok = false;
        }
        if (ok) ok = mbar_wait(&o_final[t], 0, abort_flag, p.guard, status_word(PAIR_KERNEL_ID, ROLE_EPILOGUE, t));
        if (ok) {
            tc_fence_after_sync();
            const float inv_l = (CAUSAL && m_used == -INFINITY) ? 0.0f : 1.0f / l;     // empty row: O = 0 (LSE comes out as -inf)
            // every MMA of this tile has completed, so its Q tile's shared memory is free: a private patch per warp to
            // transpose the stores
            const size_t stride = PACKED ? static_cast<size_t>(p.Hq) * D : static_cast<size_t>(D);
            const int rows_valid = min(32, Sq - qs - quad * 32);
#pragma unroll
            for (int cc = 0; cc < D / 32; ++cc) {
                uint32_t orow[32];
                tmem_ld32(tO + cc * 32, orow);
                tmem_wait_ld();
                store_rows16<F16>(orow_g - static_cast<size_t>(lane) * stride + cc * 32, stride, orow, inv_l, rows_valid,
                                sQ + t * L::TILE_BYTES + quad * STORE_SCRATCH_BYTES, lane);
            }
            // LSE in natural log: (m * scale * log2e + log2 l) * ln 2
            if (store) *lse_g = (m_used * c + log2f(l)) * 0.6931471805599453f;
        }
    }

    // -------------------------------------------------------------------------- teardown
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 9) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, PAIR_TMEM_COLS);
    }
}

template <int D, bool CAUSAL, bool PACKED, bool F16 = false>
static int launch_fwd_pair(const CUtensorMap &tq, const CUtensorMap &tk, const CUtensorMap &tv, const FwdParams &prm,
                           int n_blocks, cudaStream_t stream)
{
    using L = PairSmem<D>;
    static std::atomic<bool> configured[64];     // set-up is idempotent: two threads may both do it, neither may read a torn flag
    int dev = 0;
    cudaGetDevice(&dev);
    if (!configured[dev & 63].load(std::memory_order_acquire)) {
        cudaError_t e = cudaFuncSetAttribute(attn_fwd_pair_kernel<D, CAUSAL, PACKED, F16>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::BYTES);
        if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(fwd pair)");
        configured[dev & 63].store(true, std::memory_order_release);
    }
    attn_fwd_pair_kernel<D, CAUSAL, PACKED, F16><<<n_blocks, PAIR_THREADS, L::BYTES, stream>>>(tq, tk, tv, prm);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "attn_fwd_pair_kernel launch");
    return VT_ATTN_OK;
}

}  // namespace vt
