// Backward fused attention for sm_100a: three kernels, no atomics, every sum in a fixed order.
//
//   1. bwd_delta_kernel : Delta[b,h,i] = sum_d dO[b,h,i,d] * O[b,h,i,d]          (HBM-bound)
//   2. bwd_dkdv_kernel  : one block per (batch, KV head, 128-key tile); K and V stay in shared memory while
//                         the block walks the query heads of the group, 128 queries at a time:
//                         S^T = K Q^T, dP^T = V dO^T (tcgen05, smem x smem, N = 128: full MMA rate),
//                         P^T = exp2(S^T*c - LSE), dS^T = P^T o (dP^T - Delta) written to TMEM as bf16,
//                         then dV += P^T dO and dK += dS^T Q (tcgen05, TMEM x smem).
//   3. bwd_dq_kernel    : one block per (batch, query head, 128-query tile); walks the keys 128 at a time:
//                         S = Q K^T, dP = dO V^T, dS = P o (dP - Delta), dQ += dS K.
// What makes the tensor core wait-free in both: P depends on S alone, so S is issued ahead of dP and the
// exponentials run while the tensor core computes dP and the accumulating products of the previous step; the
// 128x128 tile is split by columns between two compute warpgroups (backward needs no row maximum, so the halves
// never have to talk to each other), each thread keeping its 64 probabilities in registers for dS.
// Block = 384 threads: warp 0 and warp 2 TMA producers, warp 1 MMA issuer, warps 4..7 and 8..11 compute.
// Recomputing S and dP in both kernels costs 7 tile products instead of 5 but every dQ, dK, dV tile has exactly
// one owner block: no cross-block reduction, bit-identical results every run.
#include <stdlib.h>

#include <mutex>

#include "bwd_common.cuh"

namespace vt {

// ----------------------------------------------------------------------------------------------
// 2. dK, dV  (key tile stationary)
// ----------------------------------------------------------------------------------------------
template <int D>
struct DkdvSmem {
    static constexpr int TILE_BYTES = TILE * D * 2;                  // a 128-row tile of K, V, Q or dO
    static constexpr int OFF_K = 0;
    static constexpr int OFF_V = OFF_K + TILE_BYTES;
    static constexpr int OFF_Q = OFF_V + TILE_BYTES;                 // [2]
    static constexpr int OFF_DO = OFF_Q + 2 * TILE_BYTES;            // [2]
    static constexpr int ROW_SLOTS = 4;                              // ring of per-iteration row vectors: -lse2[128], -delta[128]
    static constexpr int OFF_ROWS = OFF_DO + 2 * TILE_BYTES;
    static constexpr int OFF_BAR = OFF_ROWS + ROW_SLOTS * 2 * TILE * 4;
    static constexpr int BYTES = OFF_BAR + 256 + 1024;
    // TMEM columns: S^T [0,128), dP^T [128,256), dV [256,256+D), dK [256+D,256+2D).  P^T (bf16) is written over
    // S^T and dS^T over dP^T, each warpgroup inside its own WG_COLS columns (the first half of them).
    static constexpr int TMEM_COLS = 512;
};

template <int D, bool CAUSAL, bool PACKED, bool F16 = false>
__global__ void __launch_bounds__(BWD_THREADS, 1)
bwd_dkdv_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do, const BwdParams p)
{
    using L = DkdvSmem<D>;
    constexpr int NBOX = D / BOX_COLS;
    constexpr int BOX_BYTES = TILE * BOX_COLS * 2;           // 16 KB: a 64-column box of a 128-row tile

    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *sK = smem + L::OFF_K;
    uint8_t *sV = smem + L::OFF_V;
    uint8_t *sQ = smem + L::OFF_Q;
    uint8_t *sdO = smem + L::OFF_DO;
    constexpr int RS = L::ROW_SLOTS;
    float *s_rows = reinterpret_cast<float *>(smem + L::OFF_ROWS);     // [slot][-lse2 128 | -delta 128]
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L::OFF_BAR);
    uint64_t *kv_full = bars + 0;
    uint64_t *final_bar = bars + 1;
    uint64_t *s_full = bars + 2;              // S^T of the iteration is complete
    uint64_t *dp_full = bars + 3;             // dP^T of the iteration is complete
    uint64_t *p_ready = bars + 4;             // 256 arrivals: P^T written
    uint64_t *ds_ready = bars + 5;            // 256 arrivals: dS^T written
    uint64_t *q_full = bars + 6;              // [2]
    uint64_t *q_empty = bars + 8;             // [2]
    uint64_t *do_full = bars + 10;            // [2]
    uint64_t *do_empty = bars + 12;           // [2]
    uint64_t *rows_full = bars + 14;          // [RS] 32 arrivals: the row vectors of an iteration are in shared memory
    uint64_t *rows_empty = bars + 14 + RS;    // [RS] one arrival per compute warp
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 14 + 2 * RS);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    // blocks of one KV head are adjacent; under a causal mask the early key tiles are the long ones
    const int bh_kv = blockIdx.x / p.n_tiles;
    const int kt = blockIdx.x % p.n_tiles;
    const int b = bh_kv / p.Hkv;
    const int hkv = bh_kv % p.Hkv;
    const int k0 = kt * TILE;
    int Sq = p.Sq, Sk = p.Sk, q_base = 0, k_base = 0;                    // this block's sequence: lengths and first token rows
    if (PACKED) {
        q_base = p.cu_q[b];
        Sq = p.cu_q[b + 1] - q_base;
        k_base = p.cu_k[b];
        Sk = p.cu_k[b + 1] - k_base;
        if (k0 >= Sk) return;                                            // this sequence has no such key tile (whole block leaves)
    }
    const int n_qt = (Sq + TILE - 1) / TILE;                             // 128-query tiles per head
    const int off = (CAUSAL && p.bottom_right) ? Sk - Sq : 0;            // causal: query i sees the keys j <= i + off
    const int qt_start = CAUSAL ? min(max(k0 - off, 0) / TILE, n_qt) : 0;   // first query tile that can see this key tile
    const int n_qi = n_qt - qt_start;
    const int n_it = n_qi * p.G;                                         // iterations: heads of the group x query tiles
    // TMA coordinates of the 128-row tile of head hq starting at query q0
    auto q_c1 = [&](int hq, int q0) { return PACKED ? hq : q0; };
    auto q_c2 = [&](int hq, int q0) { return PACKED ? q_base + q0 : b * p.Hq + hq; };

    if (threadIdx.x == 0) {
        mbar_init(kv_full, 1);
        mbar_init(final_bar, 1);
        mbar_init(s_full, 1);
        mbar_init(dp_full, 1);
        mbar_init(p_ready, 128 * BWD_WGS);
        mbar_init(ds_ready, 128 * BWD_WGS);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&q_full[s], 1);
            mbar_init(&q_empty[s], 1);
            mbar_init(&do_full[s], 1);
            mbar_init(&do_empty[s], 1);
        }
        for (int s = 0; s < RS; ++s) {
            mbar_init(&rows_full[s], 32);
            mbar_init(&rows_empty[s], 4 * BWD_WGS);
        }
        *abort_flag = 0u;
        fence_mbar_init();
        // this thread is also the K / V / Q producer: its first loads need not wait for the block-wide sync
        prefetch_tensormap(&tm_q);
        prefetch_tensormap(&tm_k);
        prefetch_tensormap(&tm_v);
        mbar_arrive_expect_tx(kv_full, 2 * L::TILE_BYTES);
        for (int kb = 0; kb < NBOX; ++kb) {
            tma_load_3d(sK + kb * BOX_BYTES, &tm_k, kv_full, kb * BOX_COLS, PACKED ? hkv : k0, PACKED ? k_base + k0 : bh_kv);
            tma_load_3d(sV + kb * BOX_BYTES, &tm_v, kv_full, kb * BOX_COLS, PACKED ? hkv : k0, PACKED ? k_base + k0 : bh_kv);
        }
        if (n_it > 0) {
            mbar_arrive_expect_tx(&q_full[0], L::TILE_BYTES);
            for (int kb = 0; kb < NBOX; ++kb)
                tma_load_3d(sQ + kb * BOX_BYTES, &tm_q, &q_full[0], kb * BOX_COLS, q_c1(hkv * p.G, qt_start * TILE), q_c2(hkv * p.G, qt_start * TILE));
        }
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, L::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_dV = tmem_base + 256;
    const uint32_t tmem_dK = tmem_base + 256 + D;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer: the Q tiles (K, V and the first one
        // went out before the block-wide sync)
        if (lane == 0) {
            for (int it = 1; it < n_it; ++it) {
                const int sl = it & 1;
                const int hq = hkv * p.G + it / n_qi;
                const int q0 = (qt_start + it % n_qi) * TILE;
                if (!mbar_wait(&q_empty[sl], ((it >> 1) & 1) ^ 1, abort_flag, p.guard, status_word(DKDV_KERNEL_ID, ROLE_LOAD, it))) break;
                mbar_arrive_expect_tx(&q_full[sl], L::TILE_BYTES);
                for (int kb = 0; kb < NBOX; ++kb)
                    tma_load_3d(sQ + sl * L::TILE_BYTES + kb * BOX_BYTES, &tm_q, &q_full[sl], kb * BOX_COLS, q_c1(hq, q0), q_c2(hq, q0));
            }
        }
    } else if (warp == 2) {
        // ------------------------------------------------------------------ TMA producer: the dO tiles
        if (lane == 0) {
            prefetch_tensormap(&tm_do);
            for (int it = 0; it < n_it; ++it) {
                const int sl = it & 1;
                const int hq = hkv * p.G + it / n_qi;
                const int q0 = (qt_start + it % n_qi) * TILE;
                if (!mbar_wait(&do_empty[sl], ((it >> 1) & 1) ^ 1, abort_flag, p.guard, status_word(DKDV_KERNEL_ID, ROLE_LOAD, it))) break;
                mbar_arrive_expect_tx(&do_full[sl], L::TILE_BYTES);
                for (int kb = 0; kb < NBOX; ++kb)
                    tma_load_3d(sdO + sl * L::TILE_BYTES + kb * BOX_BYTES, &tm_do, &do_full[sl], kb * BOX_COLS, q_c1(hq, q0), q_c2(hq, q0));
            }
        }
    } else if (warp == 3) {
        // ------------------------------------------------------------------ row-vector producer: -LSE (log2 units), -Delta
        // The compute warps read these per query column; fetching them here, a few iterations ahead, keeps the global-load
        // latency off their critical path.  Queries past the end get -inf (P = exp2(-inf) = 0) and Delta 0.
        for (int it = 0; it < n_it; ++it) {
            const int sl = it % RS;
            if (!mbar_wait(&rows_empty[sl], ((it / RS) & 1) ^ 1, abort_flag, p.guard, status_word(DKDV_KERNEL_ID, ROLE_LOAD, it))) break;
            const int hq = hkv * p.G + it / n_qi;
            const int q0 = (qt_start + it % n_qi) * TILE;
            const size_t head = PACKED ? static_cast<size_t>(hq) * p.total_q + q_base : (static_cast<size_t>(b) * p.Hq + hq) * p.Sq;
            float nl[4], nd[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int q = q0 + e * 32 + lane;
                nl[e] = -INFINITY;
                nd[e] = 0.0f;
                if (q < Sq) {
                    nl[e] = -p.lse[head + q] * LOG2E;
                    nd[e] = -p.delta[head + q];
                }
            }
            float *dst = s_rows + sl * (2 * TILE);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                dst[e * 32 + lane] = nl[e];
                dst[TILE + e * 32 + lane] = nd[e];
            }
            mbar_arrive(&rows_full[sl]);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        // Order per iteration: dV(i), S(i+1), dK(i), dP(i+1).  S(i+1) runs while the compute warps still work on dS(i),
        // and its exponentials are taken while dK(i) and dP(i+1) run, so the tensor core does not wait for them.
        constexpr uint32_t IDESC_S = make_idesc(128, 128, fmt16<F16>(), fmt16<F16>(), 0, 0);
        constexpr uint32_t IDESC_G = make_idesc(128, D, fmt16<F16>(), fmt16<F16>(), 0, 1);   // B operand MN-major
        const uint32_t tmem_u = __shfl_sync(0xFFFFFFFFu, tmem_base, 0);    // provably warp-uniform copy
        const uint64_t dK0 = smem_desc_sw128(smem_u32(sK), 16, 1024), dV0 = smem_desc_sw128(smem_u32(sV), 16, 1024);
        bool ok = mbar_wait(kv_full, 0, abort_flag, p.guard, status_word(DKDV_KERNEL_ID, ROLE_MMA, 0xFFFF));
        auto issue_s = [&](int it) -> bool {       // S^T = K Q^T
            const int sl = it & 1;
            if (!mbar_wait(&q_full[sl], (it >> 1) & 1, abort_flag, p.guard, status_word(DKDV_KERNEL_ID, ROLE_MMA, it))) return false;
            tc_fence_after_sync();
            if (elect_one()) {
                const uint64_t dQs = smem_desc_sw128(smem_u32(sQ + sl * L::TILE_BYTES), 16, 1024);
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    const uint32_t off = (k / 4) * BOX_BYTES + (k % 4) * 32;
                    umma_ss(tmem_u, desc_advance(dK0, off), desc_advance(dQs, off), IDESC_S, k > 0 ? 1u : 0u);
                }
                umma_commit(s_full);
            }
            __syncwarp();
            return true;
        };
        auto issue_dp = [&](int it) -> bool {      // dP^T = V dO^T
            const int sl = it & 1;
            if (!mbar_wait(&do_full[sl], (it >> 1) & 1, abort_flag, p.guard, status_word(DKDV_KERNEL_ID, ROLE_MMA, it))) return false;
            tc_fence_after_sync();
            if (elect_one()) {
                const uint64_t dDOs = smem_desc_sw128(smem_u32(sdO + sl * L::TILE_BYTES), 16, 1024);
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    const uint32_t off = (k / 4) * BOX_BYTES + (k % 4) * 32;
                    umma_ss(tmem_u + 128, desc_advance(dV0, off), desc_advance(dDOs, off), IDESC_S, k > 0 ? 1u : 0u);
                }
                umma_commit(dp_full);
            }
            __syncwarp();
            return true;
        };
        if (ok && n_it > 0) ok = issue_s(0);
        if (ok && n_it > 0) ok = issue_dp(0);
        for (int it = 0; it < n_it && ok; ++it) {
            const int sl = it & 1;
            ok = mbar_wait(p_ready, it & 1, abort_flag, p.guard, status_word(DKDV_KERNEL_ID, ROLE_MMA, it));
            if (!ok) break;
            tc_fence_after_sync();
            if (elect_one()) {                     // dV += P^T dO   (dO read MN-major: 16 query rows per instruction)
                const uint64_t dDOm = smem_desc_sw128(smem_u32(sdO + sl * L::TILE_BYTES), BOX_BYTES, 1024);
#pragma unroll
                for (int k = 0; k < TILE / 16; ++k)
                    umma_ts(tmem_u + 256, tmem_u + a_col(k), desc_advance(dDOm, k * 2048), IDESC_G,
                            (it > 0 || k > 0) ? 1u : 0u);
                umma_commit(&do_empty[sl]);
            }
            __syncwarp();
            if (it + 1 < n_it) {
                ok = issue_s(it + 1);              // overwrites P^T(it): ordered behind dV(it)
                if (!ok) break;
            }
            ok = mbar_wait(ds_ready, it & 1, abort_flag, p.guard, status_word(DKDV_KERNEL_ID, ROLE_MMA, it));
            if (!ok) break;
            tc_fence_after_sync();
            if (elect_one()) {                     // dK += dS^T Q   (Q read MN-major)
                const uint64_t dQm = smem_desc_sw128(smem_u32(sQ + sl * L::TILE_BYTES), BOX_BYTES, 1024);
#pragma unroll
                for (int k = 0; k < TILE / 16; ++k)
                    umma_ts(tmem_u + 256 + D, tmem_u + 128 + a_col(k), desc_advance(dQm, k * 2048), IDESC_G,
                            (it > 0 || k > 0) ? 1u : 0u);
                umma_commit(&q_empty[sl]);
                if (it == n_it - 1) umma_commit(final_bar);
            }
            __syncwarp();
            if (it + 1 < n_it) ok = issue_dp(it + 1);     // overwrites dS^T(it): ordered behind dK(it)
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------------ compute: P^T, dS^T; epilogue
        const int wg = (warp - 4) >> 2;            // warpgroup g takes query columns [g * WG_COLS, (g + 1) * WG_COLS) of each tile
        const int quad = warp & 3;
        const int r = quad * 32 + lane;            // key row inside the tile (TMEM lane)
        const int kv = k0 + r;
        const uint32_t lane_addr = static_cast<uint32_t>(quad * 32) << 16;
        const uint32_t tS = tmem_base + lane_addr + wg * WG_COLS;
        const uint32_t tDP = tmem_base + lane_addr + 128 + wg * WG_COLS;
        const float2 c2 = make_float2(p.scale_log2e, p.scale_log2e);
        static_assert(WG_COLS == 64, "the fragment-shaped accesses below cover 64 query columns per warpgroup");
        const int cq = 2 * (lane & 3);             // this thread's column pair inside each group of 8 query columns
        const int kv_row = k0 + quad * 32 + (lane >> 2);    // its first key row (then + 8, + 16, + 24)
        bool ok = true;
        int qi = 0;                                // query tile of the iteration inside its head (it % n_qi, without the division)
        for (int it = 0; it < n_it; ++it, qi = (qi + 1 == n_qi) ? 0 : qi + 1) {
            const int q0 = (qt_start + qi) * TILE + wg * WG_COLS;          // first query column of this warpgroup
            const int rsl = it % RS;
            const float *rows = s_rows + rsl * (2 * TILE) + wg * WG_COLS;  // -lse2 of this warpgroup's columns; -delta at + TILE
            ok = mbar_wait(&rows_full[rsl], (it / RS) & 1, abort_flag, p.guard, status_word(DKDV_KERNEL_ID, ROLE_SOFTMAX, it));
            if (!ok) break;
            ok = mbar_wait(s_full, it & 1, abort_flag, p.guard, status_word(DKDV_KERNEL_ID, ROLE_SOFTMAX, it));
            if (!ok) break;
            tc_fence_after_sync();
            const bool diag = CAUSAL && (q0 + off < k0 + TILE - 1);    // some (key, query) pairs here are masked
            // Fragment-shaped TMEM accesses (see vt_ptx.cuh): per half h of the warp's 32 key rows this thread holds the
            // rows 16h + lane/4 and 16h + lane/4 + 8 at the 16 query columns 8g + 2(lane%4), + 1 (g = 0..7), so it needs the
            // per-query values of only 16 columns: 8 shared-memory loads per vector instead of 32.
            float2 nl[8];                                          // -lse2 of this thread's column pairs
#pragma unroll
            for (int g = 0; g < 8; ++g) nl[g] = *reinterpret_cast<const float2 *>(&rows[8 * g + cq]);
            float2 pr[2][8][2];                                    // [half][column group][row]: probabilities, kept for dS
            uint32_t sv[2][32];
#pragma unroll
            for (int h = 0; h < 2; ++h) tmem_ld_frag64(tS + (static_cast<uint32_t>(h * 16) << 16), sv[h]);
            tmem_wait_ld();
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                uint32_t pp[16];
#pragma unroll
                for (int g = 0; g < 8; ++g) {
#pragma unroll
                    for (int rr = 0; rr < 2; ++rr) {               // the two rows: kv_row + 16h and + 8
                        const float2 x = __ffma2_rn(make_float2(__uint_as_float(sv[h][4 * g + 2 * rr]), __uint_as_float(sv[h][4 * g + 2 * rr + 1])),
                                                    c2, nl[g]);
                        float2 e = prob_pair(2 * g + rr, x);
                        if (diag) {
                            const int kvr = kv_row + 16 * h + 8 * rr;
                            if (q0 + 8 * g + cq + off < kvr) e.x = 0.0f;
                            if (q0 + 8 * g + cq + 1 + off < kvr) e.y = 0.0f;
                        }
                        pr[h][g][rr] = e;
                        pp[2 * g + rr] = pack16<F16>(e.x, e.y);
                    }
                }
                tmem_st_frag32(tS + (static_cast<uint32_t>(h * 16) << 16), pp);   // over this warpgroup's own, already read S^T columns
            }
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(p_ready);
#pragma unroll
            for (int g = 0; g < 8; ++g) nl[g] = *reinterpret_cast<const float2 *>(&rows[TILE + 8 * g + cq]);   // now -delta
            ok = mbar_wait(dp_full, it & 1, abort_flag, p.guard, status_word(DKDV_KERNEL_ID, ROLE_SOFTMAX, it));
            if (!ok) break;
            tc_fence_after_sync();
#pragma unroll
            for (int h = 0; h < 2; ++h) tmem_ld_frag64(tDP + (static_cast<uint32_t>(h * 16) << 16), sv[h]);
            tmem_wait_ld();
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                uint32_t dd[16];
#pragma unroll
                for (int g = 0; g < 8; ++g) {
#pragma unroll
                    for (int rr = 0; rr < 2; ++rr) {
                        const float2 df = __fadd2_rn(make_float2(__uint_as_float(sv[h][4 * g + 2 * rr]), __uint_as_float(sv[h][4 * g + 2 * rr + 1])), nl[g]);
                        const float2 ds = __fmul2_rn(pr[h][g][rr], df);
                        dd[2 * g + rr] = pack16<F16>(ds.x, ds.y);
                    }
                }
                tmem_st_frag32(tDP + (static_cast<uint32_t>(h * 16) << 16), dd);
            }
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(ds_ready);
            __syncwarp();
            if (lane == 0) mbar_arrive(&rows_empty[rsl]);      // every lane of this warp has read the slot's values
        }
        // epilogue: even warpgroups write dV, odd ones dK, each its share of the columns
        const bool is_dv = (wg & 1) == 0;
        constexpr int EPI_WGS = BWD_WGS / 2;          // warpgroups per output tensor
        const int epi = wg >> 1;
        __nv_bfloat16 *out_row = (is_dv ? p.dv : p.dk) +
                                 (PACKED ? (static_cast<size_t>(k_base + kv) * p.Hkv + hkv) : (static_cast<size_t>(bh_kv) * p.Sk + kv)) * p.d;
        const bool store = kv < Sk;
        if (n_it == 0) {
            // no query can see this key tile: the gradients are zero
            if (store)
                for (int i = epi; i < p.d / 8; i += EPI_WGS) reinterpret_cast<uint4 *>(out_row)[i] = make_uint4(0, 0, 0, 0);
        } else {
            if (ok) ok = mbar_wait(final_bar, 0, abort_flag, p.guard, status_word(DKDV_KERNEL_ID, ROLE_EPILOGUE, 0));
            if (ok) {
                // tcgen05.ld is warp-collective: every lane takes part, only rows inside the tensor store
                tc_fence_after_sync();
                const uint32_t tSrc = (is_dv ? tmem_dV : tmem_dK) + lane_addr;
                const float mul = is_dv ? 1.0f : p.scale;
                // every MMA has completed, so the Q tiles' shared memory is free: each warp takes a private patch of it
                // to transpose its stores (whole sectors per instruction instead of 32 half-used ones)
                uint8_t *scratch = sQ + (warp - 4) * STORE_SCRATCH_BYTES;
                const int row0 = k0 + quad * 32;              // first key row of this warp
                const size_t stride = PACKED ? static_cast<size_t>(p.Hkv) * p.d : static_cast<size_t>(p.d);
                __nv_bfloat16 *warp_dst = out_row - static_cast<size_t>(lane) * stride;
                const int rows_valid = min(32, Sk - row0);
#pragma unroll
                for (int c = epi * (D / 32 / EPI_WGS); c < (epi + 1) * (D / 32 / EPI_WGS); ++c) {
                    uint32_t v[32];
                    tmem_ld32(tSrc + c * 32, v);
                    tmem_wait_ld();
                    store_rows16<F16>(warp_dst + c * 32, stride, v, mul, rows_valid, scratch, lane, p.d - c * 32);
                }
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, L::TMEM_COLS);
    }
}

// ----------------------------------------------------------------------------------------------
// 3. dQ  (query tile stationary)
// ----------------------------------------------------------------------------------------------
template <int D>
struct DqSmem {
    static constexpr int TILE_BYTES = TILE * D * 2;
    static constexpr int K_SLOTS = 3;          // K(j) is read by S(j) and, two steps later in issue order, by dQ(j)
    static constexpr int V_SLOTS = 2;
    static constexpr int OFF_Q = 0;
    static constexpr int OFF_DO = OFF_Q + TILE_BYTES;
    static constexpr int OFF_K = OFF_DO + TILE_BYTES;                // [K_SLOTS]
    static constexpr int OFF_V = OFF_K + K_SLOTS * TILE_BYTES;       // [V_SLOTS]
    static constexpr int OFF_BAR = OFF_V + V_SLOTS * TILE_BYTES;
    static constexpr int BYTES = OFF_BAR + 256 + 1024;
    // TMEM columns: S buffers [0,128) [128,256); dP [256,384) (dS, bf16, written over it: columns [256,288) and
    // [320,352)); dQ [384,384+D).  P never goes to tensor memory here: it stays in the compute threads' registers.
    static constexpr int TMEM_COLS = 512;
};

template <int D, bool CAUSAL, bool PACKED, bool F16 = false>
__global__ void __launch_bounds__(BWD_THREADS, 1)
bwd_dq_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
              const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do, const BwdParams p)
{
    using L = DqSmem<D>;
    constexpr int KS = L::K_SLOTS, VS = L::V_SLOTS;
    constexpr int NBOX = D / BOX_COLS;
    constexpr int BOX_BYTES = TILE * BOX_COLS * 2;           // 16 KB

    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *sQ = smem + L::OFF_Q;
    uint8_t *sdO = smem + L::OFF_DO;
    uint8_t *sK = smem + L::OFF_K;
    uint8_t *sV = smem + L::OFF_V;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L::OFF_BAR);
    uint64_t *qdo_full = bars + 0;
    uint64_t *final_bar = bars + 1;
    uint64_t *dp_full = bars + 2;
    uint64_t *ds_ready = bars + 3;            // 256 arrivals
    uint64_t *s_full = bars + 4;              // [2]
    uint64_t *k_full = bars + 6;              // [KS]
    uint64_t *k_empty = bars + 6 + KS;        // [KS]
    uint64_t *v_full = bars + 6 + 2 * KS;     // [VS]
    uint64_t *v_empty = bars + 6 + 2 * KS + VS;   // [VS]
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 6 + 2 * KS + 2 * VS);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    int bh = blockIdx.x / p.n_tiles;
    int qt = blockIdx.x % p.n_tiles;
    if (CAUSAL && p.head_group > 1) {                                    // see causal_work_item (vt_ptx.cuh)
        const int per_group = p.head_group * p.n_tiles;
        const int grp = blockIdx.x / per_group, rem = blockIdx.x - grp * per_group;
        const int gsz = min(p.head_group, static_cast<int>(gridDim.x) / p.n_tiles - grp * p.head_group);
        qt = rem / gsz;
        bh = grp * p.head_group + rem % gsz;
    }
    if (CAUSAL) qt = p.n_tiles - 1 - qt;
    const int b = bh / p.Hq;
    const int h = bh % p.Hq;
    const int hkv = h / p.G;
    const int bh_kv = b * p.Hkv + hkv;
    const int q0 = qt * TILE;
    int Sq = p.Sq, Sk = p.Sk, q_base = 0, k_base = 0;                    // this block's sequence: lengths and first token rows
    if (PACKED) {
        q_base = p.cu_q[b];
        Sq = p.cu_q[b + 1] - q_base;
        k_base = p.cu_k[b];
        Sk = p.cu_k[b + 1] - k_base;
        if (q0 >= Sq) return;                                            // this sequence has no such query tile (whole block leaves)
    }
    const int off = (CAUSAL && p.bottom_right) ? Sk - Sq : 0;            // causal: query i sees the keys j <= i + off
    int n_it = (Sk + TILE - 1) / TILE;                                   // 128-key steps; 0: no key is visible to this tile
    if (CAUSAL) n_it = (q0 + TILE - 1 + off < 0) ? 0 : min(n_it, (q0 + TILE - 1 + off) / TILE + 1);

    if (threadIdx.x == 0) {
        mbar_init(qdo_full, 1);
        mbar_init(final_bar, 1);
        mbar_init(dp_full, 1);
        mbar_init(ds_ready, 128 * BWD_WGS);
        for (int s = 0; s < 2; ++s) mbar_init(&s_full[s], 1);
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
        // this thread is also the Q / dO / K producer: its first loads need not wait for the block-wide sync
        prefetch_tensormap(&tm_q);
        prefetch_tensormap(&tm_do);
        prefetch_tensormap(&tm_k);
        mbar_arrive_expect_tx(qdo_full, 2 * L::TILE_BYTES);
        for (int kb = 0; kb < NBOX; ++kb) {
            tma_load_3d(sQ + kb * BOX_BYTES, &tm_q, qdo_full, kb * BOX_COLS, PACKED ? h : q0, PACKED ? q_base + q0 : bh);
            tma_load_3d(sdO + kb * BOX_BYTES, &tm_do, qdo_full, kb * BOX_COLS, PACKED ? h : q0, PACKED ? q_base + q0 : bh);
        }
        if (n_it > 0) {
            mbar_arrive_expect_tx(&k_full[0], L::TILE_BYTES);
            for (int kb = 0; kb < NBOX; ++kb)
                tma_load_3d(sK + kb * BOX_BYTES, &tm_k, &k_full[0], kb * BOX_COLS, PACKED ? hkv : 0, PACKED ? k_base : bh_kv);
        }
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, L::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_dQ = tmem_base + 384;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer: Q, dO, then the K tiles
        if (lane == 0) {
            for (int j = 1; j < n_it; ++j) {       // (Q, dO and the first K tile went out before the block-wide sync)
                const int sl = j % KS;
                if (!mbar_wait(&k_empty[sl], ((j / KS) & 1) ^ 1, abort_flag, p.guard, status_word(DQ_KERNEL_ID, ROLE_LOAD, j))) break;
                mbar_arrive_expect_tx(&k_full[sl], L::TILE_BYTES);
                for (int kb = 0; kb < NBOX; ++kb)
                    tma_load_3d(sK + sl * L::TILE_BYTES + kb * BOX_BYTES, &tm_k, &k_full[sl], kb * BOX_COLS,
                                PACKED ? hkv : j * TILE, PACKED ? k_base + j * TILE : bh_kv);
            }
        }
    } else if (warp == 2) {
        // ------------------------------------------------------------------ TMA producer: the V tiles
        if (lane == 0) {
            prefetch_tensormap(&tm_v);
            for (int j = 0; j < n_it; ++j) {
                const int sl = j % VS;
                if (!mbar_wait(&v_empty[sl], ((j / VS) & 1) ^ 1, abort_flag, p.guard, status_word(DQ_KERNEL_ID, ROLE_LOAD, j))) break;
                mbar_arrive_expect_tx(&v_full[sl], L::TILE_BYTES);
                for (int kb = 0; kb < NBOX; ++kb)
                    tma_load_3d(sV + sl * L::TILE_BYTES + kb * BOX_BYTES, &tm_v, &v_full[sl], kb * BOX_COLS,
                                PACKED ? hkv : j * TILE, PACKED ? k_base + j * TILE : bh_kv);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        // Order per step: dQ(j), dP(j+1), S(j+2): the scores run two steps ahead of the step whose dS is consumed, so the
        // exponentials of step j+1 are taken while dQ(j) and dP(j+1) run.
        constexpr uint32_t IDESC_S = make_idesc(128, 128, fmt16<F16>(), fmt16<F16>(), 0, 0);
        constexpr uint32_t IDESC_G = make_idesc(128, D, fmt16<F16>(), fmt16<F16>(), 0, 1);
        const uint32_t tmem_u = __shfl_sync(0xFFFFFFFFu, tmem_base, 0);    // provably warp-uniform copy
        const uint64_t dQ0 = smem_desc_sw128(smem_u32(sQ), 16, 1024), dDO0 = smem_desc_sw128(smem_u32(sdO), 16, 1024);
        bool ok = mbar_wait(qdo_full, 0, abort_flag, p.guard, status_word(DQ_KERNEL_ID, ROLE_MMA, 0xFFFF));
        if (n_it == 0) ok = false;                 // no keys: nothing to issue (Q, dO were still waited for)
        auto issue_s = [&](int j) -> bool {        // S = Q K^T into buffer j & 1
            const int sl = j % KS;
            if (!mbar_wait(&k_full[sl], (j / KS) & 1, abort_flag, p.guard, status_word(DQ_KERNEL_ID, ROLE_MMA, j))) return false;
            tc_fence_after_sync();
            if (elect_one()) {
                const uint64_t dKs = smem_desc_sw128(smem_u32(sK + sl * L::TILE_BYTES), 16, 1024);
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    const uint32_t off = (k / 4) * BOX_BYTES + (k % 4) * 32;
                    umma_ss(tmem_u + (j & 1) * TILE, desc_advance(dQ0, off), desc_advance(dKs, off), IDESC_S, k > 0 ? 1u : 0u);
                }
                umma_commit(&s_full[j & 1]);
            }
            __syncwarp();
            return true;
        };
        auto issue_dp = [&](int j) -> bool {       // dP = dO V^T
            const int sl = j % VS;
            if (!mbar_wait(&v_full[sl], (j / VS) & 1, abort_flag, p.guard, status_word(DQ_KERNEL_ID, ROLE_MMA, j))) return false;
            tc_fence_after_sync();
            if (elect_one()) {
                const uint64_t dVs = smem_desc_sw128(smem_u32(sV + sl * L::TILE_BYTES), 16, 1024);
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    const uint32_t off = (k / 4) * BOX_BYTES + (k % 4) * 32;
                    umma_ss(tmem_u + 256, desc_advance(dDO0, off), desc_advance(dVs, off), IDESC_S, k > 0 ? 1u : 0u);
                }
                umma_commit(dp_full);
                umma_commit(&v_empty[sl]);
            }
            __syncwarp();
            return true;
        };
        if (ok) ok = issue_s(0);
        if (ok) ok = issue_dp(0);
        if (ok && n_it > 1) ok = issue_s(1);
        for (int j = 0; j < n_it && ok; ++j) {
            const int sl = j % KS;
            ok = mbar_wait(ds_ready, j & 1, abort_flag, p.guard, status_word(DQ_KERNEL_ID, ROLE_MMA, j));
            if (!ok) break;
            tc_fence_after_sync();
            if (elect_one()) {                     // dQ += dS K   (K read MN-major: 16 key rows per instruction)
                const uint64_t dKm = smem_desc_sw128(smem_u32(sK + sl * L::TILE_BYTES), BOX_BYTES, 1024);
#pragma unroll
                for (int k = 0; k < TILE / 16; ++k)
                    umma_ts(tmem_u + 384, tmem_u + 256 + a_col(k), desc_advance(dKm, k * 2048), IDESC_G,
                            (j > 0 || k > 0) ? 1u : 0u);
                umma_commit(&k_empty[sl]);
                if (j == n_it - 1) umma_commit(final_bar);
            }
            __syncwarp();
            if (j + 1 < n_it) {
                ok = issue_dp(j + 1);              // overwrites dS(j): ordered behind dQ(j)
                if (!ok) break;
            }
            if (j + 2 < n_it) ok = issue_s(j + 2); // buffer j & 1: its scores were read before dS(j) was signalled
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------------ compute: P (registers), dS; epilogue
        const int wg = (warp - 4) >> 2;            // warpgroup g takes key columns [g * WG_COLS, (g + 1) * WG_COLS) of each step
        const int quad = warp & 3;
        const int r = quad * 32 + lane;
        const int row = q0 + r;
        const uint32_t lane_addr = static_cast<uint32_t>(quad * 32) << 16;
        const uint32_t tDP = tmem_base + lane_addr + 256 + wg * WG_COLS;
        float lse2 = INFINITY, dl = 0.0f;          // rows past the end: P = 0
        if (row < Sq && n_it > 0) {
            const size_t idx = PACKED ? static_cast<size_t>(h) * p.total_q + q_base + row : static_cast<size_t>(bh) * p.Sq + row;
            lse2 = p.lse[idx] * LOG2E;
            dl = p.delta[idx];
        }
        const float2 c2 = make_float2(p.scale_log2e, p.scale_log2e);
        const float2 nl2 = make_float2(-lse2, -lse2);
        const float2 ndl2 = make_float2(-dl, -dl);
        bool ok = true;
        for (int j = 0; j < n_it; ++j) {
            ok = mbar_wait(&s_full[j & 1], (j >> 1) & 1, abort_flag, p.guard, status_word(DQ_KERNEL_ID, ROLE_SOFTMAX, j));
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t tS = tmem_base + lane_addr + (j & 1) * TILE + wg * WG_COLS;
            const int c0 = j * TILE + wg * WG_COLS;                // first key column of this thread
            const bool need_mask = (j * TILE + TILE > Sk) || (CAUSAL && (j * TILE + TILE - 1 > q0 + off));
            int limit = Sk - c0;                                   // key columns >= limit contribute nothing
            if (CAUSAL) limit = min(limit, row + off - c0 + 1);
            float2 pr[WG_COLS / 2];
            uint32_t sv[WG_CHUNKS][32];
#pragma unroll
            for (int c = 0; c < WG_CHUNKS; ++c) tmem_ld32(tS + c * 32, sv[c]);
            tmem_wait_ld();
#pragma unroll
            for (int c = 0; c < WG_CHUNKS; ++c) {
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const int col = c * 32 + 2 * i;
                    const float2 x = __ffma2_rn(make_float2(__uint_as_float(sv[c][2 * i]), __uint_as_float(sv[c][2 * i + 1])), c2, nl2);
                    float2 e = prob_pair(i, x);
                    if (need_mask) {
                        if (col >= limit) e.x = 0.0f;
                        if (col + 1 >= limit) e.y = 0.0f;
                    }
                    pr[c * 16 + i] = e;
                }
            }
            ok = mbar_wait(dp_full, j & 1, abort_flag, p.guard, status_word(DQ_KERNEL_ID, ROLE_SOFTMAX, j));
            if (!ok) break;
            tc_fence_after_sync();
            uint32_t dpv[WG_CHUNKS][32];
#pragma unroll
            for (int c = 0; c < WG_CHUNKS; ++c) tmem_ld32(tDP + c * 32, dpv[c]);
            tmem_wait_ld();
#pragma unroll
            for (int c = 0; c < WG_CHUNKS; ++c) {
                uint32_t dd[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const float2 df = __fadd2_rn(make_float2(__uint_as_float(dpv[c][2 * i]), __uint_as_float(dpv[c][2 * i + 1])), ndl2);
                    const float2 ds = __fmul2_rn(pr[c * 16 + i], df);
                    dd[i] = pack16<F16>(ds.x, ds.y);
                }
                tmem_st16(tDP + c * 16, dd);       // over this thread's own, already read dP columns
            }
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(ds_ready);
        }
        const bool store = row < Sq;
        __nv_bfloat16 *dq_row = p.dq + (PACKED ? (static_cast<size_t>(q_base + row) * p.Hq + h) : (static_cast<size_t>(bh) * p.Sq + row)) * p.d;
        if (n_it == 0) {
            // a packed sequence without keys: dQ = 0 (each warpgroup clears its share of the columns)
            if (store)
                for (int i = wg; i < p.d / 8; i += BWD_WGS) reinterpret_cast<uint4 *>(dq_row)[i] = make_uint4(0, 0, 0, 0);
            ok = false;
        }
        if (ok) ok = mbar_wait(final_bar, 0, abort_flag, p.guard, status_word(DQ_KERNEL_ID, ROLE_EPILOGUE, 0));
        if (ok) {
            // the warpgroups share the dQ columns (32-column chunks; with more warpgroups than chunks the rest idle)
            tc_fence_after_sync();
            constexpr int CHUNKS = D / 32;
            constexpr int PER_WG = (CHUNKS + BWD_WGS - 1) / BWD_WGS;
            // every MMA has completed, so the Q tile's shared memory is free: a private patch per warp to transpose the stores
            uint8_t *scratch = sQ + (warp - 4) * STORE_SCRATCH_BYTES;
            const size_t stride = PACKED ? static_cast<size_t>(p.Hq) * p.d : static_cast<size_t>(p.d);
            __nv_bfloat16 *warp_dst = dq_row - static_cast<size_t>(lane) * stride;
            const int rows_valid = min(32, Sq - (q0 + quad * 32));
#pragma unroll
            for (int c = 0; c < PER_WG; ++c) {
                const int cc = wg * PER_WG + c;
                if (cc < CHUNKS) {                  // warp-uniform
                    uint32_t v[32];
                    tmem_ld32(tmem_dQ + lane_addr + cc * 32, v);
                    tmem_wait_ld();
                    store_rows16<F16>(warp_dst + cc * 32, stride, v, p.scale, rows_valid, scratch, lane, p.d - cc * 32);
                }
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, L::TMEM_COLS);
    }
}

}  // namespace vt

#include "bwd_fused.cuh"

namespace vt {

template <typename K>
static int set_smem(K kernel, int bytes, const char *what)
{
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e != cudaSuccess) return cuda_fail(e, what);
    return VT_ATTN_OK;
}

struct BwdMaps {
    CUtensorMap q128, do128, k128, v128;    // 128-row boxes
};

// B: batch size, or the number of sequences of a packed batch (then n_rows = total_q * Hq and the tile counts come from
// the longest sequence, prm.Sq / prm.Sk).
template <int D, bool CAUSAL, bool PACKED, bool F16 = false>
static int launch_bwd(const BwdMaps &m, BwdParams prm, const __nv_bfloat16 *o, const __nv_bfloat16 *d_o, float *delta, int B,
                      cudaStream_t stream)
{
    int rc;
    static std::atomic<bool> configured[64];     // set-up is idempotent: two threads may both do it, neither may read a torn flag
    int dev = 0;
    cudaGetDevice(&dev);
    if (!configured[dev & 63].load(std::memory_order_acquire)) {
        if ((rc = set_smem(bwd_dkdv_kernel<D, CAUSAL, PACKED, F16>, DkdvSmem<D>::BYTES, "cudaFuncSetAttribute(dkdv)")) != VT_ATTN_OK) return rc;
        if ((rc = set_smem(bwd_dq_kernel<D, CAUSAL, PACKED, F16>, DqSmem<D>::BYTES, "cudaFuncSetAttribute(dq)")) != VT_ATTN_OK) return rc;
        configured[dev & 63].store(true, std::memory_order_release);
    }

    const long long n_rows = PACKED ? static_cast<long long>(prm.total_q) * prm.Hq : static_cast<long long>(B) * prm.Hq * prm.Sq;
    int tpr = 1;                                      // threads per row of the Delta kernel: a power of two >= d / 8
    while (tpr * 8 < prm.d) tpr *= 2;
    const int rows_per_block = 256 / tpr;
    long long delta_blocks = (n_rows + rows_per_block - 1) / rows_per_block;
    if (delta_blocks > NUM_SMS * 32) delta_blocks = NUM_SMS * 32;
    const int db = static_cast<int>(delta_blocks), packed_hq = PACKED ? prm.Hq : 0;
    switch (tpr) {
        case 16: bwd_delta_kernel<16, F16><<<db, 256, 0, stream>>>(o, d_o, delta, n_rows, packed_hq, prm.d); break;
        case 8: bwd_delta_kernel<8, F16><<<db, 256, 0, stream>>>(o, d_o, delta, n_rows, packed_hq, prm.d); break;
        case 4: bwd_delta_kernel<4, F16><<<db, 256, 0, stream>>>(o, d_o, delta, n_rows, packed_hq, prm.d); break;
        case 2: bwd_delta_kernel<2, F16><<<db, 256, 0, stream>>>(o, d_o, delta, n_rows, packed_hq, prm.d); break;
        default: bwd_delta_kernel<1, F16><<<db, 256, 0, stream>>>(o, d_o, delta, n_rows, packed_hq, prm.d); break;
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "bwd_delta_kernel launch");

    const int n_kt = (prm.Sk + TILE - 1) / TILE;
    const int n_qt = (prm.Sq + TILE - 1) / TILE;
    prm.n_tiles = n_kt;
    bwd_dkdv_kernel<D, CAUSAL, PACKED, F16><<<n_kt * B * prm.Hkv, BWD_THREADS, DkdvSmem<D>::BYTES, stream>>>(m.q128, m.k128, m.v128, m.do128, prm);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "bwd_dkdv_kernel launch");

    prm.n_tiles = n_qt;
    // causal: the query heads are handed out in groups, longest tiles of a group first (causal_head_group).  The key-tile
    // kernel above keeps its head order: the same grouping gained 1 % there at S = 2048 and cost 1.5 % on long launches.
    prm.head_group = causal_head_group(static_cast<long long>(B) * prm.Hq, n_qt, NUM_SMS, prm.G, 4ll * prm.Sk * prm.d / prm.G);
    bwd_dq_kernel<D, CAUSAL, PACKED, F16><<<n_qt * B * prm.Hq, BWD_THREADS, DqSmem<D>::BYTES, stream>>>(m.q128, m.k128, m.v128, m.do128, prm);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "bwd_dq_kernel launch");
    return VT_ATTN_OK;
}

// ----------------------------------------------------------------------------------------------
// The five-product path (bwd_fused.cuh): workspace layout, when it is used, launches
// ----------------------------------------------------------------------------------------------
static size_t align256(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }

struct FusedPlan {
    size_t delta, acc, stats_do, stats_k, stats_v, qscale, total;     // byte offsets into the workspace; acc .. stats_v are cleared together
    size_t clear_bytes;
};

static FusedPlan fused_plan(int B, int Hq, int Hkv, int Sq, int d)
{
    FusedPlan f;
    const size_t rows = static_cast<size_t>(B) * Hq * Sq;
    size_t off = 0;
    auto take = [&off](size_t bytes) { const size_t at = off; off += align256(bytes); return at; };
    f.delta = take(rows * 4);
    f.acc = take(rows * d * 4);
    f.stats_do = take(static_cast<size_t>(B) * Hq * 4);
    f.stats_k = take(static_cast<size_t>(B) * Hkv * 4);
    f.stats_v = take(static_cast<size_t>(B) * Hkv * 4);
    f.clear_bytes = off - f.acc;
    f.qscale = take(static_cast<size_t>(B) * Hq * 4);
    f.total = off;
    return f;
}

// 0: library's choice; 1: always the two-kernel path; 2: the five-product path wherever it is built (D in (64, 128],
// batched layout).  Read from the environment variable VT_ATTN_BWD_PATH ("split" / "fused") at every call: a switch for
// tests and measurements, not part of the ABI.
static int bwd_path_override()
{
    const char *e = getenv("VT_ATTN_BWD_PATH");
    if (!e) return 0;
    if (e[0] == 's') return 1;
    if (e[0] == 'f') return 2;
    return 0;
}

// Whether vt_attn_bwd uses the five-product path for this shape (given a workspace of the size
// vt_attn_bwd_workspace_bytes states).  It is built for the 128-column kernels.  The library never picks it by itself:
// measured on the B200 it is slower than the two-kernel path on every shape tried (B = 1, 32 query heads on 8 KV heads,
// S = 16384, causal: 13.2 ms against 6.2 ms; with the red.add instructions compiled out 5.1 ms) - 64 KB of reductions
// per (query tile, key tile) pair is more than the L2 takes per SM in the time the five products need (a loop of nothing
// but these reductions on all SMs: 3.2 TB/s into HBM-resident tiles, 5.5 TB/s into tiles four blocks share).
static bool fused_wanted(int B, int Hq, int Hkv, int Sq, int Sk, int D)
{
    (void)B; (void)Hq; (void)Hkv; (void)Sq; (void)Sk;
    if (padded_head_dim(D) != 128) return false;
    return bwd_path_override() == 2;
}

template <bool CAUSAL, bool F16>
static int launch_bwd_fused(const BwdMaps &m, BwdParams prm, const __nv_bfloat16 *o, const __nv_bfloat16 *d_o, const __nv_bfloat16 *k,
                            const __nv_bfloat16 *v, uint8_t *ws, int B, cudaStream_t stream)
{
    constexpr int D = 128;
    int rc;
    static std::atomic<bool> configured[64];
    int dev = 0;
    cudaGetDevice(&dev);
    if (!configured[dev & 63].load(std::memory_order_acquire)) {
        if ((rc = set_smem(bwd_fused_kernel<D, CAUSAL, F16>, FusedSmem<D>::BYTES, "cudaFuncSetAttribute(fused)")) != VT_ATTN_OK) return rc;
        configured[dev & 63].store(true, std::memory_order_release);
    }
    const FusedPlan f = fused_plan(B, prm.Hq, prm.Hkv, prm.Sq, prm.d);
    float *delta = reinterpret_cast<float *>(ws + f.delta);
    int *acc = reinterpret_cast<int *>(ws + f.acc);
    float *stats_do = reinterpret_cast<float *>(ws + f.stats_do), *stats_k = reinterpret_cast<float *>(ws + f.stats_k);
    float *stats_v = reinterpret_cast<float *>(ws + f.stats_v), *qscale = reinterpret_cast<float *>(ws + f.qscale);
    cudaError_t e = cudaMemsetAsync(acc, 0, f.clear_bytes, stream);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync(dQ accumulator)");

    const long long n_rows = static_cast<long long>(B) * prm.Hq * prm.Sq;
    const long long n_kv_rows = static_cast<long long>(B) * prm.Hkv * prm.Sk;
    int tpr = 1;
    while (tpr * 8 < prm.d) tpr *= 2;
    const int rows_per_block = 256 / tpr;
    long long delta_blocks = (n_rows + rows_per_block - 1) / rows_per_block;
    if (delta_blocks > NUM_SMS * 32) delta_blocks = NUM_SMS * 32;
    const int db = static_cast<int>(delta_blocks);
    if (tpr == 16) bwd_delta_kernel<16, F16><<<db, 256, 0, stream>>>(o, d_o, delta, n_rows, 0, prm.d);
    else bwd_delta_kernel<8, F16><<<db, 256, 0, stream>>>(o, d_o, delta, n_rows, 0, prm.d);      // 64 < d <= 128: tpr is 16 (d > 64)
    if ((e = cudaGetLastError()) != cudaSuccess) return cuda_fail(e, "bwd_delta_kernel launch");
    auto warp_grid = [](long long rows) { long long nb = (rows + 7) / 8; return static_cast<int>(nb > NUM_SMS * 16 ? NUM_SMS * 16 : nb); };
    bwd_do_norm_kernel<F16><<<warp_grid(n_rows), 256, 0, stream>>>(d_o, stats_do, prm.Sq, prm.d, n_rows);
    if ((e = cudaGetLastError()) != cudaSuccess) return cuda_fail(e, "bwd_do_norm_kernel launch");
    bwd_kv_norm_kernel<F16><<<warp_grid(n_kv_rows), 256, 0, stream>>>(k, v, stats_k, stats_v, prm.Sk, prm.d, n_kv_rows);
    if ((e = cudaGetLastError()) != cudaSuccess) return cuda_fail(e, "bwd_kv_norm_kernel launch");
    const int n_bh = B * prm.Hq;
    bwd_qscale_kernel<<<(n_bh + 127) / 128, 128, 0, stream>>>(stats_do, stats_k, stats_v, qscale, n_bh, prm.Hq, prm.Hkv);
    if ((e = cudaGetLastError()) != cudaSuccess) return cuda_fail(e, "bwd_qscale_kernel launch");

    prm.delta = delta;
    prm.n_tiles = (prm.Sk + TILE - 1) / TILE;
    FusedParams fp;
    fp.dq_acc = acc;
    fp.qscale = qscale;
    bwd_fused_kernel<D, CAUSAL, F16><<<prm.n_tiles * B * prm.Hkv, FUSED_THREADS, FusedSmem<D>::BYTES, stream>>>(m.q128, m.k128, m.v128, m.do128, prm, fp);
    if ((e = cudaGetLastError()) != cudaSuccess) return cuda_fail(e, "bwd_fused_kernel launch");

    const long long n_vec = n_rows * prm.d / 8;
    long long cb = (n_vec + 255) / 256;
    if (cb > NUM_SMS * 32) cb = NUM_SMS * 32;
    bwd_dq_convert_kernel<F16><<<static_cast<int>(cb), 256, 0, stream>>>(acc, qscale, prm.dq, n_vec, static_cast<long long>(prm.Sq) * prm.d / 8, prm.scale);
    if ((e = cudaGetLastError()) != cudaSuccess) return cuda_fail(e, "bwd_dq_convert_kernel launch");
    return VT_ATTN_OK;
}

}  // namespace vt

extern "C" size_t vt_attn_bwd_workspace_bytes(int B, int Hq, int Hkv, int Sq, int Sk, int D)
{
    vt::Shape s{B, Hq, Hkv, Sq, Sk, D};
    if (vt::check_shape(s, 1.0f, vt::MAX_HEAD_DIM_FWD) != VT_ATTN_OK) return 0;
    if (vt::fused_wanted(B, Hq, Hkv, Sq, Sk, D)) return vt::fused_plan(B, Hq, Hkv, Sq, D).total;
    const size_t n = static_cast<size_t>(B) * Hq * Sq * sizeof(float);
    return (n + 255) & ~static_cast<size_t>(255);
}

extern "C" int vt_attn_bwd_kernel_kind(int B, int Hq, int Hkv, int Sq, int Sk, int D)
{
    vt::Shape s{B, Hq, Hkv, Sq, Sk, D};
    int rc = vt::check_shape(s, 1.0f, vt::MAX_HEAD_DIM_FWD);
    if (rc != VT_ATTN_OK) return rc;
    if (D > vt::MAX_HEAD_DIM) return 2;
    return vt::fused_wanted(B, Hq, Hkv, Sq, Sk, D) ? 1 : 0;
}

// Shared by vt_attn_bwd (bfloat16 tensors) and vt_attn_bwd_f16 (IEEE half tensors).
static int bwd_entry(bool f16, const void *q, const void *k, const void *v, const void *o, const void *d_o, const float *lse,
                           void *dq, void *dk, void *dv, int B, int Hq, int Hkv, int Sq, int Sk, int D, int causal,
                           float scale, void *workspace, size_t workspace_bytes, void *stream)
{
    using namespace vt;
    Shape s{B, Hq, Hkv, Sq, Sk, D};
    int rc = check_shape(s, scale, MAX_HEAD_DIM_FWD);
    if (rc != VT_ATTN_OK) return rc;
    if (!ptr_ok(q) || !ptr_ok(k) || !ptr_ok(v) || !ptr_ok(o) || !ptr_ok(d_o) || !ptr_ok(lse, 4) || !ptr_ok(dq) ||
        !ptr_ok(dk) || !ptr_ok(dv) || !ptr_ok(workspace))
        return VT_ATTN_ERR_INVALID_ARGUMENT;
    // The five-product path needs its larger workspace; a caller that brings only the Delta scratch (the static-scratch
    // entry point does) gets the two-kernel path, which needs nothing else.
    const size_t split_need = align256(static_cast<size_t>(B) * Hq * Sq * sizeof(float));
    const bool fused = fused_wanted(B, Hq, Hkv, Sq, Sk, D) && workspace_bytes >= fused_plan(B, Hq, Hkv, Sq, D).total &&
                       ptr_ok(workspace, 256);
    if (!fused && workspace_bytes < split_need) return VT_ATTN_ERR_WORKSPACE_TOO_SMALL;
    if (causal < 0 || causal > 2) return VT_ATTN_ERR_INVALID_ARGUMENT;
    rc = check_device();
    if (rc != VT_ATTN_OK) return rc;
    const long long max_blocks = static_cast<long long>((Sq > Sk ? Sq : Sk) + TILE - 1) / TILE * B * Hq;
    if (max_blocks > 0x7FFFFFFFll) return VT_ATTN_ERR_INVALID_ARGUMENT;

    BwdParams prm;
    prm.lse = lse;
    prm.delta = static_cast<float *>(workspace);
    prm.dq = static_cast<__nv_bfloat16 *>(dq);
    prm.dk = static_cast<__nv_bfloat16 *>(dk);
    prm.dv = static_cast<__nv_bfloat16 *>(dv);
    prm.Hq = Hq;
    prm.Hkv = Hkv;
    prm.d = D;
    const int Dp = padded_head_dim(D);      // the kernels' column count; the columns past D read as zero
    prm.G = Hq / Hkv;
    prm.Sq = Sq;
    prm.Sk = Sk;
    prm.n_tiles = 0;
    prm.cu_q = nullptr;
    prm.cu_k = nullptr;
    prm.total_q = 0;
    prm.bottom_right = (causal == 2);
    prm.head_group = 0;
    prm.scale = scale;
    prm.scale_log2e = scale * LOG2E;
    prm.guard = make_guard();
    if (!prm.guard.status) return VT_ATTN_ERR_CUDA;

    BwdMaps m;
    if ((rc = make_tensor_map(&m.q128, q, B * Hq, Sq, D, TILE)) != VT_ATTN_OK) return rc;
    if ((rc = make_tensor_map(&m.do128, d_o, B * Hq, Sq, D, TILE)) != VT_ATTN_OK) return rc;
    if ((rc = make_tensor_map(&m.k128, k, B * Hkv, Sk, D, TILE)) != VT_ATTN_OK) return rc;
    if ((rc = make_tensor_map(&m.v128, v, B * Hkv, Sk, D, TILE)) != VT_ATTN_OK) return rc;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const __nv_bfloat16 *o_ = static_cast<const __nv_bfloat16 *>(o);
    const __nv_bfloat16 *do_ = static_cast<const __nv_bfloat16 *>(d_o);
    float *delta = static_cast<float *>(workspace);
    if (D > MAX_HEAD_DIM) return launch_bwd_wide(f16, q, k, v, o, d_o, prm, delta, B, causal, st);      // 128 < D <= 256: bwd_wide.cu
    if (fused) {
        const __nv_bfloat16 *k_ = static_cast<const __nv_bfloat16 *>(k), *v_ = static_cast<const __nv_bfloat16 *>(v);
        uint8_t *ws = static_cast<uint8_t *>(workspace);
        if (f16) return causal ? launch_bwd_fused<true, true>(m, prm, o_, do_, k_, v_, ws, B, st) : launch_bwd_fused<false, true>(m, prm, o_, do_, k_, v_, ws, B, st);
        return causal ? launch_bwd_fused<true, false>(m, prm, o_, do_, k_, v_, ws, B, st) : launch_bwd_fused<false, false>(m, prm, o_, do_, k_, v_, ws, B, st);
    }
    if (f16) {
        if (Dp == 64)
            return causal ? launch_bwd<64, true, false, true>(m, prm, o_, do_, delta, B, st) : launch_bwd<64, false, false, true>(m, prm, o_, do_, delta, B, st);
        return causal ? launch_bwd<128, true, false, true>(m, prm, o_, do_, delta, B, st) : launch_bwd<128, false, false, true>(m, prm, o_, do_, delta, B, st);
    }
    if (Dp == 64)
        return causal ? launch_bwd<64, true, false>(m, prm, o_, do_, delta, B, st) : launch_bwd<64, false, false>(m, prm, o_, do_, delta, B, st);
    return causal ? launch_bwd<128, true, false>(m, prm, o_, do_, delta, B, st) : launch_bwd<128, false, false>(m, prm, o_, do_, delta, B, st);
}

extern "C" int vt_attn_bwd(const void *q, const void *k, const void *v, const void *o, const void *d_o, const float *lse,
                           void *dq, void *dk, void *dv, int B, int Hq, int Hkv, int Sq, int Sk, int D, int causal,
                           float scale, void *workspace, size_t workspace_bytes, void *stream)
{
    return bwd_entry(false, q, k, v, o, d_o, lse, dq, dk, dv, B, Hq, Hkv, Sq, Sk, D, causal, scale, workspace, workspace_bytes, stream);
}

extern "C" int vt_attn_bwd_f16(const void *q, const void *k, const void *v, const void *o, const void *d_o, const float *lse,
                           void *dq, void *dk, void *dv, int B, int Hq, int Hkv, int Sq, int Sk, int D, int causal,
                           float scale, void *workspace, size_t workspace_bytes, void *stream)
{
    return bwd_entry(true, q, k, v, o, d_o, lse, dq, dk, dv, B, Hq, Hkv, Sq, Sk, D, causal, scale, workspace, workspace_bytes, stream);
}

// Backward with V (and O, dO, dV) of their own width: the kernels of bwd_wide.cu, which take the two widths separately.
static int bwd_dv_entry(bool f16, const void *q, const void *k, const void *v, const void *o, const void *d_o, const float *lse,
                        void *dq, void *dk, void *dv, int B, int Hq, int Hkv, int Sq, int Sk, int D, int Dv, int causal,
                        float scale, void *workspace, size_t workspace_bytes, void *stream)
{
    using namespace vt;
    if (D == Dv) return bwd_entry(f16, q, k, v, o, d_o, lse, dq, dk, dv, B, Hq, Hkv, Sq, Sk, D, causal, scale, workspace, workspace_bytes, stream);
    Shape s{B, Hq, Hkv, Sq, Sk, D};
    int rc = check_shape(s, scale, MAX_HEAD_DIM_FWD);
    if (rc != VT_ATTN_OK) return rc;
    if (!head_dim_ok(Dv, MAX_HEAD_DIM_FWD)) return VT_ATTN_ERR_UNSUPPORTED;
    if (!ptr_ok(q) || !ptr_ok(k) || !ptr_ok(v) || !ptr_ok(o) || !ptr_ok(d_o) || !ptr_ok(lse, 4) || !ptr_ok(dq) ||
        !ptr_ok(dk) || !ptr_ok(dv) || !ptr_ok(workspace))
        return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (workspace_bytes < align256(static_cast<size_t>(B) * Hq * Sq * sizeof(float))) return VT_ATTN_ERR_WORKSPACE_TOO_SMALL;
    if (causal < 0 || causal > 2) return VT_ATTN_ERR_INVALID_ARGUMENT;
    rc = check_device();
    if (rc != VT_ATTN_OK) return rc;
    const long long max_blocks = static_cast<long long>((Sq > Sk ? Sq : Sk) + TILE - 1) / TILE * B * Hq;
    if (max_blocks > 0x7FFFFFFFll) return VT_ATTN_ERR_INVALID_ARGUMENT;
    BwdParams prm;
    prm.lse = lse;
    prm.delta = static_cast<float *>(workspace);
    prm.dq = static_cast<__nv_bfloat16 *>(dq);
    prm.dk = static_cast<__nv_bfloat16 *>(dk);
    prm.dv = static_cast<__nv_bfloat16 *>(dv);
    prm.Hq = Hq;
    prm.Hkv = Hkv;
    prm.d = D;
    prm.d_v = Dv;
    prm.G = Hq / Hkv;
    prm.Sq = Sq;
    prm.Sk = Sk;
    prm.n_tiles = 0;
    prm.cu_q = nullptr;
    prm.cu_k = nullptr;
    prm.total_q = 0;
    prm.bottom_right = (causal == 2);
    prm.head_group = 0;
    prm.scale = scale;
    prm.scale_log2e = scale * LOG2E;
    prm.guard = make_guard();
    if (!prm.guard.status) return VT_ATTN_ERR_CUDA;
    return launch_bwd_wide(f16, q, k, v, o, d_o, prm, static_cast<float *>(workspace), B, causal, static_cast<cudaStream_t>(stream));
}

extern "C" int vt_attn_bwd_dv(const void *q, const void *k, const void *v, const void *o, const void *d_o, const float *lse,
                              void *dq, void *dk, void *dv, int B, int Hq, int Hkv, int Sq, int Sk, int D, int Dv, int causal,
                              float scale, void *workspace, size_t workspace_bytes, void *stream)
{
    return bwd_dv_entry(false, q, k, v, o, d_o, lse, dq, dk, dv, B, Hq, Hkv, Sq, Sk, D, Dv, causal, scale, workspace, workspace_bytes, stream);
}

extern "C" int vt_attn_bwd_dv_f16(const void *q, const void *k, const void *v, const void *o, const void *d_o, const float *lse,
                                  void *dq, void *dk, void *dv, int B, int Hq, int Hkv, int Sq, int Sk, int D, int Dv, int causal,
                                  float scale, void *workspace, size_t workspace_bytes, void *stream)
{
    return bwd_dv_entry(true, q, k, v, o, d_o, lse, dq, dk, dv, B, Hq, Hkv, Sq, Sk, D, Dv, causal, scale, workspace, workspace_bytes, stream);
}

extern "C" size_t vt_attn_bwd_varlen_workspace_bytes(int Hq, int total_q)
{
    if (Hq <= 0 || total_q <= 0) return 0;
    const size_t n = static_cast<size_t>(Hq) * total_q * sizeof(float);
    return (n + 255) & ~static_cast<size_t>(255);
}

// Shared by vt_attn_bwd_varlen (bfloat16 tensors) and vt_attn_bwd_varlen_f16 (IEEE half tensors).
static int bwd_varlen_entry(bool f16, const void *q, const void *k, const void *v, const void *o, const void *d_o, const float *lse,
                            void *dq, void *dk, void *dv, const int *cu_seqlens_q, const int *cu_seqlens_k, int n_seqs,
                            int Hq, int Hkv, int total_q, int total_k, int max_sq, int max_sk, int D, int causal,
                            float scale, void *workspace, size_t workspace_bytes, void *stream)
{
    using namespace vt;
    int rc = check_varlen_shape(n_seqs, Hq, Hkv, total_q, total_k, max_sq, max_sk, D, scale);
    if (rc != VT_ATTN_OK) return rc;
    if (!ptr_ok(q) || !ptr_ok(k) || !ptr_ok(v) || !ptr_ok(o) || !ptr_ok(d_o) || !ptr_ok(lse, 4) || !ptr_ok(dq) || !ptr_ok(dk) ||
        !ptr_ok(dv) || !ptr_ok(workspace) || !ptr_ok(cu_seqlens_q, 4) || !ptr_ok(cu_seqlens_k, 4))
        return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (workspace_bytes < vt_attn_bwd_varlen_workspace_bytes(Hq, total_q)) return VT_ATTN_ERR_WORKSPACE_TOO_SMALL;
    if (causal < 0 || causal > 2) return VT_ATTN_ERR_INVALID_ARGUMENT;
    rc = check_device();
    if (rc != VT_ATTN_OK) return rc;
    const long long max_blocks = static_cast<long long>((max_sq > max_sk ? max_sq : max_sk) + TILE - 1) / TILE * n_seqs * Hq;
    if (max_blocks > 0x7FFFFFFFll) return VT_ATTN_ERR_INVALID_ARGUMENT;

    BwdParams prm;
    prm.lse = lse;
    prm.delta = static_cast<float *>(workspace);
    prm.dq = static_cast<__nv_bfloat16 *>(dq);
    prm.dk = static_cast<__nv_bfloat16 *>(dk);
    prm.dv = static_cast<__nv_bfloat16 *>(dv);
    prm.Hq = Hq;
    prm.Hkv = Hkv;
    prm.d = D;
    const int Dp = padded_head_dim(D);      // the kernels' column count; the columns past D read as zero
    prm.G = Hq / Hkv;
    prm.Sq = max_sq;
    prm.Sk = max_sk;
    prm.n_tiles = 0;
    prm.cu_q = cu_seqlens_q;
    prm.cu_k = cu_seqlens_k;
    prm.total_q = total_q;
    prm.bottom_right = (causal == 2);
    prm.head_group = 0;
    prm.scale = scale;
    prm.scale_log2e = scale * LOG2E;
    prm.guard = make_guard();
    if (!prm.guard.status) return VT_ATTN_ERR_CUDA;

    BwdMaps m;
    if ((rc = make_tensor_map_packed(&m.q128, q, total_q, Hq, D, TILE)) != VT_ATTN_OK) return rc;
    if ((rc = make_tensor_map_packed(&m.do128, d_o, total_q, Hq, D, TILE)) != VT_ATTN_OK) return rc;
    if ((rc = make_tensor_map_packed(&m.k128, k, total_k, Hkv, D, TILE)) != VT_ATTN_OK) return rc;
    if ((rc = make_tensor_map_packed(&m.v128, v, total_k, Hkv, D, TILE)) != VT_ATTN_OK) return rc;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const __nv_bfloat16 *o_ = static_cast<const __nv_bfloat16 *>(o);
    const __nv_bfloat16 *do_ = static_cast<const __nv_bfloat16 *>(d_o);
    float *delta = static_cast<float *>(workspace);
    if (f16) {
        if (Dp == 64)
            return causal ? launch_bwd<64, true, true, true>(m, prm, o_, do_, delta, n_seqs, st)
                          : launch_bwd<64, false, true, true>(m, prm, o_, do_, delta, n_seqs, st);
        return causal ? launch_bwd<128, true, true, true>(m, prm, o_, do_, delta, n_seqs, st)
                      : launch_bwd<128, false, true, true>(m, prm, o_, do_, delta, n_seqs, st);
    }
    if (Dp == 64)
        return causal ? launch_bwd<64, true, true>(m, prm, o_, do_, delta, n_seqs, st)
                      : launch_bwd<64, false, true>(m, prm, o_, do_, delta, n_seqs, st);
    return causal ? launch_bwd<128, true, true>(m, prm, o_, do_, delta, n_seqs, st)
                  : launch_bwd<128, false, true>(m, prm, o_, do_, delta, n_seqs, st);
}

extern "C" int vt_attn_bwd_varlen(const void *q, const void *k, const void *v, const void *o, const void *d_o, const float *lse,
                                  void *dq, void *dk, void *dv, const int *cu_seqlens_q, const int *cu_seqlens_k, int n_seqs,
                                  int Hq, int Hkv, int total_q, int total_k, int max_sq, int max_sk, int D, int causal,
                                  float scale, void *workspace, size_t workspace_bytes, void *stream)
{
    return bwd_varlen_entry(false, q, k, v, o, d_o, lse, dq, dk, dv, cu_seqlens_q, cu_seqlens_k, n_seqs, Hq, Hkv, total_q, total_k, max_sq, max_sk,
                            D, causal, scale, workspace, workspace_bytes, stream);
}

extern "C" int vt_attn_bwd_varlen_f16(const void *q, const void *k, const void *v, const void *o, const void *d_o, const float *lse,
                                      void *dq, void *dk, void *dv, const int *cu_seqlens_q, const int *cu_seqlens_k, int n_seqs,
                                      int Hq, int Hkv, int total_q, int total_k, int max_sq, int max_sk, int D, int causal,
                                      float scale, void *workspace, size_t workspace_bytes, void *stream)
{
    return bwd_varlen_entry(true, q, k, v, o, d_o, lse, dq, dk, dv, cu_seqlens_q, cu_seqlens_k, n_seqs, Hq, Hkv, total_q, total_k, max_sq, max_sk,
                            D, causal, scale, workspace, workspace_bytes, stream);
}

// ----------------------------------------------------------------------------------------------
// Backward without a caller-provided workspace: Delta lives in a fixed array in the device image.
// ----------------------------------------------------------------------------------------------
namespace vt {

// One copy per GPU that loads the library, held until the process exits.  Shared by every call on
// that GPU; contents persist between calls (each call overwrites the part it reads).
static __device__ __align__(256) float g_static_delta[VT_ATTN_STATIC_SCRATCH_ROWS];

// In host code `g_static_delta` is only a handle for the runtime, not a device address, so the
// address is looked up once per device (with that device current) and cached.
static int static_delta_ptr(float **out)
{
    static float *cached[64] = {};
    static std::mutex mutex;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    if (dev < 0 || dev >= 64) return VT_ATTN_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(mutex);
    if (cached[dev] == nullptr) {
        float *ptr = nullptr;
        e = cudaGetSymbolAddress(reinterpret_cast<void **>(&ptr), g_static_delta);
        if (e != cudaSuccess) return cuda_fail(e, "cudaGetSymbolAddress(static scratch)");
        if (ptr == nullptr) return VT_ATTN_ERR_CUDA;
        cached[dev] = ptr;
    }
    *out = cached[dev];
    return VT_ATTN_OK;
}

}  // namespace vt

static int bwd_static_scratch_entry(bool f16, const void *q, const void *k, const void *v, const void *o, const void *d_o,
                                    const float *lse, void *dq, void *dk, void *dv, int B, int Hq, int Hkv, int Sq,
                                    int Sk, int D, int causal, float scale, void *stream)
{
    using namespace vt;
    Shape s{B, Hq, Hkv, Sq, Sk, D};
    int rc = check_shape(s, scale);
    if (rc != VT_ATTN_OK) return rc;
    if (static_cast<long long>(B) * Hq * Sq > static_cast<long long>(VT_ATTN_STATIC_SCRATCH_ROWS))
        return VT_ATTN_ERR_STATIC_SCRATCH_TOO_SMALL;
    rc = check_device();
    if (rc != VT_ATTN_OK) return rc;
    float *scratch = nullptr;
    rc = static_delta_ptr(&scratch);
    if (rc != VT_ATTN_OK) return rc;
    return (f16 ? vt_attn_bwd_f16 : vt_attn_bwd)(q, k, v, o, d_o, lse, dq, dk, dv, B, Hq, Hkv, Sq, Sk, D, causal, scale, scratch,
                                                 static_cast<size_t>(VT_ATTN_STATIC_SCRATCH_ROWS) * sizeof(float), stream);
}

extern "C" int vt_attn_bwd_static_scratch(const void *q, const void *k, const void *v, const void *o, const void *d_o,
                                          const float *lse, void *dq, void *dk, void *dv, int B, int Hq, int Hkv, int Sq,
                                          int Sk, int D, int causal, float scale, void *stream)
{
    return bwd_static_scratch_entry(false, q, k, v, o, d_o, lse, dq, dk, dv, B, Hq, Hkv, Sq, Sk, D, causal, scale, stream);
}

extern "C" int vt_attn_bwd_static_scratch_f16(const void *q, const void *k, const void *v, const void *o, const void *d_o,
                                              const float *lse, void *dq, void *dk, void *dv, int B, int Hq, int Hkv, int Sq,
                                              int Sk, int D, int causal, float scale, void *stream)
{
    return bwd_static_scratch_entry(true, q, k, v, o, d_o, lse, dq, dk, dv, B, Hq, Hkv, Sq, Sk, D, causal, scale, stream);
}
