// Backward fused attention for head dimensions in (128, 256] (batched layout).
//
// The 128-column kernels of bwd.cu keep two 128-row operand tiles stationary in shared memory and four 128-column
// accumulators in tensor memory; at 256 columns neither fits.  Here the stationary side stays 128 rows (at 256 columns:
// 64 KB per tile) and the streamed side is cut to 64 rows, so every score tile is 128 x 64:
//
//   bwd_dkdv_wide_kernel : two blocks per (batch, KV head, 128-key tile), one per output tensor (dK and dV of 256
//       columns together would fill tensor memory).  K stays in shared memory; the query heads of the group are walked
//       64 queries at a time (Q in two slots) and S^T = K Q^T contracts over all columns in both blocks.  The dK block also
//       holds V, forms dP^T = V dO^T and dS^T and accumulates dK += dS^T Q (N = 256); the dV block only needs P^T and
//       accumulates dV += P^T dO, with two score buffers and two dO slots.  Tensors of at most 192 columns leave room
//       for both accumulators: then one block per key tile does both and forms the scores once.
//   bwd_dq_wide_kernel   : one block per (batch, query head, 128-query tile).  Q and dO stay in shared memory, K (two
//       slots) and V (one slot) stream by in tiles of 64 keys; dQ (256 columns) is accumulated in tensor memory.
//
// Same roles as in bwd.cu (warp 0 / 2 TMA producers, warp 1 MMA issuer, warp 3 row-vector producer) with ONE compute
// warpgroup (warps 4..7: a 128 x 64 tile is what one warpgroup of the 128-column kernels handles).  Every output tile
// has one owner block and every sum a fixed order, as there.  Delta comes from bwd_delta_kernel.
#include <mutex>

#include "bwd_common.cuh"

namespace vt {

constexpr int WIDE_D = 256;                          // columns the kernels are built for (the real head dimension d <= 256)
constexpr int WIDE_THREADS = 256;
constexpr int WIDE_N = 64;                           // rows of a streamed tile = columns of a score tile
constexpr int WIDE_BOXES = WIDE_D / BOX_COLS;        // 4 boxes of 64 columns per row
constexpr int BOX128_BYTES = TILE * BOX_COLS * 2;    // 16 KB: one box of a 128-row tile
constexpr int BOX64_BYTES = WIDE_N * BOX_COLS * 2;   // 8 KB: one box of a 64-row tile
constexpr int TILE128_BYTES = WIDE_BOXES * BOX128_BYTES;   // 64 KB
constexpr int TILE64_BYTES = WIDE_BOXES * BOX64_BYTES;     // 32 KB
constexpr uint32_t DKDV_WIDE_KERNEL_ID = 6;
constexpr uint32_t DQ_WIDE_KERNEL_ID = 7;

struct DkdvWideSmem {
    static constexpr int OFF_K = 0;
    static constexpr int OFF_V = OFF_K + TILE128_BYTES;
    static constexpr int OFF_Q = OFF_V + TILE128_BYTES;              // [2]
    static constexpr int OFF_DO = OFF_Q + 2 * TILE64_BYTES;          // [1]
    static constexpr int ROW_SLOTS = 2;
    static constexpr int OFF_ROWS = OFF_DO + TILE64_BYTES;           // [slot][-lse2 64 | -delta 64]
    static constexpr int OFF_BAR = OFF_ROWS + ROW_SLOTS * 2 * WIDE_N * 4;
    static constexpr int BYTES = OFF_BAR + 256;                      // no alignment slack: the kernel checks the base address
    // TMEM columns.  dK block: S^T [0,64), dP^T [64,128) (dS^T, 16-bit, over its first 32), dK [128,384).
    // dV block: two S^T buffers [0,64), [64,128) (P^T, 16-bit, over the first 32 of each), dV [128,384).
    // Block for both (widths <= 192): S^T [0,64) (P^T over its first 32), dP^T [64,128), dV [128,320), dK [320,512).
    static constexpr int TMEM_COLS = 512;
};

// grid.y = 0: the block accumulates dK of its key tile (all columns), grid.y = 1: dV.  Both walk the same queries and form
// the same scores; only the dK block needs dP and dS, only the dV block hands P to the tensor core.
template <bool CAUSAL, bool F16>
__global__ void __launch_bounds__(WIDE_THREADS, 1)
bwd_dkdv_wide_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                     const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do, const BwdParams p)
{
    using L = DkdvWideSmem;
    constexpr int RS = L::ROW_SLOTS;
    extern __shared__ __align__(1024) uint8_t smem_wide[];
    uint8_t *smem = smem_wide;
    uint8_t *sK = smem + L::OFF_K;
    uint8_t *sV = smem + L::OFF_V;
    uint8_t *sQ = smem + L::OFF_Q;
    uint8_t *sdO = smem + L::OFF_DO;
    float *s_rows = reinterpret_cast<float *>(smem + L::OFF_ROWS);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L::OFF_BAR);
    uint64_t *kv_full = bars + 0;
    uint64_t *final_bar = bars + 1;
    uint64_t *s_full = bars + 2;              // [2] (the dK block uses the first only)
    uint64_t *dp_full = bars + 4;
    // 128 arrivals each.  dK block: p_ready[0] = the scores have been read, ds_ready = dS^T is in tensor memory.  dV block:
    // p_ready[buf] = P^T is in score buffer buf - one barrier per buffer, because with the scores two iterations ahead
    // the compute warps may finish two iterations before the MMA warp looks, and a single barrier would then have gone
    // through two phases (the parity the MMA warp waits for would read as "not yet")
    uint64_t *p_ready = bars + 5;             // [2]
    uint64_t *ds_ready = bars + 7;
    uint64_t *q_full = bars + 8;              // [2]
    uint64_t *q_empty = bars + 10;            // [2]
    uint64_t *do_full = bars + 12;            // [2] (the dK block uses the first only)
    uint64_t *do_empty = bars + 14;           // [2]
    uint64_t *rows_full = bars + 16;          // [RS] 32 arrivals
    uint64_t *rows_empty = bars + 16 + RS;    // [RS] one arrival per compute warp
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 16 + 2 * RS);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    if ((smem_u32(smem_wide) & 1023u) != 0u) {           // the swizzled tiles need this, and there is no room for slack
        if (threadIdx.x == 0) atomicCAS(p.guard.status, 0u, status_word(DKDV_WIDE_KERNEL_ID, ROLE_LOAD, 0xFFFE));
        return;
    }

    // Block-uniform role.  Two blocks per key tile (gridDim.y = 2): 0 accumulates dK, 1 accumulates dV; the longer dK blocks
    // come first in the launch.  One block per key tile (gridDim.y = 1, tensors of at most 192 columns, whose two
    // accumulators fit beside S^T and dP^T): 2, both - the scores are formed once.
    const int role = (gridDim.y == 1) ? 2 : static_cast<int>(blockIdx.y);
    const bool is_dv = role == 1;                         // the dV-only block: two score buffers, two dO slots, no V, no dP
    const bool has_dv = role != 0, has_dk = role != 1;
    const int bh_kv = blockIdx.x / p.n_tiles;
    const int kt = blockIdx.x % p.n_tiles;
    const int b = bh_kv / p.Hkv;
    const int hkv = bh_kv % p.Hkv;
    const int k0 = kt * TILE;
    const int Sq = p.Sq, Sk = p.Sk;
    const int n_qt = (Sq + WIDE_N - 1) / WIDE_N;          // 64-query tiles per head
    const int off = (CAUSAL && p.bottom_right) ? Sk - Sq : 0;
    const int qt_start = CAUSAL ? min(max(k0 - off, 0) / WIDE_N, n_qt) : 0;   // first query tile with a query that sees key k0
    const int n_qi = n_qt - qt_start;
    const int n_it = n_qi * p.G;
    const int dv_w = p.d_v > 0 ? p.d_v : p.d;             // width of V, dO, dV (Q, K, dK: p.d)
    const int out_w = is_dv ? dv_w : p.d;                 // columns of this block's (first) output tensor: dV for role 1, else dK
    const uint32_t acc_k = 128 + (role == 2 ? 192 : 0);   // tensor-memory column of the dK accumulator (dV: always 128)
    const int kd = (p.d + 15) >> 4;                       // 16-column contraction steps of S^T = K Q^T that hold data
    const int kdv = (dv_w + 15) >> 4;                     // of dP^T = V dO^T

    if (threadIdx.x == 0) {
        mbar_init(kv_full, 1);
        mbar_init(final_bar, 1);
        mbar_init(&s_full[0], 1);
        mbar_init(&s_full[1], 1);
        mbar_init(dp_full, 1);
        mbar_init(&p_ready[0], 128);
        mbar_init(&p_ready[1], 128);
        mbar_init(ds_ready, 128);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&q_full[s], 1);
            mbar_init(&q_empty[s], 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(&do_full[s], 1);
            mbar_init(&do_empty[s], 1);
        }
        for (int s = 0; s < RS; ++s) {
            mbar_init(&rows_full[s], 32);
            mbar_init(&rows_empty[s], 4);
        }
        *abort_flag = 0u;
        fence_mbar_init();
        prefetch_tensormap(&tm_q);
        prefetch_tensormap(&tm_k);
        if (!is_dv) prefetch_tensormap(&tm_v);
        mbar_arrive_expect_tx(kv_full, (is_dv ? 1 : 2) * TILE128_BYTES);       // the dV block never reads V
        for (int kb = 0; kb < WIDE_BOXES; ++kb) {
            tma_load_3d(sK + kb * BOX128_BYTES, &tm_k, kv_full, kb * BOX_COLS, k0, bh_kv);
            if (!is_dv) tma_load_3d(sV + kb * BOX128_BYTES, &tm_v, kv_full, kb * BOX_COLS, k0, bh_kv);
        }
        if (n_it > 0) {
            mbar_arrive_expect_tx(&q_full[0], TILE64_BYTES);
            for (int kb = 0; kb < WIDE_BOXES; ++kb)
                tma_load_3d(sQ + kb * BOX64_BYTES, &tm_q, &q_full[0], kb * BOX_COLS, qt_start * WIDE_N, b * p.Hq + hkv * p.G);
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

    if (warp == 0) {
        if (lane == 0) {                           // Q tiles (K, V and the first one went out before the block-wide sync)
            for (int it = 1; it < n_it; ++it) {
                const int sl = it & 1;
                const int hq = hkv * p.G + it / n_qi;
                const int q0 = (qt_start + it % n_qi) * WIDE_N;
                if (!mbar_wait(&q_empty[sl], ((it >> 1) & 1) ^ 1, abort_flag, p.guard, status_word(DKDV_WIDE_KERNEL_ID, ROLE_LOAD, it))) break;
                mbar_arrive_expect_tx(&q_full[sl], TILE64_BYTES);
                for (int kb = 0; kb < WIDE_BOXES; ++kb)
                    tma_load_3d(sQ + sl * TILE64_BYTES + kb * BOX64_BYTES, &tm_q, &q_full[sl], kb * BOX_COLS, q0, b * p.Hq + hq);
            }
        }
    } else if (warp == 2) {
        if (lane == 0) {
            // dO tiles.  dK block: one slot, reloaded as soon as dP of the iteration has completed.  dV block: two slots (the
            // second in the memory the V tile would take), since dV(i + 1) follows dV(i) within a few hundred cycles.
            prefetch_tensormap(&tm_do);
            for (int it = 0; it < n_it; ++it) {
                const int hq = hkv * p.G + it / n_qi;
                const int q0 = (qt_start + it % n_qi) * WIDE_N;
                const int sl = is_dv ? (it & 1) : 0;
                uint8_t *dst = sl ? sV : sdO;
                if (!mbar_wait(&do_empty[sl], ((is_dv ? (it >> 1) : it) & 1) ^ 1, abort_flag, p.guard, status_word(DKDV_WIDE_KERNEL_ID, ROLE_LOAD, it))) break;
                mbar_arrive_expect_tx(&do_full[sl], TILE64_BYTES);
                for (int kb = 0; kb < WIDE_BOXES; ++kb)
                    tma_load_3d(dst + kb * BOX64_BYTES, &tm_do, &do_full[sl], kb * BOX_COLS, q0, b * p.Hq + hq);
            }
        }
    } else if (warp == 3) {
        // row vectors of the iteration's 64 queries: -LSE (log2 units; -inf past the end, so P = 0) and -Delta
        for (int it = 0; it < n_it; ++it) {
            const int sl = it % RS;
            if (!mbar_wait(&rows_empty[sl], ((it / RS) & 1) ^ 1, abort_flag, p.guard, status_word(DKDV_WIDE_KERNEL_ID, ROLE_LOAD, it))) break;
            const int hq = hkv * p.G + it / n_qi;
            const int q0 = (qt_start + it % n_qi) * WIDE_N;
            const size_t head = (static_cast<size_t>(b) * p.Hq + hq) * p.Sq;
            float *dst = s_rows + sl * (2 * WIDE_N);
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int q = q0 + e * 32 + lane;
                float nl = -INFINITY, nd = 0.0f;
                if (q < Sq) {
                    nl = -p.lse[head + q] * LOG2E;
                    nd = -p.delta[head + q];
                }
                dst[e * 32 + lane] = nl;
                dst[WIDE_N + e * 32 + lane] = nd;
            }
            mbar_arrive(&rows_full[sl]);
        }
    } else if (warp == 1) {
        // MMA issuer
        constexpr uint32_t IDESC_S = make_idesc(128, WIDE_N, fmt16<F16>(), fmt16<F16>(), 0, 0);
        const uint32_t IDESC_G = make_idesc(128, ((out_w + 15) >> 4) * 16, fmt16<F16>(), fmt16<F16>(), 0, 1);
        const uint32_t tmem_u = __shfl_sync(0xFFFFFFFFu, tmem_base, 0);
        const uint64_t dK0 = smem_desc_sw128(smem_u32(sK), 16, 1024), dV0 = smem_desc_sw128(smem_u32(sV), 16, 1024);
        bool ok = mbar_wait(kv_full, 0, abort_flag, p.guard, status_word(DKDV_WIDE_KERNEL_ID, ROLE_MMA, 0xFFFF));
        // S^T = K Q^T over all columns into score buffer `buf`; free_q: nothing else reads this Q tile (dV block)
        auto issue_s = [&](int it, int buf, bool free_q) -> bool {
            const int sl = it & 1;
            if (!mbar_wait(&q_full[sl], (it >> 1) & 1, abort_flag, p.guard, status_word(DKDV_WIDE_KERNEL_ID, ROLE_MMA, it))) return false;
            tc_fence_after_sync();
            if (elect_one()) {
                const uint64_t dQs = smem_desc_sw128(smem_u32(sQ + sl * TILE64_BYTES), 16, 1024);
#pragma unroll
                for (int k = 0; k < WIDE_D / 16; ++k)
                    if (k < kd)
                        umma_ss(tmem_u + buf * WIDE_N, desc_advance(dK0, (k / 4) * BOX128_BYTES + (k % 4) * 32),
                                desc_advance(dQs, (k / 4) * BOX64_BYTES + (k % 4) * 32), IDESC_S, k > 0 ? 1u : 0u);
                umma_commit(&s_full[buf]);
                if (free_q) umma_commit(&q_empty[sl]);
            }
            __syncwarp();
            return true;
        };
        if (is_dv) {
            // Per iteration: dV(i), then S(i+2) into the score buffer P^T(i) has just been read from: the scores run two
            // iterations ahead of the product that consumes their probabilities.
            if (ok && n_it > 0) ok = issue_s(0, 0, true);
            if (ok && n_it > 1) ok = issue_s(1, 1, true);
            for (int it = 0; it < n_it && ok; ++it) {
                const int dsl = it & 1;
                const uint64_t dDOm = smem_desc_sw128(smem_u32(dsl ? sV : sdO), BOX64_BYTES, 1024);      // dO as MN-major B operand, all boxes
                ok = mbar_wait(&do_full[dsl], (it >> 1) & 1, abort_flag, p.guard, status_word(DKDV_WIDE_KERNEL_ID, ROLE_MMA, it));
                if (!ok) break;
                ok = mbar_wait(&p_ready[it & 1], (it >> 1) & 1, abort_flag, p.guard, status_word(DKDV_WIDE_KERNEL_ID, ROLE_MMA, it));
                if (!ok) break;
                tc_fence_after_sync();
                if (elect_one()) {                 // dV += P^T dO   (16 query rows per instruction)
#pragma unroll
                    for (int k = 0; k < WIDE_N / 16; ++k)
                        umma_ts(tmem_u + 128, tmem_u + (it & 1) * WIDE_N + k * 8, desc_advance(dDOm, k * 2048), IDESC_G, (it > 0 || k > 0) ? 1u : 0u);
                    umma_commit(&do_empty[dsl]);
                    if (it == n_it - 1) umma_commit(final_bar);
                }
                __syncwarp();
                if (it + 2 < n_it) ok = issue_s(it + 2, it & 1, true);
            }
        } else {
            // dK block, per iteration: S(i+1) as soon as the compute warps hold S(i) in registers, dK(i), dP(i+1).
            // Block for both: dV(i) once P^T(i) is in tensor memory, S(i+1) behind it (it overwrites P^T(i)), dK(i), dP(i+1).
            const uint32_t IDESC_GV = make_idesc(128, ((dv_w + 15) >> 4) * 16, fmt16<F16>(), fmt16<F16>(), 0, 1);
            const uint64_t dDOm = smem_desc_sw128(smem_u32(sdO), BOX64_BYTES, 1024);      // dO as MN-major B operand of dV
            // dP^T = V dO^T over all columns; free_do: nothing else reads this dO tile (dK block)
            auto issue_dp = [&](int it, bool free_do) -> bool {
                if (!mbar_wait(&do_full[0], it & 1, abort_flag, p.guard, status_word(DKDV_WIDE_KERNEL_ID, ROLE_MMA, it))) return false;
                tc_fence_after_sync();
                if (elect_one()) {
                    const uint64_t dDOs = smem_desc_sw128(smem_u32(sdO), 16, 1024);
#pragma unroll
                    for (int k = 0; k < WIDE_D / 16; ++k)
                        if (k < kdv)
                            umma_ss(tmem_u + 64, desc_advance(dV0, (k / 4) * BOX128_BYTES + (k % 4) * 32),
                                    desc_advance(dDOs, (k / 4) * BOX64_BYTES + (k % 4) * 32), IDESC_S, k > 0 ? 1u : 0u);
                    umma_commit(dp_full);
                    if (free_do) umma_commit(&do_empty[0]);
                }
                __syncwarp();
                return true;
            };
            if (ok && n_it > 0) ok = issue_s(0, 0, false);
            if (ok && n_it > 0) ok = issue_dp(0, !has_dv);
            for (int it = 0; it < n_it && ok; ++it) {
                const int sl = it & 1;
                ok = mbar_wait(p_ready, it & 1, abort_flag, p.guard, status_word(DKDV_WIDE_KERNEL_ID, ROLE_MMA, it));
                if (!ok) break;
                if (has_dv) {
                    tc_fence_after_sync();
                    if (elect_one()) {                 // dV += P^T dO   (dO was read by dP(i) before: its slot is free after this)
#pragma unroll
                        for (int k = 0; k < WIDE_N / 16; ++k)
                            umma_ts(tmem_u + 128, tmem_u + k * 8, desc_advance(dDOm, k * 2048), IDESC_GV, (it > 0 || k > 0) ? 1u : 0u);
                        umma_commit(&do_empty[0]);
                    }
                    __syncwarp();
                }
                if (it + 1 < n_it) {
                    // dK block: S(i) sits in the compute warps' registers, its columns are free; both: ordered behind dV(i)
                    ok = issue_s(it + 1, 0, false);
                    if (!ok) break;
                }
                ok = mbar_wait(ds_ready, it & 1, abort_flag, p.guard, status_word(DKDV_WIDE_KERNEL_ID, ROLE_MMA, it));
                if (!ok) break;
                tc_fence_after_sync();
                if (elect_one()) {                     // dK += dS^T Q   (Q read MN-major, all boxes)
                    const uint64_t dQm = smem_desc_sw128(smem_u32(sQ + sl * TILE64_BYTES), BOX64_BYTES, 1024);
#pragma unroll
                    for (int k = 0; k < WIDE_N / 16; ++k)
                        umma_ts(tmem_u + acc_k, tmem_u + 64 + k * 8, desc_advance(dQm, k * 2048), IDESC_G, (it > 0 || k > 0) ? 1u : 0u);
                    umma_commit(&q_empty[sl]);
                    if (it == n_it - 1) umma_commit(final_bar);
                }
                __syncwarp();
                if (it + 1 < n_it) ok = issue_dp(it + 1, !has_dv);     // overwrites dS^T(i): ordered behind dK(i)
            }
        }
    } else if (warp >= 4) {
        // compute: P^T, dS^T (fragment-shaped tensor-memory accesses, see vt_ptx.cuh); epilogue
        const int quad = warp & 3;
        const int r = quad * 32 + lane;            // key row inside the tile (TMEM lane)
        const int kv = k0 + r;
        const uint32_t lane_addr = static_cast<uint32_t>(quad * 32) << 16;
        const uint32_t tDP = tmem_base + lane_addr + 64;
        const float2 c2 = make_float2(p.scale_log2e, p.scale_log2e);
        const int cq = 2 * (lane & 3);
        const int kv_row = k0 + quad * 32 + (lane >> 2);
        bool ok = true;
        int qi = 0;
        for (int it = 0; it < n_it; ++it, qi = (qi + 1 == n_qi) ? 0 : qi + 1) {
            const int q0 = (qt_start + qi) * WIDE_N;
            const int rsl = it % RS;
            const float *rows = s_rows + rsl * (2 * WIDE_N);
            const int buf = is_dv ? (it & 1) : 0;
            const uint32_t tS = tmem_base + lane_addr + buf * WIDE_N;
            ok = mbar_wait(&rows_full[rsl], (it / RS) & 1, abort_flag, p.guard, status_word(DKDV_WIDE_KERNEL_ID, ROLE_SOFTMAX, it));
            if (!ok) break;
            ok = mbar_wait(&s_full[buf], (is_dv ? (it >> 1) : it) & 1, abort_flag, p.guard, status_word(DKDV_WIDE_KERNEL_ID, ROLE_SOFTMAX, it));
            if (!ok) break;
            tc_fence_after_sync();
            const bool diag = CAUSAL && (q0 + off < k0 + TILE - 1);
            float2 nl[8];
#pragma unroll
            for (int g = 0; g < 8; ++g) nl[g] = *reinterpret_cast<const float2 *>(&rows[8 * g + cq]);
            float2 pr[2][8][2];
            uint32_t sv[2][32];
#pragma unroll
            for (int h = 0; h < 2; ++h) tmem_ld_frag64(tS + (static_cast<uint32_t>(h * 16) << 16), sv[h]);
            tmem_wait_ld();
            if (!has_dv) {                         // dK block: the scores are in registers, the next ones may overwrite their columns
                tc_fence_before_sync();
                mbar_arrive(p_ready);
            }
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                uint32_t pp[16];
#pragma unroll
                for (int g = 0; g < 8; ++g) {
#pragma unroll
                    for (int rr = 0; rr < 2; ++rr) {
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
                if (has_dv) tmem_st_frag32(tS + (static_cast<uint32_t>(h * 16) << 16), pp);
            }
            if (has_dv) {
                tmem_wait_st();
                tc_fence_before_sync();
                mbar_arrive(&p_ready[buf]);
            }
            if (has_dk) {
#pragma unroll
                for (int g = 0; g < 8; ++g) nl[g] = *reinterpret_cast<const float2 *>(&rows[WIDE_N + 8 * g + cq]);   // now -delta
                ok = mbar_wait(dp_full, it & 1, abort_flag, p.guard, status_word(DKDV_WIDE_KERNEL_ID, ROLE_SOFTMAX, it));
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
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&rows_empty[rsl]);
        }
        // epilogue: this block's tensor(s), all their columns
        const size_t key_row = static_cast<size_t>(bh_kv) * p.Sk + kv;
        if (n_it == 0) {
            if (kv < Sk) {
                if (has_dv) for (int i = 0; i < dv_w / 8; ++i) reinterpret_cast<uint4 *>(p.dv + key_row * dv_w)[i] = make_uint4(0, 0, 0, 0);
                if (has_dk) for (int i = 0; i < p.d / 8; ++i) reinterpret_cast<uint4 *>(p.dk + key_row * p.d)[i] = make_uint4(0, 0, 0, 0);
            }
        } else {
            if (ok) ok = mbar_wait(final_bar, 0, abort_flag, p.guard, status_word(DKDV_WIDE_KERNEL_ID, ROLE_EPILOGUE, 0));
            if (ok) {
                tc_fence_after_sync();
                uint8_t *scratch = sQ + (warp - 4) * STORE_SCRATCH_BYTES;     // every product has completed: the Q slots are free
                const int row0 = k0 + quad * 32;
                const int rows_valid = min(32, Sk - row0);
#pragma unroll
                for (int t = 0; t < 2; ++t) {                                  // t = 0: dV, 1: dK
                    if (t == 0 ? !has_dv : !has_dk) continue;                  // block-uniform
                    const int w_out = (t == 0) ? dv_w : p.d;
                    const size_t stride = static_cast<size_t>(w_out);
                    __nv_bfloat16 *warp_dst = (t == 0 ? p.dv : p.dk) + key_row * stride - static_cast<size_t>(lane) * stride;
                    const uint32_t tSrc = tmem_base + lane_addr + (t == 0 ? 128u : acc_k);
                    const float mul = (t == 0) ? 1.0f : p.scale;
#pragma unroll
                    for (int c = 0; c < WIDE_D / 32; ++c) {
                        if (c * 32 >= w_out) break;                        // block-uniform
                        uint32_t v[32];
                        tmem_ld32(tSrc + c * 32, v);
                        tmem_wait_ld();
                        store_rows16<F16>(warp_dst + c * 32, stride, v, mul, rows_valid, scratch, lane, w_out - c * 32);
                    }
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
// dQ, query tile stationary
// ----------------------------------------------------------------------------------------------
struct DqWideSmem {
    static constexpr int OFF_Q = 0;
    static constexpr int OFF_DO = OFF_Q + TILE128_BYTES;
    static constexpr int OFF_K = OFF_DO + TILE128_BYTES;             // [2] tiles of 64 keys
    static constexpr int OFF_V = OFF_K + 2 * TILE64_BYTES;           // [1]
    static constexpr int OFF_BAR = OFF_V + TILE64_BYTES;
    static constexpr int BYTES = OFF_BAR + 256;
    // TMEM columns: S [0,64), dP [64,128) (dS, bf16, over its first 32), dQ [128,384)
    static constexpr int TMEM_COLS = 512;
};

template <bool CAUSAL, bool F16>
__global__ void __launch_bounds__(WIDE_THREADS, 1)
bwd_dq_wide_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do, const BwdParams p)
{
    using L = DqWideSmem;
    extern __shared__ __align__(1024) uint8_t smem_wide[];
    uint8_t *smem = smem_wide;
    uint8_t *sQ = smem + L::OFF_Q;
    uint8_t *sdO = smem + L::OFF_DO;
    uint8_t *sK = smem + L::OFF_K;
    uint8_t *sV = smem + L::OFF_V;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L::OFF_BAR);
    uint64_t *qdo_full = bars + 0;
    uint64_t *final_bar = bars + 1;
    uint64_t *s_full = bars + 2;
    uint64_t *dp_full = bars + 3;
    uint64_t *ds_ready = bars + 4;            // 128 arrivals
    uint64_t *k_full = bars + 5;              // [2]
    uint64_t *k_empty = bars + 7;             // [2]
    uint64_t *v_full = bars + 9;
    uint64_t *v_empty = bars + 10;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 11);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    if ((smem_u32(smem_wide) & 1023u) != 0u) {
        if (threadIdx.x == 0) atomicCAS(p.guard.status, 0u, status_word(DQ_WIDE_KERNEL_ID, ROLE_LOAD, 0xFFFE));
        return;
    }

    const int bh = blockIdx.x / p.n_tiles;
    int qt = blockIdx.x % p.n_tiles;
    if (CAUSAL) qt = p.n_tiles - 1 - qt;                   // long (late) tiles first
    const int b = bh / p.Hq;
    const int h = bh % p.Hq;
    const int bh_kv = b * p.Hkv + h / p.G;
    const int q0 = qt * TILE;
    const int Sq = p.Sq, Sk = p.Sk;
    const int off = (CAUSAL && p.bottom_right) ? Sk - Sq : 0;
    int n_it = (Sk + WIDE_N - 1) / WIDE_N;                 // steps of 64 keys
    if (CAUSAL) n_it = (q0 + TILE - 1 + off < 0) ? 0 : min(n_it, (q0 + TILE - 1 + off) / WIDE_N + 1);
    const int kd = (p.d + 15) >> 4;                                   // contraction steps of S = Q K^T (and N / 16 of dQ)
    const int kdv = ((p.d_v > 0 ? p.d_v : p.d) + 15) >> 4;             // of dP = dO V^T

    if (threadIdx.x == 0) {
        mbar_init(qdo_full, 1);
        mbar_init(final_bar, 1);
        mbar_init(s_full, 1);
        mbar_init(dp_full, 1);
        mbar_init(ds_ready, 128);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&k_full[s], 1);
            mbar_init(&k_empty[s], 1);
        }
        mbar_init(v_full, 1);
        mbar_init(v_empty, 1);
        *abort_flag = 0u;
        fence_mbar_init();
        prefetch_tensormap(&tm_q);
        prefetch_tensormap(&tm_do);
        prefetch_tensormap(&tm_k);
        mbar_arrive_expect_tx(qdo_full, 2 * TILE128_BYTES);
        for (int kb = 0; kb < WIDE_BOXES; ++kb) {
            tma_load_3d(sQ + kb * BOX128_BYTES, &tm_q, qdo_full, kb * BOX_COLS, q0, bh);
            tma_load_3d(sdO + kb * BOX128_BYTES, &tm_do, qdo_full, kb * BOX_COLS, q0, bh);
        }
        if (n_it > 0) {
            mbar_arrive_expect_tx(&k_full[0], TILE64_BYTES);
            for (int kb = 0; kb < WIDE_BOXES; ++kb) tma_load_3d(sK + kb * BOX64_BYTES, &tm_k, &k_full[0], kb * BOX_COLS, 0, bh_kv);
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

    if (warp == 0) {
        if (lane == 0) {                           // K tiles (Q, dO and the first one went out before the block-wide sync)
            for (int j = 1; j < n_it; ++j) {
                const int sl = j & 1;
                if (!mbar_wait(&k_empty[sl], ((j >> 1) & 1) ^ 1, abort_flag, p.guard, status_word(DQ_WIDE_KERNEL_ID, ROLE_LOAD, j))) break;
                mbar_arrive_expect_tx(&k_full[sl], TILE64_BYTES);
                for (int kb = 0; kb < WIDE_BOXES; ++kb)
                    tma_load_3d(sK + sl * TILE64_BYTES + kb * BOX64_BYTES, &tm_k, &k_full[sl], kb * BOX_COLS, j * WIDE_N, bh_kv);
            }
        }
    } else if (warp == 2) {
        if (lane == 0) {                           // V tiles: one slot
            prefetch_tensormap(&tm_v);
            for (int j = 0; j < n_it; ++j) {
                if (!mbar_wait(v_empty, (j & 1) ^ 1, abort_flag, p.guard, status_word(DQ_WIDE_KERNEL_ID, ROLE_LOAD, j))) break;
                mbar_arrive_expect_tx(v_full, TILE64_BYTES);
                for (int kb = 0; kb < WIDE_BOXES; ++kb) tma_load_3d(sV + kb * BOX64_BYTES, &tm_v, v_full, kb * BOX_COLS, j * WIDE_N, bh_kv);
            }
        }
    } else if (warp == 1) {
        // MMA issuer.  Per step: dQ(j), S(j+1), dP(j+1).
        constexpr uint32_t IDESC_S = make_idesc(128, WIDE_N, fmt16<F16>(), fmt16<F16>(), 0, 0);
        const uint32_t IDESC_G = make_idesc(128, kd * 16, fmt16<F16>(), fmt16<F16>(), 0, 1);     // N = the head dimension, up to 256
        const uint32_t tmem_u = __shfl_sync(0xFFFFFFFFu, tmem_base, 0);
        const uint64_t dQ0 = smem_desc_sw128(smem_u32(sQ), 16, 1024), dDO0 = smem_desc_sw128(smem_u32(sdO), 16, 1024);
        bool ok = mbar_wait(qdo_full, 0, abort_flag, p.guard, status_word(DQ_WIDE_KERNEL_ID, ROLE_MMA, 0xFFFF));
        if (n_it == 0) ok = false;
        auto issue_s = [&](int j) -> bool {        // S = Q K^T
            const int sl = j & 1;
            if (!mbar_wait(&k_full[sl], (j >> 1) & 1, abort_flag, p.guard, status_word(DQ_WIDE_KERNEL_ID, ROLE_MMA, j))) return false;
            tc_fence_after_sync();
            if (elect_one()) {
                const uint64_t dKs = smem_desc_sw128(smem_u32(sK + sl * TILE64_BYTES), 16, 1024);
#pragma unroll
                for (int k = 0; k < WIDE_D / 16; ++k)
                    if (k < kd)
                        umma_ss(tmem_u, desc_advance(dQ0, (k / 4) * BOX128_BYTES + (k % 4) * 32),
                                desc_advance(dKs, (k / 4) * BOX64_BYTES + (k % 4) * 32), IDESC_S, k > 0 ? 1u : 0u);
                umma_commit(s_full);
            }
            __syncwarp();
            return true;
        };
        auto issue_dp = [&](int j) -> bool {       // dP = dO V^T
            if (!mbar_wait(v_full, j & 1, abort_flag, p.guard, status_word(DQ_WIDE_KERNEL_ID, ROLE_MMA, j))) return false;
            tc_fence_after_sync();
            if (elect_one()) {
                const uint64_t dVs = smem_desc_sw128(smem_u32(sV), 16, 1024);
#pragma unroll
                for (int k = 0; k < WIDE_D / 16; ++k)
                    if (k < kdv)
                        umma_ss(tmem_u + 64, desc_advance(dDO0, (k / 4) * BOX128_BYTES + (k % 4) * 32),
                                desc_advance(dVs, (k / 4) * BOX64_BYTES + (k % 4) * 32), IDESC_S, k > 0 ? 1u : 0u);
                umma_commit(dp_full);
                umma_commit(v_empty);
            }
            __syncwarp();
            return true;
        };
        if (ok) ok = issue_s(0);
        if (ok) ok = issue_dp(0);
        for (int j = 0; j < n_it && ok; ++j) {
            const int sl = j & 1;
            ok = mbar_wait(ds_ready, j & 1, abort_flag, p.guard, status_word(DQ_WIDE_KERNEL_ID, ROLE_MMA, j));
            if (!ok) break;
            tc_fence_after_sync();
            if (elect_one()) {                     // dQ += dS K   (K read MN-major over all its column boxes)
                const uint64_t dKm = smem_desc_sw128(smem_u32(sK + sl * TILE64_BYTES), BOX64_BYTES, 1024);
#pragma unroll
                for (int k = 0; k < WIDE_N / 16; ++k)
                    umma_ts(tmem_u + 128, tmem_u + 64 + k * 8, desc_advance(dKm, k * 2048), IDESC_G, (j > 0 || k > 0) ? 1u : 0u);
                umma_commit(&k_empty[sl]);
                if (j == n_it - 1) umma_commit(final_bar);
            }
            __syncwarp();
            if (j + 1 < n_it) {
                ok = issue_s(j + 1);               // the scores of step j were read before dS(j) was signalled
                if (!ok) break;
                ok = issue_dp(j + 1);              // overwrites dS(j): ordered behind dQ(j)
            }
        }
    } else if (warp >= 4) {
        // compute: P (registers), dS; epilogue.  One thread per query row, 64 key columns per step.
        const int quad = warp & 3;
        const int r = quad * 32 + lane;
        const int row = q0 + r;
        const uint32_t lane_addr = static_cast<uint32_t>(quad * 32) << 16;
        const uint32_t tS = tmem_base + lane_addr;
        const uint32_t tDP = tmem_base + lane_addr + 64;
        float lse2 = INFINITY, dl = 0.0f;          // rows past the end: P = 0
        if (row < Sq && n_it > 0) {
            const size_t idx = static_cast<size_t>(bh) * p.Sq + row;
            lse2 = p.lse[idx] * LOG2E;
            dl = p.delta[idx];
        }
        const float2 c2 = make_float2(p.scale_log2e, p.scale_log2e);
        const float2 nl2 = make_float2(-lse2, -lse2);
        const float2 ndl2 = make_float2(-dl, -dl);
        bool ok = true;
        for (int j = 0; j < n_it; ++j) {
            ok = mbar_wait(s_full, j & 1, abort_flag, p.guard, status_word(DQ_WIDE_KERNEL_ID, ROLE_SOFTMAX, j));
            if (!ok) break;
            tc_fence_after_sync();
            const int c0 = j * WIDE_N;
            const bool need_mask = (c0 + WIDE_N > Sk) || (CAUSAL && (c0 + WIDE_N - 1 > q0 + off));
            int limit = Sk - c0;
            if (CAUSAL) limit = min(limit, row + off - c0 + 1);
            float2 pr[32];
            uint32_t sv[2][32];
            tmem_ld32(tS, sv[0]);
            tmem_ld32(tS + 32, sv[1]);
            tmem_wait_ld();
#pragma unroll
            for (int c = 0; c < 2; ++c) {
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
            ok = mbar_wait(dp_full, j & 1, abort_flag, p.guard, status_word(DQ_WIDE_KERNEL_ID, ROLE_SOFTMAX, j));
            if (!ok) break;
            tc_fence_after_sync();
            tmem_ld32(tDP, sv[0]);
            tmem_ld32(tDP + 32, sv[1]);
            tmem_wait_ld();
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t dd[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const float2 df = __fadd2_rn(make_float2(__uint_as_float(sv[c][2 * i]), __uint_as_float(sv[c][2 * i + 1])), ndl2);
                    const float2 ds = __fmul2_rn(pr[c * 16 + i], df);
                    dd[i] = pack16<F16>(ds.x, ds.y);
                }
                tmem_st16(tDP + c * 16, dd);
            }
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(ds_ready);
        }
        __nv_bfloat16 *dq_row = p.dq + (static_cast<size_t>(bh) * p.Sq + row) * p.d;
        if (n_it == 0) {
            if (row < Sq)
                for (int i = 0; i < p.d / 8; ++i) reinterpret_cast<uint4 *>(dq_row)[i] = make_uint4(0, 0, 0, 0);
            ok = false;
        }
        if (ok) ok = mbar_wait(final_bar, 0, abort_flag, p.guard, status_word(DQ_WIDE_KERNEL_ID, ROLE_EPILOGUE, 0));
        if (ok) {
            tc_fence_after_sync();
            uint8_t *scratch = sK + (warp - 4) * STORE_SCRATCH_BYTES;        // every product has completed: the K slots are free
            const size_t stride = static_cast<size_t>(p.d);
            __nv_bfloat16 *warp_dst = dq_row - static_cast<size_t>(lane) * stride;
            const int rows_valid = min(32, Sq - (q0 + quad * 32));
#pragma unroll
            for (int c = 0; c < WIDE_D / 32; ++c) {
                uint32_t v[32];
                tmem_ld32(tmem_base + lane_addr + 128 + c * 32, v);
                tmem_wait_ld();
                store_rows16<F16>(warp_dst + c * 32, stride, v, p.scale, rows_valid, scratch, lane, p.d - c * 32);
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

template <bool CAUSAL, bool F16>
static int launch_wide(const CUtensorMap &q64, const CUtensorMap &do64, const CUtensorMap &k128, const CUtensorMap &v128,
                       const CUtensorMap &q128, const CUtensorMap &do128, const CUtensorMap &k64, const CUtensorMap &v64, BwdParams prm,
                       const __nv_bfloat16 *o, const __nv_bfloat16 *d_o, float *delta, int B, cudaStream_t stream)
{
    static std::atomic<bool> configured[64];
    int dev = 0;
    cudaGetDevice(&dev);
    cudaError_t e;
    if (!configured[dev & 63].load(std::memory_order_acquire)) {
        e = cudaFuncSetAttribute(bwd_dkdv_wide_kernel<CAUSAL, F16>, cudaFuncAttributeMaxDynamicSharedMemorySize, DkdvWideSmem::BYTES);
        if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(dkdv wide)");
        e = cudaFuncSetAttribute(bwd_dq_wide_kernel<CAUSAL, F16>, cudaFuncAttributeMaxDynamicSharedMemorySize, DqWideSmem::BYTES);
        if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(dq wide)");
        configured[dev & 63].store(true, std::memory_order_release);
    }
    const long long n_rows = static_cast<long long>(B) * prm.Hq * prm.Sq;
    long long delta_blocks = (n_rows + 7) / 8;                         // 32 threads per row (d / 8 <= 32 pieces), 8 rows per block
    if (delta_blocks > NUM_SMS * 32) delta_blocks = NUM_SMS * 32;
    bwd_delta_kernel<32, F16><<<static_cast<int>(delta_blocks), 256, 0, stream>>>(o, d_o, delta, n_rows, 0, prm.d_v > 0 ? prm.d_v : prm.d);
    if ((e = cudaGetLastError()) != cudaSuccess) return cuda_fail(e, "bwd_delta_kernel launch");

    prm.n_tiles = (prm.Sk + TILE - 1) / TILE;
    // a dK block and a dV block per key tile; one block for both when the two accumulators (at most 192 columns each) fit
    // beside S^T and dP^T in tensor memory
    const int dv_cols = prm.d_v > 0 ? prm.d_v : prm.d;
    const dim3 grid_kv(static_cast<unsigned>(prm.n_tiles * B * prm.Hkv), (prm.d <= 192 && dv_cols <= 192) ? 1 : 2);
    bwd_dkdv_wide_kernel<CAUSAL, F16><<<grid_kv, WIDE_THREADS, DkdvWideSmem::BYTES, stream>>>(q64, k128, v128, do64, prm);
    if ((e = cudaGetLastError()) != cudaSuccess) return cuda_fail(e, "bwd_dkdv_wide_kernel launch");

    prm.n_tiles = (prm.Sq + TILE - 1) / TILE;
    bwd_dq_wide_kernel<CAUSAL, F16><<<prm.n_tiles * B * prm.Hq, WIDE_THREADS, DqWideSmem::BYTES, stream>>>(q128, k64, v64, do128, prm);
    if ((e = cudaGetLastError()) != cudaSuccess) return cuda_fail(e, "bwd_dq_wide_kernel launch");
    return VT_ATTN_OK;
}

int launch_bwd_wide(bool f16, const void *q, const void *k, const void *v, const void *o, const void *d_o, BwdParams prm, float *delta,
                    int B, int causal, cudaStream_t stream)
{
    int rc;
    CUtensorMap q64, do64, k128, v128, q128, do128, k64, v64;
    const int D = prm.d, Dv = prm.d_v > 0 ? prm.d_v : prm.d, Sq = prm.Sq, Sk = prm.Sk;
    if ((rc = make_tensor_map(&q64, q, B * prm.Hq, Sq, D, WIDE_N)) != VT_ATTN_OK) return rc;
    if ((rc = make_tensor_map(&do64, d_o, B * prm.Hq, Sq, Dv, WIDE_N)) != VT_ATTN_OK) return rc;
    if ((rc = make_tensor_map(&k128, k, B * prm.Hkv, Sk, D, TILE)) != VT_ATTN_OK) return rc;
    if ((rc = make_tensor_map(&v128, v, B * prm.Hkv, Sk, Dv, TILE)) != VT_ATTN_OK) return rc;
    if ((rc = make_tensor_map(&q128, q, B * prm.Hq, Sq, D, TILE)) != VT_ATTN_OK) return rc;
    if ((rc = make_tensor_map(&do128, d_o, B * prm.Hq, Sq, Dv, TILE)) != VT_ATTN_OK) return rc;
    if ((rc = make_tensor_map(&k64, k, B * prm.Hkv, Sk, D, WIDE_N)) != VT_ATTN_OK) return rc;
    if ((rc = make_tensor_map(&v64, v, B * prm.Hkv, Sk, Dv, WIDE_N)) != VT_ATTN_OK) return rc;
    const __nv_bfloat16 *o_ = static_cast<const __nv_bfloat16 *>(o), *do_ = static_cast<const __nv_bfloat16 *>(d_o);
    if (f16)
        return causal ? launch_wide<true, true>(q64, do64, k128, v128, q128, do128, k64, v64, prm, o_, do_, delta, B, stream)
                      : launch_wide<false, true>(q64, do64, k128, v128, q128, do128, k64, v64, prm, o_, do_, delta, B, stream);
    return causal ? launch_wide<true, false>(q64, do64, k128, v128, q128, do128, k64, v64, prm, o_, do_, delta, B, stream)
                  : launch_wide<false, false>(q64, do64, k128, v128, q128, do128, k64, v64, prm, o_, do_, delta, B, stream);
}

}  // namespace vt
