// Backward in FIVE tile products: one key-tile-stationary kernel that forms dV, dK and the key tile's share of dQ.
//
// bwd_dkdv_kernel + bwd_dq_kernel compute S and dP twice (7 products of 128 x 128 x 128 per (query tile, key tile)
// pair for the 5 that the gradients need) because each keeps its outputs with a single owner block.  Here the block of a
// key tile also multiplies dS by its K tile and adds the 128 x D partial result into a [B, Hq, Sq, D] accumulator that
// all key-tile blocks of a head share.  The accumulator holds 32-bit FIXED-POINT integers: integer addition is
// associative, so the red.add operations of different blocks may land in any order and the sum is still the same bits
// on every run - the reduction over key tiles is deterministic without turnstiles, a launch order to respect or a block
// that waits for another.  A conversion pass turns the sums into the 16-bit dQ.
//
// Fixed-point scale.  For every query row, sum_j |dS_ij| <= max_j |dP_ij| + |Delta_i| <= 2 |dO_i| max_j |V_j| (the
// probabilities of a row sum to one; Cauchy-Schwarz), so |sum_j dS_ij K_j[c]| <= R = 2 max_i |dO_i| max_j |V_j| max |K|
// per (batch, query head).  The three maxima are taken by the Delta pass and a pass over K and V; the contributions
// are scaled by the power of two that maps 2 R (a factor two of head-room for the rounding of P and dS) to 2^29 and
// rounded to the nearest integer: one unit is R * 2^-28, i.e. ~1e-8 of the bound, three orders of magnitude below the
// bf16 rounding that dS itself carries.  No partial sum can overflow (the bound holds for any subset of the keys).
//
// Tensor memory is full (S^T, dP^T, dV, dK at 128 columns each), so the dQ partial result takes the place of dP^T as
// soon as the compute warps hold dP^T in registers, and a fourth warpgroup drains it (tcgen05.ld, scale, convert,
// red.global.add.s32) while the tensor core already works on the next products.  dS^T goes to SHARED memory (a
// 128-byte-swizzled 128 x 128 bf16 tile): it is the B operand of dQ^T = K^T dS^T and the A operand of dK += dS^T Q.
// dQ is produced transposed (head dimension on the TMEM lanes, queries on the columns) so that a warp's 32 lanes add
// into 128 contiguous bytes of an accumulator row.
//
// Block = 512 threads: warp 0 / 2 TMA producers (Q, dO), warp 1 MMA issuer, warp 3 row-vector producer, warps 4..11 two
// compute warpgroups, warps 12..15 the drain warpgroup.  D = 128 only (other head dimensions up to 128 run in it with
// zero columns); the two-kernel path remains for D <= 64, packed batches and small problems.
#pragma once

namespace vt {

constexpr int FUSED_THREADS = 512;
// Registers per thread after the roles split (setmaxnreg): 128 * producers + 256 * compute + 128 * drain <= 65536.
#ifndef VT_FUSED_COMPUTE_REGS
#define VT_FUSED_COMPUTE_REGS 128
#define VT_FUSED_DRAIN_REGS 144
#define VT_FUSED_PRODUCER_REGS 104
#endif
constexpr uint32_t FUSED_KERNEL_ID = 8;
constexpr int DQ_FIXED_BITS = 28;              // |contribution sums| * scale < 2^29 (see dq_fixed_scale)

// Power of two that maps the bound R (|dQ column sums| <= R before the softmax scale) to < 2^28; 1 when R is 0 or not finite.
__host__ __device__ __forceinline__ float dq_fixed_scale(float R)
{
    if (!(R > 0.0f) || !(R < 3.0e38f)) return 1.0f;
    int e;
    frexpf(R, &e);                              // R = m * 2^e, 0.5 <= m < 1, so R < 2^e
    return ldexpf(1.0f, DQ_FIXED_BITS - e);
}

struct FusedParams {
    int *dq_acc;                // [B, Hq, Sq, d] fixed-point sums, zero on entry
    const float *qscale;        // [B * Hq]: multiplier from dS K (fp32) to accumulator units
};

template <int D>
struct FusedSmem {
    static constexpr int TILE_BYTES = TILE * D * 2;
    static constexpr int OFF_K = 0;
    static constexpr int OFF_V = OFF_K + TILE_BYTES;
    static constexpr int OFF_Q = OFF_V + TILE_BYTES;                 // [2]
    static constexpr int OFF_DO = OFF_Q + 2 * TILE_BYTES;            // [2]
    static constexpr int OFF_DS = OFF_DO + 2 * TILE_BYTES;           // dS^T: 128 keys x 128 queries, bf16, two 64-column boxes
    static constexpr int DS_BYTES = TILE * TILE * 2;
    static constexpr int ROW_SLOTS = 2;
    static constexpr int OFF_ROWS = OFF_DS + DS_BYTES;
    static constexpr int OFF_BAR = OFF_ROWS + ROW_SLOTS * 2 * TILE * 4;
    static constexpr int BYTES = OFF_BAR + 256;                      // no alignment slack: the kernel checks the base address
    static constexpr int TMEM_COLS = 512;                            // S^T/P^T [0,128) dP^T/dQ^T [128,256) dV [256,384) dK [384,512)
};

template <int D, bool CAUSAL, bool F16 = false>
__global__ void __launch_bounds__(FUSED_THREADS, 1)
bwd_fused_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                 const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do, const BwdParams p,
                 const FusedParams fp)
{
    static_assert(D == 128, "the fused backward is built for 128 columns");
    using L = FusedSmem<D>;
    constexpr int NBOX = D / BOX_COLS;
    constexpr int BOX_BYTES = TILE * BOX_COLS * 2;           // 16 KB: a 64-column box of a 128-row tile
    constexpr int RS = L::ROW_SLOTS;

    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t *smem = smem_raw;
    uint8_t *sK = smem + L::OFF_K;
    uint8_t *sV = smem + L::OFF_V;
    uint8_t *sQ = smem + L::OFF_Q;
    uint8_t *sdO = smem + L::OFF_DO;
    uint8_t *sDS = smem + L::OFF_DS;
    float *s_rows = reinterpret_cast<float *>(smem + L::OFF_ROWS);     // [slot][-lse2 128 | -delta 128]
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L::OFF_BAR);
    uint64_t *kv_full = bars + 0;
    uint64_t *final_bar = bars + 1;
    uint64_t *s_full = bars + 2;              // S^T of the iteration is complete
    uint64_t *dp_full = bars + 3;             // dP^T of the iteration is complete (and dQ, dK of the one before)
    uint64_t *p_ready = bars + 4;             // 256 arrivals: P^T written to tensor memory
    uint64_t *ds_ready = bars + 5;            // 256 arrivals: dS^T written to shared memory, dP^T read out
    uint64_t *dq_full = bars + 6;             // the dQ^T partial result of the iteration is complete
    uint64_t *b_free = bars + 7;              // 128 arrivals: the drain warps hold it in registers
    uint64_t *q_full = bars + 8;              // [2]
    uint64_t *q_empty = bars + 10;            // [2]
    uint64_t *do_full = bars + 12;            // [2]
    uint64_t *do_empty = bars + 14;           // [2]
    uint64_t *rows_full = bars + 16;          // [RS] 32 arrivals
    uint64_t *rows_empty = bars + 16 + RS;    // [RS] one arrival per compute warp
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 16 + 2 * RS);
    volatile uint32_t *abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    // The swizzled tiles need a 1024-byte aligned base and there is no room left for slack: leave at once if the
    // dynamic shared memory does not start on such a boundary (it does on every driver seen so far).
    if ((smem_u32(smem_raw) & 1023u) != 0u) {
        if (threadIdx.x == 0) atomicCAS(p.guard.status, 0u, status_word(FUSED_KERNEL_ID, ROLE_LOAD, 0xFFFE));
        return;
    }

    const int bh_kv = blockIdx.x / p.n_tiles;
    const int kt = blockIdx.x % p.n_tiles;
    const int b = bh_kv / p.Hkv;
    const int hkv = bh_kv % p.Hkv;
    const int k0 = kt * TILE;
    const int Sq = p.Sq, Sk = p.Sk;
    const int n_qt = (Sq + TILE - 1) / TILE;
    const int off = (CAUSAL && p.bottom_right) ? Sk - Sq : 0;            // causal: query i sees the keys j <= i + off
    const int qt_start = CAUSAL ? min(max(k0 - off, 0) / TILE, n_qt) : 0;   // first query tile that can see this key tile
    const int n_qi = n_qt - qt_start;
    const int n_it = n_qi * p.G;                                         // iterations: heads of the group x query tiles

    if (threadIdx.x == 0) {
        mbar_init(kv_full, 1);
        mbar_init(final_bar, 1);
        mbar_init(s_full, 1);
        mbar_init(dp_full, 1);
        mbar_init(p_ready, 256);
        mbar_init(ds_ready, 256);
        mbar_init(dq_full, 1);
        mbar_init(b_free, 128);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&q_full[s], 1);
            mbar_init(&q_empty[s], 1);
            mbar_init(&do_full[s], 1);
            mbar_init(&do_empty[s], 1);
        }
        for (int s = 0; s < RS; ++s) {
            mbar_init(&rows_full[s], 32);
            mbar_init(&rows_empty[s], 8);
        }
        *abort_flag = 0u;
        fence_mbar_init();
        prefetch_tensormap(&tm_q);
        prefetch_tensormap(&tm_k);
        prefetch_tensormap(&tm_v);
        mbar_arrive_expect_tx(kv_full, 2 * L::TILE_BYTES);
        for (int kb = 0; kb < NBOX; ++kb) {
            tma_load_3d(sK + kb * BOX_BYTES, &tm_k, kv_full, kb * BOX_COLS, k0, bh_kv);
            tma_load_3d(sV + kb * BOX_BYTES, &tm_v, kv_full, kb * BOX_COLS, k0, bh_kv);
        }
        if (n_it > 0) {
            mbar_arrive_expect_tx(&q_full[0], L::TILE_BYTES);
            for (int kb = 0; kb < NBOX; ++kb)
                tma_load_3d(sQ + kb * BOX_BYTES, &tm_q, &q_full[0], kb * BOX_COLS, qt_start * TILE, b * p.Hq + hkv * p.G);
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
    const uint32_t tmem_dK = tmem_base + 384;

    if (warp < 4) {
        setmaxnreg_dec<VT_FUSED_PRODUCER_REGS>();
        if (warp == 0) {
            // ------------------------------------------------------------------ TMA producer: the Q tiles
            if (lane == 0) {
                for (int it = 1; it < n_it; ++it) {
                    const int sl = it & 1;
                    const int hq = hkv * p.G + it / n_qi;
                    const int q0 = (qt_start + it % n_qi) * TILE;
                    if (!mbar_wait(&q_empty[sl], ((it >> 1) & 1) ^ 1, abort_flag, p.guard, status_word(FUSED_KERNEL_ID, ROLE_LOAD, it))) break;
                    mbar_arrive_expect_tx(&q_full[sl], L::TILE_BYTES);
                    for (int kb = 0; kb < NBOX; ++kb)
                        tma_load_3d(sQ + sl * L::TILE_BYTES + kb * BOX_BYTES, &tm_q, &q_full[sl], kb * BOX_COLS, q0, b * p.Hq + hq);
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
                    if (!mbar_wait(&do_empty[sl], ((it >> 1) & 1) ^ 1, abort_flag, p.guard, status_word(FUSED_KERNEL_ID, ROLE_LOAD, it))) break;
                    mbar_arrive_expect_tx(&do_full[sl], L::TILE_BYTES);
                    for (int kb = 0; kb < NBOX; ++kb)
                        tma_load_3d(sdO + sl * L::TILE_BYTES + kb * BOX_BYTES, &tm_do, &do_full[sl], kb * BOX_COLS, q0, b * p.Hq + hq);
                }
            }
        } else if (warp == 3) {
            // ------------------------------------------------------------------ row-vector producer: -LSE (log2 units), -Delta
            for (int it = 0; it < n_it; ++it) {
                const int sl = it % RS;
                if (!mbar_wait(&rows_empty[sl], ((it / RS) & 1) ^ 1, abort_flag, p.guard, status_word(FUSED_KERNEL_ID, ROLE_LOAD, it))) break;
                const int hq = hkv * p.G + it / n_qi;
                const int q0 = (qt_start + it % n_qi) * TILE;
                const size_t head = (static_cast<size_t>(b) * p.Hq + hq) * p.Sq;
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
        } else {
            // ------------------------------------------------------------------ MMA issuer
            // Per iteration: dV(i), S(i+1), dQ(i), dK(i), dP(i+1).  S(i+1) runs while the compute warps still work on dS(i);
            // dQ(i) goes first of the two products that need dS(i) so that the drain of its result hides behind dK(i), and
            // dP(i+1) - which reuses the dQ columns - finds them free.
            constexpr uint32_t IDESC_S = make_idesc(128, 128, fmt16<F16>(), fmt16<F16>(), 0, 0);
            constexpr uint32_t IDESC_G = make_idesc(128, D, fmt16<F16>(), fmt16<F16>(), 0, 1);      // B operand MN-major
            constexpr uint32_t IDESC_Q = make_idesc(128, 128, fmt16<F16>(), fmt16<F16>(), 1, 1);    // both operands MN-major
            const uint32_t tmem_u = __shfl_sync(0xFFFFFFFFu, tmem_base, 0);    // provably warp-uniform copy
            const uint64_t dK0 = smem_desc_sw128(smem_u32(sK), 16, 1024), dV0 = smem_desc_sw128(smem_u32(sV), 16, 1024);
            const uint64_t dKm = smem_desc_sw128(smem_u32(sK), BOX_BYTES, 1024);      // K with the head dimension as M
            const uint64_t dDSk = smem_desc_sw128(smem_u32(sDS), 16, 1024);           // dS^T, queries as the K dimension
            const uint64_t dDSm = smem_desc_sw128(smem_u32(sDS), BOX_BYTES, 1024);    // dS^T, queries as N
            bool ok = mbar_wait(kv_full, 0, abort_flag, p.guard, status_word(FUSED_KERNEL_ID, ROLE_MMA, 0xFFFF));
            auto issue_s = [&](int it) -> bool {       // S^T = K Q^T
                const int sl = it & 1;
                if (!mbar_wait(&q_full[sl], (it >> 1) & 1, abort_flag, p.guard, status_word(FUSED_KERNEL_ID, ROLE_MMA, it))) return false;
                tc_fence_after_sync();
                if (elect_one()) {
                    const uint64_t dQs = smem_desc_sw128(smem_u32(sQ + sl * L::TILE_BYTES), 16, 1024);
#pragma unroll
                    for (int k = 0; k < D / 16; ++k) {
                        const uint32_t o = (k / 4) * BOX_BYTES + (k % 4) * 32;
                        umma_ss(tmem_u, desc_advance(dK0, o), desc_advance(dQs, o), IDESC_S, k > 0 ? 1u : 0u);
                    }
                    umma_commit(s_full);
                }
                __syncwarp();
                return true;
            };
            auto issue_dp = [&](int it) -> bool {      // dP^T = V dO^T
                const int sl = it & 1;
                if (!mbar_wait(&do_full[sl], (it >> 1) & 1, abort_flag, p.guard, status_word(FUSED_KERNEL_ID, ROLE_MMA, it))) return false;
                tc_fence_after_sync();
                if (elect_one()) {
                    const uint64_t dDOs = smem_desc_sw128(smem_u32(sdO + sl * L::TILE_BYTES), 16, 1024);
#pragma unroll
                    for (int k = 0; k < D / 16; ++k) {
                        const uint32_t o = (k / 4) * BOX_BYTES + (k % 4) * 32;
                        umma_ss(tmem_u + 128, desc_advance(dV0, o), desc_advance(dDOs, o), IDESC_S, k > 0 ? 1u : 0u);
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
                ok = mbar_wait(p_ready, it & 1, abort_flag, p.guard, status_word(FUSED_KERNEL_ID, ROLE_MMA, it));
                if (!ok) break;
                tc_fence_after_sync();
                if (elect_one()) {                     // dV += P^T dO   (dO read MN-major: 16 query rows per instruction)
                    const uint64_t dDOm = smem_desc_sw128(smem_u32(sdO + sl * L::TILE_BYTES), BOX_BYTES, 1024);
#pragma unroll
                    for (int k = 0; k < TILE / 16; ++k)
                        umma_ts(tmem_u + 256, tmem_u + a_col(k), desc_advance(dDOm, k * 2048), IDESC_G, (it > 0 || k > 0) ? 1u : 0u);
                    umma_commit(&do_empty[sl]);
                }
                __syncwarp();
                if (it + 1 < n_it) {
                    ok = issue_s(it + 1);              // overwrites P^T(it): ordered behind dV(it)
                    if (!ok) break;
                }
                ok = mbar_wait(ds_ready, it & 1, abort_flag, p.guard, status_word(FUSED_KERNEL_ID, ROLE_MMA, it));
                if (!ok) break;
                tc_fence_after_sync();
                if (elect_one()) {
                    // dQ^T(it) = K^T dS^T over the columns dP^T occupied (the compute warps hold dP^T in registers)
#pragma unroll
                    for (int k = 0; k < TILE / 16; ++k)
                        umma_ss(tmem_u + 128, desc_advance(dKm, k * 2048), desc_advance(dDSm, k * 2048), IDESC_Q, k > 0 ? 1u : 0u);
                    umma_commit(dq_full);
                    // dK += dS^T Q   (dS^T from shared memory, Q read MN-major)
                    const uint64_t dQm = smem_desc_sw128(smem_u32(sQ + sl * L::TILE_BYTES), BOX_BYTES, 1024);
#pragma unroll
                    for (int k = 0; k < TILE / 16; ++k) {
                        const uint32_t o = (k / 4) * BOX_BYTES + (k % 4) * 32;
                        umma_ss(tmem_u + 384, desc_advance(dDSk, o), desc_advance(dQm, k * 2048), IDESC_G, (it > 0 || k > 0) ? 1u : 0u);
                    }
                    umma_commit(&q_empty[sl]);
                    if (it == n_it - 1) umma_commit(final_bar);
                }
                __syncwarp();
                if (it + 1 < n_it) {
                    ok = mbar_wait(b_free, it & 1, abort_flag, p.guard, status_word(FUSED_KERNEL_ID, ROLE_MMA, it));
                    if (!ok) break;
                    tc_fence_after_sync();
                    ok = issue_dp(it + 1);             // into the drained dQ columns; its completion also says dK(it) is done
                }
            }
        }
    } else if (warp < 12) {
        // ------------------------------------------------------------------ compute: P^T -> tensor memory, dS^T -> shared memory; epilogue
        setmaxnreg_inc<VT_FUSED_COMPUTE_REGS>();
        const int wg = (warp - 4) >> 2;            // warpgroup g takes query columns [64 g, 64 g + 64) of each tile
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
        // dS^T in shared memory: box `wg` (64 query columns = one 128-byte row per key), 128-byte swizzle: the 16-byte chunk
        // g of key row r sits at chunk g ^ (r & 7); this thread's rows all have r & 7 == lane >> 2
        uint8_t *ds_base = sDS + wg * BOX_BYTES + (quad * 32 + (lane >> 2)) * 128 + 4 * (lane & 3);
        const int sw = lane >> 2;
        bool ok = true;
        int qi = 0;                                // query tile of the iteration inside its head (it % n_qi, without the division)
        for (int it = 0; it < n_it; ++it, qi = (qi + 1 == n_qi) ? 0 : qi + 1) {
            const int q0 = (qt_start + qi) * TILE + wg * WG_COLS;          // first query column of this warpgroup
            const int rsl = it % RS;
            const float *rows = s_rows + rsl * (2 * TILE) + wg * WG_COLS;  // -lse2 of this warpgroup's columns; -delta at + TILE
            ok = mbar_wait(&rows_full[rsl], (it / RS) & 1, abort_flag, p.guard, status_word(FUSED_KERNEL_ID, ROLE_SOFTMAX, it));
            if (!ok) break;
            ok = mbar_wait(s_full, it & 1, abort_flag, p.guard, status_word(FUSED_KERNEL_ID, ROLE_SOFTMAX, it));
            if (!ok) break;
            tc_fence_after_sync();
            const bool diag = CAUSAL && (q0 + off < k0 + TILE - 1);    // some (key, query) pairs here are masked
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
            // dP^T(it) complete also means dQ(it-1) and dK(it-1) are: the dS^T tile in shared memory may be overwritten
            ok = mbar_wait(dp_full, it & 1, abort_flag, p.guard, status_word(FUSED_KERNEL_ID, ROLE_SOFTMAX, it));
            if (!ok) break;
            tc_fence_after_sync();
#pragma unroll
            for (int h = 0; h < 2; ++h) tmem_ld_frag64(tDP + (static_cast<uint32_t>(h * 16) << 16), sv[h]);
            tmem_wait_ld();
#pragma unroll
            for (int h = 0; h < 2; ++h) {
#pragma unroll
                for (int g = 0; g < 8; ++g) {
#pragma unroll
                    for (int rr = 0; rr < 2; ++rr) {
                        const float2 df = __fadd2_rn(make_float2(__uint_as_float(sv[h][4 * g + 2 * rr]), __uint_as_float(sv[h][4 * g + 2 * rr + 1])), nl[g]);
                        const float2 ds = __fmul2_rn(pr[h][g][rr], df);
                        *reinterpret_cast<uint32_t *>(ds_base + (16 * h + 8 * rr) * 128 + ((g ^ sw) << 4)) = pack16<F16>(ds.x, ds.y);
                    }
                }
            }
            fence_proxy_async_smem();              // the MMAs read the tile through the async proxy
            tc_fence_before_sync();                // and the dP^T columns, read above, get overwritten by the next product
            mbar_arrive(ds_ready);
            __syncwarp();
            if (lane == 0) mbar_arrive(&rows_empty[rsl]);      // every lane of this warp has read the slot's values
        }
        // epilogue: warpgroup 0 writes dV, warpgroup 1 dK
        const bool is_dv = wg == 0;
        __nv_bfloat16 *out_row = (is_dv ? p.dv : p.dk) + (static_cast<size_t>(bh_kv) * p.Sk + kv) * p.d;
        const bool store = kv < Sk;
        if (n_it == 0) {
            if (store)
                for (int i = 0; i < p.d / 8; ++i) reinterpret_cast<uint4 *>(out_row)[i] = make_uint4(0, 0, 0, 0);
        } else {
            if (ok) ok = mbar_wait(final_bar, 0, abort_flag, p.guard, status_word(FUSED_KERNEL_ID, ROLE_EPILOGUE, 0));
            if (ok) {
                tc_fence_after_sync();
                const uint32_t tSrc = (is_dv ? tmem_dV : tmem_dK) + lane_addr;
                const float mul = is_dv ? 1.0f : p.scale;
                uint8_t *scratch = sQ + (warp - 4) * STORE_SCRATCH_BYTES;     // every MMA has completed: the Q tiles are free
                const int row0 = k0 + quad * 32;
                const size_t stride = static_cast<size_t>(p.d);
                __nv_bfloat16 *warp_dst = out_row - static_cast<size_t>(lane) * stride;
                const int rows_valid = min(32, Sk - row0);
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t v[32];
                    tmem_ld32(tSrc + c * 32, v);
                    tmem_wait_ld();
                    store_rows16<F16>(warp_dst + c * 32, stride, v, mul, rows_valid, scratch, lane, p.d - c * 32);
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ drain: dQ^T partial results -> fixed-point accumulator
        setmaxnreg_inc<VT_FUSED_DRAIN_REGS>();
        const int quad = warp & 3;
        const int dcol = quad * 32 + lane;         // head-dimension index (TMEM lane)
        const uint32_t tDQ = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + 128;
        bool ok = true;
        int qi = 0, hq = hkv * p.G;
        float qs = (n_it > 0) ? fp.qscale[b * p.Hq + hq] : 1.0f;
        for (int it = 0; it < n_it && ok; ++it) {
            ok = mbar_wait(dq_full, it & 1, abort_flag, p.guard, status_word(FUSED_KERNEL_ID, ROLE_EPILOGUE, it));
            if (!ok) break;
            tc_fence_after_sync();
            uint32_t v[4][32];
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld32(tDQ + c * 32, v[c]);
            tmem_wait_ld();
            tc_fence_before_sync();
            mbar_arrive(b_free);
            const int q0 = (qt_start + qi) * TILE;
            int *dst = fp.dq_acc + ((static_cast<size_t>(b) * p.Hq + hq) * p.Sq + q0) * p.d + dcol;
            const int n_valid = min(TILE, Sq - q0);                // query rows of this tile that exist
            if (dcol < p.d) {
#pragma unroll
                for (int c = 0; c < 4; ++c) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        if (c * 32 + i < n_valid) {
                            const int iv = __float2int_rn(__uint_as_float(v[c][i]) * qs);
                            asm volatile("red.global.add.s32 [%0], %1;" ::"l"(dst + static_cast<size_t>(c * 32 + i) * p.d), "r"(iv) : "memory");
                        }
                    }
                }
            }
            if (++qi == n_qi) {
                qi = 0;
                ++hq;
                if (it + 1 < n_it) qs = fp.qscale[b * p.Hq + hq];
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
// The passes around it
// ----------------------------------------------------------------------------------------------
// Non-negative floats compare like their bit patterns, and max is associative and commutative: atomicMax on the bits
// gives the same result in any order.
__device__ __forceinline__ void atomic_max_nonneg(float *addr, float v) { atomicMax(reinterpret_cast<unsigned int *>(addr), __float_as_uint(v)); }

// max over the rows of |dO_i|^2 per (batch, query head): stats[bh].  One warp per row at a time.
template <bool F16>
__global__ void __launch_bounds__(256) bwd_do_norm_kernel(const __nv_bfloat16 *__restrict__ d_o, float *__restrict__ stats, int Sq, int d, long long n_rows)
{
    const int lane = threadIdx.x & 31;
    const long long warp0 = (static_cast<long long>(blockIdx.x) * 256 + threadIdx.x) >> 5;
    const long long n_warps = (static_cast<long long>(gridDim.x) * 256) >> 5;
    for (long long row = warp0; row < n_rows; row += n_warps) {
        float acc = 0.0f;
        for (int c = lane * 8; c < d; c += 256) {
            const uint4 a = *reinterpret_cast<const uint4 *>(d_o + row * d + c);
            const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 f = unpack16<F16>(w[i]);
                acc = fmaf(f.x, f.x, acc);
                acc = fmaf(f.y, f.y, acc);
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
        if (lane == 0) atomic_max_nonneg(&stats[row / Sq], acc);
    }
}

// max_j |V_j|^2 and max |K| per (batch, KV head): stats_v[bh_kv], stats_k[bh_kv].
template <bool F16>
__global__ void __launch_bounds__(256) bwd_kv_norm_kernel(const __nv_bfloat16 *__restrict__ k, const __nv_bfloat16 *__restrict__ v,
                                                          float *__restrict__ stats_k, float *__restrict__ stats_v, int Sk, int d, long long n_rows)
{
    const int lane = threadIdx.x & 31;
    const long long warp0 = (static_cast<long long>(blockIdx.x) * 256 + threadIdx.x) >> 5;
    const long long n_warps = (static_cast<long long>(gridDim.x) * 256) >> 5;
    for (long long row = warp0; row < n_rows; row += n_warps) {
        float vv = 0.0f, kk = 0.0f;
        for (int c = lane * 8; c < d; c += 256) {
            const uint4 a = *reinterpret_cast<const uint4 *>(v + row * d + c);
            const uint4 bq = *reinterpret_cast<const uint4 *>(k + row * d + c);
            const uint32_t w[4] = {a.x, a.y, a.z, a.w};
            const uint32_t u[4] = {bq.x, bq.y, bq.z, bq.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 f = unpack16<F16>(w[i]);
                vv = fmaf(f.x, f.x, vv);
                vv = fmaf(f.y, f.y, vv);
                const float2 g = unpack16<F16>(u[i]);
                kk = fmaxf(kk, fmaxf(fabsf(g.x), fabsf(g.y)));
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            vv += __shfl_xor_sync(0xFFFFFFFFu, vv, o);
            kk = fmaxf(kk, __shfl_xor_sync(0xFFFFFFFFu, kk, o));
        }
        if (lane == 0) {
            atomic_max_nonneg(&stats_v[row / Sk], vv);
            atomic_max_nonneg(&stats_k[row / Sk], kk);
        }
    }
}

// qscale[bh] from the three maxima.
__global__ void bwd_qscale_kernel(const float *__restrict__ stats_do, const float *__restrict__ stats_k, const float *__restrict__ stats_v,
                                  float *__restrict__ qscale, int n_bh, int Hq, int Hkv)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_bh) return;
    const int b = i / Hq, h = i % Hq;
    const int kvh = b * Hkv + h / (Hq / Hkv);
    const float R = 2.0f * sqrtf(stats_do[i]) * sqrtf(stats_v[kvh]) * stats_k[kvh];
    qscale[i] = dq_fixed_scale(2.0f * R);            // a factor two of head-room for the rounded P and dS
}

// dQ (16-bit) = accumulator / qscale * softmax scale.  Eight elements per thread.
template <bool F16>
__global__ void __launch_bounds__(256) bwd_dq_convert_kernel(const int *__restrict__ acc, const float *__restrict__ qscale,
                                                             __nv_bfloat16 *__restrict__ dq, long long n_vec, long long vec_per_head, float scale)
{
    for (long long i = static_cast<long long>(blockIdx.x) * 256 + threadIdx.x; i < n_vec; i += static_cast<long long>(gridDim.x) * 256) {
        const float mul = scale / qscale[i / vec_per_head];
        const int4 a = *reinterpret_cast<const int4 *>(acc + i * 8);
        const int4 c = *reinterpret_cast<const int4 *>(acc + i * 8 + 4);
        uint4 w;
        w.x = pack16<F16>(static_cast<float>(a.x) * mul, static_cast<float>(a.y) * mul);
        w.y = pack16<F16>(static_cast<float>(a.z) * mul, static_cast<float>(a.w) * mul);
        w.z = pack16<F16>(static_cast<float>(c.x) * mul, static_cast<float>(c.y) * mul);
        w.w = pack16<F16>(static_cast<float>(c.z) * mul, static_cast<float>(c.w) * mul);
        *reinterpret_cast<uint4 *>(dq + i * 8) = w;
    }
}

}  // namespace vt
