// Forward kernel for causal (top-left aligned) sequences of moderate length: the one-tile kernel of fwd_kernel.cuh run
// over TWO query tiles of a head, one after the other, by the same block - the long tile n-1-i first, then the short tile
// i - so that every block of a head does the same amount of work (n + 1 tiles' worth of key steps) and the second
// tile's start-up (Q and K loads, the first two S = Q K^T products) runs behind the first tile's last steps and epilogue
// instead of in a fresh block.  Under a causal mask a head's tiles take 1 .. n key tiles; with one block per tile the
// short ones are mostly start-up and drain.
// The roles, the tensor-memory layout (two S buffers of 64 columns, O in [128,128+D), two blocks per SM) and the per-step
// protocol are those of attn_fwd_kernel; barrier phases and ring slots simply keep counting across the two tiles.
// Included by fwd.cu.
#pragma once
#include "fwd_kernel.cuh"

namespace vt {

constexpr uint32_t DUO_KERNEL_ID = 5;

template <int D>
struct DuoSmem {
    using F = FwdSmem<D>;
    static constexpr int OFF_SCRATCH = F::OFF_BAR + F::BAR_BYTES;      // the epilogue's store transpose (Q's memory is reloaded meanwhile)
    static constexpr int BYTES = OFF_SCRATCH + 4 * STORE_SCRATCH_BYTES + 1024;
};

// p.n_qt: query tiles per head; the grid has ceil(n_qt / 2) blocks per head.
template <int D, bool F16 = false>
__global__ void __launch_bounds__(FWD_THREADS, 2)
attn_fwd_duo_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, const FwdParams p)
{
    using L = FwdSmem<D>;
    constexpr int SL = L::KV_SLOTS;
    constexpr int NBOX = D / BOX_COLS;
    constexpr int QBOX_BYTES = TILE * BOX_COLS * 2;
    constexpr int KBOX_BYTES = BN * BOX_COLS * 2;
    constexpr int POLY_EIGHTHS = (D == 64) ? 1 : 0;

    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *sQ = smem + L::OFF_Q;
    uint8_t *sK = smem + L::OFF_K;
    uint8_t *sV = smem + L::OFF_V;
    uint8_t *s_scratch = smem + DuoSmem<D>::OFF_SCRATCH;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + L::OFF_BAR);
    uint64_t *q_full = bars + 0;             // one phase per tile
    uint64_t *o_final = bars + 1;            // one phase per tile
    uint64_t *pv_done = bars + 2;            // one phase per step
    uint64_t *s_full = bars + 3;             // [2]
    uint64_t *p_ready = bars + 5;            // [2]
    uint64_t *k_full = bars + 7;             // [SL]
    uint64_t *k_empty = bars + 7 + SL;       // [SL]
    uint64_t *v_full = bars + 7 + 2 * SL;    // [SL]
    uint64_t *v_empty = bars + 7 + 3 * SL;   // [SL]
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 7 + 4 * SL);
    volatile uint32_t *abort_flag = tmem_slot + 1;
    uint64_t *q_empty = bars + 8 + 4 * SL;   // every S product of the tile has completed: Q's memory may be reloaded
    uint64_t *o_free = bars + 9 + 4 * SL;    // 128 arrivals: the tile's O has been read out of tensor memory

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    const int n_pairs = (p.n_qt + 1) / 2;
    const int bh = blockIdx.x / n_pairs;
    const int pr = blockIdx.x % n_pairs;
    const int b = bh / p.Hq;
    const int h = bh % p.Hq;
    const int bh_kv = b * (p.Hq / p.G) + h / p.G;
    const int Sq = p.Sq, Sk = p.Sk;
    // the two tiles of this block: the long one first; a head with an odd number of tiles has one block with a single tile
    const int qt_of[2] = {p.n_qt - 1 - pr, pr};
    const int n_pass = (qt_of[0] == qt_of[1]) ? 1 : 2;
    int nt_of[2];
#pragma unroll
    for (int ps = 0; ps < 2; ++ps) nt_of[ps] = min((Sk + BN - 1) / BN, (qt_of[ps] * TILE + TILE - 1) / BN + 1);     // >= 1: key 0 is visible to every row

    constexpr int PRODUCER_THREAD = 4 * 32;
    const int n_pre = min(nt_of[0], SL);
    if (threadIdx.x == PRODUCER_THREAD) {
        mbar_init(q_full, 1);
        mbar_init(o_final, 1);
        mbar_init(pv_done, 1);
        mbar_init(q_empty, 1);
        mbar_init(o_free, 128);
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
        prefetch_tensormap(&tm_q);
        prefetch_tensormap(&tm_k);
        mbar_arrive_expect_tx(q_full, L::Q_BYTES);
        for (int kb = 0; kb < NBOX; ++kb) tma_load_3d(sQ + kb * QBOX_BYTES, &tm_q, q_full, kb * BOX_COLS, qt_of[0] * TILE, bh);
        for (int t = 0; t < n_pre; ++t) {
            mbar_arrive_expect_tx(&k_full[t], L::KV_BYTES);
            for (int kb = 0; kb < NBOX; ++kb) tma_load_3d(sK + t * L::KV_BYTES + kb * KBOX_BYTES, &tm_k, &k_full[t], kb * BOX_COLS, t * BN, bh_kv);
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
                bool ok = true;
                int g0 = 0;                                   // steps before this tile (ring slots and phases keep counting)
                for (int ps = 0; ps < n_pass && ok; ++ps) {
                    if (ps > 0) {
                        // the previous tile's S products are complete: its Q may be overwritten
                        ok = mbar_wait(q_empty, (ps - 1) & 1, abort_flag, p.guard, status_word(DUO_KERNEL_ID, ROLE_LOAD, 0xFFFF));
                        if (!ok) break;
                        mbar_arrive_expect_tx(q_full, L::Q_BYTES);
                        for (int kb = 0; kb < NBOX; ++kb) tma_load_3d(sQ + kb * QBOX_BYTES, &tm_q, q_full, kb * BOX_COLS, qt_of[ps] * TILE, bh);
                    }
                    for (int t = (ps == 0 ? n_pre : 0); t < nt_of[ps]; ++t) {
                        const int g = g0 + t, sl = g % SL;
                        if (!mbar_wait(&k_empty[sl], ((g / SL) & 1) ^ 1, abort_flag, p.guard, status_word(DUO_KERNEL_ID, ROLE_LOAD, g))) { ok = false; break; }
                        mbar_arrive_expect_tx(&k_full[sl], L::KV_BYTES);
                        for (int kb = 0; kb < NBOX; ++kb)
                            tma_load_3d(sK + sl * L::KV_BYTES + kb * KBOX_BYTES, &tm_k, &k_full[sl], kb * BOX_COLS, t * BN, bh_kv);
                    }
                    g0 += nt_of[ps];
                }
            }
        } else if (warp == 6) {
            // -------------------------------------------------------------- TMA producer: V
            if (lane == 0) {
                prefetch_tensormap(&tm_v);
                bool ok = true;
                int g0 = 0;
                for (int ps = 0; ps < n_pass && ok; ++ps) {
                    for (int t = 0; t < nt_of[ps]; ++t) {
                        const int g = g0 + t, sl = g % SL;
                        if (!mbar_wait(&v_empty[sl], ((g / SL) & 1) ^ 1, abort_flag, p.guard, status_word(DUO_KERNEL_ID, ROLE_LOAD, g))) { ok = false; break; }
                        mbar_arrive_expect_tx(&v_full[sl], L::KV_BYTES);
                        for (int kb = 0; kb < NBOX; ++kb)
                            tma_load_3d(sV + sl * L::KV_BYTES + kb * KBOX_BYTES, &tm_v, &v_full[sl], kb * BOX_COLS, t * BN, bh_kv);
                    }
                    g0 += nt_of[ps];
                }
            }
        } else if (warp == 5) {
            // -------------------------------------------------------------- MMA issuer
            constexpr uint32_t IDESC_QK = make_idesc(128, BN, fmt16<F16>(), fmt16<F16>(), 0, 0);
            // a head dimension below D (the columns past it are zero): the products skip the 16-column blocks that hold
            // nothing - fewer contraction steps for S, a narrower N for O
            const int kd = (p.d_qk + 15) >> 4;
            const uint32_t IDESC_PV = make_idesc(128, ((p.d + 15) >> 4) * 16, fmt16<F16>(), fmt16<F16>(), 0, 1);
            const uint32_t tmem_u = __shfl_sync(0xFFFFFFFFu, tmem_base, 0);
            const uint64_t dQ0 = smem_desc_sw128(smem_u32(sQ), 16, 1024);
            bool ok = true;
            int g0 = 0;
            for (int ps = 0; ps < n_pass && ok; ++ps) {
                const int n_t = nt_of[ps];
                ok = mbar_wait(q_full, ps & 1, abort_flag, p.guard, status_word(DUO_KERNEL_ID, ROLE_MMA, 0xFFFF));
                if (!ok) break;
                // S = Q K_t^T into S buffer g & 1; the tile's last one also releases Q
                auto issue_qk = [&](int t) -> bool {
                    const int g = g0 + t, sl = g % SL;
                    if (!mbar_wait(&k_full[sl], (g / SL) & 1, abort_flag, p.guard, status_word(DUO_KERNEL_ID, ROLE_MMA, g))) return false;
                    tc_fence_after_sync();
                    if (elect_one()) {
                        const uint64_t dK0 = smem_desc_sw128(smem_u32(sK + sl * L::KV_BYTES), 16, 1024);
                        const uint32_t tS = tmem_u + (g & 1) * BN;
#pragma unroll
                        for (int k = 0; k < D / 16; ++k)
                            if (k < kd)
                                umma_ss(tS, desc_advance(dQ0, (k / 4) * QBOX_BYTES + (k % 4) * 32),
                                        desc_advance(dK0, (k / 4) * KBOX_BYTES + (k % 4) * 32), IDESC_QK, k > 0 ? 1u : 0u);
                        umma_commit(&k_empty[sl]);
                        umma_commit(&s_full[g & 1]);
                        if (t == n_t - 1) umma_commit(q_empty);
                    }
                    __syncwarp();
                    return true;
                };
                ok = issue_qk(0);
                if (ok && n_t > 1) ok = issue_qk(1);
                for (int t = 0; t < n_t && ok; ++t) {
                    const int g = g0 + t, sl = g % SL;
                    ok = mbar_wait(&v_full[sl], (g / SL) & 1, abort_flag, p.guard, status_word(DUO_KERNEL_ID, ROLE_MMA, g));
                    if (!ok) break;
                    ok = mbar_wait(&p_ready[g & 1], (g >> 1) & 1, abort_flag, p.guard, status_word(DUO_KERNEL_ID, ROLE_MMA, g));
                    if (!ok) break;
                    if (ps > 0 && t == 0) {
                        // the first product of this tile overwrites O: the previous tile's epilogue must have read it
                        ok = mbar_wait(o_free, (ps - 1) & 1, abort_flag, p.guard, status_word(DUO_KERNEL_ID, ROLE_MMA, 0xFFFE));
                        if (!ok) break;
                    }
                    tc_fence_after_sync();
                    if (elect_one()) {
                        const uint64_t dV0 = smem_desc_sw128(smem_u32(sV + sl * L::KV_BYTES), KBOX_BYTES, 1024);
                        const uint32_t tP = tmem_u + (g & 1) * BN;
#pragma unroll
                        for (int k = 0; k < BN / 16; ++k)
                            umma_ts(tmem_u + 128, tP + k * 8, desc_advance(dV0, k * 2048), IDESC_PV, (t > 0 || k > 0) ? 1u : 0u);
                        umma_commit(&v_empty[sl]);
                        umma_commit(pv_done);
                        if (t == n_t - 1) umma_commit(o_final);
                    }
                    __syncwarp();
                    if (t + 2 < n_t) ok = issue_qk(t + 2);      // overwrites P of step g: ordered behind the product just issued
                }
                g0 += n_t;
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax + epilogue
        setmaxnreg_inc<SOFTMAX_REGS>();
        const int r = warp * 32 + lane;
        const uint32_t lane_addr = static_cast<uint32_t>(warp * 32) << 16;
        const float c = p.scale_log2e;
        bool ok = true;
        int g0 = 0;
        for (int ps = 0; ps < n_pass && ok; ++ps) {
            const int n_t = nt_of[ps];
            const int q0 = qt_of[ps] * TILE;
            const int row = q0 + r;
            float m_used = -INFINITY;
            float l = 0.0f;
            for (int t = 0; t < n_t; ++t) {
                const int g = g0 + t;
                const uint32_t tS = tmem_base + lane_addr + (g & 1) * BN;
                ok = mbar_wait(&s_full[g & 1], (g >> 1) & 1, abort_flag, p.guard, status_word(DUO_KERNEL_ID, ROLE_SOFTMAX, g));
                if (!ok) break;
                tc_fence_after_sync();
                uint32_t sr[2][32];
                tmem_ld32(tS, sr[0]);
                tmem_ld32(tS + 32, sr[1]);
                tmem_wait_ld();
                const int c0 = t * BN;
                const bool need_mask = (c0 + BN > Sk) || (c0 + BN - 1 > q0);
                if (need_mask) {
                    const int limit = min(Sk - c0, row - c0 + 1);      // columns >= limit are masked
#pragma unroll
                    for (int cc = 0; cc < 2; ++cc)
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (cc * 32 + i >= limit) sr[cc][i] = 0xFF800000u;   // -inf
                }
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
                    const bool moved = (m_new - m_used) * c > RESCALE_THRESHOLD;
                    if (__any_sync(0xFFFFFFFFu, moved)) {
                        // O must hold every product issued so far: wait for the product of step g - 1
                        ok = mbar_wait(pv_done, (g - 1) & 1, abort_flag, p.guard, status_word(DUO_KERNEL_ID, ROLE_SOFTMAX, g));
                        if (!ok) break;
                        tc_fence_after_sync();
                        const float alpha = fast_exp2((m_used - m_new) * c);
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
                const float2 c2 = make_float2(c, c);
                const float neg_m = -m_used * c;
                const float2 nm2 = make_float2(neg_m, neg_m);
                float2 acc[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
                for (int cc = 0; cc < 2; ++cc) {
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const float2 x = __ffma2_rn(make_float2(__uint_as_float(sr[cc][2 * i]), __uint_as_float(sr[cc][2 * i + 1])), c2, nm2);
                        float2 e;
                        if ((i & 7) < POLY_EIGHTHS) {
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
                mbar_arrive(&p_ready[g & 1]);
            }
            if (!ok) break;
            // epilogue of this tile (while it runs, the next tile's Q and K loads and first two S products proceed)
            ok = mbar_wait(o_final, ps & 1, abort_flag, p.guard, status_word(DUO_KERNEL_ID, ROLE_EPILOGUE, ps));
            if (!ok) break;
            tc_fence_after_sync();
            const float inv_l = 1.0f / l;
            __nv_bfloat16 *orow_g = p.o + (static_cast<size_t>(bh) * p.Sq + row) * p.d;
            const int rows_valid = min(32, Sq - q0 - warp * 32);
            uint32_t orow[D / 32][32];
#pragma unroll
            for (int cc = 0; cc < D / 32; ++cc) tmem_ld32(tmem_O + lane_addr + cc * 32, orow[cc]);
            tmem_wait_ld();
            if (ps + 1 < n_pass) {                 // O is in registers: the next tile's first product may overwrite it
                tc_fence_before_sync();
                mbar_arrive(o_free);
            }
#pragma unroll
            for (int cc = 0; cc < D / 32; ++cc)
                store_rows16<F16>(orow_g - static_cast<size_t>(lane) * p.d + cc * 32, p.d, orow[cc], inv_l, rows_valid,
                                  s_scratch + warp * STORE_SCRATCH_BYTES, lane, p.d - cc * 32);
            if (row < Sq) p.lse[static_cast<size_t>(bh) * p.Sq + row] = (m_used * c + log2f(l)) * 0.6931471805599453f;
            g0 += n_t;
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

template <int D, bool F16>
static int launch_fwd_duo(const CUtensorMap &tq, const CUtensorMap &tk, const CUtensorMap &tv, const FwdParams &prm,
                          int n_blocks, cudaStream_t stream)
{
    static std::atomic<bool> configured[64];     // set-up is idempotent: two threads may both do it, neither may read a torn flag
    int dev = 0;
    cudaGetDevice(&dev);
    if (!configured[dev & 63].load(std::memory_order_acquire)) {
        cudaError_t e = cudaFuncSetAttribute(attn_fwd_duo_kernel<D, F16>, cudaFuncAttributeMaxDynamicSharedMemorySize, DuoSmem<D>::BYTES);
        if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute(fwd duo)");
        configured[dev & 63].store(true, std::memory_order_release);
    }
    attn_fwd_duo_kernel<D, F16><<<n_blocks, FWD_THREADS, DuoSmem<D>::BYTES, stream>>>(tq, tk, tv, prm);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "attn_fwd_duo_kernel launch");
    return VT_ATTN_OK;
}

}  // namespace vt
