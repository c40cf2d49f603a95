// Definitions shared by the backward kernels (bwd.cu: the 64- and 128-column kernels and the single-pass kernel;
// bwd_wide.cu: head dimensions above 128): the Delta pass, the parameter block, the probability helper.
#pragma once

#include "vt_host.h"

namespace vt {

#ifndef VT_BWD_WGS
#define VT_BWD_WGS 2
#endif
constexpr int BWD_WGS = VT_BWD_WGS;                 // compute warpgroups; each takes TILE / BWD_WGS columns of a 128x128 tile
constexpr int WG_COLS = TILE / BWD_WGS;             // 32 or 64
constexpr int WG_CHUNKS = WG_COLS / 32;
constexpr int BWD_THREADS = 128 + 128 * BWD_WGS;
constexpr uint32_t DKDV_KERNEL_ID = 2;
constexpr uint32_t DQ_KERNEL_ID = 3;
constexpr float LOG2E = 1.4426950408889634f;


// ----------------------------------------------------------------------------------------------
// 1. Delta
// ----------------------------------------------------------------------------------------------
// packed_hq > 0: o and d_o are [total_q, Hq, d], so row = token * Hq + h, and Delta is laid out [Hq, total_q].
// TPR threads per row (a power of two >= d / 8), 8 elements (16 bytes) each; the threads past the row's end add zero.
template <int TPR, bool F16 = false>
__global__ void __launch_bounds__(256) bwd_delta_kernel(const __nv_bfloat16 *__restrict__ o,
                                                        const __nv_bfloat16 *__restrict__ d_o,
                                                        float *__restrict__ delta, long long n_rows, int packed_hq, int d)
{
    constexpr int ROWS_PER_BLOCK = 256 / TPR;
    const int sub = threadIdx.x % TPR;
    for (long long row = static_cast<long long>(blockIdx.x) * ROWS_PER_BLOCK + threadIdx.x / TPR; row < n_rows;
         row += static_cast<long long>(gridDim.x) * ROWS_PER_BLOCK) {
        float acc = 0.0f;
        if (sub * 8 < d) {
            const uint4 a = *reinterpret_cast<const uint4 *>(o + row * d + sub * 8);
            const uint4 b = *reinterpret_cast<const uint4 *>(d_o + row * d + sub * 8);
            const uint32_t aw[4] = {a.x, a.y, a.z, a.w};
            const uint32_t bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 fa = unpack16<F16>(aw[i]);
                const float2 fb = unpack16<F16>(bw[i]);
                acc = fmaf(fa.x, fb.x, acc);
                acc = fmaf(fa.y, fb.y, acc);
            }
        }
#pragma unroll
        for (int off = TPR / 2; off > 0; off >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, off);
        if (sub == 0) {
            const long long out = (packed_hq > 0) ? (row % packed_hq) * (n_rows / packed_hq) + row / packed_hq : row;
            delta[out] = acc;
        }
    }
}

// ----------------------------------------------------------------------------------------------
// shared bits of the two MMA kernels
// ----------------------------------------------------------------------------------------------
struct BwdParams {
    const float *lse;       // [B,Hq,Sq] natural log
    const float *delta;     // [B,Hq,Sq]
    __nv_bfloat16 *dq, *dk, *dv;
    int Hq, Hkv, G, Sq, Sk;
    int d;                  // head dimension of the tensors in global memory (<= the kernels' D; the columns between read as zero)
    int d_v = 0;            // bwd_wide.cu only: head dimension of V, O, dO, dV when it differs from that of Q, K, dQ, dK (0: the same)
    int n_tiles;            // tiles per head along the block's stationary dimension (of the longest sequence)
    float scale, scale_log2e;
    const int *cu_q;        // packed batches only: cumulative sequence lengths [n_seqs + 1], device
    const int *cu_k;
    int total_q;            // packed batches only: tokens in q
    int bottom_right;       // causal only: key j is visible to query i iff j <= i + Sk - Sq (else iff j <= i)
    int head_group;         // causal dQ kernel only: heads per scheduling group (see causal_work_item)
    Guard guard;
};

// TMEM column (relative to the 128-column tile) of the k-th group of 16 bf16 values of a tile that the compute
// warpgroups wrote, each at the start of its own WG_COLS columns: 8 columns per group, WG_COLS / 16 groups per warpgroup.
__device__ __forceinline__ constexpr uint32_t a_col(int k) { return (k / (WG_COLS / 16)) * WG_COLS + (k % (WG_COLS / 16)) * 8; }

// P = exp2(s * c - lse2) for a pair of scores; a share of the pairs (by position) goes to the FMA-pipe cubic
// so that the eight compute warps, which all take their exponentials at the same time, do not queue on the MUFU.
#ifndef VT_BWD_POLY
#define VT_BWD_POLY 2
#endif
constexpr int BWD_POLY_EIGHTHS = VT_BWD_POLY;
__device__ __forceinline__ float2 prob_pair(int i, float2 x)
{
    if ((i & 7) < BWD_POLY_EIGHTHS) return exp2_poly2(x);
    float2 e;
    e.x = fast_exp2(x.x);
    e.y = fast_exp2(x.y);
    return e;
}

// bwd_wide.cu: the backward for head dimensions in (128, 256], batched layout.  prm holds everything but n_tiles and
// delta's contents; delta: B * Hq * Sq floats of scratch.
int launch_bwd_wide(bool f16, const void *q, const void *k, const void *v, const void *o, const void *d_o, BwdParams prm, float *delta,
                    int B, int causal, cudaStream_t stream);

}  // namespace vt
