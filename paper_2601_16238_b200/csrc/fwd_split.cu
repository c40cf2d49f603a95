// Split-KV forward for low-occupancy shapes (few query tiles against many keys: decoding, small-batch prefill).
// The key steps are cut into chunks; one block per (batch, head or KV group, query tile, chunk) runs the forward kernel
// over its chunk and writes a normalised fp32 partial result with its own LSE; a merge kernel combines the chunks:
//   LSE = ln sum_s exp(LSE_s),   O = sum_s exp(LSE_s - LSE) * O_s.
// When the Sq queries of all G heads of a KV group fit one 128-row tile, the group shares a tile (row = head * Sq + query)
// and K / V are walked once per group instead of once per head.
#include "fwd_kernel.cuh"

namespace vt {

constexpr int MAX_SPLITS = 128;

// One thread per 4 output columns; the D / 4 threads of a row each recompute the row's weights (n_splits values).
// The partial results have D columns per row (the kernels' column count), the output tensor d <= D.
template <int D, bool F16 = false>
__global__ void __launch_bounds__(256) fwd_merge_kernel(const float *__restrict__ o_part, const float *__restrict__ lse_part,
                                                        __nv_bfloat16 *__restrict__ o, float *__restrict__ lse, long long n_rows,
                                                        int n_splits, int d, int packed_hq)
{
    constexpr int TPR = D / 4;
    constexpr int ROWS_PER_BLOCK = 256 / TPR;
    const int sub = threadIdx.x % TPR;
    for (long long row = static_cast<long long>(blockIdx.x) * ROWS_PER_BLOCK + threadIdx.x / TPR; row < n_rows;
         row += static_cast<long long>(gridDim.x) * ROWS_PER_BLOCK) {
        float m = -INFINITY;
        for (int s = 0; s < n_splits; ++s) m = fmaxf(m, lse_part[s * n_rows + row]);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float sum = 0.0f;
        if (m != -INFINITY) {
            for (int s = 0; s < n_splits; ++s) {
                const float w = __expf(lse_part[s * n_rows + row] - m);       // exp(-inf) = 0 for an empty chunk
                const float4 v = *reinterpret_cast<const float4 *>(o_part + (s * n_rows + row) * D + sub * 4);
                sum += w;
                acc.x = fmaf(w, v.x, acc.x);
                acc.y = fmaf(w, v.y, acc.y);
                acc.z = fmaf(w, v.z, acc.z);
                acc.w = fmaf(w, v.w, acc.w);
            }
        }
        const float inv = (sum > 0.0f) ? 1.0f / sum : 0.0f;                    // no visible key at all: O = 0, LSE = -inf
        uint2 w2;
        w2.x = pack16<F16>(acc.x * inv, acc.y * inv);
        w2.y = pack16<F16>(acc.z * inv, acc.w * inv);
        if (sub * 4 < d) *reinterpret_cast<uint2 *>(o + row * d + sub * 4) = w2;
        // packed batches: the rows are token * Hq + head, the LSE tensor is [Hq, total_q]
        const long long lrow = (packed_hq > 0) ? (row % packed_hq) * (n_rows / packed_hq) + row / packed_hq : row;
        if (sub == 0) lse[lrow] = (sum > 0.0f) ? m + logf(sum) : -INFINITY;
    }
}

static bool heads_share_a_tile(int G, int Sq) { return G > 1 && G * Sq <= TILE; }

// Number of chunks for a shape when the caller leaves the choice to the library: as many as keep all blocks in one wave
// (two blocks per SM on 148 SMs; measured best on decoding and chunked-prefill shapes - a second, partial wave costs more
// than the extra parallelism gains), at least 8 steps (512 keys) per chunk: below that a block's fixed cost and the merge
// outweigh the gain.
static int auto_splits(long long base_blocks, int n_steps)
{
    long long want = (2 * NUM_SMS) / base_blocks;
    const long long cap = n_steps / 8 > 0 ? n_steps / 8 : 1;
    if (want > cap) want = cap;
    if (want > MAX_SPLITS) want = MAX_SPLITS;
    return want < 1 ? 1 : static_cast<int>(want);
}

struct SplitPlan {
    int n_splits, chunk_steps, hpack;
    long long base_blocks;
};

static SplitPlan plan_split(int B, int Hq, int Hkv, int Sq, int Sk, int n_splits)
{
    SplitPlan pl;
    const int G = Hq / Hkv;
    pl.hpack = heads_share_a_tile(G, Sq) ? 1 : 0;
    const int n_qt = (Sq + TILE - 1) / TILE;
    pl.base_blocks = pl.hpack ? static_cast<long long>(B) * Hkv : static_cast<long long>(B) * Hq * n_qt;
    const int n_steps = (Sk + BN - 1) / BN;
    if (n_splits <= 0) n_splits = auto_splits(pl.base_blocks, n_steps);
    if (n_splits > n_steps) n_splits = n_steps;
    pl.chunk_steps = (n_steps + n_splits - 1) / n_splits;
    pl.n_splits = (n_steps + pl.chunk_steps - 1) / pl.chunk_steps;      // no chunk is empty by construction
    return pl;
}

}  // namespace vt

static size_t round_up_256(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }

extern "C" size_t vt_attn_fwd_splitkv_workspace_bytes(int B, int Hq, int Hkv, int Sq, int Sk, int D, int n_splits)
{
    using namespace vt;
    Shape s{B, Hq, Hkv, Sq, Sk, D};
    if (check_shape(s, 1.0f, MAX_HEAD_DIM_FWD) != VT_ATTN_OK || n_splits < 0 || n_splits > MAX_SPLITS) return 0;
    const SplitPlan pl = plan_split(B, Hq, Hkv, Sq, Sk, n_splits);
    const size_t n_rows = static_cast<size_t>(B) * Hq * Sq;
    return round_up_256(static_cast<size_t>(pl.n_splits) * n_rows * padded_head_dim(D) * 4) + round_up_256(static_cast<size_t>(pl.n_splits) * n_rows * 4);
}

extern "C" int vt_attn_fwd_splitkv_plan(int B, int Hq, int Hkv, int Sq, int Sk, int D, int n_splits, int *splits_used,
                                        int *heads_share_tile)
{
    using namespace vt;
    Shape s{B, Hq, Hkv, Sq, Sk, D};
    int rc = check_shape(s, 1.0f, MAX_HEAD_DIM_FWD);
    if (rc != VT_ATTN_OK) return rc;
    if (n_splits < 0 || n_splits > MAX_SPLITS) return VT_ATTN_ERR_INVALID_ARGUMENT;
    const SplitPlan pl = plan_split(B, Hq, Hkv, Sq, Sk, n_splits);
    if (splits_used) *splits_used = pl.n_splits;
    if (heads_share_tile) *heads_share_tile = pl.hpack;
    return VT_ATTN_OK;
}

namespace vt {
// The chunk kernel and the merge kernel of one head dimension and element type.
template <int DD, bool F16>
static int launch_merge(const FwdParams &prm, float *lse, long long n_rows, int n_splits, int d, int packed_hq, cudaStream_t st)
{
    const int rows_per_block = 256 / (DD / 4);
    long long mb = (n_rows + rows_per_block - 1) / rows_per_block;
    if (mb > NUM_SMS * 16) mb = NUM_SMS * 16;
    fwd_merge_kernel<DD, F16><<<static_cast<int>(mb), 256, 0, st>>>(prm.o_part, prm.lse_part, prm.o, lse, n_rows, n_splits, d, packed_hq);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? VT_ATTN_OK : cuda_fail(e, "fwd_merge_kernel launch");
}

// The same for packed batches.
template <int DD, bool F16>
static int launch_split_packed(bool causal, bool hpack, const CUtensorMap &tq, const CUtensorMap &tk, const CUtensorMap &tv, const FwdParams &prm,
                               int nb, float *lse, int n_splits, int d, cudaStream_t st)
{
    // Query tokens of a sequence past max_sq are owned by no block and get no partial result.  Their partial LSEs are
    // preset to all-ones bits (a NaN): fmaxf ignores a NaN operand, so the merge sees "no chunk saw a key" for exactly
    // those rows and writes O = 0, LSE = -inf instead of reading uninitialised scratch.  Rows that are processed get a
    // real partial LSE from every chunk's block (empty chunks write -inf), so the preset never mixes with real values.
    cudaError_t e = cudaMemsetAsync(prm.lse_part, 0xFF, static_cast<size_t>(n_splits) * prm.n_rows * sizeof(float), st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync(partial LSE)");
    int rc;
    if (hpack) rc = causal ? launch_fwd<DD, true, true, true, true, F16>(tq, tk, tv, prm, nb, st) : launch_fwd<DD, false, true, true, true, F16>(tq, tk, tv, prm, nb, st);
    else rc = causal ? launch_fwd<DD, true, true, true, false, F16>(tq, tk, tv, prm, nb, st) : launch_fwd<DD, false, true, true, false, F16>(tq, tk, tv, prm, nb, st);
    if (rc != VT_ATTN_OK) return rc;
    return launch_merge<DD, F16>(prm, lse, prm.n_rows, n_splits, d, prm.Hq, st);
}

template <int DD, bool F16>
static int launch_split(bool causal, bool hpack, const CUtensorMap &tq, const CUtensorMap &tk, const CUtensorMap &tv, const FwdParams &prm, int nb,
                        float *lse, long long n_rows, int n_splits, int d, cudaStream_t st)
{
    int rc;
    if (hpack) rc = causal ? launch_fwd<DD, true, false, true, true, F16>(tq, tk, tv, prm, nb, st) : launch_fwd<DD, false, false, true, true, F16>(tq, tk, tv, prm, nb, st);
    else rc = causal ? launch_fwd<DD, true, false, true, false, F16>(tq, tk, tv, prm, nb, st) : launch_fwd<DD, false, false, true, false, F16>(tq, tk, tv, prm, nb, st);
    if (rc != VT_ATTN_OK) return rc;
    return launch_merge<DD, F16>(prm, lse, n_rows, n_splits, d, 0, st);
}

}  // namespace vt

// Shared by vt_attn_fwd_splitkv (bfloat16 tensors) and vt_attn_fwd_splitkv_f16 (IEEE half tensors).
static int splitkv_entry(bool f16, const void *q, const void *k, const void *v, void *o, float *lse, int B, int Hq, int Hkv,
                         int Sq, int Sk, int D, int causal, float scale, int n_splits, void *workspace,
                         size_t workspace_bytes, void *stream)
{
    using namespace vt;
    Shape s{B, Hq, Hkv, Sq, Sk, D};
    int rc = check_shape(s, scale, MAX_HEAD_DIM_FWD);
    if (rc != VT_ATTN_OK) return rc;
    if (!ptr_ok(q) || !ptr_ok(k) || !ptr_ok(v) || !ptr_ok(o) || !ptr_ok(lse, 4) || !ptr_ok(workspace, 256))
        return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (causal < 0 || causal > 2 || n_splits < 0 || n_splits > MAX_SPLITS) return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (workspace_bytes < vt_attn_fwd_splitkv_workspace_bytes(B, Hq, Hkv, Sq, Sk, D, n_splits)) return VT_ATTN_ERR_WORKSPACE_TOO_SMALL;
    rc = check_device();
    if (rc != VT_ATTN_OK) return rc;

    const SplitPlan pl = plan_split(B, Hq, Hkv, Sq, Sk, n_splits);
    const long long n_rows = static_cast<long long>(B) * Hq * Sq;
    FwdParams prm;
    prm.o = static_cast<__nv_bfloat16 *>(o);
    prm.lse = lse;
    prm.Hq = Hq;
    prm.d = D;
    prm.d_qk = D;
    prm.hp_tokens = 0;
    prm.head_group = 0;
    const int Dp = padded_head_dim(D);      // the kernels' column count, also the row length of the partial results
    prm.G = Hq / Hkv;
    prm.Sq = Sq;
    prm.Sk = Sk;
    prm.n_qt = pl.hpack ? 1 : (Sq + TILE - 1) / TILE;
    prm.scale_log2e = scale * 1.4426950408889634f;
    prm.cu_q = nullptr;
    prm.cu_k = nullptr;
    prm.total_q = 0;
    prm.bottom_right = (causal == 2);
    prm.n_splits = pl.n_splits;
    prm.chunk_steps = pl.chunk_steps;
    prm.o_part = static_cast<float *>(workspace);
    prm.lse_part = reinterpret_cast<float *>(static_cast<char *>(workspace) +
                                             round_up_256(static_cast<size_t>(pl.n_splits) * n_rows * Dp * 4));
    prm.n_rows = n_rows;
    prm.guard = make_guard();
    if (!prm.guard.status) return VT_ATTN_ERR_CUDA;
    const long long n_blocks = pl.base_blocks * pl.n_splits;
    if (n_blocks > 0x7FFFFFFFll) return VT_ATTN_ERR_INVALID_ARGUMENT;

    CUtensorMap tq, tk, tv;
    if (pl.hpack) rc = make_tensor_map_heads(&tq, q, B * Hq, Sq, D, Sq, prm.G);
    else rc = make_tensor_map(&tq, q, B * Hq, Sq, D, TILE);
    if (rc != VT_ATTN_OK) return rc;
    if ((rc = make_tensor_map(&tk, k, B * Hkv, Sk, D, BN)) != VT_ATTN_OK) return rc;
    if ((rc = make_tensor_map(&tv, v, B * Hkv, Sk, D, BN)) != VT_ATTN_OK) return rc;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int nb = static_cast<int>(n_blocks);
    if (f16) {
        if (Dp == 64) return launch_split<64, true>(causal != 0, pl.hpack != 0, tq, tk, tv, prm, nb, lse, n_rows, pl.n_splits, D, st);
        if (Dp == 256) return launch_split<256, true>(causal != 0, pl.hpack != 0, tq, tk, tv, prm, nb, lse, n_rows, pl.n_splits, D, st);
        return launch_split<128, true>(causal != 0, pl.hpack != 0, tq, tk, tv, prm, nb, lse, n_rows, pl.n_splits, D, st);
    }
    if (Dp == 64) return launch_split<64, false>(causal != 0, pl.hpack != 0, tq, tk, tv, prm, nb, lse, n_rows, pl.n_splits, D, st);
    if (Dp == 256) return launch_split<256, false>(causal != 0, pl.hpack != 0, tq, tk, tv, prm, nb, lse, n_rows, pl.n_splits, D, st);
    return launch_split<128, false>(causal != 0, pl.hpack != 0, tq, tk, tv, prm, nb, lse, n_rows, pl.n_splits, D, st);
}

extern "C" int vt_attn_fwd_splitkv(const void *q, const void *k, const void *v, void *o, float *lse, int B, int Hq, int Hkv,
                                   int Sq, int Sk, int D, int causal, float scale, int n_splits, void *workspace,
                                   size_t workspace_bytes, void *stream)
{
    return splitkv_entry(false, q, k, v, o, lse, B, Hq, Hkv, Sq, Sk, D, causal, scale, n_splits, workspace, workspace_bytes, stream);
}

extern "C" int vt_attn_fwd_splitkv_f16(const void *q, const void *k, const void *v, void *o, float *lse, int B, int Hq, int Hkv,
                                       int Sq, int Sk, int D, int causal, float scale, int n_splits, void *workspace,
                                       size_t workspace_bytes, void *stream)
{
    return splitkv_entry(true, q, k, v, o, lse, B, Hq, Hkv, Sq, Sk, D, causal, scale, n_splits, workspace, workspace_bytes, stream);
}

// ----------------------------------------------------------------------------------------------
// Split-KV forward for packed batches: decoding and chunked prefill against caches of different lengths.  The plan
// (number of chunks, whether a KV group's heads share a tile) is taken from the longest sequence; the kernel cuts every
// sequence's own key steps into that many chunks; a chunk without keys writes an empty partial result (O = 0,
// LSE = -inf), which the merge ignores.
// ----------------------------------------------------------------------------------------------
namespace vt {
// Chunks for a packed batch when the caller leaves the choice to the library.  With caches of different lengths the
// blocks of a launch differ in work by the ratio of the lengths, so one wave of blocks (the choice for equal lengths)
// ends when its longest block does: about four waves of smaller blocks, and at least four chunks, let the scheduler
// even that out (measured on one decoded token per sequence, caches uniform in a 1:16 - 1:32 range: 16 sequences
// 251 -> 220 us, 64 sequences 458 -> 386 us, 128 sequences 390 -> 371 us).  `ragged`: longest / mean length > 1.25.
static int varlen_auto_splits(long long base_blocks, int n_steps, bool ragged)
{
    const int even = auto_splits(base_blocks, n_steps);
    if (!ragged) return even;
    long long want = (8 * NUM_SMS + base_blocks - 1) / base_blocks;
    if (want < 4) want = 4;
    const long long cap = n_steps / 8 > 0 ? n_steps / 8 : 1;
    if (want > 16) want = 16;                   // (beyond that the merge's share grows faster than the balance improves)
    if (want > cap) want = cap;
    return want > even ? static_cast<int>(want) : even;
}
}  // namespace vt

extern "C" size_t vt_attn_fwd_splitkv_varlen_workspace_bytes(int n_seqs, int Hq, int Hkv, int total_q, int max_sq, int max_sk, int D, int n_splits)
{
    using namespace vt;
    if (n_seqs <= 0 || Hq <= 0 || Hkv <= 0 || total_q <= 0 || max_sq <= 0 || max_sk <= 0 || Hq % Hkv != 0 || !head_dim_ok(D) || n_splits < 0 ||
        n_splits > MAX_SPLITS)
        return 0;
    if (n_splits == 0) {      // the library's choice depends on how ragged the batch is, which this query does not know: the larger of the two
        const SplitPlan p0 = plan_split(n_seqs, Hq, Hkv, max_sq, max_sk, 0);
        n_splits = varlen_auto_splits(p0.base_blocks, (max_sk + BN - 1) / BN, true);
    }
    const SplitPlan pl = plan_split(n_seqs, Hq, Hkv, max_sq, max_sk, n_splits);
    const size_t n_rows = static_cast<size_t>(total_q) * Hq;
    return round_up_256(static_cast<size_t>(pl.n_splits) * n_rows * padded_head_dim(D) * 4) + round_up_256(static_cast<size_t>(pl.n_splits) * n_rows * 4);
}

extern "C" int vt_attn_fwd_splitkv_varlen_plan(int n_seqs, int Hq, int Hkv, int total_k, int max_sq, int max_sk, int D, int n_splits,
                                               int *splits_used, int *heads_share_tile)
{
    using namespace vt;
    if (n_seqs <= 0 || Hq <= 0 || Hkv <= 0 || total_k <= 0 || max_sq <= 0 || max_sk <= 0 || Hq % Hkv != 0 || max_sk > total_k || n_splits < 0 ||
        n_splits > MAX_SPLITS)
        return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (!head_dim_ok(D)) return VT_ATTN_ERR_UNSUPPORTED;
    if (n_splits == 0) {
        const SplitPlan p0 = plan_split(n_seqs, Hq, Hkv, max_sq, max_sk, 0);
        n_splits = varlen_auto_splits(p0.base_blocks, (max_sk + BN - 1) / BN, 4ll * max_sk * n_seqs > 5ll * total_k);
    }
    const SplitPlan pl = plan_split(n_seqs, Hq, Hkv, max_sq, max_sk, n_splits);
    if (splits_used) *splits_used = pl.n_splits;
    if (heads_share_tile) *heads_share_tile = pl.hpack;
    return VT_ATTN_OK;
}

// Shared by vt_attn_fwd_splitkv_varlen (bfloat16 tensors) and vt_attn_fwd_splitkv_varlen_f16 (IEEE half tensors).
static int splitkv_varlen_entry(bool f16, const void *q, const void *k, const void *v, void *o, float *lse, const int *cu_seqlens_q,
                                const int *cu_seqlens_k, int n_seqs, int Hq, int Hkv, int total_q, int total_k, int max_sq,
                                int max_sk, int D, int causal, float scale, int n_splits, void *workspace, size_t workspace_bytes,
                                void *stream)
{
    using namespace vt;
    int rc = check_varlen_shape(n_seqs, Hq, Hkv, total_q, total_k, max_sq, max_sk, D, scale);
    if (rc != VT_ATTN_OK) return rc;
    if (!ptr_ok(q) || !ptr_ok(k) || !ptr_ok(v) || !ptr_ok(o) || !ptr_ok(lse, 4) || !ptr_ok(cu_seqlens_q, 4) || !ptr_ok(cu_seqlens_k, 4) ||
        !ptr_ok(workspace, 256))
        return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (causal < 0 || causal > 2 || n_splits < 0 || n_splits > MAX_SPLITS) return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (workspace_bytes < vt_attn_fwd_splitkv_varlen_workspace_bytes(n_seqs, Hq, Hkv, total_q, max_sq, max_sk, D, n_splits))
        return VT_ATTN_ERR_WORKSPACE_TOO_SMALL;
    rc = check_device();
    if (rc != VT_ATTN_OK) return rc;

    if (n_splits == 0) {
        const SplitPlan p0 = plan_split(n_seqs, Hq, Hkv, max_sq, max_sk, 0);
        const bool ragged = 4ll * max_sk * n_seqs > 5ll * total_k;        // longest / mean length > 1.25
        n_splits = varlen_auto_splits(p0.base_blocks, (max_sk + BN - 1) / BN, ragged);
    }
    const SplitPlan pl = plan_split(n_seqs, Hq, Hkv, max_sq, max_sk, n_splits);
    const long long n_rows = static_cast<long long>(total_q) * Hq;
    const int Dp = padded_head_dim(D);
    FwdParams prm;
    prm.o = static_cast<__nv_bfloat16 *>(o);
    prm.lse = lse;
    prm.Hq = Hq;
    prm.d = D;
    prm.d_qk = D;
    prm.hp_tokens = max_sq;
    prm.head_group = 0;
    prm.G = Hq / Hkv;
    prm.Sq = max_sq;
    prm.Sk = max_sk;
    prm.n_qt = pl.hpack ? 1 : (max_sq + TILE - 1) / TILE;
    prm.scale_log2e = scale * 1.4426950408889634f;
    prm.cu_q = cu_seqlens_q;
    prm.cu_k = cu_seqlens_k;
    prm.total_q = total_q;
    prm.bottom_right = (causal == 2);
    prm.n_splits = pl.n_splits;
    prm.chunk_steps = pl.chunk_steps;
    prm.o_part = static_cast<float *>(workspace);
    prm.lse_part = reinterpret_cast<float *>(static_cast<char *>(workspace) + round_up_256(static_cast<size_t>(pl.n_splits) * n_rows * Dp * 4));
    prm.n_rows = n_rows;
    prm.guard = make_guard();
    if (!prm.guard.status) return VT_ATTN_ERR_CUDA;
    const long long n_blocks = pl.base_blocks * pl.n_splits;
    if (n_blocks > 0x7FFFFFFFll) return VT_ATTN_ERR_INVALID_ARGUMENT;

    CUtensorMap tq, tk, tv;
    if (pl.hpack) rc = make_tensor_map_packed_heads(&tq, q, total_q, Hq, D, max_sq, prm.G);
    else rc = make_tensor_map_packed(&tq, q, total_q, Hq, D, TILE);
    if (rc != VT_ATTN_OK) return rc;
    if ((rc = make_tensor_map_packed(&tk, k, total_k, Hkv, D, BN)) != VT_ATTN_OK) return rc;
    if ((rc = make_tensor_map_packed(&tv, v, total_k, Hkv, D, BN)) != VT_ATTN_OK) return rc;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int nb = static_cast<int>(n_blocks);
    if (f16) {
        if (Dp == 64) return launch_split_packed<64, true>(causal != 0, pl.hpack != 0, tq, tk, tv, prm, nb, lse, pl.n_splits, D, st);
        return launch_split_packed<128, true>(causal != 0, pl.hpack != 0, tq, tk, tv, prm, nb, lse, pl.n_splits, D, st);
    }
    if (Dp == 64) return launch_split_packed<64, false>(causal != 0, pl.hpack != 0, tq, tk, tv, prm, nb, lse, pl.n_splits, D, st);
    return launch_split_packed<128, false>(causal != 0, pl.hpack != 0, tq, tk, tv, prm, nb, lse, pl.n_splits, D, st);
}

extern "C" int vt_attn_fwd_splitkv_varlen(const void *q, const void *k, const void *v, void *o, float *lse, const int *cu_seqlens_q,
                                          const int *cu_seqlens_k, int n_seqs, int Hq, int Hkv, int total_q, int total_k, int max_sq,
                                          int max_sk, int D, int causal, float scale, int n_splits, void *workspace, size_t workspace_bytes,
                                          void *stream)
{
    return splitkv_varlen_entry(false, q, k, v, o, lse, cu_seqlens_q, cu_seqlens_k, n_seqs, Hq, Hkv, total_q, total_k, max_sq, max_sk, D, causal,
                                scale, n_splits, workspace, workspace_bytes, stream);
}

extern "C" int vt_attn_fwd_splitkv_varlen_f16(const void *q, const void *k, const void *v, void *o, float *lse, const int *cu_seqlens_q,
                                              const int *cu_seqlens_k, int n_seqs, int Hq, int Hkv, int total_q, int total_k, int max_sq,
                                              int max_sk, int D, int causal, float scale, int n_splits, void *workspace,
                                              size_t workspace_bytes, void *stream)
{
    return splitkv_varlen_entry(true, q, k, v, o, lse, cu_seqlens_q, cu_seqlens_k, n_seqs, Hq, Hkv, total_q, total_k, max_sq, max_sk, D, causal,
                                scale, n_splits, workspace, workspace_bytes, stream);
}
