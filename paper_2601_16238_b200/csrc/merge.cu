// Merging partial attention results that cover disjoint key sets of the same queries (the per-block step of
// context-parallel ring attention; the same algebra as the split-KV merge, but one part at a time into an fp32 running
// result so that the parts can arrive over several steps):
//   LSE' = ln(e^LSE + e^LSE_part),   O' = e^(LSE - LSE') O + e^(LSE_part - LSE') O_part.
// A part that saw no key has LSE_part = -inf and leaves the running result unchanged.
#include "vt_host.h"

namespace vt {

// The kernels below give a thread 8 elements of a row (D / 8 threads per row, D a multiple of 8) and walk the
// n_rows * D / 8 pieces with a grid-stride loop.
//
// merge_partial_kernel reads and rewrites lse_acc[row] in one launch, so every thread of a row must have read the old
// value before one of them stores the new one.  The threads of a row are therefore padded to a power of two (`tpr_pad`,
// at most 32): a row then never straddles a warp, the loop bounds are the same for all lanes of a warp, and a
// __syncwarp() separates the row's loads from the store.  Lanes past the row's real D / 8 pieces only take part in the
// barrier.
__global__ void __launch_bounds__(256) merge_partial_kernel(float *__restrict__ o_acc, float *__restrict__ lse_acc,
                                                            const __nv_bfloat16 *__restrict__ o_part, const float *__restrict__ lse_part,
                                                            long long n_rows, int D, int tpr_pad, int first)
{
    const int tpr = D / 8;
    const long long n_slots = n_rows * tpr_pad;                         // a multiple of tpr_pad; rows are whole within a warp
    const long long n_warp_slots = (n_slots + 31) / 32 * 32;            // warp-uniform loop bound
    for (long long i = static_cast<long long>(blockIdx.x) * 256 + threadIdx.x; i < n_warp_slots; i += static_cast<long long>(gridDim.x) * 256) {
        const long long row = i / tpr_pad;
        const int sub = static_cast<int>(i - row * tpr_pad);
        const bool live = row < n_rows && sub < tpr;
        float wa = 0.0f, wp = 0.0f, ln = -INFINITY;
        if (live) {
            const float lp = lse_part[row];
            const float la = first ? -INFINITY : lse_acc[row];
            const float m = fmaxf(la, lp);
            if (m != -INFINITY) {                        // at least one side saw a key
                const float ea = __expf(la - m), ep = __expf(lp - m);      // exp(-inf) = 0
                const float inv = 1.0f / (ea + ep);
                wa = ea * inv;
                wp = ep * inv;
                ln = m + logf(ea + ep);
            }
        }
        __syncwarp();                                    // every lane of the row holds the old LSE before lane `sub == 0` replaces it
        if (!live) continue;
        const uint4 pv = *reinterpret_cast<const uint4 *>(o_part + row * D + sub * 8);
        const uint32_t pw[4] = {pv.x, pv.y, pv.z, pv.w};
        float4 a0 = make_float4(0.f, 0.f, 0.f, 0.f), a1 = a0;
        if (!first) {
            a0 = *reinterpret_cast<const float4 *>(o_acc + row * D + sub * 8);
            a1 = *reinterpret_cast<const float4 *>(o_acc + row * D + sub * 8 + 4);
        }
        const float2 p0 = unpack16<false>(pw[0]), p1 = unpack16<false>(pw[1]), p2 = unpack16<false>(pw[2]), p3 = unpack16<false>(pw[3]);
        a0 = make_float4(wa * a0.x + wp * p0.x, wa * a0.y + wp * p0.y, wa * a0.z + wp * p1.x, wa * a0.w + wp * p1.y);
        a1 = make_float4(wa * a1.x + wp * p2.x, wa * a1.y + wp * p2.y, wa * a1.z + wp * p3.x, wa * a1.w + wp * p3.y);
        *reinterpret_cast<float4 *>(o_acc + row * D + sub * 8) = a0;
        *reinterpret_cast<float4 *>(o_acc + row * D + sub * 8 + 4) = a1;
        if (sub == 0) lse_acc[row] = ln;
    }
}

__global__ void __launch_bounds__(256) merge_finish_kernel(const float *__restrict__ o_acc, __nv_bfloat16 *__restrict__ o, long long n_rows, int D)
{
    const int tpr = D / 8;
    const long long n_pieces = n_rows * tpr;
    for (long long i = static_cast<long long>(blockIdx.x) * 256 + threadIdx.x; i < n_pieces; i += static_cast<long long>(gridDim.x) * 256) {
        const long long row = i / tpr;
        const int sub = static_cast<int>(i - row * tpr);
        const float4 a0 = *reinterpret_cast<const float4 *>(o_acc + row * D + sub * 8);
        const float4 a1 = *reinterpret_cast<const float4 *>(o_acc + row * D + sub * 8 + 4);
        uint4 w;
        w.x = pack_bf16(a0.x, a0.y);
        w.y = pack_bf16(a0.z, a0.w);
        w.z = pack_bf16(a1.x, a1.y);
        w.w = pack_bf16(a1.z, a1.w);
        *reinterpret_cast<uint4 *>(o + row * D + sub * 8) = w;
    }
}

// acc (fp32) += part (bf16), or acc = part when `first`: the running sums of the gradient blocks in the ring backward.
__global__ void __launch_bounds__(256) accumulate_kernel(float *__restrict__ acc, const __nv_bfloat16 *__restrict__ part, long long n_rows, int D, int first)
{
    const int tpr = D / 8;
    const long long n_pieces = n_rows * tpr;
    for (long long i = static_cast<long long>(blockIdx.x) * 256 + threadIdx.x; i < n_pieces; i += static_cast<long long>(gridDim.x) * 256) {
        const long long row = i / tpr;
        const int sub = static_cast<int>(i - row * tpr);
        const uint4 pv = *reinterpret_cast<const uint4 *>(part + row * D + sub * 8);
        const float2 p0 = unpack16<false>(pv.x), p1 = unpack16<false>(pv.y), p2 = unpack16<false>(pv.z), p3 = unpack16<false>(pv.w);
        float4 a0 = make_float4(0.f, 0.f, 0.f, 0.f), a1 = a0;
        if (!first) {
            a0 = *reinterpret_cast<const float4 *>(acc + row * D + sub * 8);
            a1 = *reinterpret_cast<const float4 *>(acc + row * D + sub * 8 + 4);
        }
        *reinterpret_cast<float4 *>(acc + row * D + sub * 8) = make_float4(a0.x + p0.x, a0.y + p0.y, a0.z + p1.x, a0.w + p1.y);
        *reinterpret_cast<float4 *>(acc + row * D + sub * 8 + 4) = make_float4(a1.x + p2.x, a1.y + p2.y, a1.z + p3.x, a1.w + p3.y);
    }
}

static int pow2_at_least(int x)
{
    int p = 1;
    while (p < x) p *= 2;
    return p;
}

static int merge_grid(long long n_rows, int threads_per_row)
{
    long long nb = (n_rows * threads_per_row + 255) / 256;
    if (nb > NUM_SMS * 16) nb = NUM_SMS * 16;
    return static_cast<int>(nb);
}

}  // namespace vt

extern "C" int vt_attn_merge_partial(float *o_acc, float *lse_acc, const void *o_part, const float *lse_part, long long n_rows,
                                     int D, int first, void *stream)
{
    using namespace vt;
    if (!ptr_ok(o_acc) || !ptr_ok(lse_acc, 4) || !ptr_ok(o_part) || !ptr_ok(lse_part, 4) || n_rows <= 0) return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (!head_dim_ok(D, MAX_HEAD_DIM_FWD)) return VT_ATTN_ERR_UNSUPPORTED;
    int rc = check_device();
    if (rc != VT_ATTN_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const __nv_bfloat16 *part = static_cast<const __nv_bfloat16 *>(o_part);
    const int tpr_pad = pow2_at_least(D / 8);
    merge_partial_kernel<<<merge_grid(n_rows, tpr_pad), 256, 0, st>>>(o_acc, lse_acc, part, lse_part, n_rows, D, tpr_pad, first);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "merge_partial_kernel launch");
    return VT_ATTN_OK;
}

extern "C" int vt_attn_merge_finish(const float *o_acc, void *o, long long n_rows, int D, void *stream)
{
    using namespace vt;
    if (!ptr_ok(o_acc) || !ptr_ok(o) || n_rows <= 0) return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (!head_dim_ok(D, MAX_HEAD_DIM_FWD)) return VT_ATTN_ERR_UNSUPPORTED;
    int rc = check_device();
    if (rc != VT_ATTN_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    __nv_bfloat16 *out = static_cast<__nv_bfloat16 *>(o);
    merge_finish_kernel<<<merge_grid(n_rows, D / 8), 256, 0, st>>>(o_acc, out, n_rows, D);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "merge_finish_kernel launch");
    return VT_ATTN_OK;
}

extern "C" int vt_attn_accumulate_partial(float *acc, const void *part, long long n_rows, int D, int first, void *stream)
{
    using namespace vt;
    if (!ptr_ok(acc) || !ptr_ok(part) || n_rows <= 0) return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (!head_dim_ok(D, MAX_HEAD_DIM_FWD)) return VT_ATTN_ERR_UNSUPPORTED;
    int rc = check_device();
    if (rc != VT_ATTN_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const __nv_bfloat16 *p = static_cast<const __nv_bfloat16 *>(part);
    accumulate_kernel<<<merge_grid(n_rows, D / 8), 256, 0, st>>>(acc, p, n_rows, D, first);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "accumulate_kernel launch");
    return VT_ATTN_OK;
}
