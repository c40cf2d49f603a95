// Kernel-suite operators next to attention in the paper's microbenchmark table: RMSNorm (fwd), LayerNorm (fwd + bwd)
// and rotary position embedding (fwd).  All are streaming kernels bound by HBM bandwidth: every row is read once into
// registers with 16-byte loads (a thread's vectors are T apart, so a warp's loads are contiguous), reduced in fp32
// with warp shuffles and one shared-memory exchange, and written once.  What bounds the bandwidth a kernel reaches is the
// number of bytes it keeps in flight per SM, i.e. the share of the register file that holds loaded-but-unused data: the
// weights are therefore re-read from L1 per row instead of being kept (the compiler would hold them unpacked, 16
// registers per vector against 4 for the row itself), and the grid is one wave of blocks striding over the rows.
#include "vt_host.h"
#include "../../include/vt_suite.h"

namespace vt {

constexpr int SUITE_THREADS = 256;
constexpr int LNB_VPT = 2;                  // LayerNorm / RMSNorm backward: 16-byte vectors of a row per thread
constexpr int SUITE_BWD_BLOCKS_MAX = 4 * NUM_SMS; // LayerNorm backward: most blocks (= partial sums per column)

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
    return v;
}

// Sums NV values over the block; every thread gets the totals.  red: two buffers of NV * 32 floats of shared memory used
// in turn (`turn` flips per call), so that one barrier per call is enough: a warp can write the buffer of call k + 2
// only after every warp has passed the barrier of call k + 1, i.e. has finished reading call k's.
template <int NV>
__device__ __forceinline__ void block_sum(float (&v)[NV], float *red, uint32_t &turn)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
#pragma unroll
    for (int i = 0; i < NV; ++i) v[i] = warp_sum(v[i]);
    if (n_warps == 1) return;
    float *buf = red + (turn & 1u) * (NV * 32);
    turn ^= 1u;
    if (lane == 0)
#pragma unroll
        for (int i = 0; i < NV; ++i) buf[i * 32 + warp] = v[i];
    __syncthreads();
#pragma unroll
    for (int i = 0; i < NV; ++i) v[i] = warp_sum(lane < n_warps ? buf[i * 32 + lane] : 0.0f);
}

__device__ __forceinline__ void unpack8(const uint4 &u, float (&f)[8])
{
    const float2 a = unpack16<false>(u.x), b = unpack16<false>(u.y), c = unpack16<false>(u.z), d = unpack16<false>(u.w);
    f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y; f[4] = c.x; f[5] = c.y; f[6] = d.x; f[7] = d.y;
}

__device__ __forceinline__ uint4 pack8(const float (&f)[8])
{
    return make_uint4(pack_bf16(f[0], f[1]), pack_bf16(f[2], f[3]), pack_bf16(f[4], f[5]), pack_bf16(f[6], f[7]));
}

// The same eight values as four pairs: the norm kernels do their arithmetic two elements per instruction (fma / add / mul
// .f32x2, each half rounded like the scalar instruction), which is what keeps them off the issue-slot limit.
__device__ __forceinline__ void unpack8(const uint4 &u, float2 (&f)[4])
{
    f[0] = unpack16<false>(u.x); f[1] = unpack16<false>(u.y); f[2] = unpack16<false>(u.z); f[3] = unpack16<false>(u.w);
}

__device__ __forceinline__ uint4 pack8(const float2 (&f)[4])
{
    return make_uint4(pack_bf16(f[0].x, f[0].y), pack_bf16(f[1].x, f[1].y), pack_bf16(f[2].x, f[2].y), pack_bf16(f[3].x, f[3].y));
}

__device__ __forceinline__ float2 splat2(float v) { return make_float2(v, v); }

// ----------------------------------------------------------------------------------------------
// RMSNorm forward.  VPT: 16-byte vectors per thread (a row has nvec = cols / 8 of them, vector v of thread t is
// number v * T + t).
// ----------------------------------------------------------------------------------------------
template <int VPT, int T>
__global__ void __launch_bounds__(T) rmsnorm_fwd_kernel(const uint4 *__restrict__ x, const uint4 *__restrict__ w, uint4 *__restrict__ y,
                                                       float *__restrict__ rstd, long long rows, int nvec, float inv_cols, float eps)
{
    __shared__ float red[64];
    uint32_t turn = 0;
    const int tid = threadIdx.x, nt = blockDim.x;
    for (long long row = blockIdx.x; row < rows; row += gridDim.x) {
        const uint4 *xr = x + row * nvec;
        uint4 xv[VPT];
#pragma unroll
        for (int v = 0; v < VPT; ++v) xv[v] = (v * nt + tid < nvec) ? xr[v * nt + tid] : make_uint4(0, 0, 0, 0);
        float2 ss2 = make_float2(0.0f, 0.0f);
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            float2 f[4];
            unpack8(xv[v], f);
#pragma unroll
            for (int e = 0; e < 4; ++e) ss2 = __ffma2_rn(f[e], f[e], ss2);
        }
        float ss[1] = {ss2.x + ss2.y};
        block_sum<1>(ss, red, turn);
        const float r = 1.0f / sqrtf(ss[0] * inv_cols + eps);
        const float2 r2 = splat2(r);
        uint4 *yr = y + row * nvec;
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            if (v * nt + tid < nvec) {
                float2 f[4], g[4];
                unpack8(xv[v], f);
                unpack8(__ldg(w + v * nt + tid), g);
#pragma unroll
                for (int e = 0; e < 4; ++e) f[e] = __fmul2_rn(__fmul2_rn(f[e], r2), g[e]);
                yr[v * nt + tid] = pack8(f);
            }
        }
        if (tid == 0 && rstd) rstd[row] = r;
    }
}

// ----------------------------------------------------------------------------------------------
// LayerNorm forward: the mean first, then the variance of the centred values (both from registers).
// ----------------------------------------------------------------------------------------------
template <int VPT, int T>
__global__ void __launch_bounds__(T) layernorm_fwd_kernel(const uint4 *__restrict__ x, const uint4 *__restrict__ w, const uint4 *__restrict__ b,
                                                         uint4 *__restrict__ y, float *__restrict__ mean, float *__restrict__ rstd,
                                                         long long rows, int nvec, float inv_cols, float eps)
{
    __shared__ float red[64];
    uint32_t turn = 0;
    const int tid = threadIdx.x, nt = blockDim.x;
    for (long long row = blockIdx.x; row < rows; row += gridDim.x) {
        const uint4 *xr = x + row * nvec;
        uint4 xv[VPT];
#pragma unroll
        for (int v = 0; v < VPT; ++v) xv[v] = (v * nt + tid < nvec) ? xr[v * nt + tid] : make_uint4(0, 0, 0, 0);
        float2 s2 = make_float2(0.0f, 0.0f);
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            float2 f[4];
            unpack8(xv[v], f);
#pragma unroll
            for (int e = 0; e < 4; ++e) s2 = __fadd2_rn(s2, f[e]);
        }
        float s[1] = {s2.x + s2.y};
        block_sum<1>(s, red, turn);
        const float mu = s[0] * inv_cols;
        const float2 nmu2 = splat2(-mu);
        float2 q2 = make_float2(0.0f, 0.0f);
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            if (v * nt + tid < nvec) {                 // (the padding vectors must not add mu^2)
                float2 f[4];
                unpack8(xv[v], f);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 d = __fadd2_rn(f[e], nmu2);
                    q2 = __ffma2_rn(d, d, q2);
                }
            }
        }
        float q[1] = {q2.x + q2.y};
        block_sum<1>(q, red, turn);
        const float r = 1.0f / sqrtf(q[0] * inv_cols + eps);
        const float2 r2 = splat2(r), nmr2 = splat2(-mu * r);
        uint4 *yr = y + row * nvec;
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            if (v * nt + tid < nvec) {
                float2 f[4], g[4], h[4];
                unpack8(xv[v], f);
                unpack8(__ldg(w + v * nt + tid), g);
                unpack8(__ldg(b + v * nt + tid), h);
#pragma unroll
                for (int e = 0; e < 4; ++e) f[e] = __ffma2_rn(__ffma2_rn(f[e], r2, nmr2), g[e], h[e]);
                yr[v * nt + tid] = pack8(f);
            }
        }
        if (tid == 0) {
            if (mean) mean[row] = mu;
            if (rstd) rstd[row] = r;
        }
    }
}

// ----------------------------------------------------------------------------------------------
// LayerNorm backward.  VPT 16-byte vectors of a row per thread (a block has 1024 / VPT threads for the longest rows, fewer
// for shorter ones).  A block walks rows blockIdx.x, blockIdx.x + gridDim.x, ...; a thread owns the same columns in
// every row, so its share of dw and db accumulates in registers and is written once, as this block's partial sums
// (part: [2][gridDim.x][cols] fp32); layernorm_bwd_reduce_kernel adds the blocks in a fixed order.  The next row's x and
// dy are requested before the current row is worked on, so a block always has a row in flight.  Two vectors per thread
// (512 threads, 128 registers) measured best: with one (1024 threads, 64 registers) the compiler recomputes what it
// cannot keep across the block reduction (34 instructions per element under ncu), with four the block is too small.
// RMS: the RMSNorm backward - no mean (xh = x * rstd, no "- mean_j g" term) and no bias gradient.
// ----------------------------------------------------------------------------------------------
template <bool RMS, int VPT>
__global__ void __launch_bounds__(1024 / VPT) layernorm_bwd_kernel(const uint4 *__restrict__ x, const uint4 *__restrict__ w,
                                                                  const uint4 *__restrict__ dy, const float *__restrict__ mean,
                                                                  const float *__restrict__ rstd, uint4 *__restrict__ dx,
                                                                  float *__restrict__ part, long long rows, int nvec, float inv_cols)
{
    __shared__ float red[128];
    uint32_t turn = 0;
    const int tid = threadIdx.x, nt = blockDim.x;
    float2 aw[VPT][4], ab[VPT][4];
#pragma unroll
    for (int v = 0; v < VPT; ++v)
#pragma unroll
        for (int e = 0; e < 4; ++e) aw[v][e] = ab[v][e] = make_float2(0.0f, 0.0f);
    const uint4 zero = make_uint4(0, 0, 0, 0);
    long long row = blockIdx.x;
    uint4 xv[VPT], gv[VPT];
    float mu = 0.0f, r = 0.0f;
#pragma unroll
    for (int v = 0; v < VPT; ++v) xv[v] = gv[v] = zero;
    if (row < rows) {
#pragma unroll
        for (int v = 0; v < VPT; ++v)
            if (v * nt + tid < nvec) {
                xv[v] = x[row * nvec + v * nt + tid];
                gv[v] = dy[row * nvec + v * nt + tid];
            }
        mu = RMS ? 0.0f : mean[row];
        r = rstd[row];
    }
    while (row < rows) {
        const long long next = row + gridDim.x;
        uint4 xn[VPT], gn[VPT];
        float mun = 0.0f, rn = 0.0f;
#pragma unroll
        for (int v = 0; v < VPT; ++v) xn[v] = gn[v] = zero;
        if (next < rows) {
#pragma unroll
            for (int v = 0; v < VPT; ++v)
                if (v * nt + tid < nvec) {
                    xn[v] = x[next * nvec + v * nt + tid];
                    gn[v] = dy[next * nvec + v * nt + tid];
                }
            mun = RMS ? 0.0f : mean[next];
            rn = rstd[next];
        }
        float2 xh[VPT][4], g[VPT][4];
        float2 s0 = make_float2(0.0f, 0.0f), s1 = make_float2(0.0f, 0.0f);   // sum_j g, sum_j g * xh   (vectors past the row's end hold dy = 0, w = 0: they add nothing)
        const float2 r2 = splat2(r), nmr2 = splat2(-mu * r);
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            float2 f[4], d[4];
            unpack8(xv[v], f);
            unpack8(gv[v], d);
            unpack8((v * nt + tid < nvec) ? __ldg(w + v * nt + tid) : zero, g[v]);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                xh[v][e] = __ffma2_rn(f[e], r2, nmr2);
                g[v][e] = __fmul2_rn(g[v][e], d[e]);
                s0 = __fadd2_rn(s0, g[v][e]);
                s1 = __ffma2_rn(g[v][e], xh[v][e], s1);
                aw[v][e] = __ffma2_rn(d[e], xh[v][e], aw[v][e]);
                if (!RMS) ab[v][e] = __fadd2_rn(ab[v][e], d[e]);
            }
        }
        float s[2] = {s0.x + s0.y, s1.x + s1.y};
        block_sum<2>(s, red, turn);
        const float m1 = RMS ? 0.0f : s[0] * inv_cols, m2 = s[1] * inv_cols;
        const float2 c1 = splat2(-r * m1), c2 = splat2(-r * m2);
#pragma unroll
        for (int v = 0; v < VPT; ++v)
            if (v * nt + tid < nvec) {
                float2 f[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) f[e] = __ffma2_rn(xh[v][e], c2, __ffma2_rn(g[v][e], r2, c1));
                dx[row * nvec + v * nt + tid] = pack8(f);
            }
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            xv[v] = xn[v];
            gv[v] = gn[v];
        }
        mu = mun; r = rn;
        row = next;
    }
    const size_t cols = static_cast<size_t>(nvec) * 8;
#pragma unroll
    for (int v = 0; v < VPT; ++v)
        if (v * nt + tid < nvec) {
            const size_t c = static_cast<size_t>(v * nt + tid) * 8;
            float *pw = part + static_cast<size_t>(blockIdx.x) * cols + c;
            float *pb = part + (static_cast<size_t>(gridDim.x) + blockIdx.x) * cols + c;
            *reinterpret_cast<float4 *>(pw) = make_float4(aw[v][0].x, aw[v][0].y, aw[v][1].x, aw[v][1].y);
            *reinterpret_cast<float4 *>(pw + 4) = make_float4(aw[v][2].x, aw[v][2].y, aw[v][3].x, aw[v][3].y);
            if (!RMS) {
                *reinterpret_cast<float4 *>(pb) = make_float4(ab[v][0].x, ab[v][0].y, ab[v][1].x, ab[v][1].y);
                *reinterpret_cast<float4 *>(pb + 4) = make_float4(ab[v][2].x, ab[v][2].y, ab[v][3].x, ab[v][3].y);
            }
        }
}

// dw, db = the blocks' partial sums added in a fixed order: thread (tx, ty) of a 32 x 32 block adds the partial rows
// ty, ty + 32, ... of its 4 columns, then the 32 sums are added in order of ty.  blockIdx.y: 0 = dw, 1 = db.
__global__ void __launch_bounds__(1024) layernorm_bwd_reduce_kernel(const float *__restrict__ part, float *dw, float *db,
                                                                  int n_blocks, int cols)
{
    __shared__ float4 sm[32][32];
    const int tx = threadIdx.x, ty = threadIdx.y;
    const int q = blockIdx.x * 32 + tx;                        // group of 4 columns
    const int which = blockIdx.y;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (q * 4 < cols) {
        const float *src = part + static_cast<size_t>(which) * n_blocks * cols + static_cast<size_t>(q) * 4;
#pragma unroll 8
        for (int b = ty; b < n_blocks; b += 32) {
            const float4 v = *reinterpret_cast<const float4 *>(src + static_cast<size_t>(b) * cols);
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
    }
    sm[ty][tx] = acc;
    __syncthreads();
    if (ty == 0 && q * 4 < cols) {
        for (int i = 1; i < 32; ++i) {
            const float4 v = sm[i][tx];
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
        *reinterpret_cast<float4 *>((which ? db : dw) + static_cast<size_t>(q) * 4) = acc;
    }
}

// ----------------------------------------------------------------------------------------------
// Rotary embedding.  The tables: one thread per (position, pair), double precision.
// ----------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) rope_tables_kernel(float *__restrict__ cos_t, float *__restrict__ sin_t, int S, int half, double base)
{
    const long long i = static_cast<long long>(blockIdx.x) * 256 + threadIdx.x;
    if (i >= static_cast<long long>(S) * half) return;
    const int s = static_cast<int>(i / half), p = static_cast<int>(i % half);
    const double inv_freq = pow(base, -static_cast<double>(p) / static_cast<double>(half));      // base^(-2p/D)
    double sn, cs;
    sincos(static_cast<double>(s) * inv_freq, &sn, &cs);
    cos_t[i] = static_cast<float>(cs);
    sin_t[i] = static_cast<float>(sn);
}

// A thread takes 8 pairs: elements [8j, 8j + 8) of the first half of a row and the same of the second half, at one
// position s, and keeps that position's 8 cosines and sines in registers for every head it walks (blockIdx.y strides
// over the heads), so the tables cost one read per gridDim.y heads.  hv = D / 16 vector pairs per row.
__global__ void __launch_bounds__(256) rope_apply_kernel(const uint4 *__restrict__ x, const float4 *__restrict__ cos_t, const float4 *__restrict__ sin_t,
                                                        uint4 *__restrict__ y, long long n_heads, int S, int hv, float sign)
{
    const int i = blockIdx.x * 256 + threadIdx.x;            // (s, j)
    if (i >= S * hv) return;
    const int s = i / hv, j = i - s * hv;
    float c[8], sn[8];
    {
        const float4 c0 = cos_t[2 * i], c1 = cos_t[2 * i + 1], s0 = sin_t[2 * i], s1 = sin_t[2 * i + 1];
        c[0] = c0.x; c[1] = c0.y; c[2] = c0.z; c[3] = c0.w; c[4] = c1.x; c[5] = c1.y; c[6] = c1.z; c[7] = c1.w;
        sn[0] = s0.x; sn[1] = s0.y; sn[2] = s0.z; sn[3] = s0.w; sn[4] = s1.x; sn[5] = s1.y; sn[6] = s1.z; sn[7] = s1.w;
#pragma unroll
        for (int e = 0; e < 8; ++e) sn[e] *= sign;
    }
    for (long long h = blockIdx.y; h < n_heads; h += gridDim.y) {
        const size_t base = (static_cast<size_t>(h) * S + s) * (2 * hv) + j;
        float a[8], b[8], oa[8], ob[8];
        unpack8(x[base], a);
        unpack8(x[base + hv], b);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            oa[e] = a[e] * c[e] - b[e] * sn[e];
            ob[e] = b[e] * c[e] + a[e] * sn[e];
        }
        y[base] = pack8(oa);
        y[base + hv] = pack8(ob);
    }
}

// Threads per block and vectors per thread for a row of nvec 16-byte vectors (nvec <= 8 * SUITE_THREADS).
static void row_plan(int nvec, int *threads, int *vpt)
{
    int t = 32;
    while (t < SUITE_THREADS && t < nvec) t *= 2;
    int v = 1;
    while (v * t < nvec) v *= 2;
    *threads = t;
    *vpt = v;
}

static int row_grid(long long rows, int threads)
{
    const long long per_sm = 2048 / threads;
    const long long cap = static_cast<long long>(NUM_SMS) * (per_sm > 16 ? 16 : per_sm);
    return static_cast<int>(rows < cap ? rows : cap);
}

}  // namespace vt

using namespace vt;

static int norm_args_ok(const void *x, const void *w, const void *y, long long rows, int cols, int max_cols)
{
    if (!ptr_ok(x) || !ptr_ok(w) || !ptr_ok(y) || rows <= 0 || cols <= 0) return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (cols % 8 != 0 || cols > max_cols) return VT_ATTN_ERR_UNSUPPORTED;
    return VT_ATTN_OK;
}

extern "C" int vt_suite_rmsnorm_fwd(const void *x, const void *w, void *y, float *rstd, long long rows, int cols, float eps, void *stream)
{
    int rc = norm_args_ok(x, w, y, rows, cols, 65536);
    if (rc != VT_ATTN_OK) return rc;
    if (!(eps >= 0.0f) || !isfinite(eps) || (rstd && !ptr_ok(rstd, 4))) return VT_ATTN_ERR_INVALID_ARGUMENT;
    if ((rc = check_device()) != VT_ATTN_OK) return rc;
    const int nvec = cols / 8;
    const float inv = 1.0f / static_cast<float>(cols);
    const uint4 *xp = static_cast<const uint4 *>(x), *wp = static_cast<const uint4 *>(w);
    uint4 *yp = static_cast<uint4 *>(y);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (nvec > 8 * SUITE_THREADS) {
        rmsnorm_fwd_kernel<8, 1024><<<row_grid(rows, 1024), 1024, 0, st>>>(xp, wp, yp, rstd, rows, nvec, inv, eps);
    } else {
        int t, v;
        row_plan(nvec, &t, &v);
        const int g = row_grid(rows, t);
        switch (v) {
            case 1: rmsnorm_fwd_kernel<1, SUITE_THREADS><<<g, t, 0, st>>>(xp, wp, yp, rstd, rows, nvec, inv, eps); break;
            case 2: rmsnorm_fwd_kernel<2, SUITE_THREADS><<<g, t, 0, st>>>(xp, wp, yp, rstd, rows, nvec, inv, eps); break;
            case 4: rmsnorm_fwd_kernel<4, SUITE_THREADS><<<g, t, 0, st>>>(xp, wp, yp, rstd, rows, nvec, inv, eps); break;
            default: rmsnorm_fwd_kernel<8, SUITE_THREADS><<<g, t, 0, st>>>(xp, wp, yp, rstd, rows, nvec, inv, eps); break;
        }
    }
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? VT_ATTN_OK : cuda_fail(e, "rmsnorm_fwd_kernel launch");
}

extern "C" int vt_suite_layernorm_fwd(const void *x, const void *w, const void *b, void *y, float *mean, float *rstd, long long rows,
                                      int cols, float eps, void *stream)
{
    int rc = norm_args_ok(x, w, y, rows, cols, 65536);
    if (rc != VT_ATTN_OK) return rc;
    if (!ptr_ok(b) || !(eps >= 0.0f) || !isfinite(eps) || (mean && !ptr_ok(mean, 4)) || (rstd && !ptr_ok(rstd, 4)))
        return VT_ATTN_ERR_INVALID_ARGUMENT;
    if ((rc = check_device()) != VT_ATTN_OK) return rc;
    const int nvec = cols / 8;
    const float inv = 1.0f / static_cast<float>(cols);
    const uint4 *xp = static_cast<const uint4 *>(x), *wp = static_cast<const uint4 *>(w), *bp = static_cast<const uint4 *>(b);
    uint4 *yp = static_cast<uint4 *>(y);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (nvec > 8 * SUITE_THREADS) {
        layernorm_fwd_kernel<8, 1024><<<row_grid(rows, 1024), 1024, 0, st>>>(xp, wp, bp, yp, mean, rstd, rows, nvec, inv, eps);
    } else {
        int t, v;
        row_plan(nvec, &t, &v);
        const int g = row_grid(rows, t);
        switch (v) {
            case 1: layernorm_fwd_kernel<1, SUITE_THREADS><<<g, t, 0, st>>>(xp, wp, bp, yp, mean, rstd, rows, nvec, inv, eps); break;
            case 2: layernorm_fwd_kernel<2, SUITE_THREADS><<<g, t, 0, st>>>(xp, wp, bp, yp, mean, rstd, rows, nvec, inv, eps); break;
            case 4: layernorm_fwd_kernel<4, SUITE_THREADS><<<g, t, 0, st>>>(xp, wp, bp, yp, mean, rstd, rows, nvec, inv, eps); break;
            default: layernorm_fwd_kernel<8, SUITE_THREADS><<<g, t, 0, st>>>(xp, wp, bp, yp, mean, rstd, rows, nvec, inv, eps); break;
        }
    }
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? VT_ATTN_OK : cuda_fail(e, "layernorm_fwd_kernel launch");
}

// LayerNorm backward launch shape: `threads` = the row's vectors rounded up to a power of two (32 .. 1024), of which a
// block has threads / LNB_VPT; blocks = what is resident at once (1024 / threads per SM), at most SUITE_BWD_BLOCKS_MAX
// (each block costs a partial row of dw and db).
static void bwd_plan(int cols, int *threads, int *max_blocks)
{
    int t = 32;
    while (t < cols / 8) t *= 2;
    int nb = NUM_SMS * (1024 / t);
    if (nb > SUITE_BWD_BLOCKS_MAX) nb = SUITE_BWD_BLOCKS_MAX;
    *threads = t;
    *max_blocks = nb;
}

extern "C" size_t vt_suite_layernorm_bwd_workspace_bytes(int cols)
{
    if (cols <= 0 || cols % 8 != 0 || cols > 8192) return 0;
    int t, nb;
    bwd_plan(cols, &t, &nb);
    return static_cast<size_t>(2) * nb * cols * sizeof(float);
}

extern "C" int vt_suite_layernorm_bwd(const void *x, const void *w, const void *dy, const float *mean, const float *rstd, void *dx,
                                      float *dw, float *db, long long rows, int cols, void *workspace, size_t workspace_bytes, void *stream)
{
    int rc = norm_args_ok(x, w, dx, rows, cols, 8192);
    if (rc != VT_ATTN_OK) return rc;
    if (!ptr_ok(dy) || !ptr_ok(mean, 4) || !ptr_ok(rstd, 4) || !ptr_ok(dw) || !ptr_ok(db) || !ptr_ok(workspace)) return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (workspace_bytes < vt_suite_layernorm_bwd_workspace_bytes(cols)) return VT_ATTN_ERR_WORKSPACE_TOO_SMALL;
    if ((rc = check_device()) != VT_ATTN_OK) return rc;
    int t, nb;
    bwd_plan(cols, &t, &nb);
    const int g = static_cast<int>(rows < nb ? rows : nb);
    float *part = static_cast<float *>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    layernorm_bwd_kernel<false, LNB_VPT><<<g, t / LNB_VPT < 32 ? 32 : t / LNB_VPT, 0, st>>>(static_cast<const uint4 *>(x), static_cast<const uint4 *>(w), static_cast<const uint4 *>(dy), mean, rstd,
                                                 static_cast<uint4 *>(dx), part, rows, cols / 8, 1.0f / static_cast<float>(cols));
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "layernorm_bwd_kernel launch");
    layernorm_bwd_reduce_kernel<<<dim3((cols / 4 + 31) / 32, 2), dim3(32, 32), 0, st>>>(part, dw, db, g, cols);
    e = cudaGetLastError();
    return e == cudaSuccess ? VT_ATTN_OK : cuda_fail(e, "layernorm_bwd_reduce_kernel launch");
}

extern "C" int vt_suite_rmsnorm_bwd(const void *x, const void *w, const void *dy, const float *rstd, void *dx, float *dw, long long rows, int cols,
                                    void *workspace, size_t workspace_bytes, void *stream)
{
    int rc = norm_args_ok(x, w, dx, rows, cols, 8192);
    if (rc != VT_ATTN_OK) return rc;
    if (!ptr_ok(dy) || !ptr_ok(rstd, 4) || !ptr_ok(dw) || !ptr_ok(workspace)) return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (workspace_bytes < vt_suite_layernorm_bwd_workspace_bytes(cols)) return VT_ATTN_ERR_WORKSPACE_TOO_SMALL;
    if ((rc = check_device()) != VT_ATTN_OK) return rc;
    int t, nb;
    bwd_plan(cols, &t, &nb);
    const int g = static_cast<int>(rows < nb ? rows : nb);
    float *part = static_cast<float *>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    layernorm_bwd_kernel<true, LNB_VPT><<<g, t / LNB_VPT < 32 ? 32 : t / LNB_VPT, 0, st>>>(static_cast<const uint4 *>(x), static_cast<const uint4 *>(w), static_cast<const uint4 *>(dy), nullptr, rstd,
                                                static_cast<uint4 *>(dx), part, rows, cols / 8, 1.0f / static_cast<float>(cols));
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "layernorm_bwd_kernel<rms> launch");
    layernorm_bwd_reduce_kernel<<<dim3((cols / 4 + 31) / 32, 1), dim3(32, 32), 0, st>>>(part, dw, dw, g, cols);      // (only dw: blockIdx.y = 0)
    e = cudaGetLastError();
    return e == cudaSuccess ? VT_ATTN_OK : cuda_fail(e, "layernorm_bwd_reduce_kernel launch");
}

extern "C" int vt_suite_rope_tables(float *cos_t, float *sin_t, int S, int D, double base, void *stream)
{
    if (!ptr_ok(cos_t) || !ptr_ok(sin_t) || S <= 0 || D <= 0 || !(base > 0.0) || !isfinite(base)) return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (D % 16 != 0 || D > 512) return VT_ATTN_ERR_UNSUPPORTED;
    int rc = check_device();
    if (rc != VT_ATTN_OK) return rc;
    const long long n = static_cast<long long>(S) * (D / 2);
    if (n > 0x7FFFFFFFll) return VT_ATTN_ERR_INVALID_ARGUMENT;
    rope_tables_kernel<<<static_cast<int>((n + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(cos_t, sin_t, S, D / 2, base);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? VT_ATTN_OK : cuda_fail(e, "rope_tables_kernel launch");
}

extern "C" int vt_suite_rope_apply(const void *x, const float *cos_t, const float *sin_t, void *y, long long n_heads, int S, int D, int inverse,
                                   void *stream)
{
    if (!ptr_ok(x) || !ptr_ok(cos_t) || !ptr_ok(sin_t) || !ptr_ok(y) || n_heads <= 0 || S <= 0 || D <= 0) return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (D % 16 != 0 || D > 512) return VT_ATTN_ERR_UNSUPPORTED;
    const int hv = D / 16;
    if (static_cast<long long>(S) * hv > 0x7FFFFFFFll - 256) return VT_ATTN_ERR_INVALID_ARGUMENT;
    int rc = check_device();
    if (rc != VT_ATTN_OK) return rc;
    const int bx = (S * hv + 255) / 256;
    long long gy = (4 * NUM_SMS + bx - 1) / bx;          // enough blocks for a few per SM; the rest of the heads are walked by stride
    if (gy > n_heads) gy = n_heads;
    if (gy > 65535) gy = 65535;
    if (gy < 1) gy = 1;
    rope_apply_kernel<<<dim3(bx, static_cast<unsigned>(gy)), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4 *>(x), reinterpret_cast<const float4 *>(cos_t), reinterpret_cast<const float4 *>(sin_t),
        static_cast<uint4 *>(y), n_heads, S, hv, inverse ? -1.0f : 1.0f);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? VT_ATTN_OK : cuda_fail(e, "rope_apply_kernel launch");
}

// ----------------------------------------------------------------------------------------------
// Softmax, cross-entropy and AdamW (the suite's "softmax/loss" and "optimizers").
// ----------------------------------------------------------------------------------------------
namespace vt {

constexpr float SUITE_LOG2E = 1.4426950408889634f;
constexpr float SUITE_LN2 = 0.6931471805599453f;

__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, off));
    return v;
}

// Block-wide maximum; same single-barrier scheme as block_sum (red: two buffers of 32 floats).
__device__ __forceinline__ float block_max(float v, float *red, uint32_t &turn)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    v = warp_max(v);
    if (n_warps == 1) return v;
    float *buf = red + (turn & 1u) * 32;
    turn ^= 1u;
    if (lane == 0) buf[warp] = v;
    __syncthreads();
    return warp_max(lane < n_warps ? buf[lane] : -INFINITY);
}

// Row softmax from registers: maximum, exponentials (exp2 form) and their sum, one normalising pass.
template <int VPT, int T>
__global__ void __launch_bounds__(T) softmax_fwd_kernel(const uint4 *__restrict__ x, uint4 *__restrict__ y, long long rows, int nvec)
{
    __shared__ float red[128];
    uint32_t turn = 0;
    const int tid = threadIdx.x, nt = blockDim.x;
    for (long long row = blockIdx.x; row < rows; row += gridDim.x) {
        const uint4 *xr = x + row * nvec;
        float f[VPT][8];
        float mx = -INFINITY;
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
            if (v * nt + tid < nvec) {
                unpack8(xr[v * nt + tid], f[v]);
#pragma unroll
                for (int e = 0; e < 8; ++e) mx = fmaxf(mx, f[v][e]);
            }
        }
        mx = block_max(mx, red, turn);
        const float nm = (mx == -INFINITY) ? 0.0f : -mx * SUITE_LOG2E;      // (a row of -inf: exp2(-inf) = 0 everywhere, 0 / 0 below)
        float s[1] = {0.0f};
#pragma unroll
        for (int v = 0; v < VPT; ++v)
            if (v * nt + tid < nvec)
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    f[v][e] = exp2f(fmaf(f[v][e], SUITE_LOG2E, nm));
                    s[0] += f[v][e];
                }
        block_sum<1>(s, red + 64, turn);
        const float inv = 1.0f / s[0];
        uint4 *yr = y + row * nvec;
#pragma unroll
        for (int v = 0; v < VPT; ++v)
            if (v * nt + tid < nvec) {
#pragma unroll
                for (int e = 0; e < 8; ++e) f[v][e] *= inv;
                yr[v * nt + tid] = pack8(f[v]);
            }
    }
}

// Cross-entropy forward: one block per row at a time; a thread walks its vectors once, keeping a running maximum and the
// sum of exponentials about it (rescaled when the maximum moves), and picks up the target's logit when it passes it.
// The pairs (maximum, sum) are then merged over the block.  Any row length.
__global__ void __launch_bounds__(256) cross_entropy_fwd_kernel(const uint4 *__restrict__ x, const int *__restrict__ targets, float *__restrict__ loss,
                                                               float *__restrict__ lse_out, long long rows, int nvec)
{
    __shared__ float red[192];                            // the maximum's two buffers of 32, then the sums' two of 64
    uint32_t turn = 0;
    const int tid = threadIdx.x;
    for (long long row = blockIdx.x; row < rows; row += gridDim.x) {
        const uint4 *xr = x + row * nvec;
        const int tgt = targets[row];
        float m = -INFINITY, s = 0.0f, xt = 0.0f;
#pragma unroll 4
        for (int v = tid; v < nvec; v += 256) {
            float f[8];
            unpack8(xr[v], f);
            float m8 = f[0];
#pragma unroll
            for (int e = 1; e < 8; ++e) m8 = fmaxf(m8, f[e]);
            if (m8 > m) {
                s *= exp2f((m - m8) * SUITE_LOG2E);       // (m = -inf at first: s = 0 stays 0)
                m = m8;
            }
            const float nm = (m == -INFINITY) ? 0.0f : -m * SUITE_LOG2E;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                s += exp2f(fmaf(f[e], SUITE_LOG2E, nm));
                xt = (v * 8 + e == tgt) ? f[e] : xt;
            }
        }
        const float mb = block_max(m, red, turn);
        float t[2] = {(m == -INFINITY) ? 0.0f : s * exp2f((m - mb) * SUITE_LOG2E), xt};
        block_sum<2>(t, red + 64, turn);
        if (tid == 0) {
            const float l = mb + log2f(t[0]) * SUITE_LN2;
            lse_out[row] = l;
            loss[row] = l - t[1];
        }
    }
}

// Cross-entropy backward: dlogits = (exp(x - lse) - [column == target]) * dloss, elementwise with three per-row scalars.
__global__ void __launch_bounds__(256) cross_entropy_bwd_kernel(const uint4 *__restrict__ x, const int *__restrict__ targets, const float *__restrict__ lse,
                                                               const float *__restrict__ dloss, uint4 *__restrict__ dx, long long rows, int nvec)
{
    const long long n = rows * nvec;
    for (long long i = static_cast<long long>(blockIdx.x) * 256 + threadIdx.x; i < n; i += static_cast<long long>(gridDim.x) * 256) {
        const long long row = i / nvec;
        const int v = static_cast<int>(i - row * nvec);
        const float nl = -lse[row] * SUITE_LOG2E, dl = dloss[row];
        const int tgt = targets[row];
        float f[8];
        unpack8(x[i], f);
#pragma unroll
        for (int e = 0; e < 8; ++e) f[e] = (exp2f(fmaf(f[e], SUITE_LOG2E, nl)) - ((v * 8 + e == tgt) ? 1.0f : 0.0f)) * dl;
        dx[i] = pack8(f);
    }
}

// Cross-entropy forward and backward by one block per row: the forward's walk over the row (running maximum and sum of
// exponentials), then a second walk that writes the gradient.  The second read of the row comes from L2 (a row is
// 2 * cols bytes, the rows all resident blocks work on stay far below the 126 MB), so HBM sees the logits once and the
// gradient once: two thirds of the traffic of the two separate kernels.  Many small blocks per SM rather than the row in
// the registers of one large block: the phases of different rows overlap (a 1024-thread block per SM holding the row
// in registers was measured at 3.3 - 3.5 TB/s, no better than the two kernels).  Any row length.
__global__ void __launch_bounds__(256) cross_entropy_fwd_bwd_kernel(const uint4 *x, const int *__restrict__ targets,
                                                                   const float *__restrict__ dloss, float *__restrict__ loss,
                                                                   float *__restrict__ lse_out, uint4 *dx, long long rows, int nvec)   // (dx may be x)
{
    __shared__ float red[192];
    uint32_t turn = 0;
    const int tid = threadIdx.x;
    for (long long row = blockIdx.x; row < rows; row += gridDim.x) {
        const uint4 *xr = x + row * nvec;
        const int tgt = targets[row];
        float m = -INFINITY, s = 0.0f, xt = 0.0f;
#pragma unroll 4
        for (int v = tid; v < nvec; v += 256) {
            float f[8];
            unpack8(xr[v], f);
            float m8 = f[0];
#pragma unroll
            for (int e = 1; e < 8; ++e) m8 = fmaxf(m8, f[e]);
            if (m8 > m) {
                s *= exp2f((m - m8) * SUITE_LOG2E);
                m = m8;
            }
            const float nm = (m == -INFINITY) ? 0.0f : -m * SUITE_LOG2E;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                s += exp2f(fmaf(f[e], SUITE_LOG2E, nm));
                xt = (v * 8 + e == tgt) ? f[e] : xt;
            }
        }
        const float mb = block_max(m, red, turn);
        float t[2] = {(m == -INFINITY) ? 0.0f : s * exp2f((m - mb) * SUITE_LOG2E), xt};
        block_sum<2>(t, red + 64, turn);
        const float l = mb + log2f(t[0]) * SUITE_LN2;
        if (tid == 0) {
            lse_out[row] = l;
            loss[row] = l - t[1];
        }
        const float nl = -l * SUITE_LOG2E, dl = dloss[row];
        uint4 *dr = dx + row * nvec;
#pragma unroll 4
        for (int v = tid; v < nvec; v += 256) {
            float f[8];
            unpack8(xr[v], f);
#pragma unroll
            for (int e = 0; e < 8; ++e) f[e] = (exp2f(fmaf(f[e], SUITE_LOG2E, nl)) - ((v * 8 + e == tgt) ? 1.0f : 0.0f)) * dl;
            dr[v] = pack8(f);
        }
    }
}

// AdamW, four elements per thread: fp32 parameters and moments, bf16 gradients.
__global__ void __launch_bounds__(256) adamw_kernel(float4 *__restrict__ p, const uint2 *__restrict__ g, float4 *__restrict__ m, float4 *__restrict__ v,
                                                   long long n4, float decay, float b1, float b2, float step_size, float inv_sqrt_bc2, float eps)
{
    for (long long i = static_cast<long long>(blockIdx.x) * 256 + threadIdx.x; i < n4; i += static_cast<long long>(gridDim.x) * 256) {
        const float4 pp = p[i], mm = m[i], vv = v[i];
        const uint2 gw = g[i];
        const float2 g01 = unpack16<false>(gw.x), g23 = unpack16<false>(gw.y);
        const float gg[4] = {g01.x, g01.y, g23.x, g23.y};
        float pa[4] = {pp.x, pp.y, pp.z, pp.w}, ma[4] = {mm.x, mm.y, mm.z, mm.w}, va[4] = {vv.x, vv.y, vv.z, vv.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            ma[e] = fmaf(b1, ma[e], (1.0f - b1) * gg[e]);
            va[e] = fmaf(b2, va[e], (1.0f - b2) * gg[e] * gg[e]);
            pa[e] = pa[e] * decay - step_size * ma[e] / (sqrtf(va[e]) * inv_sqrt_bc2 + eps);
        }
        p[i] = make_float4(pa[0], pa[1], pa[2], pa[3]);
        m[i] = make_float4(ma[0], ma[1], ma[2], ma[3]);
        v[i] = make_float4(va[0], va[1], va[2], va[3]);
    }
}

}  // namespace vt

extern "C" int vt_suite_softmax_fwd(const void *x, void *y, long long rows, int cols, void *stream)
{
    if (!ptr_ok(x) || !ptr_ok(y) || rows <= 0 || cols <= 0) return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (cols % 8 != 0 || cols > 65536) return VT_ATTN_ERR_UNSUPPORTED;
    int rc = check_device();
    if (rc != VT_ATTN_OK) return rc;
    const int nvec = cols / 8;
    const uint4 *xp = static_cast<const uint4 *>(x);
    uint4 *yp = static_cast<uint4 *>(y);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (nvec > 8 * SUITE_THREADS) {
        softmax_fwd_kernel<8, 1024><<<row_grid(rows, 1024), 1024, 0, st>>>(xp, yp, rows, nvec);
    } else {
        int t, v;
        row_plan(nvec, &t, &v);
        const int g = row_grid(rows, t);
        switch (v) {
            case 1: softmax_fwd_kernel<1, SUITE_THREADS><<<g, t, 0, st>>>(xp, yp, rows, nvec); break;
            case 2: softmax_fwd_kernel<2, SUITE_THREADS><<<g, t, 0, st>>>(xp, yp, rows, nvec); break;
            case 4: softmax_fwd_kernel<4, SUITE_THREADS><<<g, t, 0, st>>>(xp, yp, rows, nvec); break;
            default: softmax_fwd_kernel<8, SUITE_THREADS><<<g, t, 0, st>>>(xp, yp, rows, nvec); break;
        }
    }
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? VT_ATTN_OK : cuda_fail(e, "softmax_fwd_kernel launch");
}

extern "C" int vt_suite_cross_entropy_fwd(const void *logits, const int *targets, float *loss, float *lse, long long rows, int cols, void *stream)
{
    if (!ptr_ok(logits) || !ptr_ok(targets, 4) || !ptr_ok(loss, 4) || !ptr_ok(lse, 4) || rows <= 0 || cols <= 0) return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (cols % 8 != 0) return VT_ATTN_ERR_UNSUPPORTED;
    int rc = check_device();
    if (rc != VT_ATTN_OK) return rc;
    const long long cap = static_cast<long long>(NUM_SMS) * 8;
    cross_entropy_fwd_kernel<<<static_cast<int>(rows < cap ? rows : cap), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4 *>(logits), targets, loss, lse, rows, cols / 8);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? VT_ATTN_OK : cuda_fail(e, "cross_entropy_fwd_kernel launch");
}

extern "C" int vt_suite_cross_entropy_bwd(const void *logits, const int *targets, const float *lse, const float *dloss, void *dlogits, long long rows,
                                          int cols, void *stream)
{
    if (!ptr_ok(logits) || !ptr_ok(targets, 4) || !ptr_ok(lse, 4) || !ptr_ok(dloss, 4) || !ptr_ok(dlogits) || rows <= 0 || cols <= 0)
        return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (cols % 8 != 0) return VT_ATTN_ERR_UNSUPPORTED;
    int rc = check_device();
    if (rc != VT_ATTN_OK) return rc;
    const long long n = rows * (cols / 8), cap = static_cast<long long>(NUM_SMS) * 16;
    long long nb = (n + 255) / 256;
    if (nb > cap) nb = cap;
    cross_entropy_bwd_kernel<<<static_cast<int>(nb), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4 *>(logits), targets, lse, dloss, static_cast<uint4 *>(dlogits), rows, cols / 8);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? VT_ATTN_OK : cuda_fail(e, "cross_entropy_bwd_kernel launch");
}

extern "C" int vt_suite_cross_entropy_fwd_bwd(const void *logits, const int *targets, const float *dloss, float *loss, float *lse, void *dlogits,
                                              long long rows, int cols, void *stream)
{
    if (!ptr_ok(logits) || !ptr_ok(targets, 4) || !ptr_ok(dloss, 4) || !ptr_ok(loss, 4) || !ptr_ok(lse, 4) || !ptr_ok(dlogits) || rows <= 0 || cols <= 0)
        return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (cols % 8 != 0) return VT_ATTN_ERR_UNSUPPORTED;
    int rc = check_device();
    if (rc != VT_ATTN_OK) return rc;
    const long long cap = static_cast<long long>(NUM_SMS) * 8;
    cross_entropy_fwd_bwd_kernel<<<static_cast<int>(rows < cap ? rows : cap), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4 *>(logits), targets, dloss, loss, lse, static_cast<uint4 *>(dlogits), rows, cols / 8);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? VT_ATTN_OK : cuda_fail(e, "cross_entropy_fwd_bwd_kernel launch");
}

extern "C" int vt_suite_adamw_step(float *p, const void *g, float *m, float *v, long long n, int step, float lr, float beta1, float beta2, float eps,
                                   float weight_decay, void *stream)
{
    if (!ptr_ok(p) || !ptr_ok(g, 8) || !ptr_ok(m) || !ptr_ok(v) || n <= 0 || step < 1) return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (!(lr >= 0.0f) || !(beta1 >= 0.0f && beta1 < 1.0f) || !(beta2 >= 0.0f && beta2 < 1.0f) || !(eps >= 0.0f) || !(weight_decay >= 0.0f) ||
        !isfinite(lr) || !isfinite(eps) || !isfinite(weight_decay))
        return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (n % 4 != 0) return VT_ATTN_ERR_UNSUPPORTED;
    int rc = check_device();
    if (rc != VT_ATTN_OK) return rc;
    // the bias corrections in double precision on the host; the kernel gets lr / (1 - b1^t) and 1 / sqrt(1 - b2^t)
    const double bc1 = 1.0 - pow(static_cast<double>(beta1), step), bc2 = 1.0 - pow(static_cast<double>(beta2), step);
    const long long n4 = n / 4, cap = static_cast<long long>(NUM_SMS) * 16;
    long long nb = (n4 + 255) / 256;
    if (nb > cap) nb = cap;
    adamw_kernel<<<static_cast<int>(nb), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        reinterpret_cast<float4 *>(p), static_cast<const uint2 *>(g), reinterpret_cast<float4 *>(m), reinterpret_cast<float4 *>(v), n4,
        1.0f - lr * weight_decay, beta1, beta2, static_cast<float>(lr / bc1), static_cast<float>(1.0 / sqrt(bc2)), eps);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? VT_ATTN_OK : cuda_fail(e, "adamw_kernel launch");
}
