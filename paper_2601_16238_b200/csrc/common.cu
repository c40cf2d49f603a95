// Status codes, argument checks, tensor-map encoding and the device status word.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <mutex>

#include "vt_host.h"

namespace vt {

// One word per device that loads the library: 0 = clean, else where a bounded wait gave up.
__device__ unsigned int g_status_word = 0;

static thread_local char t_last_error[256] = "";

int cuda_fail(cudaError_t e, const char *what)
{
    snprintf(t_last_error, sizeof(t_last_error), "%s: %s", what, cudaGetErrorString(e));
    return VT_ATTN_ERR_CUDA;
}

int cu_fail(CUresult r, const char *what)
{
    snprintf(t_last_error, sizeof(t_last_error), "%s: CUresult %d", what, static_cast<int>(r));
    return VT_ATTN_ERR_CUDA;
}

int check_shape(const Shape &s, float scale, int max_d)
{
    if (s.B <= 0 || s.Hq <= 0 || s.Hkv <= 0 || s.Sq <= 0 || s.Sk <= 0 || s.D <= 0) return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (s.Hq % s.Hkv != 0) return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (s.Sq > (1 << 24) || s.Sk > (1 << 24)) return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (static_cast<long long>(s.B) * s.Hq > 0x7FFFFFFFll) return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (!(scale > 0.0f) || !isfinite(scale)) return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (!head_dim_ok(s.D, max_d)) return VT_ATTN_ERR_UNSUPPORTED;
    return VT_ATTN_OK;
}

static std::mutex g_mutex;
static int g_device_cc[64];           // 0 = unknown, else major*10+minor
static unsigned int *g_status_ptr[64];

int check_device()
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    if (dev < 0 || dev >= 64) return VT_ATTN_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_device_cc[dev] == 0) {
        int major = 0, minor = 0;
        e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
        if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceGetAttribute");
        e = cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev);
        if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceGetAttribute");
        g_device_cc[dev] = major * 10 + minor;
    }
    return (g_device_cc[dev] / 10 == 10) ? VT_ATTN_OK : VT_ATTN_ERR_UNSUPPORTED;
}

unsigned int *status_word_ptr()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_status_ptr[dev] == nullptr) {
        void *p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_status_word);
        if (e != cudaSuccess) {
            cuda_fail(e, "cudaGetSymbolAddress(status word)");
            return nullptr;
        }
        g_status_ptr[dev] = static_cast<unsigned int *>(p);
    }
    return g_status_ptr[dev];
}

Guard make_guard()
{
    Guard g;
    g.status = status_word_ptr();
    g.limit_ns = DEFAULT_WAIT_LIMIT_NS;
    return g;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

// Encoding a tensor map costs about a microsecond of host time, which matters for the small
// shapes whose kernels run for a few microseconds.  A map depends only on (base, BH, S, D,
// box_rows), so recent ones are kept in a small cache.  A stale entry cannot do harm: the same key
// always encodes to the same 128 bytes.
struct MapKey {
    const void *base;
    int BH, S, D, box_rows;      // packed maps: BH = -H, S = total
    bool operator==(const MapKey &o) const { return base == o.base && BH == o.BH && S == o.S && D == o.D && box_rows == o.box_rows; }
};
constexpr int MAP_CACHE_SIZE = 64;
static MapKey g_map_keys[MAP_CACHE_SIZE];
static CUtensorMap g_map_vals[MAP_CACHE_SIZE];
static int g_map_count = 0, g_map_next = 0;
static std::mutex g_map_mutex;

static int make_map_cached(CUtensorMap *map, const MapKey &key, const cuuint64_t (&dims)[3], const cuuint64_t (&strides)[2],
                           const cuuint32_t (&box)[3])
{
    {
        std::lock_guard<std::mutex> lock(g_map_mutex);
        for (int i = 0; i < g_map_count; ++i)
            if (g_map_keys[i] == key) {
                *map = g_map_vals[i];
                return VT_ATTN_OK;
            }
    }
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) {
        snprintf(t_last_error, sizeof(t_last_error), "cuTensorMapEncodeTiled entry point not found");
        return VT_ATTN_ERR_CUDA;
    }
    cuuint32_t estr[3] = {1u, 1u, 1u};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(key.base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cu_fail(r, "cuTensorMapEncodeTiled");
    {
        std::lock_guard<std::mutex> lock(g_map_mutex);
        const int slot = (g_map_count < MAP_CACHE_SIZE) ? g_map_count++ : (g_map_next++ % MAP_CACHE_SIZE);
        g_map_keys[slot] = key;
        g_map_vals[slot] = *map;
    }
    return VT_ATTN_OK;
}

int make_tensor_map(CUtensorMap *map, const void *base, int BH, int S, int D, int box_rows)
{
    const cuuint64_t dims[3] = {static_cast<cuuint64_t>(D), static_cast<cuuint64_t>(S), static_cast<cuuint64_t>(BH)};
    const cuuint64_t strides[2] = {static_cast<cuuint64_t>(D) * 2ull, static_cast<cuuint64_t>(S) * D * 2ull};
    const cuuint32_t box[3] = {static_cast<cuuint32_t>(BOX_COLS), static_cast<cuuint32_t>(box_rows), 1u};
    return make_map_cached(map, MapKey{base, BH, S, D, box_rows}, dims, strides, box);
}

int make_tensor_map_packed(CUtensorMap *map, const void *base, int total, int H, int D, int box_rows)
{
    const cuuint64_t dims[3] = {static_cast<cuuint64_t>(D), static_cast<cuuint64_t>(H), static_cast<cuuint64_t>(total)};
    const cuuint64_t strides[2] = {static_cast<cuuint64_t>(D) * 2ull, static_cast<cuuint64_t>(H) * D * 2ull};
    const cuuint32_t box[3] = {static_cast<cuuint32_t>(BOX_COLS), 1u, static_cast<cuuint32_t>(box_rows)};
    return make_map_cached(map, MapKey{base, -H, total, D, box_rows}, dims, strides, box);
}

int make_tensor_map_heads(CUtensorMap *map, const void *base, int BH, int S, int D, int rows, int heads)
{
    const cuuint64_t dims[3] = {static_cast<cuuint64_t>(D), static_cast<cuuint64_t>(S), static_cast<cuuint64_t>(BH)};
    const cuuint64_t strides[2] = {static_cast<cuuint64_t>(D) * 2ull, static_cast<cuuint64_t>(S) * D * 2ull};
    const cuuint32_t box[3] = {static_cast<cuuint32_t>(BOX_COLS), static_cast<cuuint32_t>(rows), static_cast<cuuint32_t>(heads)};
    return make_map_cached(map, MapKey{base, BH, S, D, -(heads * 65536 + rows)}, dims, strides, box);
}

int make_tensor_map_packed_heads(CUtensorMap *map, const void *base, int total, int H, int D, int tokens, int heads)
{
    const cuuint64_t dims[3] = {static_cast<cuuint64_t>(D), static_cast<cuuint64_t>(H), static_cast<cuuint64_t>(total)};
    const cuuint64_t strides[2] = {static_cast<cuuint64_t>(D) * 2ull, static_cast<cuuint64_t>(H) * D * 2ull};
    const cuuint32_t box[3] = {static_cast<cuuint32_t>(BOX_COLS), static_cast<cuuint32_t>(heads), static_cast<cuuint32_t>(tokens)};
    return make_map_cached(map, MapKey{base, -H, total, D, -(heads * 65536 + tokens)}, dims, strides, box);
}

int check_varlen_shape(int n_seqs, int Hq, int Hkv, int total_q, int total_k, int max_sq, int max_sk, int D, float scale)
{
    if (n_seqs <= 0 || Hq <= 0 || Hkv <= 0 || total_q <= 0 || total_k <= 0 || max_sq <= 0 || max_sk <= 0 || D <= 0)
        return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (Hq % Hkv != 0 || max_sq > total_q || max_sk > total_k) return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (max_sq > (1 << 24) || max_sk > (1 << 24)) return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (static_cast<long long>(n_seqs) * Hq > 0x7FFFFFFFll) return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (!(scale > 0.0f) || !isfinite(scale)) return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (!head_dim_ok(D)) return VT_ATTN_ERR_UNSUPPORTED;
    return VT_ATTN_OK;
}

}  // namespace vt

extern "C" {

int vt_attn_abi_version(void) { return VT_ATTN_ABI_VERSION; }

const char *vt_attn_status_string(int status)
{
    switch (status) {
        case VT_ATTN_OK: return "ok";
        case VT_ATTN_ERR_INVALID_ARGUMENT: return "invalid argument";
        case VT_ATTN_ERR_UNSUPPORTED: return "unsupported head dimension or device";
        case VT_ATTN_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case VT_ATTN_ERR_CUDA: return "CUDA call failed";
        case VT_ATTN_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel expired";
        case VT_ATTN_ERR_STATIC_SCRATCH_TOO_SMALL:
            return "B*Hq*Sq exceeds the built-in scratch of vt_attn_bwd_static_scratch; use vt_attn_bwd with a workspace";
        default: return "unknown status";
    }
}

const char *vt_attn_last_cuda_error(void) { return vt::t_last_error; }

int vt_attn_device_status(unsigned int *detail, void *stream)
{
    unsigned int *p = vt::status_word_ptr();
    if (!p) return VT_ATTN_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    unsigned int word = 0;
    cudaError_t e = cudaMemcpyAsync(&word, p, sizeof(word), cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return vt::cuda_fail(e, "cudaMemcpyAsync(status)");
    e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return vt::cuda_fail(e, "cudaStreamSynchronize");
    if (detail) *detail = word;
    if (word != 0) {
        e = cudaMemsetAsync(p, 0, sizeof(word), s);
        if (e != cudaSuccess) return vt::cuda_fail(e, "cudaMemsetAsync(status)");
        e = cudaStreamSynchronize(s);
        if (e != cudaSuccess) return vt::cuda_fail(e, "cudaStreamSynchronize");
        return VT_ATTN_ERR_DEVICE_TIMEOUT;
    }
    return VT_ATTN_OK;
}

int vt_attn_device_status_async(unsigned int *word_host, void *stream)
{
    if (!word_host) return VT_ATTN_ERR_INVALID_ARGUMENT;
    unsigned int *p = vt::status_word_ptr();
    if (!p) return VT_ATTN_ERR_CUDA;
    cudaError_t e = cudaMemcpyAsync(word_host, p, sizeof(unsigned int), cudaMemcpyDeviceToHost, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return vt::cuda_fail(e, "cudaMemcpyAsync(status)");
    return VT_ATTN_OK;
}

int vt_attn_device_status_clear(void *stream)
{
    unsigned int *p = vt::status_word_ptr();
    if (!p) return VT_ATTN_ERR_CUDA;
    cudaError_t e = cudaMemsetAsync(p, 0, sizeof(unsigned int), static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return vt::cuda_fail(e, "cudaMemsetAsync(status)");
    return VT_ATTN_OK;
}

}  // extern "C"
