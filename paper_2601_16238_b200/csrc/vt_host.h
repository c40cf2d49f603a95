// Host-side helpers shared by the entry points: argument checks, tensor-map encoding,
// the per-device status word and CUDA error bookkeeping.  Internal to the library.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <atomic>

#include "../../include/vt_attn.h"
#include "vt_ptx.cuh"

namespace vt {

constexpr int TILE = 128;                 // query rows and key rows per tile
constexpr int BOX_COLS = 64;              // 16-bit elements per 128-byte swizzled row
constexpr int NUM_SMS = 148;              // B200: grid sizes and dispatch thresholds are stated in multiples of this
constexpr unsigned long long DEFAULT_WAIT_LIMIT_NS = 2000000000ull;   // 2 s per wait

// Head dimensions: multiples of 8 (rows stay 16-byte aligned) up to 128, in the forward kernels up to 256.  The kernels are
// built for 64, 128 and (forward only) 256 columns; any other dimension runs in the next larger one: the TMA boxes read
// the columns past the row's end as zero, which adds nothing to S = Q K^T, and the epilogues store only the real columns.
constexpr int MAX_HEAD_DIM = 128;          // packed and split-KV entry points, the one-pass kernels
constexpr int MAX_HEAD_DIM_FWD = 256;      // batched forward and backward (the backward above 128 columns: bwd_wide.cu)
inline bool head_dim_ok(int D, int max_d = MAX_HEAD_DIM) { return D >= 8 && D <= max_d && D % 8 == 0; }
inline int padded_head_dim(int D) { return D <= 64 ? 64 : (D <= 128 ? 128 : 256); }

// Heads per scheduling group of a causal launch (causal_work_item in vt_ptx.cuh); 0: one head after the other.
// heads x n_items work items (a head's items are 1 .. n_items tiles long), `slots` blocks resident on the GPU at one
// time, G: query heads that share a KV head; bytes_per_head: what the items of one head read of the tensors they walk.
// Larger groups end the launch on shorter items, but the blocks resident at one time then spread over more heads: with
// at most NUM_SMS / 8 heads in a group every head keeps eight or more of its items resident, which walk its K / V
// together, and the group's tensors are held to 96 MB (they are read as a moving window, so this is generous).  The heads
// are divided evenly: a small last group would end the launch like no grouping at all.  A group holds whole KV groups.
// What grouping can save is part of one longest item per SM; a launch that lasts more than eight of those is left in
// head order (measured: nothing to gain there, and the wider spread of the reads costs a little under the power cap).
inline int causal_head_group(long long heads, int n_items, int slots, int G, long long bytes_per_head)
{
    long long cap = NUM_SMS / 8;
    const long long budget = 96ll << 20;
    if (bytes_per_head > 0 && cap * bytes_per_head > budget) cap = budget / bytes_per_head;
    if (heads <= 1 || cap <= 1 || heads * n_items > 16ll * slots) return 0;
    const long long n_groups = (heads + cap - 1) / cap;
    long long group = (heads + n_groups - 1) / n_groups;
    if (G > 1 && group > G) group = (group + G - 1) / G * G;
    return static_cast<int>(group < heads ? group : heads);
}

struct Shape {
    int B, Hq, Hkv, Sq, Sk, D;
};

// VT_ATTN_OK, or the error a bad shape / scale maps to.
int check_shape(const Shape &s, float scale, int max_d = MAX_HEAD_DIM);

// true when p is non-null and aligned to `align` bytes
inline bool ptr_ok(const void *p, size_t align = 16)
{
    return p != nullptr && (reinterpret_cast<uintptr_t>(p) % align) == 0;
}

// Records a CUDA error for vt_attn_last_cuda_error and returns VT_ATTN_ERR_CUDA.
int cuda_fail(cudaError_t e, const char *what);
int cu_fail(CUresult r, const char *what);

// VT_ATTN_OK if the current device is compute capability 10.x.
int check_device();

// Device address of the current device's status word (set up once per device), or nullptr.
unsigned int *status_word_ptr();

Guard make_guard();

// Tensor map over a bf16 tensor [BH, S, D] (D innermost): box = 64 columns x box_rows rows
// x 1, 128-byte swizzle, out-of-range rows read as zero.
int make_tensor_map(CUtensorMap *map, const void *base, int BH, int S, int D, int box_rows);

// Tensor map over a packed bf16 tensor [total, H, D] (token-major): seen as (D, H, total) with boxes of
// 64 columns x 1 head x box_rows tokens, so a box lands in shared memory exactly like a box of the map above.
// Tokens past `total` read as zero; tokens of the next sequence do not (the kernels mask them).
int make_tensor_map_packed(CUtensorMap *map, const void *base, int total, int H, int D, int box_rows);

// Tensor map over a bf16 tensor [BH, S, D] whose box spans `rows` rows of `heads` consecutive heads (64 columns x rows x
// heads, rows * heads <= 128): in shared memory the box is a tile whose row index is head * rows + row.
int make_tensor_map_heads(CUtensorMap *map, const void *base, int BH, int S, int D, int rows, int heads);

// Tensor map over a packed bf16 tensor [total, H, D] whose box spans `heads` consecutive heads of `tokens` consecutive
// tokens (64 columns x heads x tokens, heads * tokens <= 128): in shared memory the row index is token * heads + head.
int make_tensor_map_packed_heads(CUtensorMap *map, const void *base, int total, int H, int D, int tokens, int heads);

// Checks shared by the variable-length entry points.
int check_varlen_shape(int n_seqs, int Hq, int Hkv, int total_q, int total_k, int max_sq, int max_sk, int D, float scale);

}  // namespace vt
