/*
 * vt_attn.h — C ABI of the B200 (sm_100a) fused-attention library.
 *
 * The paper describes a versioned, stable C ABI through which dynamically loaded
 * operator plugins reach its runtime (section "Interoperability and extension
 * points") but prints no signatures.  This header is that idea applied to the one
 * operator the paper benchmarks against torch scaled_dot_product_attention
 * (kernel-microbenchmark table, rows "Attention (fwd)" and "Attention (bwd)").
 *
 * Conventions shared by every entry point
 *   - Plain C types only.  Unless a parameter says "host", every data pointer is a
 *     DEVICE pointer to memory on the current CUDA device, 16-byte aligned.
 *   - Tensor layout is row-major [B, H, S, D] with D innermost and no padding.
 *     Q, O, dO, dQ use H = Hq; K, V, dK, dV use H = Hkv.  Query head h reads KV head
 *     h / (Hq / Hkv) (consecutive query heads share one KV head).
 *   - Element type of Q, K, V, O, dO, dQ, dK, dV is bfloat16 (fp16 in the two *_f16 entry points); LSE is float.
 *   - Products accumulate in fp32.
 *   - causal selects the mask: 0 none; 1 key j is visible to query i iff j <= i
 *     (top-left aligned, also when Sq != Sk: key 0 is always visible, no row is
 *     empty; this is the mask of the paper's benchmark rows, which are square);
 *     2 key j is visible iff j <= i + (Sk - Sq) (bottom-right aligned: the queries
 *     are the last Sq positions of a sequence of Sk keys - chunked prefill or
 *     decoding against a cache; the paper has no counterpart, its shapes have
 *     Sq == Sk where 1 and 2 coincide).  With causal = 2 and Sk < Sq the first
 *     Sq - Sk query rows see no key: they get O = 0, LSE = -inf and contribute
 *     nothing to any gradient.  Any other value: VT_ATTN_ERR_INVALID_ARGUMENT.
 *   - The caller owns every buffer.  The library allocates no device memory and
 *     keeps no state between calls apart from a per-device status word, a cache of
 *     tensor-map descriptors and (for the *_host entry points) two streams per device.
 *   - Calls enqueue work on `stream` (a cudaStream_t passed as void*, NULL = the
 *     legacy default stream) and return without synchronising.
 *   - Return value: VT_ATTN_OK or a negative VT_ATTN_ERR_* code.  Nothing throws.
 *     On an argument, shape or workspace error nothing has been launched.  After
 *     VT_ATTN_ERR_CUDA (a launch or a driver call failed part-way through an entry point
 *     that enqueues several kernels) the outputs are undefined.
 *   - Threads: calls from different host threads are safe on different streams.  The
 *     *_host entry points serialise their enqueueing inside the library (one call at a
 *     time forks onto the library's two streams and joins back), and two such calls
 *     that are in flight together on one device must not share a staging area.
 *   - Supported: D a multiple of 8 in [8, 128]; in the entry points that take
 *     [B, H, S, D] tensors (vt_attn_fwd, vt_attn_bwd, their _f16 twins, vt_attn_fwd_splitkv)
 *     and the merge entry points up to 256.  The kernels are built for 64, 128 and 256
 *     columns; another D runs in the next larger one at that one's cost, its rows are still
 *     D elements long in memory.  B, Hq, Hkv, Sq, Sk >= 1; Hq % Hkv == 0;
 *     B * Hq and B * Hkv at most 2^31 - 1; Sq, Sk at most 2^24; scale finite, > 0.
 */
#ifndef VT_ATTN_H_
#define VT_ATTN_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

#define VT_ATTN_ABI_VERSION 1

#define VT_ATTN_OK 0
#define VT_ATTN_ERR_INVALID_ARGUMENT (-1)    /* null/misaligned pointer, bad shape or scale */
#define VT_ATTN_ERR_UNSUPPORTED (-2)         /* head dim not a multiple of 8 in [8,256] ([8,128] in the packed entry points); device is not sm_100 */
#define VT_ATTN_ERR_WORKSPACE_TOO_SMALL (-3) /* workspace_bytes below vt_attn_bwd_workspace_bytes */
#define VT_ATTN_ERR_CUDA (-4)                /* a CUDA runtime / driver call failed */
#define VT_ATTN_ERR_DEVICE_TIMEOUT (-5)      /* reported by vt_attn_device_status only */
#define VT_ATTN_ERR_STATIC_SCRATCH_TOO_SMALL (-6) /* shape needs more than the built-in scratch */

/* ABI version the library was built with (compare with VT_ATTN_ABI_VERSION). */
int vt_attn_abi_version(void);

/* Static, human-readable text for a status code.  Never NULL. */
const char *vt_attn_status_string(int status);

/* Text of the last CUDA error seen by the calling thread inside this library ("" if none). */
const char *vt_attn_last_cuda_error(void);

/*
 * Forward pass ("Attention (fwd)" row of the kernel-microbenchmark table;
 * flash-attention-style stabilised softmax as in the debugging-episodes table,
 * row "log2 vs ln scaling"):
 *
 *   s_ij = scale * <Q[b,h,i,:], K[b,g,j,:]>,  masked as `causal` says (see above)
 *   LSE[b,h,i] = ln sum_j exp(s_ij)                       (natural log)
 *   O[b,h,i,:] = sum_j exp(s_ij - LSE[b,h,i]) * V[b,g,j,:]
 *
 * q [B,Hq,Sq,D], k and v [B,Hkv,Sk,D] : bf16, read only.
 * o [B,Hq,Sq,D] bf16 and lse [B,Hq,Sq] float : fully overwritten.
 */
int vt_attn_fwd(const void *q, const void *k, const void *v,
                void *o, float *lse,
                int B, int Hq, int Hkv, int Sq, int Sk, int D,
                int causal, float scale, void *stream);

/*
 * vt_attn_fwd with the rotary position embedding of the QUERIES applied inside the kernel
 * (the paper's kernel microbenchmark table has "Rotary (fwd)" as a row of its own; this takes
 * the query half of that operator into the attention kernel's load path, saving its pass
 * over Q in global memory).  q is unrotated; every query tile is rotated in shared memory, in
 * fp32 and rounded to bf16, before the first product: "rotate-half" convention, element i of a
 * head pairs with element i + D/2, query i of the sequence sits at position q_pos0 + i:
 *     q'[i] = q[i] cos[pos][i] - q[i + D/2] sin[pos][i],   q'[i + D/2] = q[i + D/2] cos[pos][i] + q[i] sin[pos][i]
 * k_rotated must hold the ALREADY rotated keys (vt_suite_rope_apply): a key tile is read by
 * every query tile of its head, rotating it inside the kernel would repeat the work each time.
 * rope_cos, rope_sin: float [rope_positions, D/2] (vt_suite_rope_tables), device, 16-byte
 * aligned; q_pos0 + Sq <= rope_positions.  D must be 64 or 128.  Everything else as vt_attn_fwd.
 */
int vt_attn_fwd_rope(const void *q, const void *k_rotated, const void *v,
                     const float *rope_cos, const float *rope_sin,
                     void *o, float *lse,
                     int B, int Hq, int Hkv, int Sq, int Sk, int D,
                     int causal, float scale, int q_pos0, int rope_positions, void *stream);

/*
 * Bytes of device scratch vt_attn_bwd needs for this shape (0 on an invalid shape).
 * The scratch holds Delta[b,h,i] = sum_d dO*O in fp32 and, for the shapes that take the
 * single-pass backward (vt_attn_bwd_kernel_kind), a 32-bit accumulator per element of dQ
 * plus a few per-head scalars.  Its contents on entry are ignored; every word that is
 * read is written first by the same call.
 */
size_t vt_attn_bwd_workspace_bytes(int B, int Hq, int Hkv, int Sq, int Sk, int D);

/*
 * Which kernels vt_attn_bwd runs for a shape when it is given the workspace size stated
 * above (host-only, launches nothing; a negative VT_ATTN_ERR_* for an invalid shape):
 *   0  three kernels: Delta, then one kernel per key tile for dK / dV and one per query tile
 *      for dQ; each output tile has one owner block (7 tile products per tile pair);
 *   1  the single-pass backward, built for 64 < D <= 128: one kernel per key tile forms dK,
 *      dV and that tile's share of dQ (5 tile products per tile pair); the shares are summed
 *      in 32-bit fixed point, scaled per (batch, head) from bounds on dO, K and V, so the sum
 *      does not depend on the order in which the blocks add and dQ is the same bits on every
 *      run; a last pass rounds it to the tensors' type.  Six kernels and one memset per call.
 *   2  D above 128 (up to 256): Delta, a dK / dV kernel that keeps 128 keys stationary and
 *      walks the queries 64 at a time, once per half of the output columns, and a dQ kernel
 *      that keeps 128 queries stationary and walks the keys 64 at a time.
 * For D <= 128 the library itself always answers 0: on the B200 the reductions of 1 cost more than the two
 * products they save.  The environment variable VT_ATTN_BWD_PATH=fused (read at every call)
 * selects 1 wherever it is built, for measurements and tests; =split or unset selects 0.  A
 * call whose workspace only holds Delta (vt_attn_bwd_static_scratch does this) takes 0 too.
 */
int vt_attn_bwd_kernel_kind(int B, int Hq, int Hkv, int Sq, int Sk, int D);

/*
 * Backward pass ("Attention (bwd)" row of the same table).  With P recomputed from
 * the forward's LSE, P_ij = exp(s_ij - LSE_i):
 *
 *   Delta_i = sum_d dO[i,d] * O[i,d]
 *   dS_ij   = P_ij * (<dO_i, V_j> - Delta_i)
 *   dQ_i    = scale * sum_j dS_ij K_j
 *   dK_j    = scale * sum_{h in group} sum_i dS_ij Q_i
 *   dV_j    =         sum_{h in group} sum_i P_ij  dO_i
 *
 * q, k, v, o, d_o (bf16) and lse (float) are read only; o and lse must be the
 * outputs of vt_attn_fwd on the same q, k, v, causal and scale.
 * dq [B,Hq,Sq,D], dk and dv [B,Hkv,Sk,D] (bf16) are fully overwritten; every sum
 * is taken in a fixed order or in integer arithmetic, so repeated calls give
 * bit-identical results.
 * workspace: device scratch of at least vt_attn_bwd_workspace_bytes(...) bytes,
 * 256-byte aligned, owned by the caller, not shared with a concurrent call.
 */
int vt_attn_bwd(const void *q, const void *k, const void *v,
                const void *o, const void *d_o, const float *lse,
                void *dq, void *dk, void *dv,
                int B, int Hq, int Hkv, int Sq, int Sk, int D,
                int causal, float scale,
                void *workspace, size_t workspace_bytes, void *stream);

/*
 * Backward pass for callers that cannot allocate device memory.  (The paper has no
 * counterpart; this is an addition of this library.)
 *
 * Some callers have nowhere to get the scratch buffer vt_attn_bwd asks for: code that
 * runs under a framework whose allocator it must not re-enter (an allocator hook, a
 * destructor, a signal-like callback), code inside a memory pool that is already fixed
 * or exhausted, or a plugin host that only hands out the tensors of the operator's
 * signature.  For them the Delta scratch lives in a fixed array inside the library's
 * device image instead: VT_ATTN_STATIC_SCRATCH_ROWS floats (4 MiB), which every GPU
 * that loads the library holds until the process exits.
 *
 * Same inputs, outputs, formulas and error behaviour as vt_attn_bwd, minus the two
 * workspace arguments.  Differences:
 *   - B * Hq * Sq must not exceed VT_ATTN_STATIC_SCRATCH_ROWS, otherwise the call
 *     returns VT_ATTN_ERR_STATIC_SCRATCH_TOO_SMALL and launches nothing.
 *   - The call itself makes no cudaMalloc, cudaFree or other allocating call.
 *   - The first call on each device looks up the array's device address (the device
 *     must be current).  Make that first call outside any stream capture.
 *   - All calls on one device share the one array, and it keeps whatever the last
 *     call left there.  Nothing in it has to start at zero: each call writes every
 *     Delta value it later reads.  Two calls whose kernels may overlap on the GPU
 *     (different streams, no ordering between them) race on the array and give
 *     wrong gradients; order them, or use vt_attn_bwd with separate workspaces.
 */
#define VT_ATTN_STATIC_SCRATCH_ROWS (1 << 20)
int vt_attn_bwd_static_scratch(const void *q, const void *k, const void *v,
                               const void *o, const void *d_o, const float *lse,
                               void *dq, void *dk, void *dv,
                               int B, int Hq, int Hkv, int Sq, int Sk, int D,
                               int causal, float scale, void *stream);
/* The same on IEEE half tensors (vt_attn_bwd_f16 with the library's array); shares the array with the call above. */
int vt_attn_bwd_static_scratch_f16(const void *q, const void *k, const void *v,
                                   const void *o, const void *d_o, const float *lse,
                                   void *dq, void *dk, void *dv,
                                   int B, int Hq, int Hkv, int Sq, int Sk, int D,
                                   int causal, float scale, void *stream);

/*
 * Variable-length ("packed") batches: the ragged batches of real training loops, where
 * documents of different lengths are concatenated instead of padded.  The paper's
 * attention rows use a fixed "batch 32, sequence length 2048" shape (kernel
 * microbenchmark table) and name ragged cases only as "small-batch GQA prefill";
 * the operation is the same attention, applied to every sequence on its own.
 *
 * Layout: q, o [total_q, Hq, D]; k, v [total_k, Hkv, D] (token-major, bf16);
 * lse [Hq, total_q] (float).  Sequence i owns the token rows
 * [cu_seqlens_q[i], cu_seqlens_q[i+1]) of q / o and [cu_seqlens_k[i], cu_seqlens_k[i+1])
 * of k / v.  cu_seqlens_*: DEVICE int32 arrays of n_seqs + 1 entries, starting at 0,
 * non-decreasing, ending at total_q / total_k (not checked: they live on the device).
 * max_sq / max_sk: at least the longest query / key sequence; tokens of a sequence
 * beyond them are not processed.  causal: as above with i, j, Sq, Sk taken inside the
 * sequence (1: j <= i; 2: j <= i + Sk_seq - Sq_seq).  A sequence without queries costs
 * nothing; one without keys gets O = 0 and LSE = -inf.
 */
int vt_attn_fwd_varlen(const void *q, const void *k, const void *v, void *o, float *lse,
                       const int *cu_seqlens_q, const int *cu_seqlens_k,
                       int n_seqs, int Hq, int Hkv, int total_q, int total_k,
                       int max_sq, int max_sk, int D,
                       int causal, float scale, void *stream);

/*
 * vt_attn_fwd with V (and O) of their own head dimension Dv, e.g. Q, K of 192 columns against V of
 * 128: q [B, Hq, Sq, D], k [B, Hkv, Sk, D], v [B, Hkv, Sk, Dv], o [B, Hq, Sq, Dv], bfloat16;
 * D and Dv multiples of 8 in [8, 256].  Runs in the kernel built for the larger of the two (rounded
 * up to 64, 128 or 256 columns).  Its backward is vt_attn_bwd_dv.
 */
int vt_attn_fwd_dv(const void *q, const void *k, const void *v, void *o, float *lse,
                   int B, int Hq, int Hkv, int Sq, int Sk, int D, int Dv,
                   int causal, float scale, void *stream);
/* The same on IEEE half tensors. */
int vt_attn_fwd_dv_f16(const void *q, const void *k, const void *v, void *o, float *lse,
                       int B, int Hq, int Hkv, int Sq, int Sk, int D, int Dv,
                       int causal, float scale, void *stream);

/*
 * The backward of vt_attn_fwd_dv: V, O, dO and dV have Dv columns, Q, K, dQ and dK have D (both
 * multiples of 8 up to 256, e.g. 192 / 128; the paper has no counterpart).  Same formulas,
 * buffers and workspace (vt_attn_bwd_workspace_bytes(B, Hq, Hkv, Sq, Sk, D)) as vt_attn_bwd, to
 * which the call forwards when Dv == D; other pairs run in the kernels built for head
 * dimensions above 128 (vt_attn_bwd_kernel_kind 2), whatever their size.
 */
int vt_attn_bwd_dv(const void *q, const void *k, const void *v,
                   const void *o, const void *d_o, const float *lse,
                   void *dq, void *dk, void *dv,
                   int B, int Hq, int Hkv, int Sq, int Sk, int D, int Dv,
                   int causal, float scale,
                   void *workspace, size_t workspace_bytes, void *stream);
int vt_attn_bwd_dv_f16(const void *q, const void *k, const void *v,
                       const void *o, const void *d_o, const float *lse,
                       void *dq, void *dk, void *dv,
                       int B, int Hq, int Hkv, int Sq, int Sk, int D, int Dv,
                       int causal, float scale,
                       void *workspace, size_t workspace_bytes, void *stream);

/*
 * Which forward kernel vt_attn_fwd / vt_attn_fwd_f16 launch for a shape: 0 the one-tile kernel
 * (one 128-row query tile per block, 64-key steps), 1 the two-tile kernel (two query tiles per
 * block side by side, 128-key steps; long D = 128 sequences), 2 the one-tile kernel run over a
 * long and a short query tile per block, one after the other (causal masks whose blocks then
 * fill the SMs in a single even wave).  Host-only, launches nothing; a negative
 * VT_ATTN_ERR_* code for a bad shape.  Kernels 0 and 2 give the same bits; kernel 1 agrees with
 * them within the tolerances, not bit for bit.
 */
int vt_attn_fwd_kernel_kind(int B, int Hq, int Hkv, int Sq, int Sk, int D, int causal);

/*
 * IEEE half (fp16) tensors: vt_attn_fwd_f16 / vt_attn_bwd_f16 are vt_attn_fwd / vt_attn_bwd with
 * every 16-bit tensor (q, k, v, o, d_o, dq, dk, dv) in fp16 instead of bfloat16; everything else -
 * layouts, masks, LSE in float, workspace (vt_attn_bwd_workspace_bytes), determinism, errors - is
 * the same.  Products still accumulate in fp32; P and dS are rounded to fp16 for the second GEMM of
 * each pair (values below 6e-5 lose precision there, below 6e-8 they vanish - fp16's subnormal
 * range - which bfloat16 does not have).  The paper benchmarks bf16 only; this is an extension.
 * The host-buffer and static-scratch variants exist for bfloat16 only.
 */
int vt_attn_fwd_f16(const void *q, const void *k, const void *v,
                    void *o, float *lse,
                    int B, int Hq, int Hkv, int Sq, int Sk, int D,
                    int causal, float scale, void *stream);
int vt_attn_bwd_f16(const void *q, const void *k, const void *v,
                    const void *o, const void *d_o, const float *lse,
                    void *dq, void *dk, void *dv,
                    int B, int Hq, int Hkv, int Sq, int Sk, int D,
                    int causal, float scale,
                    void *workspace, size_t workspace_bytes, void *stream);

/* The packed and split-KV entry points for fp16 tensors: the same arguments as vt_attn_fwd_varlen,
 * vt_attn_bwd_varlen and vt_attn_fwd_splitkv (whose workspace-size and plan queries serve both). */
int vt_attn_fwd_varlen_f16(const void *q, const void *k, const void *v, void *o, float *lse,
                           const int *cu_seqlens_q, const int *cu_seqlens_k,
                           int n_seqs, int Hq, int Hkv, int total_q, int total_k,
                           int max_sq, int max_sk, int D,
                           int causal, float scale, void *stream);
int vt_attn_bwd_varlen_f16(const void *q, const void *k, const void *v,
                           const void *o, const void *d_o, const float *lse,
                           void *dq, void *dk, void *dv,
                           const int *cu_seqlens_q, const int *cu_seqlens_k,
                           int n_seqs, int Hq, int Hkv, int total_q, int total_k,
                           int max_sq, int max_sk, int D,
                           int causal, float scale,
                           void *workspace, size_t workspace_bytes, void *stream);
int vt_attn_fwd_splitkv_f16(const void *q, const void *k, const void *v, void *o, float *lse,
                            int B, int Hq, int Hkv, int Sq, int Sk, int D,
                            int causal, float scale, int n_splits,
                            void *workspace, size_t workspace_bytes, void *stream);

/*
 * Split-KV forward: the same result as vt_attn_fwd (same arguments, layouts and masks),
 * computed with the keys cut into chunks that run as separate thread blocks and are then
 * merged (LSE = ln sum_s exp(LSE_s), O = sum_s exp(LSE_s - LSE) O_s).  For shapes with few
 * query tiles against many keys - decoding, small-batch prefill - where vt_attn_fwd would
 * leave most SMs idle; the paper reports exactly this regime (small-batch GQA prefill) as
 * the one where its kernel falls behind, and has no split kernel of its own.  When the Sq
 * queries of the Hq / Hkv heads that share a KV head fit one 128-row tile
 * ((Hq / Hkv) * Sq <= 128, Hq > Hkv) they are processed as one tile, so K and V are read
 * once per KV head.
 * n_splits: number of chunks, 1..128, or 0 to let the library choose (as many as keep all
 * blocks in one wave of two per SM, at least 512 keys per chunk; 1 when the shape fills the
 * GPU by itself); it is clamped so that no chunk is empty.
 * workspace: DEVICE scratch, 256-byte aligned, at least
 * vt_attn_fwd_splitkv_workspace_bytes(...) bytes for the same shape and n_splits
 * (n_splits partial outputs in fp32 and their LSEs); contents undefined afterwards.
 * The merged result differs from vt_attn_fwd's only by fp32 rounding of the merge; it is
 * bit-identical from run to run for a given n_splits.
 * Errors: as vt_attn_fwd, plus VT_ATTN_ERR_WORKSPACE_TOO_SMALL, and
 * VT_ATTN_ERR_INVALID_ARGUMENT for n_splits outside 0..128.
 */
size_t vt_attn_fwd_splitkv_workspace_bytes(int B, int Hq, int Hkv, int Sq, int Sk, int D, int n_splits);
int vt_attn_fwd_splitkv(const void *q, const void *k, const void *v, void *o, float *lse,
                        int B, int Hq, int Hkv, int Sq, int Sk, int D,
                        int causal, float scale, int n_splits,
                        void *workspace, size_t workspace_bytes, void *stream);
/* What vt_attn_fwd_splitkv will do for a shape: chunks actually used, and whether the heads
 * of a KV group share a tile (1) or not (0).  Host-only, launches nothing. */
int vt_attn_fwd_splitkv_plan(int B, int Hq, int Hkv, int Sq, int Sk, int D, int n_splits,
                             int *splits_used, int *heads_share_tile);

/*
 * vt_attn_fwd_splitkv for packed batches (the layouts of vt_attn_fwd_varlen): decoding or chunked
 * prefill against caches of different lengths.  The number of chunks, and whether the heads of a KV
 * group share a tile (Hq / Hkv * max_sq <= 128), are planned from the longest sequence
 * (vt_attn_fwd_splitkv_plan(n_seqs, Hq, Hkv, max_sq, max_sk, D, n_splits, ...) tells); every
 * sequence's own keys are then cut into that many chunks.  A sequence
 * without queries costs nothing; one without keys (or whose rows see none) gets O = 0, LSE = -inf,
 * and so do the query tokens of a sequence longer than max_sq (vt_attn_fwd_varlen leaves those
 * untouched; pass a max_sq that covers the longest sequence).
 * workspace: device memory of at least vt_attn_fwd_splitkv_varlen_workspace_bytes(...) bytes,
 * 256-byte aligned, contents undefined afterwards.  bfloat16; D a multiple of 8 in [8, 128].
 */
size_t vt_attn_fwd_splitkv_varlen_workspace_bytes(int n_seqs, int Hq, int Hkv, int total_q,
                                                  int max_sq, int max_sk, int D, int n_splits);
/* The number of chunks the call below uses (n_splits = 0: the library's choice, which for packed
 * batches also depends on how far the longest sequence is from the mean, max_sk * n_seqs / total_k),
 * and whether the heads of a KV group share a tile.  Host-only. */
int vt_attn_fwd_splitkv_varlen_plan(int n_seqs, int Hq, int Hkv, int total_k, int max_sq, int max_sk,
                                    int D, int n_splits, int *splits_used, int *heads_share_tile);
int vt_attn_fwd_splitkv_varlen(const void *q, const void *k, const void *v, void *o, float *lse,
                               const int *cu_seqlens_q, const int *cu_seqlens_k,
                               int n_seqs, int Hq, int Hkv, int total_q, int total_k,
                               int max_sq, int max_sk, int D,
                               int causal, float scale, int n_splits,
                               void *workspace, size_t workspace_bytes, void *stream);
/* The same on IEEE half tensors (same workspace size and plan). */
int vt_attn_fwd_splitkv_varlen_f16(const void *q, const void *k, const void *v, void *o, float *lse,
                                   const int *cu_seqlens_q, const int *cu_seqlens_k,
                                   int n_seqs, int Hq, int Hkv, int total_q, int total_k,
                                   int max_sq, int max_sk, int D,
                                   int causal, float scale, int n_splits,
                                   void *workspace, size_t workspace_bytes, void *stream);

/*
 * Merging partial results over disjoint key sets (one step of context-parallel "ring" attention,
 * where the keys of a long sequence live on several GPUs and visit the queries block by block;
 * the paper leaves multi-GPU attention open and has no counterpart).  o_part [n_rows, D] bf16 and
 * lse_part [n_rows] are the outputs of a forward call over one block of keys; o_acc [n_rows, D]
 * float and lse_acc [n_rows] float hold the running result (caller-owned DEVICE buffers):
 *   LSE' = ln(e^LSE + e^LSE_part),   O' = e^(LSE - LSE') O + e^(LSE_part - LSE') O_part.
 * first != 0 initialises the running result from the part instead of reading it.  A part with
 * LSE_part = -inf (no visible key) leaves the result unchanged; if nothing has been seen the
 * result stays O = 0, LSE = -inf.  vt_attn_merge_finish rounds o_acc to bf16 into o.
 * n_rows = B * Hq * Sq of the forward calls (same row order); D a multiple of 8 in [8, 256].
 */
int vt_attn_merge_partial(float *o_acc, float *lse_acc, const void *o_part, const float *lse_part,
                          long long n_rows, int D, int first, void *stream);
int vt_attn_merge_finish(const float *o_acc, void *o, long long n_rows, int D, void *stream);
/* acc [n_rows, D] float += part [n_rows, D] bf16 (acc = part when first != 0): the running sums of
 * the per-block gradients in the ring backward, where each block's dQ / dK / dV contribution comes
 * out of vt_attn_bwd in bf16.  vt_attn_merge_finish rounds the sums to bf16. */
int vt_attn_accumulate_partial(float *acc, const void *part, long long n_rows, int D, int first, void *stream);

/* Bytes of device scratch vt_attn_bwd_varlen needs (Delta, [Hq, total_q] floats); 0 if invalid. */
size_t vt_attn_bwd_varlen_workspace_bytes(int Hq, int total_q);

/*
 * Backward of vt_attn_fwd_varlen: same layouts; d_o, dq like q; dk, dv like k.  dq, dk,
 * dv are fully overwritten (rows of sequences that see nothing get zeros); results are
 * bit-identical from run to run.  workspace as for vt_attn_bwd.
 */
int vt_attn_bwd_varlen(const void *q, const void *k, const void *v,
                       const void *o, const void *d_o, const float *lse,
                       void *dq, void *dk, void *dv,
                       const int *cu_seqlens_q, const int *cu_seqlens_k,
                       int n_seqs, int Hq, int Hkv, int total_q, int total_k,
                       int max_sq, int max_sk, int D,
                       int causal, float scale,
                       void *workspace, size_t workspace_bytes, void *stream);

/*
 * Bytes of device staging the *_host entry points need for this shape
 * (with_backward != 0 adds room for dO, dQ, dK, dV and the backward scratch).
 */
size_t vt_attn_host_staging_bytes(int B, int Hq, int Hkv, int Sq, int Sk, int D, int with_backward);

/*
 * Forward pass on HOST buffers: q_host, k_host, v_host are copied to the device
 * staging area, vt_attn_fwd runs there, and O and LSE are copied back to o_host
 * and lse_host.  The problem is cut into up to 16 chunks of whole (batch, KV head)
 * groups that alternate between two streams owned by the library (created on the
 * first call on a device and kept), so that one chunk's kernels overlap the next
 * chunk's copies in and the previous chunk's copies out; those streams start after
 * the work already enqueued on `stream` and `stream` continues after them, so the
 * call is ordered on `stream` like any other (the library takes a lock while it enqueues,
 * so calls from several host threads are safe; each call in flight needs its own staging).  Host buffers must be pinned for the
 * copies to be asynchronous and to overlap; the results are valid after the caller
 * synchronises `stream`.  Results are the same bits as vt_attn_fwd on the whole
 * problem whenever the chunks get the same kernel (see vt_attn_fwd_kernel_kind).
 * staging: DEVICE memory of at least vt_attn_host_staging_bytes(..., 0) bytes,
 * 256-byte aligned, owned by the caller.
 */
int vt_attn_fwd_host(const void *q_host, const void *k_host, const void *v_host,
                     void *o_host, float *lse_host,
                     int B, int Hq, int Hkv, int Sq, int Sk, int D,
                     int causal, float scale,
                     void *staging, size_t staging_bytes, void *stream);

/*
 * Forward and backward on HOST buffers in one call: copies q, k, v, d_o in, runs
 * vt_attn_fwd then vt_attn_bwd in the staging area, copies o, lse, dq, dk, dv out,
 * chunk by chunk on the library's two streams as described for vt_attn_fwd_host.
 * staging: at least vt_attn_host_staging_bytes(..., 1) bytes of DEVICE memory.
 */
int vt_attn_fwd_bwd_host(const void *q_host, const void *k_host, const void *v_host,
                         const void *d_o_host,
                         void *o_host, float *lse_host,
                         void *dq_host, void *dk_host, void *dv_host,
                         int B, int Hq, int Hkv, int Sq, int Sk, int D,
                         int causal, float scale,
                         void *staging, size_t staging_bytes, void *stream);

/*
 * The two calls above on IEEE half tensors (vt_attn_fwd_f16 / vt_attn_bwd_f16 in the
 * staging area); the staging size is the same.
 */
int vt_attn_fwd_host_f16(const void *q_host, const void *k_host, const void *v_host,
                         void *o_host, float *lse_host,
                         int B, int Hq, int Hkv, int Sq, int Sk, int D,
                         int causal, float scale,
                         void *staging, size_t staging_bytes, void *stream);
int vt_attn_fwd_bwd_host_f16(const void *q_host, const void *k_host, const void *v_host,
                             const void *d_o_host,
                             void *o_host, float *lse_host,
                             void *dq_host, void *dk_host, void *dv_host,
                             int B, int Hq, int Hkv, int Sq, int Sk, int D,
                             int causal, float scale,
                             void *staging, size_t staging_bytes, void *stream);

/*
 * Every wait inside the kernels is bounded.  If one expires, the kernel records
 * where in a per-device status word, lets all its warps leave, and returns
 * normally; outputs of that launch are then undefined.  The word is sticky: the
 * first expired wait stays recorded until it is cleared.
 *
 * vt_attn_device_status is the convenient, BLOCKING form (the one entry point of this
 * library that synchronises): it waits for `stream`, reads the word of the current
 * device, clears it if set (waiting once more), and returns VT_ATTN_OK or
 * VT_ATTN_ERR_DEVICE_TIMEOUT.  detail (host, may be NULL) receives the raw word: bits
 * 0-7 kernel id, 8-15 waiting role, 16-31 tile index.  Not for use during stream capture.
 * Kernel ids: 1 one-tile forward, 2 dK/dV, 3 dQ, 4 two-tile forward, 5 forward with two tiles
 * in sequence, 6 / 7 dK/dV and dQ above 128 columns, 8 single-pass backward, 9 self-test.
 *
 * vt_attn_device_status_async and vt_attn_device_status_clear are the non-blocking
 * pieces for callers that own their synchronisation points: the first enqueues a copy
 * of the word into *word_host (host memory, pinned for the copy to be asynchronous;
 * valid once the caller has synchronised `stream`; 0 = no wait expired), the second
 * enqueues the reset of the word.  Neither synchronises.
 */
int vt_attn_device_status(unsigned int *detail, void *stream);
int vt_attn_device_status_async(unsigned int *word_host, void *stream);
int vt_attn_device_status_clear(void *stream);

/*
 * Static facts about the build, written to info[0..n) (host): [0] ABI version,
 * [1] query-tile rows, [2] keys per step of the one-tile forward kernel, [3] its threads
 * per block, [4] its dynamic shared memory bytes at D=128, [5] its tensor-memory columns
 * per block (the two-tile kernel used for long D=128 sequences: 128 keys per step, 384
 * threads, all 512 columns), [6] number of kernels launched by vt_attn_fwd, [7] by
 * vt_attn_bwd.
 * Returns the number of entries written (at most n).
 */
int vt_attn_get_info(int *info, int n);

/*
 * Self-test of the tensor-core building blocks on one 128 x 128 tile (called by the
 * test-suite, not by the product path; the paper has no counterpart): S = Q K^T in
 * fp32, then O = P V with P = S * p_scale rounded to bf16.
 * q, k, v: bf16 [128, D]; s_out: float [128,128]; o_out: float [128, D].
 */
int vt_attn_selftest_tile(const void *q, const void *k, const void *v,
                          float *s_out, float *o_out, int D, float p_scale, void *stream);

/*
 * Self-test of the bounded-wait path (test-suite only; the paper has no counterpart):
 * launches one warp that waits on a barrier nothing ever signals, with a limit of
 * limit_ms milliseconds (1..1000).  The kernel returns normally once the limit has
 * passed and vt_attn_device_status then reports VT_ATTN_ERR_DEVICE_TIMEOUT.
 */
int vt_attn_selftest_timeout(unsigned int limit_ms, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* VT_ATTN_H_ */
