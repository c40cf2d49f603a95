// Forward attention with the rotary position embedding of the queries applied inside the kernel (fwd_kernel.cuh, ROPE
// flag).  The paper lists "Rotary (fwd)" as its own row of the kernel microbenchmark table; this entry point takes
// the query half of that operator into the attention kernel's load path, where it costs no pass over Q in global memory.
#include "fwd_kernel.cuh"

extern "C" int vt_attn_fwd_rope(const void *q, const void *k_rotated, const void *v, const float *rope_cos, const float *rope_sin,
                                void *o, float *lse, int B, int Hq, int Hkv, int Sq, int Sk, int D, int causal, float scale,
                                int q_pos0, int rope_positions, void *stream)
{
    using namespace vt;
    Shape s{B, Hq, Hkv, Sq, Sk, D};
    int rc = check_shape(s, scale, MAX_HEAD_DIM_FWD);
    if (rc != VT_ATTN_OK) return rc;
    if (D != 64 && D != 128) return VT_ATTN_ERR_UNSUPPORTED;
    if (!ptr_ok(q) || !ptr_ok(k_rotated) || !ptr_ok(v) || !ptr_ok(o) || !ptr_ok(lse, 4) || !ptr_ok(rope_cos) || !ptr_ok(rope_sin))
        return VT_ATTN_ERR_INVALID_ARGUMENT;
    if (causal < 0 || causal > 2 || q_pos0 < 0 || rope_positions < 1 || static_cast<long long>(q_pos0) + Sq > rope_positions)
        return VT_ATTN_ERR_INVALID_ARGUMENT;
    rc = check_device();
    if (rc != VT_ATTN_OK) return rc;

    FwdParams prm;
    prm.o = static_cast<__nv_bfloat16 *>(o);
    prm.lse = lse;
    prm.Hq = Hq;
    prm.d = D;
    prm.d_qk = D;
    prm.hp_tokens = 0;
    prm.G = Hq / Hkv;
    prm.Sq = Sq;
    prm.Sk = Sk;
    prm.n_qt = (Sq + TILE - 1) / TILE;
    prm.scale_log2e = scale * 1.4426950408889634f;
    prm.cu_q = nullptr;
    prm.cu_k = nullptr;
    prm.total_q = 0;
    prm.bottom_right = (causal == 2);
    prm.n_splits = 1;
    prm.chunk_steps = 0;
    prm.o_part = nullptr;
    prm.lse_part = nullptr;
    prm.n_rows = 0;
    prm.rope_cos = rope_cos;
    prm.rope_sin = rope_sin;
    prm.rope_pos0 = q_pos0;
    prm.guard = make_guard();
    if (!prm.guard.status) return VT_ATTN_ERR_CUDA;
    const long long n_blocks = static_cast<long long>(prm.n_qt) * B * Hq;
    if (n_blocks > 0x7FFFFFFFll) return VT_ATTN_ERR_INVALID_ARGUMENT;
    prm.head_group = causal_head_group(static_cast<long long>(B) * Hq, prm.n_qt, 2 * NUM_SMS, prm.G, 4ll * Sk * D / prm.G);

    CUtensorMap tq, tk, tv;
    if ((rc = make_tensor_map(&tq, q, B * Hq, Sq, D, TILE)) != VT_ATTN_OK) return rc;
    if ((rc = make_tensor_map(&tk, k_rotated, B * Hkv, Sk, D, BN)) != VT_ATTN_OK) return rc;
    if ((rc = make_tensor_map(&tv, v, B * Hkv, Sk, D, BN)) != VT_ATTN_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int nb = static_cast<int>(n_blocks);
    if (D == 64)
        return causal ? launch_fwd<64, true, false, false, false, false, true>(tq, tk, tv, prm, nb, st)
                      : launch_fwd<64, false, false, false, false, false, true>(tq, tk, tv, prm, nb, st);
    return causal ? launch_fwd<128, true, false, false, false, false, true>(tq, tk, tv, prm, nb, st)
                  : launch_fwd<128, false, false, false, false, false, true>(tq, tk, tv, prm, nb, st);
}
