/*
 * fp64 CPU oracle for scaled-dot-product attention, forward and backward.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow definition that the
 * GPU library is checked against.  It shares no code with the GPU path and must
 * never be called from it.
 *
 * What it computes.  The paper names the operation only through its baseline,
 * torch scaled_dot_product_attention (caption of the kernel-microbenchmark
 * table, "Attention (fwd)/(bwd)" rows) and says the kernel uses a
 * flash-attention-style stabilised formulation (debugging-episodes table, row
 * "log2 vs ln scaling").  Flash attention is an exact re-ordering of the plain
 * definition, so the oracle is that definition written out, per (b, h, i):
 *
 *   g      = h / (Hq / Hkv)                                 (GQA head map)
 *   s_ij   = scale * sum_d Q[b,h,i,d] * K[b,g,j,d]          (j > i masked if causal)
 *   m_i    = max_j s_ij ;  l_i = sum_j exp(s_ij - m_i)
 *   LSE_i  = m_i + ln(l_i)                                  (natural log)
 *   P_ij   = exp(s_ij - LSE_i)
 *   O_i    = sum_j P_ij * V[b,g,j,:]
 *
 * and, for a given dO,
 *
 *   Delta_i = sum_d dO[i,d] * O[i,d]
 *   dP_ij   = sum_d dO[i,d] * V[g,j,d]
 *   dS_ij   = P_ij * (dP_ij - Delta_i)
 *   dQ_i    = scale * sum_j dS_ij * K[g,j,:]
 *   dK_j    = scale * sum_{h in group g} sum_i dS_ij * Q[h,i,:]
 *   dV_j    =         sum_{h in group g} sum_i P_ij  * dO[h,i,:]
 *
 * Two-pass softmax (max, then sum), one query row at a time, no S x S matrix is
 * ever stored.  `causal` selects the mask:
 *   0  none;
 *   1  top-left aligned: key j is visible to query i iff j <= i (torch's is_causal; key 0 is
 *      always visible, no row is empty);
 *   2  bottom-right aligned: key j is visible to query i iff j <= i + (Sk - Sq), the alignment
 *      used when the Sq queries are the LAST positions of a sequence of Sk keys (chunked
 *      prefill, decoding against a cache).  An extension beyond the paper, which only runs
 *      Sq == Sk, where the two alignments coincide.  With Sk < Sq the first Sq - Sk rows see
 *      no key: their softmax is empty, and by convention O = 0, LSE = -inf and every gradient
 *      contribution of the row is 0.
 *
 * All tensors are double, row-major [B, H, S, D] (D innermost).
 * Parallelism: OpenMP over (b, g); every (b, g) pair owns its dK/dV slice, so
 * no atomics are needed and the result does not depend on the thread count.
 */
#include <math.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double dot(const double *a, const double *b, int n)
{
    double acc = 0.0;
#pragma omp simd reduction(+ : acc)
    for (int d = 0; d < n; ++d) acc += a[d] * b[d];
    return acc;
}

/* number of keys visible to query row i (they are always keys 0 .. n-1) */
static int visible_keys(int i, int Sq, int Sk, int causal)
{
    if (!causal) return Sk;
    int n = i + 1;
    if (causal == 2) n += Sk - Sq;
    if (n < 0) n = 0;
    return (n < Sk) ? n : Sk;
}

/*
 * One query row: fills p[0..n) with the softmax probabilities over the n
 * visible keys and returns LSE.  qrow: [D]; kmat: [Sk, D].
 */
static double softmax_row(const double *qrow, const double *kmat, int n, int D,
                          double scale, double *p)
{
    if (n <= 0) return -INFINITY;          /* empty softmax: nothing to fill */
    double m = -INFINITY;
    for (int j = 0; j < n; ++j) {
        p[j] = scale * dot(qrow, kmat + (size_t)j * D, D);
        if (p[j] > m) m = p[j];
    }
    double l = 0.0;
    for (int j = 0; j < n; ++j) l += exp(p[j] - m);
    double lse = m + log(l);
    for (int j = 0; j < n; ++j) p[j] = exp(p[j] - lse);
    return lse;
}

int attn_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Sets the number of OpenMP threads later calls use (n >= 1); returns the value now in force.  Threading only decides
 * which core computes which (b, g) slice, never the arithmetic inside one: a test checks the results are the same bits. */
int attn_oracle_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n >= 1) omp_set_num_threads(n);
    return omp_get_max_threads();
#else
    (void)n;
    return 1;
#endif
}

static int bad_shape(int B, int Hq, int Hkv, int Sq, int Sk, int D)
{
    return B <= 0 || Hq <= 0 || Hkv <= 0 || Sq <= 0 || Sk <= 0 || D <= 0 || (Hq % Hkv) != 0;
}

static int bad_mask(int causal) { return causal < 0 || causal > 2; }

/* Forward.  o: [B,Hq,Sq,D], lse: [B,Hq,Sq].  Returns 0, or -1 on a bad shape. */
int attn_oracle_fwd(const double *q, const double *k, const double *v,
                    double *o, double *lse,
                    int B, int Hq, int Hkv, int Sq, int Sk, int D,
                    int causal, double scale)
{
    if (bad_shape(B, Hq, Hkv, Sq, Sk, D) || bad_mask(causal)) return -1;
    const int G = Hq / Hkv;
    int status = 0;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        for (int h = 0; h < Hq; ++h) {
            const int g = h / G;
            const double *kmat = k + ((size_t)b * Hkv + g) * Sk * D;
            const double *vmat = v + ((size_t)b * Hkv + g) * Sk * D;
            double *p = (double *)malloc(sizeof(double) * (size_t)Sk);
            if (!p) { status = -2; continue; }
            for (int i = 0; i < Sq; ++i) {
                const size_t row = ((size_t)b * Hq + h) * Sq + i;
                const int n = visible_keys(i, Sq, Sk, causal);
                lse[row] = softmax_row(q + row * D, kmat, n, D, scale, p);
                double *orow = o + row * D;
                for (int d = 0; d < D; ++d) orow[d] = 0.0;
                for (int j = 0; j < n; ++j) {
                    const double pj = p[j];
                    const double *vrow = vmat + (size_t)j * D;
                    for (int d = 0; d < D; ++d) orow[d] += pj * vrow[d];
                }
            }
            free(p);
        }
    }
    return status;
}

/*
 * Probabilities of one (b, h) head, dense: p_out is [Sq, Sk], masked entries 0.
 * Exists so that tests can pin the softmax itself (rows sum to one).
 */
int attn_oracle_probs(const double *q, const double *k, double *p_out,
                      int B, int Hq, int Hkv, int Sq, int Sk, int D,
                      int causal, double scale, int b, int h)
{
    if (bad_shape(B, Hq, Hkv, Sq, Sk, D) || bad_mask(causal) || b < 0 || b >= B || h < 0 || h >= Hq) return -1;
    const int g = h / (Hq / Hkv);
    const double *kmat = k + ((size_t)b * Hkv + g) * Sk * D;
    for (int i = 0; i < Sq; ++i) {
        const size_t row = ((size_t)b * Hq + h) * Sq + i;
        const int n = visible_keys(i, Sq, Sk, causal);
        double *p = p_out + (size_t)i * Sk;
        softmax_row(q + row * D, kmat, n, D, scale, p);
        for (int j = n; j < Sk; ++j) p[j] = 0.0;
    }
    return 0;
}

/*
 * Backward.  Recomputes its own fp64 P and O from q, k, v (it never sees the
 * GPU's O or LSE).  dq: [B,Hq,Sq,D]; dk, dv: [B,Hkv,Sk,D]; delta (optional,
 * may be NULL): [B,Hq,Sq].
 */
int attn_oracle_bwd(const double *q, const double *k, const double *v, const double *d_o,
                    double *dq, double *dk, double *dv, double *delta,
                    int B, int Hq, int Hkv, int Sq, int Sk, int D,
                    int causal, double scale)
{
    if (bad_shape(B, Hq, Hkv, Sq, Sk, D) || bad_mask(causal)) return -1;
    const int G = Hq / Hkv;
    int status = 0;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        for (int g = 0; g < Hkv; ++g) {
            const size_t kvoff = ((size_t)b * Hkv + g) * Sk * D;
            const double *kmat = k + kvoff;
            const double *vmat = v + kvoff;
            double *dkmat = dk + kvoff;
            double *dvmat = dv + kvoff;
            memset(dkmat, 0, sizeof(double) * (size_t)Sk * D);
            memset(dvmat, 0, sizeof(double) * (size_t)Sk * D);
            double *p = (double *)malloc(sizeof(double) * (size_t)Sk);
            double *orow = (double *)malloc(sizeof(double) * (size_t)D);
            if (!p || !orow) { status = -2; free(p); free(orow); continue; }
            for (int h = g * G; h < (g + 1) * G; ++h) {
                for (int i = 0; i < Sq; ++i) {
                    const size_t row = ((size_t)b * Hq + h) * Sq + i;
                    const double *qrow = q + row * D;
                    const double *dorow = d_o + row * D;
                    double *dqrow = dq + row * D;
                    const int n = visible_keys(i, Sq, Sk, causal);
                    softmax_row(qrow, kmat, n, D, scale, p);
                    /* O_i = sum_j P_ij V_j */
                    for (int d = 0; d < D; ++d) orow[d] = 0.0;
                    for (int j = 0; j < n; ++j) {
                        const double pj = p[j];
                        const double *vrow = vmat + (size_t)j * D;
                        for (int d = 0; d < D; ++d) orow[d] += pj * vrow[d];
                    }
                    const double delta_i = dot(dorow, orow, D);
                    if (delta) delta[row] = delta_i;
                    for (int d = 0; d < D; ++d) dqrow[d] = 0.0;
                    for (int j = 0; j < n; ++j) {
                        const double *krow = kmat + (size_t)j * D;
                        const double *vrow = vmat + (size_t)j * D;
                        double *dkrow = dkmat + (size_t)j * D;
                        double *dvrow = dvmat + (size_t)j * D;
                        const double pj = p[j];
                        const double dp = dot(dorow, vrow, D);
                        const double ds = pj * (dp - delta_i);
                        for (int d = 0; d < D; ++d) {
                            dqrow[d] += scale * ds * krow[d];
                            dkrow[d] += scale * ds * qrow[d];
                            dvrow[d] += pj * dorow[d];
                        }
                    }
                }
            }
            free(p);
            free(orow);
        }
    }
    return status;
}
