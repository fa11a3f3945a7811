/*
 * CPU oracle for exact softmax attention, forward and backward, in float64.
 *
 * THIS IS TEST INFRASTRUCTURE.  It exists to define what the CUDA library must
 * compute; it is slow on purpose, shares no code with the CUDA path, and must
 * never be used by it.  Only the test-suite, the smoke check and the benchmark's
 * CPU-baseline leg call into this file.
 *
 * What is computed (paper notation on the left, names used here on the right;
 * the paper's S = A1 X is our pre-projected query Q, its A2 is K, its h = A3 Y is V):
 *
 *   A = exp(Q K^T * scale)          Definition B.3 (A(X)), the 1/sqrt(d) factor is
 *                                   the part of X the caller keeps explicit
 *   l = A 1                         Definition B.4
 *   f = diag(l)^-1 A        -> P    Definition B.5 (the matrix form printed there
 *                                   lacks the inverse; the row form and every
 *                                   algorithm use diag(l)^-1, which is what we take)
 *   O = f h                         Definition B.7, Definition 3.1
 *   q = dO h^T              -> dP   Definition B.8
 *   v = (dO o O) 1          -> D    Definition B.9, second matrix form
 *   p = f o q - diag(v) f   -> dS   Definition B.9
 *   dQ = scale * p K, dK = scale * p^T Q   chain rule through Definition 3.2
 *                                   (dL/dX = A1^T p A2 with Q = A1 X, K = A2)
 *   dV = f^T dO                     O is linear in h (Remark after Definition 3.2)
 *
 * The saved row statistic is LSE = ln l, evaluated as m + ln sum exp(s - m) with
 * m the row maximum, which is the same number as ln l whenever exp(s) does not
 * overflow.  A masked score is excluded from the row (it is "minus infinity", not
 * zero).  A row with no kept entry has O = 0, LSE = -inf and contributes nothing to
 * any gradient.
 *
 * Layout: every tensor is [batch, heads, n, d] contiguous doubles; LSE is
 * [batch, heads, n].  Functions are independent per (batch, head).
 *
 * attn_oracle_fwd / attn_oracle_bwd stream one row at a time (memory O(n)), so they
 * also serve the long-sequence workloads.  attn_oracle_dense forms, row by row and
 * without the max shift, the n x n matrices that Definitions B.3 - B.9 name (A, f, q, p)
 * and the vectors l and (f o q) 1; it is a second implementation that the tests compare
 * the first one with on small inputs.
 *
 * The attention weights (the paper's own gradient target):
 *   attn_oracle_project      S = A1 X and h = A3 Y, the two products of phase 1 of the
 *                            large-cache algorithm (Appendix D): out = A W per unit
 *   attn_oracle_weight_grad  dL/dX = A1^T p A2 (Definition 3.2) given G = p A2, i.e. the
 *                            plain product g = A^T G; with G = f^T dO it is dL/dY
 *                            (O = f A3 Y is linear in Y).  Units that share a weight
 *                            matrix add their gradients.
 * Unit u (= batch index * heads + head) uses weight matrix u mod weight_units, so
 * weight_units is 1 (one matrix for all), heads (shared over the batch) or batch*heads.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { MASK_NONE = 0, MASK_CAUSAL = 1, MASK_BLOCK = 2, MASK_ELEMENT = 3, MASK_BLOCK_CAUSAL = 4 };

typedef struct {
    int kind;            /* MASK_* */
    int block;           /* block edge for MASK_BLOCK, MASK_BLOCK_CAUSAL */
    const uint8_t *bits; /* MASK_BLOCK(_CAUSAL): [mask_heads][nb][nb]; MASK_ELEMENT: [mask_heads][n][n]; 1 = keep */
    int mask_heads;      /* 1: shared by every (batch, head); else batch*heads */
} mask_t;

static int kept(const mask_t *m, int n, long bh, int i, int j)
{
    switch (m->kind) {
    case MASK_NONE:
        return 1;
    case MASK_CAUSAL:
        return j <= i;
    case MASK_BLOCK:
    case MASK_BLOCK_CAUSAL: {   /* the latter: kept by the block mask AND j <= i */
        int nb = (n + m->block - 1) / m->block;
        long mh = m->mask_heads == 1 ? 0 : bh;
        if (m->kind == MASK_BLOCK_CAUSAL && j > i) return 0;
        return m->bits[(mh * nb + i / m->block) * nb + j / m->block] != 0;
    }
    case MASK_ELEMENT: {
        long mh = m->mask_heads == 1 ? 0 : bh;
        return m->bits[(mh * n + i) * (long)n + j] != 0;
    }
    }
    return 0;
}

static double dot(const double *a, const double *b, int d)
{
    double s = 0.0;
    for (int c = 0; c < d; ++c) s += a[c] * b[c];
    return s;
}

int attn_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Forward: O and LSE (Definitions B.3-B.7). */
void attn_oracle_fwd(const double *Q, const double *K, const double *V, int n, int d, int heads, int batch,
                     int mask_kind, int block, const uint8_t *mask_bits, int mask_heads, double scale,
                     double *O, double *LSE)
{
    mask_t mk = { mask_kind, block, mask_bits, mask_heads };
    long BH = (long)batch * heads;
#pragma omp parallel
    {
        double *s = (double *)malloc(sizeof(double) * (size_t)n);
#pragma omp for collapse(2) schedule(dynamic, 8)
        for (long bh = 0; bh < BH; ++bh) {
            for (int i = 0; i < n; ++i) {
                const double *q = Q + (bh * n + i) * d;
                const double *Kh = K + bh * n * d, *Vh = V + bh * n * d;
                double *o = O + (bh * n + i) * d;
                double m = -INFINITY;
                for (int j = 0; j < n; ++j) {
                    if (!kept(&mk, n, bh, i, j)) continue;
                    s[j] = scale * dot(q, Kh + (long)j * d, d);
                    if (s[j] > m) m = s[j];
                }
                for (int c = 0; c < d; ++c) o[c] = 0.0;
                if (m == -INFINITY) { /* no kept entry in this row */
                    LSE[bh * n + i] = -INFINITY;
                    continue;
                }
                double l = 0.0;
                for (int j = 0; j < n; ++j)
                    if (kept(&mk, n, bh, i, j)) l += exp(s[j] - m);
                double lse = m + log(l);
                LSE[bh * n + i] = lse;
                for (int j = 0; j < n; ++j) {
                    if (!kept(&mk, n, bh, i, j)) continue;
                    double p = exp(s[j] - lse);
                    const double *v = Vh + (long)j * d;
                    for (int c = 0; c < d; ++c) o[c] += p * v[c];
                }
            }
        }
        free(s);
    }
}

/* Backward given the forward's O and LSE (the large-cache algorithm's premise:
 * l and O are available from the forward pass).  D = rowsum(dO o O); dS = P o (dP - D). */
void attn_oracle_bwd(const double *Q, const double *K, const double *V, const double *O, const double *dO,
                     const double *LSE, int n, int d, int heads, int batch,
                     int mask_kind, int block, const uint8_t *mask_bits, int mask_heads, double scale,
                     double *dQ, double *dK, double *dV)
{
    mask_t mk = { mask_kind, block, mask_bits, mask_heads };
    long BH = (long)batch * heads;
    double *D = (double *)malloc(sizeof(double) * (size_t)(BH * n));
#pragma omp parallel for schedule(static)
    for (long r = 0; r < BH * n; ++r) D[r] = dot(dO + r * d, O + r * d, d);

    /* dQ_i = scale * sum_j dS_ij K_j : one query row at a time */
#pragma omp parallel for collapse(2) schedule(dynamic, 8)
    for (long bh = 0; bh < BH; ++bh) {
        for (int i = 0; i < n; ++i) {
            long r = bh * n + i;
            double *dq = dQ + r * d;
            for (int c = 0; c < d; ++c) dq[c] = 0.0;
            if (LSE[r] == -INFINITY) continue;
            for (int j = 0; j < n; ++j) {
                if (!kept(&mk, n, bh, i, j)) continue;
                const double *k = K + (bh * n + j) * d;
                double p = exp(scale * dot(Q + r * d, k, d) - LSE[r]);
                double dp = dot(dO + r * d, V + (bh * n + j) * d, d);
                double ds = p * (dp - D[r]);
                for (int c = 0; c < d; ++c) dq[c] += scale * ds * k[c];
            }
        }
    }
    /* dK_j = scale * sum_i dS_ij Q_i ; dV_j = sum_i P_ij dO_i : one key row at a time */
#pragma omp parallel for collapse(2) schedule(dynamic, 8)
    for (long bh = 0; bh < BH; ++bh) {
        for (int j = 0; j < n; ++j) {
            long rj = bh * n + j;
            double *dk = dK + rj * d, *dv = dV + rj * d;
            for (int c = 0; c < d; ++c) dk[c] = dv[c] = 0.0;
            for (int i = 0; i < n; ++i) {
                long r = bh * n + i;
                if (!kept(&mk, n, bh, i, j) || LSE[r] == -INFINITY) continue;
                const double *q = Q + r * d, *g = dO + r * d;
                double p = exp(scale * dot(q, K + rj * d, d) - LSE[r]);
                double dp = dot(g, V + rj * d, d);
                double ds = p * (dp - D[r]);
                for (int c = 0; c < d; ++c) {
                    dv[c] += p * g[c];
                    dk[c] += scale * ds * q[c];
                }
            }
        }
    }
    free(D);
}

/* One head, the dense n x n matrices of the definitions, unshifted, one query row at a time:
 *   A_ij = exp(scale q_i . k_j) on kept entries, 0 elsewhere     (Definition B.3)
 *   l_i  = sum_j A_ij                                            (Definition B.4)
 *   f_ij = A_ij / l_i                                            (Definition B.5, the form with the inverse)
 *   q_ij = dO_i . V_j                                            (Definition B.8)
 *   v_i  = sum_j f_ij q_ij
 *   p_ij = f_ij (q_ij - v_i)                                     (Definition B.9, row form)
 * Outputs (any may be NULL): l [n], f [n*n], q [n*n], p [n*n], v_fq [n] = (f o q) 1.          */
void attn_oracle_dense(const double *Q, const double *K, const double *V, const double *dO, int n, int d,
                       int mask_kind, int block, const uint8_t *mask_bits, double scale,
                       double *l_out, double *f_out, double *q_out, double *p_out, double *v_fq_out)
{
    mask_t mk = { mask_kind, block, mask_bits, 1 };
    double *f = (double *)calloc((size_t)n, sizeof(double));
    double *q = (double *)calloc((size_t)n, sizeof(double));
    for (int i = 0; i < n; ++i) {
        double l = 0.0, v = 0.0;
        for (int j = 0; j < n; ++j) {
            f[j] = kept(&mk, n, 0, i, j) ? exp(scale * dot(Q + (long)i * d, K + (long)j * d, d)) : 0.0;
            l += f[j];
        }
        for (int j = 0; j < n; ++j) {
            f[j] = l > 0.0 ? f[j] / l : 0.0;
            q[j] = dot(dO + (long)i * d, V + (long)j * d, d);
            v += f[j] * q[j];
        }
        if (l_out) l_out[i] = l;
        if (v_fq_out) v_fq_out[i] = v;
        for (int j = 0; j < n; ++j) {
            size_t e = (size_t)i * n + j;
            if (f_out) f_out[e] = f[j];
            if (q_out) q_out[e] = q[j];
            if (p_out) p_out[e] = f[j] * (q[j] - v);
        }
    }
    free(f); free(q);
}

/* out_u = A_u W_{u mod weight_units}; A, out: [units][n][d]; W: [weight_units][d][d], row = input
 * feature, column = output feature (S = A1 X and h = A3 Y of Appendix D, phase 1). */
void attn_oracle_project(const double *A, const double *W, double *out, int n, int d, long units, long weight_units)
{
#pragma omp parallel for schedule(static)
    for (long r = 0; r < units * n; ++r) {
        const long u = r / n;
        const double *a = A + r * d;
        const double *w = W + (u % weight_units) * (long)d * d;
        double *o = out + r * d;
        for (int c = 0; c < d; ++c) {
            double acc = 0.0;
            for (int k = 0; k < d; ++k) acc += a[k] * w[(long)k * d + c];
            o[c] = acc;
        }
    }
}

/* g_w = sum over the units u with u mod weight_units = w of A_u^T G_u; A, G: [units][n][d];
 * g: [weight_units][d][d] (Definition 3.2 with G = p A2: g = A1^T p A2). */
void attn_oracle_weight_grad(const double *A, const double *G, double *g, int n, int d, long units, long weight_units)
{
    for (long w = 0; w < weight_units; ++w)
        for (int a = 0; a < d; ++a)
            for (int b = 0; b < d; ++b) {
                double acc = 0.0;
                for (long u = w; u < units; u += weight_units)
                    for (int i = 0; i < n; ++i)
                        acc += A[(u * n + i) * d + a] * G[(u * n + i) * d + b];
                g[(w * d + a) * d + b] = acc;
            }
}
