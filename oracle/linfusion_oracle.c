/*
 * fp64 CPU oracle for normalized, non-causal generalized linear attention.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * attention computes.  It shares no code with the CUDA library and is never on
 * the product path: only the tests, the smoke check and the benchmark's
 * CPU-baseline leg call it.
 *
 * Notation follows the paper.  With the role map of Eq. 3-4 (C <-> Q, B <-> K,
 * X <-> V) and the gates absorbed into f' and g' (Prop. 2 / Prop. 3), one
 * (batch, head) slab holds Q = f'(X), K = g'(X) in R^{n x d} and V in R^{n x d}:
 *
 *   state        H = phi(K)^T V            in R^{d x d}   ("S" below; g'(X)^T X of Prop. 2)
 *   normalizer   Z = sum_j phi(K_j)        in R^{1 x d}   ("z";  Eq. 5 without the causal scan)
 *   output       Y_i = phi(Q_i) H / (sum_c phi(Q_ic) Z_c + eps)   (C' = C / sum(C * Z) of Eq. 5)
 *
 * phi is the non-negative activation of Sec. 2.2; the paper gives no closed
 * form, the reading used here is phi(x) = elu(x) + 1.  eps is not in the paper;
 * it is added once to the full denominator.  No activation is applied to V and
 * there is no 1/sqrt(d') scaling.
 *
 * The linear form equals the attention-matrix form exactly (associativity,
 * Prop. 2), so two routines are given: oracle_linear (state, then apply) and
 * oracle_quadratic (explicit n x n weights M_ij, row-normalized as Sec. 2.2
 * requires: sum_k M_ik = 1 up to eps).  The second exists to pin the first.
 *
 * All arrays are dense row-major doubles: q, k, v, y are [slabs][n][d];
 * S is [slabs][d][d] (row = feature c of K, column = channel e of V);
 * z is [slabs][d].  Sums run in index order; threads only split independent
 * outputs (rows of S, rows of Y), never a single sum.
 */
#include <math.h>
#include <stddef.h>
#include <stdlib.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_PHI_ELU_PLUS_ONE = 0, ORACLE_PHI_IDENTITY = 1 };

/* Non-negative activation (Sec. 2.2): elu(x) + 1 = x + 1 for x > 0, exp(x) otherwise. */
double oracle_phi(double x, int phi_kind)
{
    if (phi_kind == ORACLE_PHI_IDENTITY) return x;
    return x > 0.0 ? x + 1.0 : exp(x);
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* State and normalizer of one or more slabs: S = phi(K)^T V, z = sum_j phi(K_j)
 * (Prop. 2's g'(X)^T X; Eq. 5's Z with the scan replaced by the full sum). */
void oracle_state(const double* k, const double* v, long slabs, long n, int d,
                  int phi_kind, double* S, double* z)
{
    long rows = slabs * (long)d;
#pragma omp parallel for schedule(static)
    for (long r = 0; r < rows; ++r) {
        long s = r / d;
        int c = (int)(r % d);
        const double* ks = k + (size_t)s * n * d;
        const double* vs = v + (size_t)s * n * d;
        double* Srow = S + ((size_t)s * d + c) * d;
        double zc = 0.0;
        for (int e = 0; e < d; ++e) Srow[e] = 0.0;
        for (long j = 0; j < n; ++j) {
            double p = oracle_phi(ks[(size_t)j * d + c], phi_kind);
            zc += p;
            for (int e = 0; e < d; ++e) Srow[e] += p * vs[(size_t)j * d + e];
        }
        z[(size_t)s * d + c] = zc;
    }
}

/* Apply: Y_i = phi(Q_i) S / (phi(Q_i) . z + eps)   (Prop. 2 output with Eq. 5's division). */
void oracle_apply(const double* q, const double* S, const double* z, long slabs, long n,
                  int d, double eps, int phi_kind, double* y)
{
    long rows = slabs * n;
#pragma omp parallel for schedule(static)
    for (long r = 0; r < rows; ++r) {
        long s = r / n;
        const double* qi = q + (size_t)r * d;
        const double* Ss = S + (size_t)s * d * d;
        const double* zs = z + (size_t)s * d;
        double* yi = y + (size_t)r * d;
        double den = 0.0;
        for (int e = 0; e < d; ++e) yi[e] = 0.0;
        for (int c = 0; c < d; ++c) {
            double p = oracle_phi(qi[c], phi_kind);
            den += p * zs[c];
            for (int e = 0; e < d; ++e) yi[e] += p * Ss[(size_t)c * d + e];
        }
        den += eps;
        for (int e = 0; e < d; ++e) yi[e] /= den;
    }
}

/* Apply without the normalizer: Y_i = phi(Q_i) S, i.e. Y = f'(X) g'(X)^T X of Prop. 2 before
 * Eq. 5's division is put on top (the "without normalization" rows of the ablation in Tab. 2). */
void oracle_apply_unnormalized(const double* q, const double* S, long slabs, long n, int d,
                               int phi_kind, double* y)
{
    long rows = slabs * n;
#pragma omp parallel for schedule(static)
    for (long r = 0; r < rows; ++r) {
        long s = r / n;
        const double* qi = q + (size_t)r * d;
        const double* Ss = S + (size_t)s * d * d;
        double* yi = y + (size_t)r * d;
        for (int e = 0; e < d; ++e) yi[e] = 0.0;
        for (int c = 0; c < d; ++c) {
            double p = oracle_phi(qi[c], phi_kind);
            for (int e = 0; e < d; ++e) yi[e] += p * Ss[(size_t)c * d + e];
        }
    }
}

/* The whole path in its linear form.  Returns 0, or -1 if scratch memory cannot be had. */
int oracle_linear(const double* q, const double* k, const double* v, long slabs, long n,
                  int d, double eps, int phi_kind, double* y)
{
    double* S = (double*)malloc(sizeof(double) * (size_t)slabs * d * d);
    double* z = (double*)malloc(sizeof(double) * (size_t)slabs * d);
    if (!S || !z) { free(S); free(z); return -1; }
    oracle_state(k, v, slabs, n, d, phi_kind, S, z);
    oracle_apply(q, S, z, slabs, n, d, eps, phi_kind, y);
    free(S);
    free(z);
    return 0;
}

/* The attention-matrix form: M_ij = w_ij / (sum_k w_ik + eps), w_ij = phi(Q_i) . phi(K_j),
 * Y = M V (Eq. 4 with the mask dropped, rows normalized as in Sec. 2.2).  O(n^2 d): tiny n only.
 * If m_out is not NULL it receives the n x n matrix M of every slab, [slabs][n][n]. */
void oracle_quadratic(const double* q, const double* k, const double* v, long slabs, long n,
                      int d, double eps, int phi_kind, double* y, double* m_out)
{
    for (long s = 0; s < slabs; ++s) {
        const double* qs = q + (size_t)s * n * d;
        const double* ks = k + (size_t)s * n * d;
        const double* vs = v + (size_t)s * n * d;
        double* ys = y + (size_t)s * n * d;
        double* w = (double*)malloc(sizeof(double) * (size_t)n);
        for (long i = 0; i < n; ++i) {
            double rowsum = 0.0;
            for (long j = 0; j < n; ++j) {
                double wij = 0.0;
                for (int c = 0; c < d; ++c)
                    wij += oracle_phi(qs[(size_t)i * d + c], phi_kind) *
                           oracle_phi(ks[(size_t)j * d + c], phi_kind);
                w[j] = wij;
                rowsum += wij;
            }
            rowsum += eps;
            for (int e = 0; e < d; ++e) {
                double acc = 0.0;
                for (long j = 0; j < n; ++j) acc += (w[j] / rowsum) * vs[(size_t)j * d + e];
                ys[(size_t)i * d + e] = acc;
            }
            if (m_out)
                for (long j = 0; j < n; ++j)
                    m_out[((size_t)s * n + i) * n + j] = w[j] / rowsum;
        }
        free(w);
    }
}
