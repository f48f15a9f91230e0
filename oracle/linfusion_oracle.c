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
 * The feature width of Q and K may differ from the channel width of V (Prop. 3: f' and g' may
 * widen the features to d' while the values keep d).  Every routine therefore takes two widths:
 * dk (= d', columns of Q and K, rows of S, length of z) and dv (= d, columns of V and Y, columns
 * of S).  dk = dv is the case the released model uses.
 *
 * All arrays are dense row-major doubles: q, k are [slabs][n][dk]; v, y are [slabs][n][dv];
 * S is [slabs][dk][dv] (row = feature c of K, column = channel e of V);
 * z is [slabs][dk].  Sums run in index order; threads only split independent
 * outputs (rows of S, rows of Y), never a single sum.
 *
 * The second half of the file states the producers of Q, K, V from the layer input X
 * (Sec. 3.1, implementation details; Eq. 2 for V): oracle_linear_map, oracle_layernorm,
 * oracle_leaky_relu and oracle_mlp_producer.
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
void oracle_state(const double* k, const double* v, long slabs, long n, int dk, int dv,
                  int phi_kind, double* S, double* z)
{
    long rows = slabs * (long)dk;
#pragma omp parallel for schedule(static)
    for (long r = 0; r < rows; ++r) {
        long s = r / dk;
        int c = (int)(r % dk);
        const double* ks = k + (size_t)s * n * dk;
        const double* vs = v + (size_t)s * n * dv;
        double* Srow = S + ((size_t)s * dk + c) * dv;
        double zc = 0.0;
        for (int e = 0; e < dv; ++e) Srow[e] = 0.0;
        for (long j = 0; j < n; ++j) {
            double p = oracle_phi(ks[(size_t)j * dk + c], phi_kind);
            zc += p;
            for (int e = 0; e < dv; ++e) Srow[e] += p * vs[(size_t)j * dv + e];
        }
        z[(size_t)s * dk + c] = zc;
    }
}

/* Apply: Y_i = phi(Q_i) S / (phi(Q_i) . z + eps)   (Prop. 2 output with Eq. 5's division). */
void oracle_apply(const double* q, const double* S, const double* z, long slabs, long n,
                  int dk, int dv, double eps, int phi_kind, double* y)
{
    long rows = slabs * n;
#pragma omp parallel for schedule(static)
    for (long r = 0; r < rows; ++r) {
        long s = r / n;
        const double* qi = q + (size_t)r * dk;
        const double* Ss = S + (size_t)s * dk * dv;
        const double* zs = z + (size_t)s * dk;
        double* yi = y + (size_t)r * dv;
        double den = 0.0;
        for (int e = 0; e < dv; ++e) yi[e] = 0.0;
        for (int c = 0; c < dk; ++c) {
            double p = oracle_phi(qi[c], phi_kind);
            den += p * zs[c];
            for (int e = 0; e < dv; ++e) yi[e] += p * Ss[(size_t)c * dv + e];
        }
        den += eps;
        for (int e = 0; e < dv; ++e) yi[e] /= den;
    }
}

/* Apply without the normalizer: Y_i = phi(Q_i) S, i.e. Y = f'(X) g'(X)^T X of Prop. 2 before
 * Eq. 5's division is put on top (the "without normalization" rows of the ablation in Tab. 2). */
void oracle_apply_unnormalized(const double* q, const double* S, long slabs, long n, int dk, int dv,
                               int phi_kind, double* y)
{
    long rows = slabs * n;
#pragma omp parallel for schedule(static)
    for (long r = 0; r < rows; ++r) {
        long s = r / n;
        const double* qi = q + (size_t)r * dk;
        const double* Ss = S + (size_t)s * dk * dv;
        double* yi = y + (size_t)r * dv;
        for (int e = 0; e < dv; ++e) yi[e] = 0.0;
        for (int c = 0; c < dk; ++c) {
            double p = oracle_phi(qi[c], phi_kind);
            for (int e = 0; e < dv; ++e) yi[e] += p * Ss[(size_t)c * dv + e];
        }
    }
}

/* The whole path in its linear form.  Returns 0, or -1 if scratch memory cannot be had. */
int oracle_linear(const double* q, const double* k, const double* v, long slabs, long n,
                  int dk, int dv, double eps, int phi_kind, double* y)
{
    double* S = (double*)malloc(sizeof(double) * (size_t)slabs * dk * dv);
    double* z = (double*)malloc(sizeof(double) * (size_t)slabs * dk);
    if (!S || !z) { free(S); free(z); return -1; }
    oracle_state(k, v, slabs, n, dk, dv, phi_kind, S, z);
    oracle_apply(q, S, z, slabs, n, dk, dv, eps, phi_kind, y);
    free(S);
    free(z);
    return 0;
}

/* The attention-matrix form: M_ij = w_ij / (sum_k w_ik + eps), w_ij = phi(Q_i) . phi(K_j),
 * Y = M V (Eq. 4 with the mask dropped, rows normalized as in Sec. 2.2).  O(n^2 d): tiny n only.
 * If m_out is not NULL it receives the n x n matrix M of every slab, [slabs][n][n]. */
void oracle_quadratic(const double* q, const double* k, const double* v, long slabs, long n,
                      int dk, int dv, double eps, int phi_kind, double* y, double* m_out)
{
    for (long s = 0; s < slabs; ++s) {
        const double* qs = q + (size_t)s * n * dk;
        const double* ks = k + (size_t)s * n * dk;
        const double* vs = v + (size_t)s * n * dv;
        double* ys = y + (size_t)s * n * dv;
        double* w = (double*)malloc(sizeof(double) * (size_t)n);
        for (long i = 0; i < n; ++i) {
            double rowsum = 0.0;
            for (long j = 0; j < n; ++j) {
                double wij = 0.0;
                for (int c = 0; c < dk; ++c)
                    wij += oracle_phi(qs[(size_t)i * dk + c], phi_kind) *
                           oracle_phi(ks[(size_t)j * dk + c], phi_kind);
                w[j] = wij;
                rowsum += wij;
            }
            rowsum += eps;
            for (int e = 0; e < dv; ++e) {
                double acc = 0.0;
                for (long j = 0; j < n; ++j) acc += (w[j] / rowsum) * vs[(size_t)j * dv + e];
                ys[(size_t)i * dv + e] = acc;
            }
            if (m_out)
                for (long j = 0; j < n; ++j)
                    m_out[((size_t)s * n + i) * n + j] = w[j] / rowsum;
        }
        free(w);
    }
}

/* ------------------------------------------------------------------------------------------
 * Producers of Q, K, V from the layer input X (Sec. 3.1, implementation details; Eq. 2).
 *
 *   V = X W_V                                               (Eq. 2)
 *   Q = f'(X),  K = g'(X),   each  X W_lin + LeakyReLU(LayerNorm(X W_1 + b_1))
 *
 * i.e. an MLP made of a linear branch and a non-linear branch with one Linear-LayerNorm-LeakyReLU
 * block, the two results added.  The paper initializes the linear branch with the attention's
 * W_Q (W_K) and the non-linear branch's OUTPUT with zero; with this block that is a LayerNorm
 * whose scale and shift start at zero, so f'(X) = X W_Q at initialization.  Readings where the
 * text is silent: the linear branch has no bias (the projections it is initialized from have
 * none); the block's Linear has a bias b_1; LayerNorm runs over the whole feature vector of a
 * token (all heads, before the split into heads), biased variance, epsilon inside the root,
 * per-feature scale gamma and shift beta; LeakyReLU's negative slope is a parameter (0.01 in
 * the tests).  X is [n][c_in]; W is [c_in][c_out]; outputs are [n][c_out].
 * ------------------------------------------------------------------------------------------ */

/* out = X W (+ bias).  bias may be NULL. */
void oracle_linear_map(const double* x, const double* w, const double* bias, long n, int c_in,
                       int c_out, double* out)
{
#pragma omp parallel for schedule(static)
    for (long i = 0; i < n; ++i) {
        for (int o = 0; o < c_out; ++o) {
            double acc = 0.0;
            for (int c = 0; c < c_in; ++c) acc += x[(size_t)i * c_in + c] * w[(size_t)c * c_out + o];
            out[(size_t)i * c_out + o] = acc + (bias ? bias[o] : 0.0);
        }
    }
}

/* Row-wise layer normalization: out_io = (p_io - mean_i) / sqrt(var_i + ln_eps) * gamma_o + beta_o,
 * mean and (biased) variance taken over the c features of row i. */
void oracle_layernorm(const double* p, const double* gamma, const double* beta, double ln_eps,
                      long n, int c, double* out)
{
#pragma omp parallel for schedule(static)
    for (long i = 0; i < n; ++i) {
        const double* row = p + (size_t)i * c;
        double mean = 0.0, var = 0.0;
        for (int o = 0; o < c; ++o) mean += row[o];
        mean /= (double)c;
        for (int o = 0; o < c; ++o) var += (row[o] - mean) * (row[o] - mean);
        var /= (double)c;
        double inv = 1.0 / sqrt(var + ln_eps);
        for (int o = 0; o < c; ++o) out[(size_t)i * c + o] = (row[o] - mean) * inv * gamma[o] + beta[o];
    }
}

/* LeakyReLU: x for x >= 0, slope * x otherwise. */
double oracle_leaky_relu(double x, double slope) { return x >= 0.0 ? x : slope * x; }

/* f'(X) (or g'(X)): X W_lin + LeakyReLU(LayerNorm(X W_1 + b_1; gamma, beta)).
 * Returns 0, or -1 if scratch memory cannot be had. */
int oracle_mlp_producer(const double* x, const double* w_lin, const double* w_1, const double* b_1,
                        const double* gamma, const double* beta, double ln_eps, double slope,
                        long n, int c_in, int c_out, double* out)
{
    double* pre = (double*)malloc(sizeof(double) * (size_t)n * c_out);
    double* nrm = (double*)malloc(sizeof(double) * (size_t)n * c_out);
    if (!pre || !nrm) { free(pre); free(nrm); return -1; }
    oracle_linear_map(x, w_1, b_1, n, c_in, c_out, pre);
    oracle_layernorm(pre, gamma, beta, ln_eps, n, c_out, nrm);
    oracle_linear_map(x, w_lin, NULL, n, c_in, c_out, out);
    for (size_t t = 0; t < (size_t)n * c_out; ++t) out[t] += oracle_leaky_relu(nrm[t], slope);
    free(pre);
    free(nrm);
    return 0;
}
