/*
 * CPU fp64 oracle for the guided layer objective of GuidedQuant.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing in the product path may call this file;
 * it shares no code, header, table or helper with the CUDA library.  It is
 * written to be checked against the paper by eye: every function is the
 * paper's definition as plain loops in fp64, with no blocking, fusion or
 * reordering beyond a transposed copy of X (so that a column is contiguous)
 * and an OpenMP split of the outermost independent index.
 *
 * Inputs are the exact bit patterns handed to the GPU (bf16 as uint16_t,
 * fp32 weights); both widen to fp64 without rounding.
 *
 * Notation (paper, Section 2 "Preliminaries" and Section 3.2):
 *   n tokens, X in R^{n x d_in}, dl/dZ in R^{n x d_out}, g groups,
 *   J_k = {m k, ..., m (k+1) - 1} with m = d_out / g (0-based; Algorithm 1, grouping step).
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double bf16_to_f64(uint16_t b)
{
    uint32_t u = ((uint32_t)b) << 16;   /* bf16 is the top half of an fp32 */
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/*
 * Algorithm 1, saliency step (and the averaged-squared-gradient form under Eq. 7):
 *   s_k[i] = 1/|J_k| * sum_{j in J_k} (grad_scale * dl/dZ[i][j])^2
 * grad_scale is the constant the paper multiplies gradients by (10^3 in its
 * experiments, Section 3.2); it is applied to the gradient before squaring.
 * grad: [n][ld_grad] bf16 bits, s: [g][ld_s] fp64.  Returns 0, or -1 on bad sizes.
 */
int gq_oracle_saliency(const uint16_t *grad, int64_t n, int64_t d_out, int64_t ld_grad,
                       int32_t g, double grad_scale, double *s, int64_t ld_s)
{
    if (g < 1 || d_out < 1 || d_out % g != 0 || ld_grad < d_out || ld_s < n) return -1;
    const int64_t m = d_out / g;
    for (int32_t k = 0; k < g; ++k) {
#pragma omp parallel for schedule(static)
        for (int64_t i = 0; i < n; ++i) {
            double acc = 0.0;
            for (int64_t j = m * k; j < m * (k + 1); ++j) {
                double gij = grad_scale * bf16_to_f64(grad[i * ld_grad + j]);
                acc += gij * gij;
            }
            s[(int64_t)k * ld_s + i] = acc / (double)m;
        }
    }
    return 0;
}

/*
 * The same saliency for a gradient as a backward pass hands it over (Section 3.2: only the averaged squared
 * gradients of a layer are kept): a [batch][seq][d_out] array with element strides (stride_b, stride_t, 1),
 * stored as bf16 (dtype 0), IEEE half (dtype 1) or fp32 (dtype 2); token i = b * seq + t.  Every input value
 * widens to fp64 without rounding.  s: [g][ld_s] fp64.  Returns 0, or -1 on bad sizes / an unknown dtype.
 */
static double half_to_f64(uint16_t h)
{
    const int sign = (h >> 15) & 1, expo = (h >> 10) & 0x1f, frac = h & 0x3ff;
    double v;
    if (expo == 0) v = (double)frac / 1024.0 / 16384.0;                       /* subnormal: frac * 2^-24 */
    else if (expo == 31) v = frac ? (0.0 / 0.0) : (1.0 / 0.0);
    else {
        v = 1.0 + (double)frac / 1024.0;
        for (int e = expo; e > 15; --e) v *= 2.0;
        for (int e = expo; e < 15; ++e) v *= 0.5;
    }
    return sign ? -v : v;
}

int gq_oracle_saliency_strided(const void *grad, int32_t dtype, int64_t batch, int64_t seq, int64_t d_out,
                               int64_t stride_b, int64_t stride_t, int32_t g, double grad_scale, double *s,
                               int64_t ld_s)
{
    if (g < 1 || d_out < 1 || d_out % g != 0 || batch < 0 || seq < 0 || ld_s < batch * seq) return -1;
    if (dtype < 0 || dtype > 2) return -1;
    const int64_t m = d_out / g;
    for (int32_t k = 0; k < g; ++k) {
#pragma omp parallel for schedule(static)
        for (int64_t i = 0; i < batch * seq; ++i) {
            const int64_t b = i / seq, t = i % seq;
            const int64_t base = b * stride_b + t * stride_t;
            double acc = 0.0;
            for (int64_t j = m * k; j < m * (k + 1); ++j) {
                double v;
                if (dtype == 0) v = bf16_to_f64(((const uint16_t *)grad)[base + j]);
                else if (dtype == 1) v = half_to_f64(((const uint16_t *)grad)[base + j]);
                else v = (double)((const float *)grad)[base + j];
                const double gij = grad_scale * v;
                acc += gij * gij;
            }
            s[(int64_t)k * ld_s + i] = acc / (double)m;
        }
    }
    return 0;
}

/*
 * Algorithm 1, Hessian step:  H_k = X^T Diag(s_k) X, i.e.
 *   H_k[a][b] (+)= sum_{i=1..n} s_k[i] * X[i][a] * X[i][b]      for all a, b.
 * No 1/n factor (Section 3.2 writes the unguided case as H = X^T X).
 * The whole d_in x d_in matrix is computed entry by entry (no use of symmetry).
 * X: [n][ld_x] bf16 bits, s: [g][ld_s] fp64, H: [g][d_in][d_in] fp64, ADDED to
 * (so a caller can stream token chunks; zero H first for a single shot).
 * Returns 0, -1 on bad sizes, -2 if out of memory.
 */
int gq_oracle_hessian_accumulate(const uint16_t *X, int64_t n, int64_t d_in, int64_t ld_x,
                                 const double *s, int64_t ld_s, int32_t g, double *H)
{
    if (g < 1 || d_in < 1 || ld_x < d_in || ld_s < n || n < 0) return -1;
    if (n == 0) return 0;
    double *Xt = (double *)malloc(sizeof(double) * (size_t)d_in * (size_t)n);   /* Xt[a][i] = X[i][a] */
    if (!Xt) return -2;
    for (int64_t i = 0; i < n; ++i)
        for (int64_t a = 0; a < d_in; ++a)
            Xt[a * n + i] = bf16_to_f64(X[i * ld_x + a]);

    int fail = 0;
    for (int32_t k = 0; k < g; ++k) {
        const double *sk = s + (int64_t)k * ld_s;
        double *Hk = H + (int64_t)k * d_in * d_in;
#pragma omp parallel
        {
            double *col = (double *)malloc(sizeof(double) * (size_t)n);   /* s_k[i] * X[i][a] */
            if (!col) {
#pragma omp atomic write
                fail = 1;
            }
#pragma omp for schedule(dynamic, 4)
            for (int64_t a = 0; a < d_in; ++a) {
                if (!col) continue;
                for (int64_t i = 0; i < n; ++i) col[i] = sk[i] * Xt[a * n + i];
                for (int64_t b = 0; b < d_in; ++b) {
                    const double *xb = Xt + b * n;
                    double acc = 0.0;
                    for (int64_t i = 0; i < n; ++i) acc += col[i] * xb[i];
                    Hk[a * d_in + b] += acc;
                }
            }
            free(col);
        }
    }
    free(Xt);
    return fail ? -2 : 0;
}

/*
 * Eq. 7 (the objective after the averaging approximation):
 *   loss_k = sum_{j in J_k} (w_j - what_j)^T H_k (w_j - what_j),   total = sum_k loss_k.
 * W, What: [d_out][d_in] fp32, row j = output channel j (the paper's column w_j).
 * H: [g][d_in][d_in] fp64 (all entries are read).  loss: [g + 1], loss[g] = total.
 */
int gq_oracle_objective(const float *W, const float *What, int64_t d_in, int64_t d_out,
                        const double *H, int32_t g, double *loss)
{
    if (g < 1 || d_out < 1 || d_out % g != 0 || d_in < 1) return -1;
    const int64_t m = d_out / g;
    double total = 0.0;
    for (int32_t k = 0; k < g; ++k) {
        const double *Hk = H + (int64_t)k * d_in * d_in;
        double lk = 0.0;
        int fail = 0;
#pragma omp parallel reduction(+ : lk)
        {
            double *delta = (double *)malloc(sizeof(double) * (size_t)d_in);
            if (!delta) {
#pragma omp atomic write
                fail = 1;
            }
#pragma omp for schedule(static)
            for (int64_t j = m * k; j < m * (k + 1); ++j) {
                if (!delta) continue;
                for (int64_t a = 0; a < d_in; ++a)
                    delta[a] = (double)W[j * d_in + a] - (double)What[j * d_in + a];
                double q = 0.0;
                for (int64_t a = 0; a < d_in; ++a) {
                    double row = 0.0;
                    for (int64_t b = 0; b < d_in; ++b) row += Hk[a * d_in + b] * delta[b];
                    q += delta[a] * row;
                }
                lk += q;
            }
            free(delta);
        }
        if (fail) return -2;
        loss[k] = lk;
        total += lk;
    }
    loss[g] = total;
    return 0;
}

/*
 * Two consequences of the definition H_k = X^T Diag(s_k) X (Algorithm 1, Hessian step) that need only
 * O(n d_in) work per group and can therefore be evaluated at full size, where the d_in x d_in matrix
 * cannot: its diagonal and its action on a vector.  Both are ADDED to, token chunk after token chunk.
 *
 *   diag[k][a]   (+)= sum_i s_k[i] * X[i][a]^2                                (= H_k[a][a])
 */
int gq_oracle_hessian_diag(const uint16_t *X, int64_t n, int64_t d_in, int64_t ld_x,
                           const double *s, int64_t ld_s, int32_t g, double *diag)
{
    if (g < 1 || d_in < 1 || ld_x < d_in || ld_s < n || n < 0) return -1;
    for (int32_t k = 0; k < g; ++k) {
        const double *sk = s + (int64_t)k * ld_s;
        double *dk = diag + (int64_t)k * d_in;
        /* the entries a are independent: threads take runs of 64 of them and walk the tokens in order */
#pragma omp parallel for schedule(static)
        for (int64_t a0 = 0; a0 < d_in; a0 += 64) {
            const int64_t a1 = a0 + 64 < d_in ? a0 + 64 : d_in;
            for (int64_t i = 0; i < n; ++i)
                for (int64_t a = a0; a < a1; ++a) {
                    const double x = bf16_to_f64(X[i * ld_x + a]);
                    dk[a] += sk[i] * x * x;
                }
        }
    }
    return 0;
}

/*
 *   out[k][v][a] (+)= sum_i s_k[i] * (sum_b X[i][b] V[v][b]) * X[i][a]        (= (H_k V[v])[a])
 * V: [nv][d_in] fp64 probe vectors, out: [g][nv][d_in] fp64.  Returns 0, -1 on bad sizes, -2 if out of memory.
 */
int gq_oracle_hessian_apply(const uint16_t *X, int64_t n, int64_t d_in, int64_t ld_x,
                            const double *s, int64_t ld_s, int32_t g, const double *V, int32_t nv,
                            double *out)
{
    if (g < 1 || d_in < 1 || ld_x < d_in || ld_s < n || n < 0 || nv < 1) return -1;
    if (n == 0) return 0;
    double *y = (double *)malloc(sizeof(double) * (size_t)n * (size_t)nv);      /* y[v][i] = x_i . V[v] */
    if (!y) return -2;
    for (int32_t v = 0; v < nv; ++v) {
#pragma omp parallel for schedule(static)
        for (int64_t i = 0; i < n; ++i) {
            double acc = 0.0;
            for (int64_t b = 0; b < d_in; ++b) acc += bf16_to_f64(X[i * ld_x + b]) * V[(int64_t)v * d_in + b];
            y[(int64_t)v * n + i] = acc;
        }
    }
    for (int32_t k = 0; k < g; ++k) {
        const double *sk = s + (int64_t)k * ld_s;
        for (int32_t v = 0; v < nv; ++v) {
            const double *yv = y + (int64_t)v * n;
            double *ov = out + ((int64_t)k * nv + v) * d_in;
#pragma omp parallel for schedule(static)
            for (int64_t a0 = 0; a0 < d_in; a0 += 64) {
                const int64_t a1 = a0 + 64 < d_in ? a0 + 64 : d_in;
                for (int64_t i = 0; i < n; ++i) {
                    const double wi = sk[i] * yv[i];
                    for (int64_t a = a0; a < a1; ++a) ov[a] += wi * bf16_to_f64(X[i * ld_x + a]);
                }
            }
        }
    }
    free(y);
    return 0;
}

/* Number of OpenMP threads the loops above will use (reported by the benchmark). */
#ifdef _OPENMP
#include <omp.h>
int gq_oracle_threads(void) { return omp_get_max_threads(); }
#else
int gq_oracle_threads(void) { return 1; }
#endif
