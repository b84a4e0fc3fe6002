/*
 * CPU fp64 oracle for cyclic coordinate descent on the layer objective
 * (GuidedQuant, Section 4.2 "LNQ Algorithm", Eq. 10, and Appendix B.2
 * "Efficient Implementation of CD Algorithm in LNQ", Algorithms 3 and 4).
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing in the product path may call this file;
 * it shares no code, header, table or helper with the CUDA library.
 *
 * Problem (fixed codebooks, Eq. 9 with the guided Hessians of Eq. 7): for every
 * group k and every output channel j in J_k minimise
 *     (what_j - w_j)^T H_k (what_j - w_j)     over what_j in {c^(j)_1..c^(j)_m}^{d_in}
 * by cyclic CD: coordinates i = 1..d_in in order, each set to its exact minimiser
 *     Round_j( W_ij - sum_{c != i} H_ic / H_ii * (What_cj - W_cj) )               (Eq. 10).
 *
 * Array conventions are those of the C-ABI library: W, W_hat are [d_out][d_in]
 * (row j = the paper's column w_j), H is [g][d_in][d_in] full symmetric,
 * codebook is [d_out][m], codes Q are [d_out][d_in] (0-based index into the
 * channel's codebook).  Inputs are fp32 bit patterns widened exactly; all
 * arithmetic is fp64.
 *
 * How the sums of Eq. 10 are carried (derived from Eq. 10, not taken from the printed pseudo-code).
 * Write Ht = diag(H)^-1 H and E = What - W.  Coordinate i needs  t_i = sum_{c != i} Ht_ic E_c  with the
 * E_c of the moment at which i is visited: E_c already updated in this cycle for c < i, still the
 * previous cycle's for c > i.  Split the sum at i:
 *     t_i = sum_{c > i} Ht_ic E_c(old)  +  sum_{c < i} Ht_ic E_c(new).
 * The first part is known before the cycle starts; it is formed for all i at once as
 * B = StrictUpper(Ht) E.  The second part grows as the cycle proceeds: once coordinate c has been
 * decided, Ht_ic E_c(new) is owed to every later coordinate i > c.  Paying that debt immediately, row
 * by row, is the plain form (block size >= d_in).  With a block size b the debt of a coordinate is paid
 * at once only to the later coordinates of its own block, and the whole block's debt to everything
 * after the block is paid in one matrix product when the block is finished.  Each B_i has received
 * exactly the same terms by the time coordinate i is visited, so the decisions do not depend on b.
 *
 * Readings where the paper is silent or at odds with itself:
 *  - Round_j ties: the smaller codebook index wins.
 *  - Algorithms 3/4 write the in-loop correction as U_{(i+1):,i} with U the STRICT UPPER
 *    part of Htilde = diag(H)^-1 H, whose entries below the diagonal are zero; what Eq. 10
 *    requires there is Htilde_{(i+1):,i} (the entries of Htilde below the diagonal), and that
 *    is what is used.  U keeps its printed meaning in B = U (What - W).
 *  - The last block of Algorithm 4 is shorter when b does not divide d_in.
 *  - H_ii <= 0 (a feature that never fired): the row of Htilde is taken as zero, i.e. the
 *    coordinate is rounded to the codebook value nearest to W_ij.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

static int32_t round_idx(double x, const float *cb, int32_t m)
{
    int32_t best = 0;
    double bd = fabs(x - (double)cb[0]);
    for (int32_t q = 1; q < m; ++q) {
        const double dq = fabs(x - (double)cb[q]);
        if (dq < bd) { bd = dq; best = q; }      /* strict: ties keep the smaller index */
    }
    return best;
}

/*
 * Cyclic CD with the sums carried as described above (the scheme of Algorithm 4; with b >= d_in that of
 * Algorithm 3), `cycles` cycles, block size b.
 * W_hat is read as the feasible starting point and overwritten; Q receives the codes.
 * Returns 0, or -1 on bad sizes / allocation failure.
 */
int gq_oracle_cd(const float *W, float *W_hat, int32_t *Q, const float *codebook, int32_t m,
                 int64_t d_in, int64_t d_out, const float *H, int32_t g, int32_t cycles, int64_t b)
{
    if (g < 1 || d_out < 1 || d_in < 1 || d_out % g != 0 || m < 1 || b < 1 || cycles < 0) return -1;
    const int64_t mk = d_out / g;
    int rc = 0;
    for (int32_t k = 0; k < g && rc == 0; ++k) {
        const float *Hk = H + (size_t)k * d_in * d_in;
        /* Htilde = diag(H)^-1 H, row by row */
        double *Ht = (double *)malloc(sizeof(double) * d_in * d_in);
        double *B = (double *)malloc(sizeof(double) * d_in * mk);    /* [d_in][mk] */
        double *E = (double *)malloc(sizeof(double) * d_in * mk);    /* What - W, [d_in][mk] */
        if (!Ht || !B || !E) { free(Ht); free(B); free(E); return -1; }
        for (int64_t r = 0; r < d_in; ++r) {
            const double hrr = (double)Hk[r * d_in + r];
            for (int64_t c = 0; c < d_in; ++c) Ht[r * d_in + c] = hrr > 0.0 ? (double)Hk[r * d_in + c] / hrr : 0.0;
        }
        for (int32_t cyc = 0; cyc < cycles; ++cyc) {
            for (int64_t i = 0; i < d_in; ++i)
                for (int64_t j = 0; j < mk; ++j)
                    E[i * mk + j] = (double)W_hat[(k * mk + j) * d_in + i] - (double)W[(k * mk + j) * d_in + i];
            /* the part of every t_i that is known before the cycle: B = StrictUpper(Ht) E */
#pragma omp parallel for schedule(static)
            for (int64_t r = 0; r < d_in; ++r)
                for (int64_t j = 0; j < mk; ++j) {
                    double acc = 0.0;
                    for (int64_t c = r + 1; c < d_in; ++c) acc += Ht[r * d_in + c] * E[c * mk + j];
                    B[r * mk + j] = acc;
                }
            for (int64_t s = 0; s < d_in; s += b) {
                const int64_t e = s + b < d_in ? s + b : d_in;
                for (int64_t i = s; i < e; ++i) {
                    /* Eq. 10 for coordinate i of every channel: Round_j(W_ij - t_i) */
                    for (int64_t j = 0; j < mk; ++j) {
                        const int64_t ch = k * mk + j;
                        const double target = (double)W[ch * d_in + i] - B[i * mk + j];
                        const int32_t q = round_idx(target, codebook + ch * m, m);
                        Q[ch * d_in + i] = q;
                        W_hat[ch * d_in + i] = codebook[ch * m + q];
                        E[i * mk + j] = (double)codebook[ch * m + q] - (double)W[ch * d_in + i];
                    }
                    /* coordinate i's debt to the later coordinates of its own block */
                    for (int64_t r = i + 1; r < e; ++r)
                        for (int64_t j = 0; j < mk; ++j) B[r * mk + j] += Ht[r * d_in + i] * E[i * mk + j];
                }
                /* the finished block's debt to every coordinate after it, in one product */
#pragma omp parallel for schedule(static)
                for (int64_t r = e; r < d_in; ++r)
                    for (int64_t j = 0; j < mk; ++j) {
                        double acc = 0.0;
                        for (int64_t c = s; c < e; ++c) acc += Ht[r * d_in + c] * E[c * mk + j];
                        B[r * mk + j] += acc;
                    }
            }
        }
        free(Ht); free(B); free(E);
    }
    return rc;
}
