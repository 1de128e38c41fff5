/*
 * ORACLE -- TEST INFRASTRUCTURE ONLY.  Nothing on the product path may call this.
 *
 * Plain per-token Semidirect Fourier Delta Attention recurrence in complex
 * double precision, written straight from the definition of the layer
 * (Section 3, Eq. "sfda" and the output equation below it):
 *
 *     Lambda_t = diag(alpha_t * exp(i theta_t))
 *     S_t      = (I - beta_t k_t k_t^*) Lambda_t S_{t-1} + beta_t k_t v_t^*
 *     o_t      = S_t^* q_t
 *
 * Reading of the storage (stated by the workload, not by the paper): the key
 * space is R^{2m} ~ C^m with real channel 2j = Re and 2j+1 = Im of complex
 * coordinate j (the aligned 2x2 blocks of Prop. "Complex phases are real block
 * rotations"); v is real, so v^* = v^T; S is m x d_v complex, stored as 2m real
 * rows (row 2j = Re, row 2j+1 = Im of complex row j).
 *
 * No blocking, no reordering, no fusion: one token at a time, every step in the
 * order the equation states it (phase-decay, erase, write, read).
 * Sequences are independent; OpenMP only distributes whole sequences.
 */
#include <complex.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * q, k      : [N, T, 2m]   real pairs (Re, Im) of the complex query / key
 * v         : [N, T, dv]   real values
 * alpha     : [N, T, m]    decay per complex coordinate
 * theta     : [N, T, m]    phase per complex coordinate (radians)
 * beta      : [N, T]       step size
 * S0        : [N, 2m, dv]  initial state (paired rows) or NULL for zero
 * o_re,o_im : [N, T, dv]   real and imaginary part of o_t = S_t^* q_t
 * S_T       : [N, 2m, dv]  final state (paired rows), may be NULL
 * returns 0, or -1 when scratch allocation fails.
 */
int oracle_sfda_recurrence(const double *q, const double *k, const double *v,
                           const double *alpha, const double *theta,
                           const double *beta, const double *S0,
                           double *o_re, double *o_im, double *S_T,
                           long N, long T, int m, int dv)
{
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (long n = 0; n < N; ++n) {
        double complex *S = malloc(sizeof(double complex) * (size_t)m * dv);
        double complex *c = malloc(sizeof(double complex) * (size_t)dv);
        double complex *kc = malloc(sizeof(double complex) * (size_t)m);
        double complex *qc = malloc(sizeof(double complex) * (size_t)m);
        if (!S || !c || !kc || !qc) {
            failed = 1;
            free(S); free(c); free(kc); free(qc);
            continue;
        }
        for (int j = 0; j < m; ++j)
            for (int x = 0; x < dv; ++x)
                S[(size_t)j * dv + x] = S0
                    ? S0[((size_t)n * 2 * m + 2 * j) * dv + x] +
                      I * S0[((size_t)n * 2 * m + 2 * j + 1) * dv + x]
                    : 0.0;

        for (long t = 0; t < T; ++t) {
            const double *qt = q + ((size_t)n * T + t) * 2 * m;
            const double *kt = k + ((size_t)n * T + t) * 2 * m;
            const double *vt = v + ((size_t)n * T + t) * dv;
            const double *at = alpha + ((size_t)n * T + t) * m;
            const double *tt = theta + ((size_t)n * T + t) * m;
            const double bt = beta[(size_t)n * T + t];

            for (int j = 0; j < m; ++j) {
                kc[j] = kt[2 * j] + I * kt[2 * j + 1];
                qc[j] = qt[2 * j] + I * qt[2 * j + 1];
            }
            /* S <- Lambda_t S */
            for (int j = 0; j < m; ++j) {
                const double complex lam = at[j] * cexp(I * tt[j]);
                for (int x = 0; x < dv; ++x)
                    S[(size_t)j * dv + x] *= lam;
            }
            /* c <- k^* (Lambda_t S_{t-1})   (row vector, conjugate on k) */
            for (int x = 0; x < dv; ++x) {
                double complex acc = 0.0;
                for (int j = 0; j < m; ++j)
                    acc += conj(kc[j]) * S[(size_t)j * dv + x];
                c[x] = acc;
            }
            /* S <- S - beta k c + beta k v^T */
            for (int j = 0; j < m; ++j)
                for (int x = 0; x < dv; ++x)
                    S[(size_t)j * dv + x] += kc[j] * (bt * (vt[x] - c[x]));
            /* o_t <- S_t^* q_t   (conjugate transpose on the UPDATED state) */
            for (int x = 0; x < dv; ++x) {
                double complex acc = 0.0;
                for (int j = 0; j < m; ++j)
                    acc += conj(S[(size_t)j * dv + x]) * qc[j];
                o_re[((size_t)n * T + t) * dv + x] = creal(acc);
                o_im[((size_t)n * T + t) * dv + x] = cimag(acc);
            }
        }
        if (S_T)
            for (int j = 0; j < m; ++j)
                for (int x = 0; x < dv; ++x) {
                    S_T[((size_t)n * 2 * m + 2 * j) * dv + x] = creal(S[(size_t)j * dv + x]);
                    S_T[((size_t)n * 2 * m + 2 * j + 1) * dv + x] = cimag(S[(size_t)j * dv + x]);
                }
        free(S); free(c); free(kc); free(qc);
    }
    return failed ? -1 : 0;
}
