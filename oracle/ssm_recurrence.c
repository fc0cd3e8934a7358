/*
 * TEST INFRASTRUCTURE ONLY -- fp64 CPU oracle, never part of the product path.
 *
 * Sequential per-token Mamba-2 selective state-space recurrence, exactly as the
 * paper states it (Section 3.1 "State-Space (Mamba) Layers" and appendix
 * "State-Space Recurrence", the state-update and output equations):
 *
 *     S_t = Abar_t * S_{t-1} + x_t (Delta_t b_t)^T ,   y_t = S_t c_t ,
 *
 * with S_t in R^{p x n} per head, Abar_t a scalar per head in (0,1), and b_t, c_t
 * shared by the heads of one group.  The paper writes Abar_t = exp(-Delta_t A)
 * with A > 0; this file takes the stored parameter with its sign, A_h < 0, and
 * forms Abar_t = exp(Delta_t * A_h), the same number.
 *
 * No chunking, no blocking, no reordering: one token after the other.  The only
 * parallelism is OpenMP over heads, which are independent problems.
 *
 * Layouts (row-major, fp64): x [T,H,p], dt [T,H], A [H], B,C [T,G,n],
 * D [H] or NULL (optional skip term y_t += D_h x_t, absent from the paper's
 * recurrence and off by default), S0 [H,p,n] or NULL (zero initial state),
 * y [T,H,p], Sfinal [H,p,n] or NULL.  Head h belongs to group h / (H/G).
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>

int ssm_recurrence_f64(long T, long H, long p, long n, long G,
                       const double *x, const double *dt, const double *A,
                       const double *B, const double *C, const double *D,
                       const double *S0, double *y, double *Sfinal)
{
    if (T < 0 || H <= 0 || p <= 0 || n <= 0 || G <= 0 || H % G != 0) return -1;
    const long heads_per_group = H / G;
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (long h = 0; h < H; ++h) {
        const long g = h / heads_per_group;
        double *S = (double *)malloc(sizeof(double) * (size_t)(p * n));
        if (!S) { failed = 1; continue; }
        if (S0) memcpy(S, S0 + h * p * n, sizeof(double) * (size_t)(p * n));
        else    memset(S, 0, sizeof(double) * (size_t)(p * n));
        for (long t = 0; t < T; ++t) {
            const double delta = dt[t * H + h];
            const double abar = exp(delta * A[h]);          /* decay in (0,1) */
            const double *b = B + (t * G + g) * n;
            const double *c = C + (t * G + g) * n;
            const double *xt = x + (t * H + h) * p;
            double *yt = y + (t * H + h) * p;
            for (long i = 0; i < p; ++i) {
                double *Si = S + i * n;
                const double xi = xt[i];
                double acc = 0.0;
                for (long k = 0; k < n; ++k) {
                    Si[k] = abar * Si[k] + xi * (delta * b[k]);  /* state update */
                    acc += Si[k] * c[k];                         /* y_t = S_t c_t */
                }
                yt[i] = acc + (D ? D[h] * xi : 0.0);
            }
        }
        if (Sfinal) memcpy(Sfinal + h * p * n, S, sizeof(double) * (size_t)(p * n));
        free(S);
    }
    return failed ? -2 : 0;
}
