/*
 * ORACLE — TEST INFRASTRUCTURE ONLY.  Not part of the product path.
 *
 * Plain fp64 one-sided (Hestenes) Jacobi SVD of a P x d KV page (P <= d).
 *
 * The paper's page factor format (Eq. 2) is the rank-r truncated SVD of the
 * page, X ~= L R with L = U_r (P x r, orthonormal columns) and
 * R = Sigma_r W_r^T (r x d).  The paper states (Section 3.3, paragraph after
 * Eq. 3) that its Gram-matrix route reaches exactly these factors, so the
 * oracle computes the plain definition instead, by a route that deliberately
 * differs from the GPU's Gram + two-sided Jacobi:
 *
 *   keep X = U * Y with U orthogonal (P x P); rotate pairs of rows of Y until
 *   all rows are mutually orthogonal.  Then the row norms of Y are the singular
 *   values, the matching columns of U are the left singular vectors, and the
 *   rows of Y are sigma_i * w_i^T.
 *
 * No blocking, no reordering, no early truncation.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>

/*
 * X      : P x d row-major input page (not modified)
 * U      : P x P row-major output, orthogonal
 * Y      : P x d row-major output, rows mutually orthogonal, X = U * Y
 * sigma  : P singular values in the row order of Y (NOT sorted)
 * order  : P indices sorting sigma descending, ties by lower index
 * returns the number of sweeps used, or -1 if max_sweeps was reached
 * while rotations were still being applied.
 */
int pkvo_page_svd(const double *X, int P, int d, double *U, double *Y,
                  double *sigma, int *order, int max_sweeps, double eps)
{
    memcpy(Y, X, sizeof(double) * (size_t)P * (size_t)d);
    memset(U, 0, sizeof(double) * (size_t)P * (size_t)P);
    for (int i = 0; i < P; ++i) U[i * P + i] = 1.0;

    int sweeps = 0, converged = 0;
    while (sweeps < max_sweeps) {
        int rotations = 0;
        for (int i = 0; i < P - 1; ++i) {
            for (int j = i + 1; j < P; ++j) {
                double *yi = Y + (size_t)i * d, *yj = Y + (size_t)j * d;
                double a = 0.0, b = 0.0, c = 0.0;
                for (int k = 0; k < d; ++k) {
                    a += yi[k] * yi[k];
                    b += yj[k] * yj[k];
                    c += yi[k] * yj[k];
                }
                if (fabs(c) <= eps * sqrt(a * b)) continue;
                ++rotations;
                /* tan of the rotation angle that zeroes y_i . y_j: the smaller
                 * root of t^2 + 2*zeta*t - 1 = 0 */
                double zeta = (b - a) / (2.0 * c);
                double t = (zeta >= 0.0 ? 1.0 : -1.0) / (fabs(zeta) + sqrt(1.0 + zeta * zeta));
                double cs = 1.0 / sqrt(1.0 + t * t), sn = cs * t;
                for (int k = 0; k < d; ++k) {
                    double p = yi[k], q = yj[k];
                    yi[k] = cs * p - sn * q;
                    yj[k] = sn * p + cs * q;
                }
                for (int k = 0; k < P; ++k) {
                    double p = U[k * P + i], q = U[k * P + j];
                    U[k * P + i] = cs * p - sn * q;
                    U[k * P + j] = sn * p + cs * q;
                }
            }
        }
        ++sweeps;
        if (rotations == 0) { converged = 1; break; }
    }

    for (int i = 0; i < P; ++i) {
        double s = 0.0;
        const double *yi = Y + (size_t)i * d;
        for (int k = 0; k < d; ++k) s += yi[k] * yi[k];
        sigma[i] = sqrt(s);
        order[i] = i;
    }
    /* stable insertion sort: descending sigma, ties keep the lower index first */
    for (int i = 1; i < P; ++i) {
        int oi = order[i];
        int j = i - 1;
        while (j >= 0 && sigma[order[j]] < sigma[oi]) { order[j + 1] = order[j]; --j; }
        order[j + 1] = oi;
    }
    return converged ? sweeps : -1;
}

/*
 * Batched form: n_pages independent pages stored back to back.  Pages are
 * independent (the paper's point), so the loop is an OpenMP parallel-for; each
 * page runs exactly the routine above.  sweeps[p] receives its return value.
 */
void pkvo_batch_page_svd(const double *X, long n_pages, int P, int d, double *U,
                         double *Y, double *sigma, int *order, int *sweeps,
                         int max_sweeps, double eps)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (long p = 0; p < n_pages; ++p) {
        sweeps[p] = pkvo_page_svd(X + (size_t)p * P * d, P, d, U + (size_t)p * P * P,
                                  Y + (size_t)p * P * d, sigma + (size_t)p * P,
                                  order + (size_t)p * P, max_sweeps, eps);
    }
}

int pkvo_max_threads(void);
#ifdef _OPENMP
#include <omp.h>
int pkvo_max_threads(void) { return omp_get_max_threads(); }
#else
int pkvo_max_threads(void) { return 1; }
#endif
