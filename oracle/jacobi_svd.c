/*
 * TEST INFRASTRUCTURE -- CPU oracle, double precision.  Not part of the product path:
 * only tests, the smoke check and the CPU-baseline leg of the benchmark may call it.
 * Shares no code with the CUDA library.
 *
 * Thin singular value decomposition by the textbook one-sided (Hestenes) Jacobi method.
 * Spectral ATOMO (Section 5 of the paper) takes the atoms of a layer gradient X to be the
 * rank-one terms of  X = sum_{i<=r} sigma_i u_i v_i^T ; the paper does not name an SVD
 * routine, so the oracle uses the simplest one whose result is the SVD by definition:
 * plane rotations that make the r short-side vectors mutually orthogonal.
 *
 *   B  (r x L, row-major): the r vectors of length L = max(m, n)   (rows of G, or of G^T)
 *   Jt (r x r, row-major): identity at the start; every rotation of rows (p, q) of B is
 *                          repeated on rows (p, q) of Jt, so that  B_end = Jt * B_start.
 *   At convergence the rows of B are orthogonal: row i = sigma_i * (long-side vector i)^T,
 *   and row i of Jt is the short-side vector i.
 *
 * No blocking, no reordering beyond the row-cyclic sweep (p < q), no BLAS.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>

static void rotate_rows(double *x, double *y, long len, double c, double s)
{
    for (long k = 0; k < len; ++k) {
        double xp = x[k], xq = y[k];
        x[k] = c * xp - s * xq;
        y[k] = s * xp + c * xq;
    }
}

/*
 * G      : m x n, row-major, double (the fp32 gradient widened by the caller)
 * U      : m x r, row-major (column i = left singular vector i)
 * sigma  : r, descending
 * V      : n x r, row-major (column i = right singular vector i)
 * tol    : a pair is rotated when |<b_p,b_q>| > tol * ||b_p|| * ||b_q||
 * returns the number of sweeps used (the last one rotated nothing), or -1 if
 * max_sweeps sweeps did not reach that state, or -2 on allocation failure.
 */
int oracle_jacobi_svd(const double *G, int m, int n, double *U, double *sigma, double *V,
                      double tol, int max_sweeps)
{
    const int tall = m > n;           /* short side is the column count */
    const int r = tall ? n : m;
    const long L = tall ? m : n;
    double *B = (double *)malloc(sizeof(double) * (size_t)r * (size_t)L);
    double *Jt = (double *)calloc((size_t)r * (size_t)r, sizeof(double));
    double *nrm = (double *)malloc(sizeof(double) * (size_t)r);
    int *order = (int *)malloc(sizeof(int) * (size_t)r);
    if (!B || !Jt || !nrm || !order) { free(B); free(Jt); free(nrm); free(order); return -2; }

    if (!tall) {
        memcpy(B, G, sizeof(double) * (size_t)m * (size_t)n);
    } else {
        for (int i = 0; i < m; ++i)
            for (int j = 0; j < n; ++j)
                B[(long)j * L + i] = G[(long)i * n + j];
    }
    for (int i = 0; i < r; ++i) Jt[(long)i * r + i] = 1.0;

    int sweeps = -1;
    for (int sw = 1; sw <= max_sweeps; ++sw) {
        long rotations = 0;
        for (int p = 0; p < r - 1; ++p) {
            for (int q = p + 1; q < r; ++q) {
                double *bp = B + (long)p * L, *bq = B + (long)q * L;
                double alpha = 0.0, beta = 0.0, gamma = 0.0;
                for (long k = 0; k < L; ++k) {
                    alpha += bp[k] * bp[k];
                    beta += bq[k] * bq[k];
                    gamma += bp[k] * bq[k];
                }
                if (fabs(gamma) <= tol * sqrt(alpha * beta)) continue;
                double zeta = (beta - alpha) / (2.0 * gamma);
                double t = (zeta >= 0.0 ? 1.0 : -1.0) / (fabs(zeta) + sqrt(1.0 + zeta * zeta));
                double c = 1.0 / sqrt(1.0 + t * t);
                double s = c * t;
                rotate_rows(bp, bq, L, c, s);
                rotate_rows(Jt + (long)p * r, Jt + (long)q * r, r, c, s);
                ++rotations;
            }
        }
        if (rotations == 0) { sweeps = sw; break; }
    }

    for (int i = 0; i < r; ++i) {
        double a = 0.0;
        const double *bi = B + (long)i * L;
        for (long k = 0; k < L; ++k) a += bi[k] * bi[k];
        nrm[i] = sqrt(a);
        order[i] = i;
    }
    /* stable insertion sort, descending singular value, ties keep the lower index first */
    for (int i = 1; i < r; ++i) {
        int oi = order[i];
        int j = i - 1;
        while (j >= 0 && nrm[order[j]] < nrm[oi]) { order[j + 1] = order[j]; --j; }
        order[j + 1] = oi;
    }

    for (int k = 0; k < r; ++k) {
        const int i = order[k];
        const double sg = nrm[i];
        const double *bi = B + (long)i * L;
        const double *ji = Jt + (long)i * r;
        sigma[k] = sg;
        /* reporting convention: largest-magnitude component of the short-side vector > 0 */
        double big = 0.0;
        for (int a = 0; a < r; ++a) if (fabs(ji[a]) > fabs(big)) big = ji[a];
        const double sgn = big < 0.0 ? -1.0 : 1.0;
        double *shortv = tall ? V : U;     /* (short dim) x r */
        double *longv = tall ? U : V;      /* (long dim)  x r */
        for (int a = 0; a < r; ++a) shortv[(long)a * r + k] = sgn * ji[a];
        for (long a = 0; a < L; ++a) longv[a * r + k] = sg > 0.0 ? sgn * bi[a] / sg : 0.0;
    }
    free(B); free(Jt); free(nrm); free(order);
    return sweeps;
}
