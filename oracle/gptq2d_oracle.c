/* Plain-C restatement of the sequential sweeps of two-sided adaptive rounding.
 *
 * TEST INFRASTRUCTURE ONLY: built into liboracle_gptq2d.so and called from the
 * test-suite, the smoke check and the benchmark's CPU-baseline leg.  It shares
 * nothing with the CUDA path.  Single-threaded, fp64, row-major arrays with
 * leading dimension = number of columns, 0-based indices.
 *
 * Each routine follows the paper's steps in the paper's order:
 *   oracle_vec_sweep   Algorithm 1 on vec(X) (column-major) with the feedback
 *                      coefficient F[(i,j),(i',j')] = L[i][i'] * U[j'][j] of Eq. 10
 *                      formed on the fly -- the quartic definition.
 *   oracle_alg3        Algorithm 3 (GPTQ-2D) literally, anti-diagonal by anti-diagonal.
 *   oracle_nested      Algorithm 5 (nested, column-major).
 * Rounding is nearbyint in the default rounding mode (ties to even).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* Algorithm 1 over coordinates k_begin <= k < k_end of vec(X), k = j*m + i.
 * Y (m x n) is the running corrected matrix: the caller initialises it to X before
 * the first call; a later call continues where the previous one stopped. */
void oracle_vec_sweep(int m, int n, double *Y, const double *L, const double *U,
                      int64_t *Z, double *E, int64_t k_begin, int64_t k_end)
{
    for (int64_t k = k_begin; k < k_end; ++k) {
        int jp = (int)(k / m), ip = (int)(k % m);
        double y = Y[(size_t)ip * n + jp];
        double z = nearbyint(y);
        double e = z - y;
        Z[(size_t)ip * n + jp] = (int64_t)z;
        E[(size_t)ip * n + jp] = e;
        /* y_{k:} += F_{k:,k} e : every coordinate (i,j) with vec index >= k.  The
         * coefficient L[i][ip]*U[jp][j] vanishes for i < ip (L lower) -- it is
         * still multiplied out, as the one-dimensional sweep does not know. */
        for (int j = jp; j < n; ++j) {
            double u = U[(size_t)jp * n + j] * e;
            int i0 = (j == jp) ? ip : 0;
            for (int i = i0; i < m; ++i)
                Y[(size_t)i * n + j] += L[(size_t)i * m + ip] * u;
        }
    }
}

/* Algorithm 3, stages s_begin <= s < s_end (s = i + j, 0-based).  Y and C carry the
 * state: caller sets Y = X and C = 0 before stage 0. */
void oracle_alg3(int m, int n, double *Y, double *C, const double *L, const double *U,
                 int64_t *Z, double *E, int s_begin, int s_end)
{
    for (int s = s_begin; s < s_end; ++s) {
        int lo = s - n + 1 > 0 ? s - n + 1 : 0;
        int hi = s < m - 1 ? s : m - 1;
        for (int i = lo; i <= hi; ++i) {
            int j = s - i;
            double y = Y[(size_t)i * n + j];
            double z = nearbyint(y);
            double e = z - y;
            Z[(size_t)i * n + j] = (int64_t)z;
            E[(size_t)i * n + j] = e;
            C[(size_t)i * n + j] += e;                       /* L[i][i] = 1 */
            for (int r = i + 1; r < m; ++r) {
                double mm = L[(size_t)r * m + i] * e;
                C[(size_t)r * n + j] += mm;                  /* fold      */
                Y[(size_t)r * n + j] += mm;                  /* push down */
            }
        }
        for (int i = lo; i <= hi; ++i) {
            int j = s - i;
            double c = C[(size_t)i * n + j];
            for (int q = j + 1; q < n; ++q)
                Y[(size_t)i * n + q] += c * U[(size_t)j * n + q];   /* push right */
        }
    }
}

/* Algorithm 5.  Y is initialised to X by the caller and is overwritten. */
void oracle_nested(int m, int n, double *Y, const double *L, const double *U,
                   int64_t *Z, double *E)
{
    double *y = (double *)malloc(sizeof(double) * (size_t)m);
    for (int j = 0; j < n; ++j) {
        for (int i = 0; i < m; ++i) y[i] = Y[(size_t)i * n + j];
        for (int i = 0; i < m; ++i) {
            double z = nearbyint(y[i]);
            double e = z - y[i];
            Z[(size_t)i * n + j] = (int64_t)z;
            E[(size_t)i * n + j] = e;
            for (int r = i; r < m; ++r) y[r] += L[(size_t)r * m + i] * e;
        }
        for (int i = 0; i < m; ++i) {
            double d = y[i] - Y[(size_t)i * n + j];
            for (int q = j; q < n; ++q)
                Y[(size_t)i * n + q] += d * U[(size_t)j * n + q];
        }
    }
    free(y);
}
