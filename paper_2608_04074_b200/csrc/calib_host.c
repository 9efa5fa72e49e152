/*
 * Host-side (offline) codebook training: Lloyd / k-means per coefficient group, float64.
 *
 * Follows Algorithm 3 ("Codebook training") and the calibration paragraph of App. B: one
 * codebook of K centroids per group of g transform coefficients, a fixed number of
 * iterations, empty clusters reseeded from the points that are currently served worst.
 * The paper does not fix every detail; this implementation takes:
 *   - assignment: exact Euclidean nearest centroid, the lowest index wins a tie;
 *   - update: centroid = float64 mean of its cell;
 *   - the m-th empty cluster (ascending index) is moved to the point with the m-th largest
 *     distance to its assigned centroid.
 * Calibration is not on the GPU hot path; it produces the tables the library loads.
 *
 * Groups are independent and run in parallel under OpenMP when available.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <float.h>

static void lloyd_one_group(const double* X, long n, int g, double* C, int k, int iters,
                            int32_t* assign, double* dist, double* distortion)
{
    double* sum = (double*)malloc(sizeof(double) * (size_t)k * g);
    long* cnt = (long*)malloc(sizeof(long) * (size_t)k);
    for (int it = 0; it < iters; ++it) {
        double total = 0.0;
        for (long j = 0; j < n; ++j) {
            const double* x = X + j * g;
            double best = DBL_MAX;
            int bi = 0;
            for (int c = 0; c < k; ++c) {
                const double* cc = C + (long)c * g;
                double s = 0.0;
                for (int i = 0; i < g; ++i) {
                    double e = x[i] - cc[i];
                    s += e * e;
                }
                if (s < best) { best = s; bi = c; }
            }
            assign[j] = bi;
            dist[j] = best;
            total += best;
        }
        if (distortion) distortion[it] = total;
        memset(sum, 0, sizeof(double) * (size_t)k * g);
        memset(cnt, 0, sizeof(long) * (size_t)k);
        for (long j = 0; j < n; ++j) {
            int c = assign[j];
            cnt[c]++;
            for (int i = 0; i < g; ++i) sum[(long)c * g + i] += X[j * g + i];
        }
        int n_empty = 0;
        for (int c = 0; c < k; ++c) {
            if (cnt[c] > 0) {
                for (int i = 0; i < g; ++i) C[(long)c * g + i] = sum[(long)c * g + i] / (double)cnt[c];
            } else {
                n_empty++;
            }
        }
        if (n_empty > 0) {
            /* m-th empty cluster takes the point with the m-th largest current distance */
            int m = 0;
            char* taken = (char*)calloc((size_t)n, 1);
            for (int c = 0; c < k && m < n_empty; ++c) {
                if (cnt[c] > 0) continue;
                long arg = -1;
                double worst = -1.0;
                for (long j = 0; j < n; ++j) {
                    if (!taken[j] && dist[j] > worst) { worst = dist[j]; arg = j; }
                }
                if (arg >= 0) {
                    taken[arg] = 1;
                    for (int i = 0; i < g; ++i) C[(long)c * g + i] = X[arg * g + i];
                }
                m++;
            }
            free(taken);
        }
    }
    free(sum);
    free(cnt);
}

/*
 * X: [n_groups][n][g] float64 training subvectors, C: [n_groups][k][g] float64 initial centroids,
 * overwritten with the trained codebooks.  distortion: [n_groups][iters] summed squared error
 * measured at the assignment step of each iteration (may be NULL).
 */
void novakv_calib_lloyd(const double* X, int n_groups, long n, int g, double* C, int k,
                        int iters, double* distortion)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int G = 0; G < n_groups; ++G) {
        int32_t* assign = (int32_t*)malloc(sizeof(int32_t) * (size_t)n);
        double* dist = (double*)malloc(sizeof(double) * (size_t)n);
        lloyd_one_group(X + (long)G * n * g, n, g, C + (long)G * k * g, k, iters, assign, dist,
                        distortion ? distortion + (long)G * iters : NULL);
        free(assign);
        free(dist);
    }
}
