/* CPU oracle for the HARP apply path, plain C, fp64 -- TEST INFRASTRUCTURE.
 *
 * Only the tests, the smoke check and the benchmark's CPU baseline load this
 * library.  It shares no code with the CUDA library.
 *
 * Scalar loops over (row, stage, block), written from the index form of a stride
 * stage (Lemma 1: X[alpha, r, beta] = x[alpha*b*s + r*s + beta]) and the stage
 * order of Algorithm 1 / Eq. 8 (stage 0, stride 1, first):
 *
 *   forward:   u_i = sign_i * x_i;  v_i = u_{perm[i]};
 *              for t = 0..m-1, for every (alpha, beta), c = alpha*s_t + beta:
 *                 z[base + j*s_t] = sum_i v[base + i*s_t] * K_t[c][i][j],
 *                 base = alpha*b_t*s_t + beta
 *   transpose: stages t = m-1..0 with K_t[c][j][i], then w[perm[i]] = v_i,
 *              then x_i = sign_i * w_i.
 *
 * blocks: one flat fp64 array, stage after stage, stage t = [d/b_t][b_t][b_t].
 * Rows are independent; OpenMP spreads rows over threads and changes no
 * arithmetic.  Pinned by tests against the numpy oracle, which is itself pinned
 * against dense constructions.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int harp_oracle_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

static void stage_row(double *v, double *z, int64_t d, int64_t b, int64_t s,
                      const double *K, int transposed) {
    int64_t g = d / (b * s);
    for (int64_t alpha = 0; alpha < g; ++alpha) {
        for (int64_t beta = 0; beta < s; ++beta) {
            int64_t c = alpha * s + beta;
            int64_t base = alpha * b * s + beta;
            const double *Kc = K + c * b * b;
            for (int64_t j = 0; j < b; ++j) {
                double acc = 0.0;
                for (int64_t i = 0; i < b; ++i) {
                    double k = transposed ? Kc[j * b + i] : Kc[i * b + j];
                    acc += v[base + i * s] * k;
                }
                z[base + j * s] = acc;
            }
        }
    }
    memcpy(v, z, (size_t)d * sizeof(double));
}

/* x: [n_rows][d] fp64, in place.  perm / signs may be NULL.  Returns 0, or -1 on
 * allocation failure. */
int harp_oracle_apply(int64_t d, int32_t m, const int32_t *radices, const int64_t *perm,
                      const double *signs, const double *blocks, double *x, int64_t n_rows,
                      int transposed) {
    int64_t *stride = (int64_t *)malloc(sizeof(int64_t) * (size_t)m);
    int64_t *offset = (int64_t *)malloc(sizeof(int64_t) * (size_t)m);
    if (!stride || !offset) { free(stride); free(offset); return -1; }
    int64_t s = 1, off = 0;
    for (int32_t t = 0; t < m; ++t) {
        stride[t] = s;
        offset[t] = off;
        s *= radices[t];
        off += d * radices[t];            /* (d/b) * b * b */
    }
    int fail = 0;
#pragma omp parallel
    {
        double *v = (double *)malloc(sizeof(double) * (size_t)d);
        double *z = (double *)malloc(sizeof(double) * (size_t)d);
        if (!v || !z) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp barrier
        if (!fail) {
#pragma omp for schedule(static)
            for (int64_t r = 0; r < n_rows; ++r) {
                double *row = x + r * d;
                if (!transposed) {
                    for (int64_t i = 0; i < d; ++i) {
                        int64_t src = perm ? perm[i] : i;
                        v[i] = (signs ? signs[src] : 1.0) * row[src];
                    }
                    for (int32_t t = 0; t < m; ++t)
                        stage_row(v, z, d, radices[t], stride[t], blocks + offset[t], 0);
                    memcpy(row, v, (size_t)d * sizeof(double));
                } else {
                    memcpy(v, row, (size_t)d * sizeof(double));
                    for (int32_t t = m - 1; t >= 0; --t)
                        stage_row(v, z, d, radices[t], stride[t], blocks + offset[t], 1);
                    for (int64_t i = 0; i < d; ++i) {
                        int64_t dst = perm ? perm[i] : i;
                        row[dst] = (signs ? signs[dst] : 1.0) * v[i];
                    }
                }
            }
        }
        free(v);
        free(z);
    }
    free(stride);
    free(offset);
    return fail ? -1 : 0;
}
