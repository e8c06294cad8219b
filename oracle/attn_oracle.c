/*
 * fp64 CPU oracle for one decode step of attention over a gathered KV cache.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference that the
 * CUDA library is checked against; it shares no code with that library and the
 * library never calls it.  Only tests, the smoke check and the CPU-baseline leg
 * of the benchmark load it.
 *
 * What it computes (the decode self-attention whose operation count the paper
 * gives as 4*BS*ctx*h1 in its T_compute^d formula, Section IV-C "Decode Stage
 * Processing Time": 2*ctx*h1 for q.K^T and 2*ctx*h1 for p.V per sequence):
 *
 *   for every sequence s (n_s >= 1 tokens) and query head h (KV head g = h / (Hq/Hkv)):
 *     score_i = (sum_j q[s][h][j] * K[s][i][g][j]) / sqrt(d)        i = 0 .. n_s-1
 *     m       = max_i score_i
 *     w_i     = exp(score_i - m)
 *     Z       = sum_i w_i
 *     out[s][h][j] = (sum_i w_i * V[s][i][g][j]) / Z
 *
 * K and V arrive already gathered in logical token order (the caller gathers
 * them from its own record of what was appended), converted exactly to fp64.
 * There is no blocking, no splitting and no reordering: one pass per step above,
 * in index order.  The OpenMP pragma only distributes independent (s, h) pairs.
 *
 * Pinned by tests/test_oracle_pins.py (brute force without max subtraction,
 * context-length-1, row sums, closed forms, invariances, library softmax).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/*
 * q       [n_seqs][Hq][d]
 * K, V    rows of [Hkv][d]; sequence s owns rows row_off[s] .. row_off[s]+lens[s]-1
 * out     [n_seqs][Hq][d]
 * weights NULL, or for sequence s and head h the n_s normalised weights w_i/Z at
 *         weights[row_off[s]*Hq + h*lens[s] + i]
 * n_threads <= 0 means the OpenMP default.
 * Returns 0, or -1 on a bad argument (a length < 1, Hq not a multiple of Hkv),
 * or -2 when a scratch allocation fails.
 */
int oracle_attn_decode(const double *q, const double *K, const double *V,
                       const int64_t *row_off, const int32_t *lens,
                       int n_seqs, int Hq, int Hkv, int d,
                       double *out, double *weights, int n_threads)
{
    if (n_seqs < 0 || Hq < 1 || Hkv < 1 || d < 1 || Hq % Hkv != 0) return -1;
    for (int s = 0; s < n_seqs; ++s)
        if (lens[s] < 1) return -1;
    const int G = Hq / Hkv;
    const double inv_sqrt_d = 1.0 / sqrt((double)d);
    int failed = 0;
    /* thread count for this call only (a global omp_set_num_threads would outlast it) */
    int team = 1;
#ifdef _OPENMP
    team = n_threads > 0 ? n_threads : omp_get_max_threads();
#else
    (void)n_threads;
    (void)team;
#endif
#pragma omp parallel for schedule(dynamic, 1) num_threads(team)
    for (long sh = 0; sh < (long)n_seqs * Hq; ++sh) {
        const int s = (int)(sh / Hq);
        const int h = (int)(sh % Hq);
        const int g = h / G;
        const int n = lens[s];
        const double *qv = q + ((size_t)s * Hq + h) * d;
        double *w = (double *)malloc((size_t)n * sizeof(double));
        if (!w) {
#pragma omp atomic write
            failed = 1;
            continue;
        }
        /* scores */
        for (int i = 0; i < n; ++i) {
            const double *k = K + ((size_t)(row_off[s] + i) * Hkv + g) * d;
            double acc = 0.0;
            for (int j = 0; j < d; ++j) acc += qv[j] * k[j];
            w[i] = acc * inv_sqrt_d;
        }
        /* softmax with the maximum subtracted */
        double m = w[0];
        for (int i = 1; i < n; ++i)
            if (w[i] > m) m = w[i];
        double Z = 0.0;
        for (int i = 0; i < n; ++i) {
            w[i] = exp(w[i] - m);
            Z += w[i];
        }
        /* weighted sum of V */
        double *o = out + ((size_t)s * Hq + h) * d;
        for (int j = 0; j < d; ++j) o[j] = 0.0;
        for (int i = 0; i < n; ++i) {
            const double *v = V + ((size_t)(row_off[s] + i) * Hkv + g) * d;
            for (int j = 0; j < d; ++j) o[j] += w[i] * v[j];
        }
        for (int j = 0; j < d; ++j) o[j] /= Z;
        if (weights) {
            double *wo = weights + (size_t)row_off[s] * Hq + (size_t)h * n;
            for (int i = 0; i < n; ++i) wo[i] = w[i] / Z;
        }
        free(w);
    }
    return failed ? -2 : 0;
}

/* Threads the OpenMP runtime would use for the loop above (1 without OpenMP). */
int oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
