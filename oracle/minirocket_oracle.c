/*
 * MINIROCKET oracle: a plain, slow CPU statement of the transform the paper names as the extension of its
 * GPU implementation (Section 2, paragraph on MINIROCKET; Section 6, last sentence).
 *
 * TEST INFRASTRUCTURE ONLY, like rocket_oracle.c: nothing on the product path may call, link or import this
 * file, and it shares no code with the CUDA path.
 *
 * The paper describes MINIROCKET in words only: two-valued ("binary") kernels from a predetermined set, so
 * that the convolution needs additions only; biases sampled from the input data; PPV as the only pooled
 * feature.  What is computed here, in double precision on the fp32 inputs promoted to double:
 *
 *   convolution   z_i = sum_{c in S} sum_{j<9} w_j * xpad[c][i + (j - 4) d],  w_j = 2 on the kernel's three
 *                 taps and -1 on the other six, xpad = x inside [0, L) and 0 outside; outputs i in [0, L)
 *                 for a padded combination, [4d, L - 4d) otherwise
 *   bias          of feature f: the quantile q_f of the outputs of one chosen training example, with linear
 *                 interpolation between the two nearest order statistics (position q (n - 1) of the sorted
 *                 outputs)
 *   feature       PPV against the bias (Eq. 1-2 with z - bias in place of z): #{ i : z_i > bias_f } / n
 *
 * Parity pins (tests/test_oracle_minirocket.py): every feature equals the PPV that rocket_oracle.c gives for
 * the ROCKET kernel with the same weights, dilation, padding and bias -b; the quantile against numpy's and
 * hand-worked values; constant inputs (all outputs zero); brute force in pure Python.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>

typedef struct {
    int C, L, F, n_combos;
    const int32_t *taps;           /* [84][3] */
    const int32_t *dilation, *kernel_index, *padded, *num_channels; /* [n_combos] */
    const int32_t *channel_idx;    /* ragged */
    const int64_t *channel_offset; /* [n_combos + 1] */
    const int32_t *feature_offset; /* [n_combos + 1] */
} mini_params;

static double xpad(const float *x, int L, int64_t t) { return (t >= 0 && t < L) ? (double)x[t] : 0.0; }

static double weight(const mini_params *P, int kernel, int j) {
    const int32_t *t = P->taps + 3 * kernel;
    return (j == t[0] || j == t[1] || j == t[2]) ? 2.0 : -1.0;
}

/* One conv output of combination c on example Xn[C][L]. */
static double conv_at(const mini_params *P, int c, const float *Xn, int64_t i) {
    const int d = P->dilation[c], kernel = P->kernel_index[c];
    const int32_t *S = P->channel_idx + P->channel_offset[c];
    double z = 0.0;
    for (int q = 0; q < P->num_channels[c]; ++q) {
        const float *x = Xn + (int64_t)S[q] * P->L;
        for (int j = 0; j < 9; ++j) z += weight(P, kernel, j) * xpad(x, P->L, i + (int64_t)(j - 4) * d);
    }
    return z;
}

static void out_range(const mini_params *P, int c, int64_t *first, int64_t *last) {
    const int64_t d = P->dilation[c];
    *first = P->padded[c] ? 0 : 4 * d;
    *last = P->padded[c] ? P->L : P->L - 4 * d;
}

/* z over the output range of combination c on example n; returns the number of outputs (z may be NULL). */
int64_t minirocket_oracle_conv(const mini_params *P, const float *X, int n, int c, double *z) {
    int64_t first, last;
    out_range(P, c, &first, &last);
    if (z) {
        const float *Xn = X + (int64_t)n * P->C * P->L;
        for (int64_t i = first; i < last; ++i) z[i - first] = conv_at(P, c, Xn, i);
    }
    return last - first;
}

static int cmp_double(const void *a, const void *b) {
    const double x = *(const double *)a, y = *(const double *)b;
    return (x > y) - (x < y);
}

/* Biases: feature f of combination c reads the quantile q[f] of the outputs of example example[c]. */
void minirocket_oracle_fit(const mini_params *P, const float *X, const int32_t *example, const double *q, double *bias) {
#pragma omp parallel for schedule(dynamic, 1)
    for (int c = 0; c < P->n_combos; ++c) {
        const int64_t n = minirocket_oracle_conv(P, X, example[c], c, NULL);
        double *z = (double *)malloc((size_t)n * sizeof(double));
        minirocket_oracle_conv(P, X, example[c], c, z);
        qsort(z, (size_t)n, sizeof(double), cmp_double);
        for (int f = P->feature_offset[c]; f < P->feature_offset[c + 1]; ++f) {
            const double pos = q[f] * (double)(n - 1);
            const int64_t lo = (int64_t)floor(pos);
            const int64_t hi = lo + 1 < n ? lo + 1 : lo;
            bias[f] = z[lo] + (pos - (double)lo) * (z[hi] - z[lo]);
        }
        free(z);
    }
}

/* Features [N][F], plus per feature the counts above bias + eps and within eps of the bias (any may be NULL). */
void minirocket_oracle_transform(const mini_params *P, const float *X, int N, const double *bias, double eps,
                                 double *feat, int64_t *pos_eps, int64_t *amb) {
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int n = 0; n < N; ++n)
        for (int c = 0; c < P->n_combos; ++c) {
            const float *Xn = X + (int64_t)n * P->C * P->L;
            int64_t first, last;
            out_range(P, c, &first, &last);
            const int f0 = P->feature_offset[c], f1 = P->feature_offset[c + 1];
            for (int f = f0; f < f1; ++f) {
                const int64_t e = (int64_t)n * P->F + f;
                if (feat) feat[e] = 0.0;
                if (pos_eps) pos_eps[e] = 0;
                if (amb) amb[e] = 0;
            }
            for (int64_t i = first; i < last; ++i) {
                const double z = conv_at(P, c, Xn, i);
                for (int f = f0; f < f1; ++f) {
                    const int64_t e = (int64_t)n * P->F + f;
                    if (feat && z > bias[f]) feat[e] += 1.0;              /* Eq. 1 against the bias */
                    if (pos_eps && z > bias[f] + eps) ++pos_eps[e];
                    if (amb && fabs(z - bias[f]) <= eps) ++amb[e];
                }
            }
            if (feat)
                for (int f = f0; f < f1; ++f) feat[(int64_t)n * P->F + f] /= (double)(last - first);   /* Eq. 2 */
        }
}
