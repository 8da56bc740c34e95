/*
 * ROCKET transform oracle: a plain, slow CPU statement of what the transform computes.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing on the product path may call, link or import this
 * file; it exists so that tests and the benchmark's CPU-baseline leg have an independent
 * result to compare the CUDA path with.  It shares no code with the CUDA path.
 *
 * Everything is the definition written out, in double precision on the fp32 inputs
 * promoted to double, with no blocking, fusion or reordering:
 *
 *   convolution   Section 3, step (1), with the kernel parameters of Section 3.1:
 *                 z_i = b + sum_q sum_j W[q][j] * xpad[S[q]][i - p + j*d],  0 <= i < n,
 *                 n = L + 2p - (len-1)d, xpad = x inside [0, L) and 0 outside.
 *   PPV           Eq. 1-2:  (1/n) * #{ i : z_i > 0 }       (strict inequality)
 *   max           Section 3, step (2): max_i z_i (second pooled feature of ROCKET)
 *   softPPV       Eq. 3-4:  (1/n) * sum_i 1 / (1 + exp(-(lambda*z_i + shift)));
 *                 Eq. 3 as printed has shift = +3, the prose describes shift = -3;
 *                 the shift is therefore an argument.
 *   backward      chain rule through Eq. 3-4 and the convolution (the paper states the
 *                 capability only):  gz_i = gP*(lambda/n)*h_i*(1-h_i) + gM*[i == argmax],
 *                 db = sum_n sum_i gz_i,  dW[q][j] = sum_n sum_i gz_i * xpad[S[q]][i-p+j*d].
 *
 * Parity pins (tests/test_oracle_*.py): numpy.correlate on zero-stuffed kernels, moving
 * sums, constant-input closed forms, impulse response, scaling laws, sigma(shift) at
 * lambda = 0, soft -> hard as lambda grows, brute force in pure Python, central finite
 * differences for the backward pass.  No function here is parity-unpinned.
 *
 * Parallelism: OpenMP over (example, kernel) pairs in the forward pass and over kernels in
 * the backward pass; each output element is still computed by one thread in program order.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>

#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int K, C, L;
    const int32_t *length, *dilation, *padding, *num_channels;
    const int32_t *channel_idx; /* ragged, sum m            */
    const float *weights;       /* ragged, sum m*len, [q][j] */
    const float *bias;
    const int64_t *channel_offset; /* [K+1] prefix sums of m     */
    const int64_t *weight_offset;  /* [K+1] prefix sums of m*len */
} oracle_params;

int rocket_oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void rocket_oracle_set_threads(int t) {
#ifdef _OPENMP
    if (t > 0) omp_set_num_threads(t);
#else
    (void)t;
#endif
}

static double xpad(const float *x, int L, int64_t t) { return (t >= 0 && t < L) ? (double)x[t] : 0.0; }

/* One conv output z_i of kernel k on example Xn[C][L] (Section 3 step (1), Section 3.1). */
static double conv_at(const oracle_params *P, int k, const float *Xn, int64_t i) {
    const int len = P->length[k], d = P->dilation[k], p = P->padding[k], m = P->num_channels[k];
    const int32_t *S = P->channel_idx + P->channel_offset[k];
    const float *W = P->weights + P->weight_offset[k];
    double z = (double)P->bias[k];
    for (int q = 0; q < m; ++q) {
        const float *x = Xn + (int64_t)S[q] * P->L;
        for (int j = 0; j < len; ++j) z += (double)W[q * len + j] * xpad(x, P->L, i - p + (int64_t)j * d);
    }
    return z;
}

static int64_t out_len(const oracle_params *P, int k) {
    return (int64_t)P->L + 2 * (int64_t)P->padding[k] - ((int64_t)P->length[k] - 1) * P->dilation[k];
}

/* z[0..n) of kernel k on example n; returns n.  z may be NULL to query the length. */
int64_t rocket_oracle_conv(const oracle_params *P, const float *X, int n, int k, double *z) {
    const int64_t nout = out_len(P, k);
    if (z) {
        const float *Xn = X + (int64_t)n * P->C * P->L;
        for (int64_t i = 0; i < nout; ++i) z[i] = conv_at(P, k, Xn, i);
    }
    return nout;
}

/*
 * Pooled features for a list of (example, kernel) pairs.  All outputs have one entry per
 * pair; any output pointer may be NULL.
 *   ppv     Eq. 1-2                        maxv    max_i z_i
 *   soft    Eq. 3-4 with (lambda, shift)   argmax  lowest index attaining the max
 *   pos_eps #{ i : z_i >  amb_eps }        amb     #{ i : |z_i| <= amb_eps }
 *   gap     max minus the second-largest value (0 when n == 1)
 */
void rocket_oracle_forward_pairs(const oracle_params *P, const float *X, int64_t npairs,
                                 const int32_t *pair_n, const int32_t *pair_k, double lambda, double shift,
                                 double amb_eps, double *ppv, double *maxv, double *soft, int32_t *argmax,
                                 int64_t *pos_eps, int64_t *amb, double *gap) {
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t e = 0; e < npairs; ++e) {
        const int n = pair_n[e], k = pair_k[e];
        const float *Xn = X + (int64_t)n * P->C * P->L;
        const int64_t nout = out_len(P, k);
        int64_t cnt = 0, cnt_eps = 0, cnt_amb = 0, arg = 0;
        double best = -INFINITY, second = -INFINITY, hsum = 0.0;
        for (int64_t i = 0; i < nout; ++i) {
            const double z = conv_at(P, k, Xn, i);
            if (z > 0.0) ++cnt;                                    /* Eq. 1: H(z) = 1 iff z > 0 */
            if (z > amb_eps) ++cnt_eps;
            if (fabs(z) <= amb_eps) ++cnt_amb;
            if (z > best) { second = best; best = z; arg = i; }
            else if (z > second) second = z;
            hsum += 1.0 / (1.0 + exp(-(lambda * z + shift)));      /* Eq. 3 */
        }
        if (ppv) ppv[e] = (double)cnt / (double)nout;              /* Eq. 2 */
        if (maxv) maxv[e] = best;
        if (soft) soft[e] = hsum / (double)nout;                   /* Eq. 4 */
        if (argmax) argmax[e] = (int32_t)arg;
        if (pos_eps) pos_eps[e] = cnt_eps;
        if (amb) amb[e] = cnt_amb;
        if (gap) gap[e] = (nout > 1) ? best - second : 0.0;
    }
}

/*
 * Backward of L = sum_{n,k} gP[n,k]*softPPV[n,k] + gM[n,k]*MAX[n,k] w.r.t. weights and biases.
 * g is [N][2K] interleaved (gP, gM); argmax is [N][K]; examples listed in ex[0..nex) are summed.
 * Kernels ks[0..nk) are processed; dW/db are written (not accumulated) for those kernels only,
 * dW in the ragged layout of the weights, db indexed by kernel.
 */
void rocket_oracle_backward(const oracle_params *P, const float *X, int nex, const int32_t *ex, int nk,
                            const int32_t *ks, double lambda, double shift, const float *g,
                            const int32_t *argmax, double *dW, double *db) {
#pragma omp parallel for schedule(dynamic, 1)
    for (int kk = 0; kk < nk; ++kk) {
        const int k = ks[kk];
        const int len = P->length[k], d = P->dilation[k], p = P->padding[k], m = P->num_channels[k];
        const int32_t *S = P->channel_idx + P->channel_offset[k];
        double *dWk = dW + P->weight_offset[k];
        const int64_t nout = out_len(P, k);
        for (int t = 0; t < m * len; ++t) dWk[t] = 0.0;
        db[k] = 0.0;
        for (int e = 0; e < nex; ++e) {
            const int n = ex[e];
            const float *Xn = X + (int64_t)n * P->C * P->L;
            const double gP = (double)g[((int64_t)n * P->K + k) * 2];
            const double gM = (double)g[((int64_t)n * P->K + k) * 2 + 1];
            const int64_t A = argmax[(int64_t)n * P->K + k];
            for (int64_t i = 0; i < nout; ++i) {
                const double z = conv_at(P, k, Xn, i);
                const double h = 1.0 / (1.0 + exp(-(lambda * z + shift)));
                double gz = gP * (lambda / (double)nout) * h * (1.0 - h);
                if (i == A) gz += gM;
                db[k] += gz;
                for (int q = 0; q < m; ++q) {
                    const float *x = Xn + (int64_t)S[q] * P->L;
                    for (int j = 0; j < len; ++j) dWk[q * len + j] += gz * xpad(x, P->L, i - p + (int64_t)j * d);
                }
            }
        }
    }
}
