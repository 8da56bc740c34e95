/*
 * Half-precision form of the ROCKET transform oracle (the paper's remark in Section 5 that FP16 compute could
 * speed the transform up): what the hard transform computes when the samples, the weights and the biases are
 * binary16 numbers and every multiply-add of the convolution rounds once to binary16.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing on the product path may call, link or import this file.  It shares no code
 * with the CUDA path.
 *
 *   inputs        X, W, b given as floats whose values are binary16 numbers (the caller rounds them, round to
 *                 nearest even; values that are not binary16 numbers are refused)
 *   convolution   Section 3, step (1), Section 3.1, in this order: z starts at b; the kernel's channels are taken
 *                 in the order of its channel list, inside a channel the taps j = 0 .. len - 1; every step is one
 *                 fused multiply-add z <- round16(z + W[q][j] * xpad[S[q]][i - p + j d]) (exact product and sum,
 *                 ONE rounding to the nearest binary16 number, ties to even, subnormals kept)
 *   PPV           Eq. 1-2 on those z: (1/n) #{ i : z_i > 0 }
 *   max           Section 3, step (2): max_i z_i (a binary16 number, returned exactly)
 *
 * The arithmetic is exact integer arithmetic: every finite binary16 number is an integer multiple of 2^-24 below
 * 2^16 in size, a product of two is a multiple of 2^-48 below 2^32, so product + addend fit 128-bit integers in
 * units of 2^-48; the rounding is done on that integer.
 *
 * Parity pins (tests/test_oracle_f16.py): integer-valued cases that never round (equal to the double-precision
 * oracle), hand-worked roundings (a tie, a fused step that an unfused one would get wrong), a brute force with
 * rational arithmetic and a table of all binary16 numbers, and the standard error bound against the
 * double-precision oracle.  No function here is parity-unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>

typedef struct {
    int K, C, L;
    const int32_t *length, *dilation, *padding, *num_channels;
    const int32_t *channel_idx;
    const float *weights;
    const float *bias;
    const int64_t *channel_offset;
    const int64_t *weight_offset;
} oracle_params;

/* v as a multiple of 2^-24; *ok is cleared when v is no finite binary16 number */
static int64_t units_of(float v, int *ok) {
    const double s = (double)v * 16777216.0;   /* exact: a power of two */
    const int64_t u = (int64_t)s;
    if ((double)u != s) { *ok = 0; return 0; }
    const int64_t a = u < 0 ? -u : u;
    if (a >= ((int64_t)65520 << 24)) { *ok = 0; return 0; }
    if (a != 0) {
        int h = 63 - __builtin_clzll((unsigned long long)a);   /* value = a 2^-24, leading bit 2^(h-24) */
        const int drop = h - 10 > 0 ? h - 10 : 0;                /* 11 significant bits */
        if (a & (((int64_t)1 << drop) - 1)) { *ok = 0; return 0; }
    }
    return u;
}

/* S in units of 2^-48 -> nearest binary16 number in units of 2^-24 (ties to even); *ok cleared on overflow */
static int64_t round16(__int128 S, int *ok) {
    const int neg = S < 0;
    unsigned __int128 a = neg ? (unsigned __int128)(-S) : (unsigned __int128)S;
    if (a == 0) return 0;
    int h = 0;
    { const uint64_t hi = (uint64_t)(a >> 64), lo = (uint64_t)a; h = hi ? 127 - __builtin_clzll(hi) : 63 - __builtin_clzll(lo); }
    int shift = h - 10;            /* keep 11 significant bits ...                          */
    if (shift < 24) shift = 24;    /* ... but never finer than the subnormal spacing 2^-24 */
    unsigned __int128 q = a >> shift;
    const unsigned __int128 rem = a & (((unsigned __int128)1 << shift) - 1), half = (unsigned __int128)1 << (shift - 1);
    if (rem > half || (rem == half && (q & 1))) ++q;
    const unsigned __int128 r = q << (shift - 24);   /* units of 2^-24 */
    if (r >= ((unsigned __int128)65520 << 24)) { *ok = 0; return 0; }
    return neg ? -(int64_t)r : (int64_t)r;
}

static int64_t out_len(const oracle_params *P, int k) {
    return (int64_t)P->L + 2 * (int64_t)P->padding[k] - ((int64_t)P->length[k] - 1) * P->dilation[k];
}

/*
 * Pooled features of the half-precision transform for a list of (example, kernel) pairs; one entry per pair.
 * count = #{ i : z_i > 0 }, ppv = count / n, maxv = max_i z_i, argmax = lowest index attaining it.  z_out, when
 * not NULL, receives the z of the FIRST pair only (n values, for the pins).  Returns 0, or 1 when an input is no
 * binary16 number or an intermediate result overflows binary16.
 */
int rocket_oracle_f16_forward_pairs(const oracle_params *P, const float *X, int64_t npairs, const int32_t *pair_n,
                                    const int32_t *pair_k, int64_t *count, double *ppv, double *maxv, int32_t *argmax,
                                    double *z_out) {
    int all_ok = 1;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t e = 0; e < npairs; ++e) {
        int ok = 1;
        const int n = pair_n[e], k = pair_k[e];
        const float *Xn = X + (int64_t)n * P->C * P->L;
        const int len = P->length[k], d = P->dilation[k], p = P->padding[k], m = P->num_channels[k];
        const int32_t *S = P->channel_idx + P->channel_offset[k];
        const float *W = P->weights + P->weight_offset[k];
        const int64_t nout = out_len(P, k);
        const int64_t b = units_of(P->bias[k], &ok);
        int64_t cnt = 0, arg = 0, best = INT64_MIN;
        for (int64_t i = 0; i < nout; ++i) {
            int64_t z = b;
            for (int q = 0; q < m; ++q) {
                const float *x = Xn + (int64_t)S[q] * P->L;
                for (int j = 0; j < len; ++j) {
                    const int64_t t = i - p + (int64_t)j * d;
                    const int64_t xv = (t >= 0 && t < P->L) ? units_of(x[t], &ok) : 0;
                    const int64_t wv = units_of(W[q * len + j], &ok);
                    z = round16((__int128)wv * (__int128)xv + ((__int128)z << 24), &ok);
                }
            }
            if (z > 0) ++cnt;
            if (z > best) { best = z; arg = i; }
            if (z_out && e == 0) z_out[i] = (double)z / 16777216.0;
        }
        if (count) count[e] = cnt;
        if (ppv) ppv[e] = (double)cnt / (double)nout;
        if (maxv) maxv[e] = (double)best / 16777216.0;
        if (argmax) argmax[e] = (int32_t)arg;
        if (!ok) {
#pragma omp atomic write
            all_ok = 0;
        }
    }
    return all_ok ? 0 : 1;
}
