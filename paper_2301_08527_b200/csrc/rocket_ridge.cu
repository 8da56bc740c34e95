// Ridge regressor on the pooled features (Section 3, step (3); Section 3.3): fit and predict on the
// device, so that features never have to leave it.
//
// Fit, with an intercept that is not penalised: centre the columns of F [N][P] and y, solve the dual
// system (Fc Fc^T + alpha I) a = yc (N x N, N examples << P features), w = Fc^T a,
// b = mean(y) - mean(F) . w.  The Gram matrix, its Cholesky factor and the two triangular solves are
// kept in double precision: the features are fp32 data, everything derived from them is not rounded
// to fp32 before w and b are stored.
#include <algorithm>
#include <cstdint>

#include "rocket_internal.h"

namespace rocket {
namespace {

constexpr int kRThreads = 256;

// mu[p] = mean over the N rows of F[.][p]; one thread per column, rows coalesced across the warp.
__global__ void __launch_bounds__(kRThreads)
ridge_colmean_kernel(const float* __restrict__ F, int N, int P, double* __restrict__ mu) {
    const int p = blockIdx.x * kRThreads + threadIdx.x;
    if (p >= P) return;
    double s = 0.0;
    for (int i = 0; i < N; ++i) s += (double)F[(size_t)i * P + p];
    mu[p] = s / (double)N;
}

// ybar = mean(y); one block.
__global__ void __launch_bounds__(kRThreads)
ridge_ymean_kernel(const float* __restrict__ y, int N, double* __restrict__ ybar) {
    __shared__ double red[kRThreads];
    double s = 0.0;
    for (int i = threadIdx.x; i < N; i += kRThreads) s += (double)y[i];
    red[threadIdx.x] = s;
    __syncthreads();
    for (int o = kRThreads / 2; o > 0; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) *ybar = red[0] / (double)N;
}

// G[i][j] = sum_p (F[i][p] - mu[p]) (F[j][p] - mu[p]) (+ alpha on the diagonal), lower triangle and
// its mirror.  One block per 32 x 32 tile with bi >= bj; the feature axis goes through shared memory
// in pieces of 32 (centred on the way in); every thread owns a 2 x 2 piece of the tile.
constexpr int kGT = 32, kGP = 32;
__global__ void __launch_bounds__(kRThreads)
ridge_gram_kernel(const float* __restrict__ F, int N, int P, const double* __restrict__ mu, double alpha,
                  double* __restrict__ G) {
    const int bi = blockIdx.y, bj = blockIdx.x;
    if (bj > bi) return;
    __shared__ double A[kGT][kGP + 1], B[kGT][kGP + 1];
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;   // 16 x 16 threads, 2 x 2 outputs each
    double acc[2][2] = {{0.0, 0.0}, {0.0, 0.0}};
    for (int p0 = 0; p0 < P; p0 += kGP) {
        for (int e = threadIdx.x; e < kGT * kGP; e += kRThreads) {
            const int r = e / kGP, c = e % kGP, p = p0 + c;
            const int ia = bi * kGT + r, ib = bj * kGT + r;
            const double m = p < P ? mu[p] : 0.0;
            A[r][c] = (ia < N && p < P) ? (double)F[(size_t)ia * P + p] - m : 0.0;
            B[r][c] = (ib < N && p < P) ? (double)F[(size_t)ib * P + p] - m : 0.0;
        }
        __syncthreads();
#pragma unroll 8
        for (int c = 0; c < kGP; ++c) {
            const double a0 = A[2 * ty][c], a1 = A[2 * ty + 1][c], b0 = B[2 * tx][c], b1 = B[2 * tx + 1][c];
            acc[0][0] += a0 * b0; acc[0][1] += a0 * b1; acc[1][0] += a1 * b0; acc[1][1] += a1 * b1;
        }
        __syncthreads();
    }
    for (int u = 0; u < 2; ++u)
        for (int v = 0; v < 2; ++v) {
            const int i = bi * kGT + 2 * ty + u, j = bj * kGT + 2 * tx + v;
            if (i < N && j < N) {
                const double g = acc[u][v] + (i == j ? alpha : 0.0);
                G[(size_t)i * N + j] = g;
                G[(size_t)j * N + i] = g;
            }
        }
}

// In-place Cholesky factor (lower triangle, G = L L^T) and the two triangular solves, one block.
// Right-looking, column by column; status: 0 = ok, 1 = a pivot was not positive.
__global__ void __launch_bounds__(1024)
ridge_cholesky_solve_kernel(double* __restrict__ G, int N, const float* __restrict__ y, const double* __restrict__ ybar,
                            double* __restrict__ a, int* __restrict__ status) {
    __shared__ double pivot;
    __shared__ int bad;
    __shared__ double col[ROCKET_RIDGE_MAX_EXAMPLES];   // column k of L below the diagonal
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    if (threadIdx.x == 0) bad = 0;
    __syncthreads();
    for (int k = 0; k < N; ++k) {
        if (threadIdx.x == 0) {
            const double d = G[(size_t)k * N + k];
            if (!(d > 0.0)) bad = 1;
            pivot = d > 0.0 ? sqrt(d) : 1.0;
            G[(size_t)k * N + k] = pivot;
        }
        __syncthreads();
        const double inv = 1.0 / pivot;
        for (int i = k + 1 + threadIdx.x; i < N; i += blockDim.x) {
            const double l = G[(size_t)i * N + k] * inv;
            G[(size_t)i * N + k] = l;
            col[i] = l;
        }
        __syncthreads();
        // trailing update of the lower triangle: G[i][j] -= L[i][k] L[j][k], k < j <= i (a warp per row)
        for (int i = k + 1 + warp; i < N; i += nwarps) {
            const double li = col[i];
            double* __restrict__ row = G + (size_t)i * N;
            for (int j = k + 1 + lane; j <= i; j += 32) row[j] -= li * col[j];
        }
        __syncthreads();
    }
    // L z = yc (forward), then L^T a = z (backward); a holds z in between
    for (int i = threadIdx.x; i < N; i += blockDim.x) a[i] = (double)y[i] - *ybar;
    __syncthreads();
    for (int k = 0; k < N; ++k) {
        if (threadIdx.x == 0) a[k] /= G[(size_t)k * N + k];
        __syncthreads();
        const double zk = a[k];
        for (int i = k + 1 + threadIdx.x; i < N; i += blockDim.x) a[i] -= G[(size_t)i * N + k] * zk;
        __syncthreads();
    }
    for (int k = N - 1; k >= 0; --k) {
        if (threadIdx.x == 0) a[k] /= G[(size_t)k * N + k];
        __syncthreads();
        const double ak = a[k];
        for (int i = threadIdx.x; i < k; i += blockDim.x) a[i] -= G[(size_t)k * N + i] * ak;
        __syncthreads();
    }
    if (threadIdx.x == 0) *status = bad;
}

// w[p] = sum_i a[i] (F[i][p] - mu[p]); one thread per feature.  Also part[block] = sum_p mu[p] w[p].
__global__ void __launch_bounds__(kRThreads)
ridge_weights_kernel(const float* __restrict__ F, int N, int P, const double* __restrict__ mu,
                     const double* __restrict__ a, float* __restrict__ w, double* __restrict__ part) {
    __shared__ double red[kRThreads];
    const int p = blockIdx.x * kRThreads + threadIdx.x;
    double s = 0.0, m = 0.0;
    if (p < P) {
        m = mu[p];
        for (int i = 0; i < N; ++i) s += a[i] * ((double)F[(size_t)i * P + p] - m);
        w[p] = (float)s;
    }
    red[threadIdx.x] = p < P ? m * (double)(float)s : 0.0;   // the intercept matches the stored fp32 weights
    __syncthreads();
    for (int o = kRThreads / 2; o > 0; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) part[blockIdx.x] = red[0];
}

// b = ybar - sum of the partial dot products, in block order (run-to-run identical).
__global__ void ridge_intercept_kernel(const double* __restrict__ part, int nparts, const double* __restrict__ ybar,
                                       float* __restrict__ b) {
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        double s = 0.0;
        for (int i = 0; i < nparts; ++i) s += part[i];
        *b = (float)(*ybar - s);
    }
}

// yhat[n] = b + sum_p F[n][p] w[p]; one block per example, products summed in double.
__global__ void __launch_bounds__(kRThreads)
ridge_predict_kernel(const float* __restrict__ F, int P, const float* __restrict__ w, const float* __restrict__ b,
                     float* __restrict__ yhat) {
    __shared__ double red[kRThreads];
    const float* __restrict__ f = F + (size_t)blockIdx.x * P;
    double s = 0.0;
    for (int p = threadIdx.x; p < P; p += kRThreads) s += (double)f[p] * (double)w[p];
    red[threadIdx.x] = s;
    __syncthreads();
    for (int o = kRThreads / 2; o > 0; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) yhat[blockIdx.x] = (float)(red[0] + (double)*b);
}

int status_of(cudaError_t e) {
    if (e == cudaSuccess) return ROCKET_OK;
    cudaGetLastError();
    return e == cudaErrorMemoryAllocation ? ROCKET_ENOMEM : ROCKET_ECUDA;
}

}  // namespace
}  // namespace rocket

using namespace rocket;

extern "C" int rocket_ridge_fit(const float* feat_dev, int N, int P, const float* y_dev, float alpha, float* w_dev,
                                float* b_dev, void* cuda_stream) {
    if (!feat_dev || !y_dev || !w_dev || !b_dev || N < 1 || P < 1) return ROCKET_EINVAL;
    if (!(alpha >= 0.0f) || !(alpha < 3.0e38f)) return ROCKET_EINVAL;
    if (N > ROCKET_RIDGE_MAX_EXAMPLES) return ROCKET_EUNSUPPORTED;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int nparts = (P + kRThreads - 1) / kRThreads;
    // workspace: mu[P], G[N][N], a[N], part[nparts], ybar, status
    const size_t doubles = (size_t)P + (size_t)N * N + (size_t)N + (size_t)nparts + 1;
    char* ws = nullptr;
    cudaError_t e = rocket::device_malloc(reinterpret_cast<void**>(&ws), doubles * sizeof(double) + 16);
    if (e != cudaSuccess) return status_of(e);
    double* mu = reinterpret_cast<double*>(ws);
    double* G = mu + P;
    double* a = G + (size_t)N * N;
    double* part = a + N;
    double* ybar = part + nparts;
    int* status = reinterpret_cast<int*>(ybar + 1);
    const int tiles = (N + kGT - 1) / kGT;
    ridge_colmean_kernel<<<nparts, kRThreads, 0, stream>>>(feat_dev, N, P, mu);
    ridge_ymean_kernel<<<1, kRThreads, 0, stream>>>(y_dev, N, ybar);
    ridge_gram_kernel<<<dim3(tiles, tiles), kRThreads, 0, stream>>>(feat_dev, N, P, mu, (double)alpha, G);
    ridge_cholesky_solve_kernel<<<1, 1024, 0, stream>>>(G, N, y_dev, ybar, a, status);
    ridge_weights_kernel<<<nparts, kRThreads, 0, stream>>>(feat_dev, N, P, mu, a, w_dev, part);
    ridge_intercept_kernel<<<1, 32, 0, stream>>>(part, nparts, ybar, b_dev);
    count_launch(6);
    int host_status = 0;
    e = cudaGetLastError();
    if (e == cudaSuccess) e = cudaMemcpyAsync(&host_status, status, sizeof(int), cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    cudaFree(ws);
    if (e != cudaSuccess) return status_of(e);
    return host_status == 0 ? ROCKET_OK : ROCKET_EINVAL;
}

extern "C" int rocket_ridge_predict(const float* feat_dev, int N, int P, const float* w_dev, const float* b_dev,
                                    float* yhat_dev, void* cuda_stream) {
    if (N < 0 || P < 1) return ROCKET_EINVAL;
    if (N == 0) return ROCKET_OK;
    if (!feat_dev || !w_dev || !b_dev || !yhat_dev) return ROCKET_EINVAL;
    ridge_predict_kernel<<<(unsigned)N, kRThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(feat_dev, P, w_dev, b_dev,
                                                                                              yhat_dev);
    count_launch();
    return status_of(cudaGetLastError());
}
