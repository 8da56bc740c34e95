// Generic kernels: one thread block per (example, kernel), inputs read straight from global
// memory with a range test per tap.  They accept every kernel the handle accepts (any length
// up to 11, any L, no alignment demands) and serve what the fast path does not cover.
#include <algorithm>
#include <cfloat>
#include <climits>

#include "rocket_internal.h"

namespace rocket {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxTaps = ROCKET_MAX_LENGTH * ROCKET_MAX_CHANNELS_PER_KERNEL;

struct KernelShape {
    int len, d, p, m;
    int64_t nout;
};

__device__ __forceinline__ float sigmoidf_fast(float v) { return __fdividef(1.0f, 1.0f + __expf(-v)); }

// Loads kernel k's parameters into shared memory (weights, channel row offsets) and returns its shape.
__device__ __forceinline__ KernelShape load_kernel(const DeviceParams& dp, int k, float* sW, int* sS) {
    KernelShape s;
    s.len = dp.length[k]; s.d = dp.dilation[k]; s.p = dp.padding[k]; s.m = dp.num_channels[k];
    s.nout = (int64_t)dp.L + 2 * (int64_t)s.p - (int64_t)(s.len - 1) * s.d;
    const int co = dp.channel_offset[k], wo = dp.weight_offset[k];
    for (int t = threadIdx.x; t < s.m * s.len; t += kThreads) sW[t] = dp.weights[wo + t];
    for (int t = threadIdx.x; t < s.m; t += kThreads) sS[t] = dp.channel_idx[co + t];
    __syncthreads();
    return s;
}

// z_i of Section 3 step (1): bias plus the dilated, zero-padded multichannel correlation.
__device__ __forceinline__ float conv_at(const KernelShape& s, const float* __restrict__ Xn, int L,
                                         const float* sW, const int* sS, float b, int i) {
    float z = b;
    for (int q = 0; q < s.m; ++q) {
        const float* __restrict__ x = Xn + (int64_t)sS[q] * L;
        const float* w = sW + q * s.len;
        for (int j = 0; j < s.len; ++j) {
            const int t = i - s.p + j * s.d;
            if (t >= 0 && t < L) z = fmaf(w[j], __ldg(x + t), z);
        }
    }
    return z;
}

template <bool SOFT>
__global__ void __launch_bounds__(kThreads)
generic_forward_kernel(DeviceParams dp, const float* __restrict__ X, float lambda, float shift,
                       float* __restrict__ feat, int32_t* __restrict__ argmax, const int32_t* __restrict__ klist,
                       int nk) {
    __shared__ float sW[kMaxTaps];
    __shared__ int sS[ROCKET_MAX_CHANNELS_PER_KERNEL];
    __shared__ float rsum[kWarps], rmax[kWarps];
    __shared__ int rcnt[kWarps], rarg[kWarps];

    const int64_t e = blockIdx.x;
    const int n = (int)(e / nk);
    const int k = klist ? klist[e % nk] : (int)(e % nk);
    const KernelShape s = load_kernel(dp, k, sW, sS);
    const float* Xn = X + (int64_t)n * dp.C * dp.L;
    const float b = dp.bias[k];
    const int nout = (int)s.nout;

    int cnt = 0, arg = INT_MAX;
    float mx = -FLT_MAX, hs = 0.0f;
    for (int i = threadIdx.x; i < nout; i += kThreads) {
        const float z = conv_at(s, Xn, dp.L, sW, sS, b, i);
        if (SOFT) hs += sigmoidf_fast(fmaf(lambda, z, shift));   // Eq. 3
        else cnt += (z > 0.0f) ? 1 : 0;                            // Eq. 1
        if (z > mx) { mx = z; arg = i; }
    }
    // warp then block reduction; ties on the max resolve to the lowest index
    for (int o = 16; o > 0; o >>= 1) {
        cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
        hs += __shfl_xor_sync(0xffffffffu, hs, o);
        const float om = __shfl_xor_sync(0xffffffffu, mx, o);
        const int oa = __shfl_xor_sync(0xffffffffu, arg, o);
        if (om > mx || (om == mx && oa < arg)) { mx = om; arg = oa; }
    }
    const int w = threadIdx.x >> 5;
    if ((threadIdx.x & 31) == 0) { rcnt[w] = cnt; rsum[w] = hs; rmax[w] = mx; rarg[w] = arg; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int v = 1; v < kWarps; ++v) {
            cnt += rcnt[v]; hs += rsum[v];
            if (rmax[v] > mx || (rmax[v] == mx && rarg[v] < arg)) { mx = rmax[v]; arg = rarg[v]; }
        }
        float* f = feat + ((int64_t)n * dp.K + k) * 2;
        f[0] = SOFT ? hs / (float)nout : (float)cnt / (float)nout;  // Eq. 4 / Eq. 2
        f[1] = mx;
        if (SOFT && argmax) argmax[(int64_t)n * dp.K + k] = arg;
    }
}

constexpr int kTile = 1024;  // outputs whose gz is held in shared memory at a time

__global__ void __launch_bounds__(kThreads)
generic_backward_kernel(DeviceParams dp, int64_t n_weights, const float* __restrict__ X, float lambda,
                        float shift, const float* __restrict__ dfeat, const int32_t* __restrict__ argmax,
                        float* __restrict__ scratch, const int32_t* __restrict__ klist, int nk) {
    __shared__ float sW[kMaxTaps];
    __shared__ int sS[ROCKET_MAX_CHANNELS_PER_KERNEL];
    __shared__ float sgz[kTile];
    __shared__ float rdb[kWarps];

    const int64_t e = blockIdx.x;
    const int n = (int)(e / nk);
    const int k = klist ? klist[e % nk] : (int)(e % nk);
    const KernelShape s = load_kernel(dp, k, sW, sS);
    const float* Xn = X + (int64_t)n * dp.C * dp.L;
    const float b = dp.bias[k];
    const int nout = (int)s.nout;
    const float gP = dfeat[((int64_t)n * dp.K + k) * 2] * (lambda / (float)nout);
    const float gM = dfeat[((int64_t)n * dp.K + k) * 2 + 1];
    const int A = argmax[(int64_t)n * dp.K + k];
    const int taps = s.m * s.len;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    constexpr int kPerWarp = (kMaxTaps + kWarps - 1) / kWarps;
    float acc[kPerWarp];
#pragma unroll
    for (int v = 0; v < kPerWarp; ++v) acc[v] = 0.0f;
    float dbias = 0.0f;

    for (int base = 0; base < nout; base += kTile) {
        const int cnt = min(kTile, nout - base);
        __syncthreads();
        for (int u = threadIdx.x; u < cnt; u += kThreads) {
            const int i = base + u;
            const float z = conv_at(s, Xn, dp.L, sW, sS, b, i);
            const float h = sigmoidf_fast(fmaf(lambda, z, shift));
            float gz = gP * h * (1.0f - h);
            if (i == A) gz += gM;
            sgz[u] = gz;
            dbias += gz;
        }
        __syncthreads();
#pragma unroll
        for (int v = 0; v < kPerWarp; ++v) {
            const int t = warp + v * kWarps;  // tap (q, j)
            if (t < taps) {
                const int q = t / s.len, j = t - q * s.len;
                const float* __restrict__ x = Xn + (int64_t)sS[q] * dp.L;
                const int off = base - s.p + j * s.d;
                float a = acc[v];
                for (int u = lane; u < cnt; u += 32) {
                    const int tt = off + u;
                    if (tt >= 0 && tt < dp.L) a = fmaf(sgz[u], __ldg(x + tt), a);
                }
                acc[v] = a;
            }
        }
    }
    float* out = scratch + (int64_t)n * (n_weights + dp.K);
#pragma unroll
    for (int v = 0; v < kPerWarp; ++v) {
        float a = acc[v];
        for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        const int t = warp + v * kWarps;
        if (lane == 0 && t < taps) out[dp.weight_offset[k] + t] = a;
    }
    for (int o = 16; o > 0; o >>= 1) dbias += __shfl_xor_sync(0xffffffffu, dbias, o);
    if (lane == 0) rdb[warp] = dbias;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.0f;
        for (int v = 0; v < kWarps; ++v) t += rdb[v];
        out[n_weights + k] = t;
    }
}

// dW/db = sum over examples of the per-example partials, in example order (run-to-run identical).
__global__ void __launch_bounds__(kThreads)
reduce_examples_kernel(const float* __restrict__ scratch, int N, int64_t n_weights, int K,
                       float* __restrict__ dW, float* __restrict__ db) {
    const int64_t width = n_weights + K;
    const int64_t t = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (t >= width) return;
    float a = 0.0f;
    for (int n = 0; n < N; ++n) a += scratch[(int64_t)n * width + t];
    if (t < n_weights) dW[t] = a;
    else db[t - n_weights] = a;
}

// The same sum for a list of kernels only (one block per listed kernel): the other entries of dW / db belong
// to someone else and are left alone.
__global__ void __launch_bounds__(kThreads)
reduce_examples_list_kernel(const float* __restrict__ scratch, int N, int64_t n_weights, DeviceParams dp,
                            const int32_t* __restrict__ klist, float* __restrict__ dW, float* __restrict__ db) {
    const int k = klist[blockIdx.x];
    const int64_t width = n_weights + dp.K;
    const int wo = dp.weight_offset[k], taps = dp.weight_offset[k + 1] - wo;
    for (int t = threadIdx.x; t <= taps; t += kThreads) {
        const int64_t col = t < taps ? (int64_t)wo + t : n_weights + k;
        float a = 0.0f;
        for (int n = 0; n < N; ++n) a += scratch[(int64_t)n * width + col];
        if (t < taps) dW[wo + t] = a;
        else db[k] = a;
    }
}

// Per-channel feature scaling of raw 8-bit intensities (Sections 4.1 and 4.3).
__global__ void __launch_bounds__(kThreads)
normalise_u8_kernel(const uint8_t* __restrict__ X, int64_t total, int L, int C, const float* __restrict__ mean,
                    const float* __restrict__ inv_std, float* __restrict__ out) {
    for (int64_t e = (int64_t)blockIdx.x * kThreads + threadIdx.x; e < total; e += (int64_t)gridDim.x * kThreads) {
        const int c = (int)((e / L) % C);
        out[e] = ((float)X[e] - mean[c]) * inv_std[c];
    }
}

}  // namespace

cudaError_t launch_normalise_u8(const uint8_t* X, int64_t rows, int L, int C, const float* mean, const float* inv_std,
                                float* out, cudaStream_t stream) {
    const int64_t total = rows * L;
    if (total == 0) return cudaSuccess;
    const unsigned grid = (unsigned)std::min<int64_t>((total + kThreads - 1) / kThreads, 148 * 16);
    normalise_u8_kernel<<<grid, kThreads, 0, stream>>>(X, total, L, C, mean, inv_std, out);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_generic_forward(const DeviceParams& dp, const float* X, int N, bool soft, float lambda,
                                   float shift, float* feat, int32_t* argmax, cudaStream_t stream,
                                   const int32_t* klist, int nk) {
    if (!klist) nk = dp.K;
    const int64_t blocks = (int64_t)N * nk;
    if (blocks == 0) return cudaSuccess;
    if (blocks > 0x7fffffffll) return cudaErrorInvalidConfiguration;
    if (soft) generic_forward_kernel<true><<<(unsigned)blocks, kThreads, 0, stream>>>(dp, X, lambda, shift, feat, argmax, klist, nk);
    else generic_forward_kernel<false><<<(unsigned)blocks, kThreads, 0, stream>>>(dp, X, lambda, shift, feat, argmax, klist, nk);
    count_launch();
    return cudaGetLastError();
}

size_t generic_backward_scratch_floats(int N, int64_t n_weights, int K) {
    return (size_t)N * (size_t)(n_weights + K);
}

cudaError_t launch_generic_backward(const DeviceParams& dp, int64_t n_weights, const float* X, int N,
                                    float lambda, float shift, const float* dfeat, const int32_t* argmax,
                                    float* scratch, float* dW, float* db, cudaStream_t stream, const int32_t* klist,
                                    int nk) {
    if (!klist) nk = dp.K;
    if (nk == 0) return cudaSuccess;
    const int64_t blocks = (int64_t)N * nk;
    if (blocks > 0x7fffffffll) return cudaErrorInvalidConfiguration;
    if (blocks > 0) {
        generic_backward_kernel<<<(unsigned)blocks, kThreads, 0, stream>>>(dp, n_weights, X, lambda, shift, dfeat,
                                                                           argmax, scratch, klist, nk);
        count_launch();
        cudaError_t err = cudaGetLastError();
        if (err != cudaSuccess) return err;
    }
    if (klist) {
        reduce_examples_list_kernel<<<(unsigned)nk, kThreads, 0, stream>>>(scratch, N, n_weights, dp, klist, dW, db);
    } else {
        const int64_t width = n_weights + dp.K;
        reduce_examples_kernel<<<(unsigned)((width + kThreads - 1) / kThreads), kThreads, 0, stream>>>(
            scratch, N, n_weights, dp.K, dW, db);
    }
    count_launch();
    return cudaGetLastError();
}

}  // namespace rocket
