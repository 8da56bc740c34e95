// Benchmark-only helper (not part of the transform library): measures what the FP32 FMA pipes of the
// current device sustain on dependent chains held in registers, once with scalar fma.rn.f32 and once with
// the packed two-wide fma.rn.f32x2 the transform's inner loop uses.  The result is the third denominator of
// the benchmark's roofline figures, beside SMs x 128 lanes x 2 flop x clock at the maximum and at the
// observed SM clock.  A third chain uses the packed half-precision fma.rn.f16x2: the rate a reduced-precision
// form of the transform (the paper's remark in Section 5) would have to live on.
#include <cuda_runtime.h>

#include <cstdint>

namespace {

typedef unsigned long long u64;

__device__ __forceinline__ u64 pack2(float lo, float hi) {
    u64 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}

// 16 independent chains per thread; every iteration issues one fused multiply-add per chain.
// The same 16 chains with packed half-precision fused multiply-adds (two per instruction and lane).
__global__ void __launch_bounds__(512, 1) fma_chain_f16x2_kernel(float* out, int iters) {
    unsigned p[16], a2, b2;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(a2) : "f"(0.999f), "f"(0.999f));
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(b2) : "f"(-1e-3f), "f"(1e-3f));
#pragma unroll
    for (int i = 0; i < 16; ++i) asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(p[i]) : "f"(1.0f - i * 0.01f), "f"(threadIdx.x * 1e-3f + i));
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < 16; ++i) asm volatile("fma.rn.f16x2 %0, %0, %1, %2;" : "+r"(p[i]) : "r"(a2), "r"(b2));
    }
    unsigned acc = 0;
#pragma unroll
    for (int i = 0; i < 16; ++i) acc ^= p[i];
    out[blockIdx.x * blockDim.x + threadIdx.x] = (float)acc;
}

template <bool PACKED>
__global__ void __launch_bounds__(512, 1) fma_chain_kernel(float* out, int iters) {
    const float a = 0.999f, b = 1e-3f;
    float s[16];
    u64 p[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        s[i] = threadIdx.x * 1e-3f + i;
        p[i] = pack2(s[i], 1.0f - s[i]);
    }
    const u64 a2 = pack2(a, a), b2 = pack2(b, -b);
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            if (PACKED) asm volatile("fma.rn.f32x2 %0, %0, %1, %2;" : "+l"(p[i]) : "l"(a2), "l"(b2));
            else asm volatile("fma.rn.f32 %0, %0, %1, %2;" : "+f"(s[i]) : "f"(a), "f"(b));
        }
    }
    float acc = 0.0f;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        float lo, hi;
        asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(p[i]));
        acc += s[i] + lo + hi;
    }
    out[blockIdx.x * blockDim.x + threadIdx.x] = acc;
}

// KIND 0: scalar fp32, 1: packed fp32, 2: packed fp16
template <int KIND>
int time_chain(int sms, float* out, double* tflops) {
    constexpr bool PACKED = KIND != 0;
    const int iters = 20000;
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return -1;
    double best = 0.0;
    for (int rep = 0; rep < 4; ++rep) {   // the first repetition warms up
        cudaEventRecord(e0);
        if (KIND == 2) fma_chain_f16x2_kernel<<<sms, 512>>>(out, iters);
        else fma_chain_kernel<KIND == 1><<<sms, 512>>>(out, iters);
        cudaEventRecord(e1);
        if (cudaEventSynchronize(e1) != cudaSuccess) return -1;
        float ms = 0.0f;
        cudaEventElapsedTime(&ms, e0, e1);
        const double flop = 2.0 * (PACKED ? 2.0 : 1.0) * 16.0 * iters * 512.0 * sms;
        if (rep > 0 && ms > 0.0f) best = flop / (ms * 1e-3) / 1e12 > best ? flop / (ms * 1e-3) / 1e12 : best;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    *tflops = best;
    return 0;
}

}  // namespace

// Returns 0 on success; *scalar_tflops and *packed_tflops receive the sustained FP32 FMA rates (2 flop per
// fused multiply-add) of the current device.
extern "C" int fma_peak_measure(double* scalar_tflops, double* packed_tflops) {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return -1;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return -1;
    float* out = nullptr;
    if (cudaMalloc(&out, (size_t)sms * 512 * sizeof(float)) != cudaSuccess) return -1;
    int rc = time_chain<0>(sms, out, scalar_tflops);
    if (rc == 0) rc = time_chain<1>(sms, out, packed_tflops);
    cudaFree(out);
    return cudaGetLastError() == cudaSuccess ? rc : -1;
}

// The sustained rate of packed half-precision fused multiply-adds (fma.rn.f16x2), in TFLOP/s.
extern "C" int fma_peak_measure_f16x2(double* packed_f16_tflops) {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return -1;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return -1;
    float* out = nullptr;
    if (cudaMalloc(&out, (size_t)sms * 512 * sizeof(float)) != cudaSuccess) return -1;
    const int rc = time_chain<2>(sms, out, packed_f16_tflops);
    cudaFree(out);
    return cudaGetLastError() == cudaSuccess ? rc : -1;
}
