// Internal declarations shared by the translation units of the ROCKET transform library.
#pragma once

#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>
#include <mutex>
#include <vector>

#include "rocket.h"

namespace rocket {

// Device-side view of the ragged kernel parameters (all pointers are device pointers).
struct DeviceParams {
    int K, C, L;
    const int32_t* length;
    const int32_t* dilation;
    const int32_t* padding;
    const int32_t* num_channels;
    const int32_t* channel_offset;  // [K+1]
    const int32_t* weight_offset;   // [K+1]
    const int32_t* channel_idx;
    const float* weights;
    const float* bias;
};

struct HostParams {
    int K = 0, C = 0, L = 0;
    std::vector<int32_t> length, dilation, padding, num_channels, channel_idx;
    std::vector<int32_t> channel_offset, weight_offset;  // [K+1]
    std::vector<float> weights, bias;
    double conv_flops = 0.0, conv_outputs = 0.0;
};

extern std::atomic<int64_t> g_launch_count;
inline void count_launch(int n = 1) { g_launch_count.fetch_add(n, std::memory_order_relaxed); }

// Every device allocation of the library goes through here, so that a caller (and the tests) can
// tell whether a call allocated: rocket_device_alloc_count reports the number made so far.
extern std::atomic<int64_t> g_alloc_count;
inline cudaError_t device_malloc(void** ptr, size_t bytes) {
    g_alloc_count.fetch_add(1, std::memory_order_relaxed);
    return cudaMalloc(ptr, bytes);
}

// Draws K kernels by the rules of Section 3.1 with the counter-based generator.
void generate_host_params(uint64_t seed, int K, int C, int L, HostParams& out);

// ---- generic kernels (any length <= 11, any shape, no alignment demands) -------------------
// Forward: one block per (example, kernel).  soft = false: PPV + max; soft = true: softPPV + max
// (+ argmax when argmax != nullptr).  klist (device, nk entries) restricts the pass to those
// kernels; nullptr means all K.
cudaError_t launch_generic_forward(const DeviceParams& dp, const float* X, int N, bool soft, float lambda,
                                   float shift, float* feat, int32_t* argmax, cudaStream_t stream,
                                   const int32_t* klist = nullptr, int nk = 0);
// Backward: per-example partial gradients into scratch[N][nW + K], then a fixed-order sum over n.
size_t generic_backward_scratch_floats(int N, int64_t n_weights, int K);
// x[i] = (v[i] - mean[c]) * inv_std[c] for [rows][L] 8-bit samples, c = row % C (mean, inv_std on the device).
cudaError_t launch_normalise_u8(const uint8_t* X, int64_t rows, int L, int C, const float* mean, const float* inv_std,
                                float* out, cudaStream_t stream);
// klist (device, nk entries) restricts the pass to those kernels, whose dW / db entries alone are written.
cudaError_t launch_generic_backward(const DeviceParams& dp, int64_t n_weights, const float* X, int N,
                                    float lambda, float shift, const float* dfeat, const int32_t* argmax,
                                    float* scratch, float* dW, float* db, cudaStream_t stream,
                                    const int32_t* klist = nullptr, int nk = 0);

}  // namespace rocket

namespace rocket { namespace fast { struct FastState; } }

// Grow-only device buffer owned by a handle.
struct DeviceBuffer {
    void* ptr = nullptr;
    size_t bytes = 0;
    cudaError_t reserve(size_t need) {
        if (need <= bytes) return cudaSuccess;
        if (ptr) cudaFree(ptr);
        ptr = nullptr; bytes = 0;
        cudaError_t e = rocket::device_malloc(&ptr, need);
        if (e == cudaSuccess) bytes = need;
        else ptr = nullptr;
        return e;
    }
    void release() { if (ptr) cudaFree(ptr); ptr = nullptr; bytes = 0; }
};

struct rocket_params {
    rocket::HostParams host;
    int path = 0;                 // 0 = automatic, 1 = generic kernels only
    mutable std::mutex mu;        // guards the lazy upload and the grow-only buffers below
    mutable int device = -1;      // device of the first device call; -1 until then
    mutable void* dev_blob = nullptr;  // one allocation holding every parameter array
    mutable rocket::DeviceParams dp{};
    mutable DeviceBuffer scratch; // backward partial sums
    mutable DeviceBuffer u8_x, u8_norm;   // 8-bit input outside the fast path: normalised fp32 copy, mean / inv_std
    mutable std::vector<float> u8_norm_host;
    rocket::fast::FastState* fast = nullptr;   // fast-path launch plan and its device-side state
    DeviceBuffer stage_u8, stage_x, stage_feat, stage_arg, stage_g, stage_dw;  // host-call staging
    cudaStream_t host_stream = nullptr;
    cudaStream_t copy_stream = nullptr;        // host forms: uploads run ahead of the kernels on this stream
    std::vector<cudaEvent_t> copy_events;      // one per chunk of a host-form call
};
