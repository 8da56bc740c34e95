// Allocation-free variant of the soft backward pass: the per-example partial sums live in a
// file-scope device array instead of a cudaMalloc'ed workspace, for callers that must not
// allocate (real-time loops, fixed memory pools, streams being recorded by someone else).
#include <mutex>

#include "rocket_internal.h"

namespace {

// Part of the library image: every GPU that loads the library holds these 16 MiB until exit.
static __device__ __align__(256) float g_noalloc_scratch[ROCKET_NOALLOC_MAX_SCRATCH_FLOATS];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
float* g_scratch_addr[kMaxDevices] = {};  // device address of the array, per device ordinal

// In host code `g_noalloc_scratch` is only a stand-in symbol, not a device address; the address
// a kernel can use comes from cudaGetSymbolAddress, once per device, with that device current.
int scratch_address(int device, float** out) {
    if (device < 0 || device >= kMaxDevices) return ROCKET_EUNSUPPORTED;
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g_scratch_addr[device]) {
        void* addr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&addr, g_noalloc_scratch);
        if (e != cudaSuccess || !addr) {
            cudaGetLastError();
            return ROCKET_ECUDA;
        }
        g_scratch_addr[device] = static_cast<float*>(addr);
    }
    *out = g_scratch_addr[device];
    return ROCKET_OK;
}

}  // namespace

extern "C" int rocket_transform_soft_backward_noalloc(const rocket_params_t* p, const float* X_dev, int N, int C,
                                                      int L, float lambda, float shift, const float* dfeat_dev,
                                                      const int32_t* argmax_dev, float* dW_dev, float* db_dev,
                                                      void* cuda_stream) {
    if (!p || N < 0) return ROCKET_EINVAL;
    if (C != p->host.C || L != p->host.L) return ROCKET_ESHAPE;
    if (!(lambda == lambda) || !(shift == shift)) return ROCKET_EINVAL;
    if (!dW_dev || !db_dev) return ROCKET_EINVAL;
    if (N > 0 && (!X_dev || !dfeat_dev || !argmax_dev)) return ROCKET_EINVAL;
    int device = -1;
    rocket::DeviceParams dp;
    {   // the binding of a handle happens under its mutex: read what it wrote under the same mutex
        std::lock_guard<std::mutex> lk(p->mu);
        device = p->device;
        dp = p->dp;
    }
    if (device < 0) return ROCKET_EINVAL;  // not bound yet: binding would allocate
    const int64_t nW = (int64_t)p->host.weights.size();
    if ((int64_t)N * p->host.K > 0x7fffffffll) return ROCKET_EUNSUPPORTED;
    if (rocket::generic_backward_scratch_floats(N, nW, p->host.K) > (size_t)ROCKET_NOALLOC_MAX_SCRATCH_FLOATS)
        return ROCKET_EUNSUPPORTED;

    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) { cudaGetLastError(); return ROCKET_ECUDA; }
    if (prev != device && cudaSetDevice(device) != cudaSuccess) { cudaGetLastError(); return ROCKET_ECUDA; }
    float* scratch = nullptr;
    int st = scratch_address(device, &scratch);
    if (st == ROCKET_OK) {
        cudaError_t e = rocket::launch_generic_backward(dp, nW, X_dev, N, lambda, shift, dfeat_dev, argmax_dev,
                                                        scratch, dW_dev, db_dev, static_cast<cudaStream_t>(cuda_stream));
        if (e != cudaSuccess) { cudaGetLastError(); st = ROCKET_ECUDA; }
    }
    if (prev != device) cudaSetDevice(prev);
    return st;
}
