// C ABI of the ROCKET transform library: parameter handles, validation, dispatch.
#include <algorithm>
#include <cstring>
#include <functional>
#include <new>

#include "rocket_fast.h"
#include "rocket_internal.h"

namespace rocket {
std::atomic<int64_t> g_launch_count{0};
std::atomic<int64_t> g_alloc_count{0};
}

using namespace rocket;

namespace {

int64_t n_weights_of(const rocket_params* p) { return (int64_t)p->host.weights.size(); }

int finish_host_params(HostParams& hp) {
    const int K = hp.K;
    hp.channel_offset.assign(K + 1, 0);
    hp.weight_offset.assign(K + 1, 0);
    hp.conv_flops = 0.0; hp.conv_outputs = 0.0;
    int64_t co = 0, wo = 0;
    for (int k = 0; k < K; ++k) {
        const int64_t len = hp.length[k], d = hp.dilation[k], p = hp.padding[k], m = hp.num_channels[k];
        if (len < 1 || len > ROCKET_MAX_LENGTH || d < 1 || p < 0) return ROCKET_EINVAL;
        if (m < 1 || m > std::min<int64_t>(hp.C, ROCKET_MAX_CHANNELS_PER_KERNEL)) return ROCKET_EINVAL;
        const int64_t nout = (int64_t)hp.L + 2 * p - (len - 1) * d;
        if (nout < 1 || (len - 1) * d + 1 > 0x3fffffffll || p > 0x3fffffffll) return ROCKET_EINVAL;
        // the kernels index outputs with 32-bit counters that step past the end by up to a block's width
        if (nout > 0x40000000ll) return ROCKET_EUNSUPPORTED;
        co += m; wo += m * len;
        if (wo > 0x7fffffffll) return ROCKET_EUNSUPPORTED;
        hp.channel_offset[k + 1] = (int32_t)co;
        hp.weight_offset[k + 1] = (int32_t)wo;
        hp.conv_flops += 2.0 * (double)len * (double)m * (double)nout;
        hp.conv_outputs += (double)nout;
    }
    return ROCKET_OK;
}

int validate_channels(const HostParams& hp) {
    for (int k = 0; k < hp.K; ++k) {
        const int32_t* S = hp.channel_idx.data() + hp.channel_offset[k];
        const int m = hp.num_channels[k];
        for (int a = 0; a < m; ++a) {
            if (S[a] < 0 || S[a] >= hp.C) return ROCKET_EINVAL;
            for (int b = 0; b < a; ++b) if (S[a] == S[b]) return ROCKET_EINVAL;
        }
    }
    return ROCKET_OK;
}

size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

// Uploads the host arrays into one device allocation on the current device and fills p->dp.
// Runs once per handle, at its first device call.
int ensure_device(const rocket_params* p) {
    std::lock_guard<std::mutex> lk(p->mu);
    if (p->device >= 0) return ROCKET_OK;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return ROCKET_ECUDA; }
    const HostParams& h = p->host;
    struct Part { const void* src; size_t bytes; size_t off; };
    Part parts[9] = {
        {h.length.data(), h.length.size() * 4, 0},         {h.dilation.data(), h.dilation.size() * 4, 0},
        {h.padding.data(), h.padding.size() * 4, 0},       {h.num_channels.data(), h.num_channels.size() * 4, 0},
        {h.channel_offset.data(), h.channel_offset.size() * 4, 0},
        {h.weight_offset.data(), h.weight_offset.size() * 4, 0},
        {h.channel_idx.data(), h.channel_idx.size() * 4, 0}, {h.weights.data(), h.weights.size() * 4, 0},
        {h.bias.data(), h.bias.size() * 4, 0}};
    size_t total = 0;
    for (auto& pt : parts) { pt.off = total; total += align256(pt.bytes); }
    cudaError_t e = device_malloc(&p->dev_blob, std::max<size_t>(total, 256));
    if (e != cudaSuccess) { cudaGetLastError(); p->dev_blob = nullptr; return e == cudaErrorMemoryAllocation ? ROCKET_ENOMEM : ROCKET_ECUDA; }
    char* base = static_cast<char*>(p->dev_blob);
    for (auto& pt : parts)
        if (pt.bytes && cudaMemcpy(base + pt.off, pt.src, pt.bytes, cudaMemcpyHostToDevice) != cudaSuccess) {
            cudaGetLastError();
            cudaFree(p->dev_blob);
            p->dev_blob = nullptr;
            return ROCKET_ECUDA;
        }
    DeviceParams& d = p->dp;
    d.K = h.K; d.C = h.C; d.L = h.L;
    d.length = reinterpret_cast<const int32_t*>(base + parts[0].off);
    d.dilation = reinterpret_cast<const int32_t*>(base + parts[1].off);
    d.padding = reinterpret_cast<const int32_t*>(base + parts[2].off);
    d.num_channels = reinterpret_cast<const int32_t*>(base + parts[3].off);
    d.channel_offset = reinterpret_cast<const int32_t*>(base + parts[4].off);
    d.weight_offset = reinterpret_cast<const int32_t*>(base + parts[5].off);
    d.channel_idx = reinterpret_cast<const int32_t*>(base + parts[6].off);
    d.weights = reinterpret_cast<const float*>(base + parts[7].off);
    d.bias = reinterpret_cast<const float*>(base + parts[8].off);
    if (p->fast->host.enabled) {
        cudaError_t pe = fast::upload_plan(*p->fast);
        if (pe != cudaSuccess) {
            cudaGetLastError();
            cudaFree(p->dev_blob);
            p->dev_blob = nullptr;
            return pe == cudaErrorMemoryAllocation ? ROCKET_ENOMEM : ROCKET_ECUDA;
        }
    }
    p->device = dev;
    return ROCKET_OK;
}

int finish_handle(rocket_params* p, rocket_params_t** out) {
    int st = finish_host_params(p->host);
    if (st == ROCKET_OK) st = validate_channels(p->host);
    if (st == ROCKET_OK) {
        try {
            p->fast = new fast::FastState();
            fast::build_plan(p->host, fast::kSplitDefault, p->fast->host);
        } catch (const std::bad_alloc&) {
            st = ROCKET_ENOMEM;
        }
    }
    if (st != ROCKET_OK) { rocket_params_destroy(p); return st; }
    *out = p;
    return ROCKET_OK;
}

int check_call(const rocket_params* p, const void* X, int N, int C, int L) {
    if (!p || N < 0) return ROCKET_EINVAL;
    if (C != p->host.C || L != p->host.L) return ROCKET_ESHAPE;
    if (N > 0 && !X) return ROCKET_EINVAL;
    if ((int64_t)N * p->host.K > 0x7fffffffll) return ROCKET_EUNSUPPORTED;
    return ROCKET_OK;
}

int cuda_status(cudaError_t e) {
    if (e == cudaSuccess) return ROCKET_OK;
    cudaGetLastError();
    return e == cudaErrorMemoryAllocation ? ROCKET_ENOMEM : ROCKET_ECUDA;
}

// Makes the handle's device current for the duration of a call.
struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; cudaGetLastError(); return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) { ok = false; cudaGetLastError(); }
    }
    ~DeviceGuard() { if (ok && prev >= 0) cudaSetDevice(prev); }
};

}  // namespace

extern "C" {

const char* rocket_strerror(int status) {
    switch (status) {
        case ROCKET_OK: return "success";
        case ROCKET_EINVAL: return "invalid argument";
        case ROCKET_ESHAPE: return "C or L differ from the parameter handle's";
        case ROCKET_EUNSUPPORTED: return "unsupported size or configuration";
        case ROCKET_ENOMEM: return "out of memory";
        case ROCKET_ECUDA: return "CUDA error";
        default: return "unknown status";
    }
}

int rocket_params_generate(uint64_t seed, int K, int C, int L, rocket_params_t** out) {
    if (!out || K < 1 || C < 1 || L < ROCKET_MAX_LENGTH) return ROCKET_EINVAL;
    rocket_params* p = new (std::nothrow) rocket_params();
    if (!p) return ROCKET_ENOMEM;
    try {
        generate_host_params(seed, K, C, L, p->host);
    } catch (const std::bad_alloc&) {
        delete p;
        return ROCKET_ENOMEM;
    }
    return finish_handle(p, out);
}

int rocket_params_from_arrays(int K, int C, int L, const int32_t* length, const int32_t* dilation,
                              const int32_t* padding, const int32_t* num_channels, const int32_t* channel_idx,
                              const float* weights, const float* bias, rocket_params_t** out) {
    if (!out || K < 1 || C < 1 || L < 1) return ROCKET_EINVAL;
    if (!length || !dilation || !padding || !num_channels || !channel_idx || !weights || !bias) return ROCKET_EINVAL;
    rocket_params* p = new (std::nothrow) rocket_params();
    if (!p) return ROCKET_ENOMEM;
    try {
        HostParams& h = p->host;
        h.K = K; h.C = C; h.L = L;
        h.length.assign(length, length + K);
        h.dilation.assign(dilation, dilation + K);
        h.padding.assign(padding, padding + K);
        h.num_channels.assign(num_channels, num_channels + K);
        h.bias.assign(bias, bias + K);
        // sizes of the ragged arrays follow from the per-kernel counts; validate those first
        int64_t nch = 0, nw = 0;
        for (int k = 0; k < K; ++k) {
            if (length[k] < 1 || length[k] > ROCKET_MAX_LENGTH || num_channels[k] < 1 ||
                num_channels[k] > ROCKET_MAX_CHANNELS_PER_KERNEL || num_channels[k] > C) {
                delete p;
                return ROCKET_EINVAL;
            }
            nch += num_channels[k];
            nw += (int64_t)num_channels[k] * length[k];
        }
        h.channel_idx.assign(channel_idx, channel_idx + nch);
        h.weights.assign(weights, weights + nw);
    } catch (const std::bad_alloc&) {
        delete p;
        return ROCKET_ENOMEM;
    }
    return finish_handle(p, out);
}

int rocket_params_counts(const rocket_params_t* p, int* K, int* C, int* L, int64_t* n_channel_idx,
                         int64_t* n_weights) {
    if (!p) return ROCKET_EINVAL;
    if (K) *K = p->host.K;
    if (C) *C = p->host.C;
    if (L) *L = p->host.L;
    if (n_channel_idx) *n_channel_idx = (int64_t)p->host.channel_idx.size();
    if (n_weights) *n_weights = (int64_t)p->host.weights.size();
    return ROCKET_OK;
}

int rocket_params_host_view(const rocket_params_t* p, const int32_t** length, const int32_t** dilation,
                            const int32_t** padding, const int32_t** num_channels, const int32_t** channel_idx,
                            const float** weights, const float** bias) {
    if (!p) return ROCKET_EINVAL;
    if (length) *length = p->host.length.data();
    if (dilation) *dilation = p->host.dilation.data();
    if (padding) *padding = p->host.padding.data();
    if (num_channels) *num_channels = p->host.num_channels.data();
    if (channel_idx) *channel_idx = p->host.channel_idx.data();
    if (weights) *weights = p->host.weights.data();
    if (bias) *bias = p->host.bias.data();
    return ROCKET_OK;
}

int rocket_params_work(const rocket_params_t* p, double* conv_flops_per_example, double* conv_outputs_per_example) {
    if (!p) return ROCKET_EINVAL;
    if (conv_flops_per_example) *conv_flops_per_example = p->host.conv_flops;
    if (conv_outputs_per_example) *conv_outputs_per_example = p->host.conv_outputs;
    return ROCKET_OK;
}

void rocket_params_destroy(rocket_params_t* p) {
    if (!p) return;
    if (p->device >= 0) {
        DeviceGuard g(p->device);
        if (p->dev_blob) cudaFree(p->dev_blob);
        if (p->fast) fast::release_fast_state(*p->fast);
        p->scratch.release();
        p->u8_x.release(); p->u8_norm.release(); p->stage_u8.release();
        p->stage_x.release(); p->stage_feat.release(); p->stage_arg.release();
        p->stage_g.release(); p->stage_dw.release();
        if (p->host_stream) cudaStreamDestroy(p->host_stream);
        if (p->copy_stream) cudaStreamDestroy(p->copy_stream);
        for (cudaEvent_t ev : p->copy_events) cudaEventDestroy(ev);
        cudaGetLastError();
    }
    delete p->fast;
    delete p;
}

int rocket_params_bind_device(const rocket_params_t* p) {
    if (!p) return ROCKET_EINVAL;
    return ensure_device(p);
}

int rocket_params_device_status(const rocket_params_t* p, int* wait_timeouts) {
    if (!p || !wait_timeouts) return ROCKET_EINVAL;
    *wait_timeouts = 0;
    if (p->device < 0 || !p->fast->dev.error_flag) return ROCKET_OK;
    DeviceGuard g(p->device);
    if (!g.ok) return ROCKET_ECUDA;
    return cuda_status(cudaMemcpy(wait_timeouts, p->fast->dev.error_flag, sizeof(int), cudaMemcpyDeviceToHost));
}

int rocket_params_set_weights(rocket_params_t* p, const float* weights, const float* bias) {
    if (!p || !weights || !bias) return ROCKET_EINVAL;
    const size_t nw = p->host.weights.size(), nb = p->host.bias.size();
    for (size_t i = 0; i < nw; ++i)
        if (!(weights[i] - weights[i] == 0.0f)) return ROCKET_EINVAL;
    for (size_t i = 0; i < nb; ++i)
        if (!(bias[i] - bias[i] == 0.0f)) return ROCKET_EINVAL;
    std::lock_guard<std::mutex> lk(p->mu);
    p->host.weights.assign(weights, weights + nw);
    p->host.bias.assign(bias, bias + nb);
    if (p->fast)
        for (fast::KRec& f : p->fast->host.krec) fast::fill_record_weights(p->host, f);
    if (p->device < 0) return ROCKET_OK;
    DeviceGuard g(p->device);
    if (!g.ok) return ROCKET_ECUDA;
    // work that still reads the old values finishes first
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess && nw) e = cudaMemcpy(const_cast<float*>(p->dp.weights), weights, nw * sizeof(float), cudaMemcpyHostToDevice);
    if (e == cudaSuccess && nb) e = cudaMemcpy(const_cast<float*>(p->dp.bias), bias, nb * sizeof(float), cudaMemcpyHostToDevice);
    if (e == cudaSuccess && p->fast) e = fast::upload_records(*p->fast);
    return cuda_status(e);
}

int rocket_params_set_path(rocket_params_t* p, int path) {
    if (!p || path < 0 || path > 1) return ROCKET_EINVAL;
    p->path = path;
    return ROCKET_OK;
}

int rocket_params_set_profiling(rocket_params_t* p, int enable) {
    if (!p || enable < 0 || enable > 1) return ROCKET_EINVAL;
    p->fast->profile = enable != 0;
    if (!enable) p->fast->ev_chunks = 0;
    return ROCKET_OK;
}

int rocket_params_last_profile(const rocket_params_t* p, double* ms_small_dilations, double* ms_large_dilations,
                               double* flops_small_dilations, double* flops_large_dilations) {
    if (!p) return ROCKET_EINVAL;
    if (flops_small_dilations) *flops_small_dilations = p->fast->host.flops_s;
    if (flops_large_dilations) *flops_large_dilations = p->fast->host.flops_t;
    if (ms_small_dilations) *ms_small_dilations = 0.0;
    if (ms_large_dilations) *ms_large_dilations = 0.0;
    if (p->fast->ev_chunks == 0 || p->device < 0) return ROCKET_OK;
    DeviceGuard g(p->device);
    if (!g.ok) return ROCKET_ECUDA;
    const std::vector<cudaEvent_t>& evs = p->fast->evs;
    const int chunks = p->fast->ev_chunks;
    cudaError_t e = cudaEventSynchronize(evs[3 * chunks - 1]);
    if (e != cudaSuccess) return cuda_status(e);
    double ms_s = 0.0, ms_t = 0.0;
    for (int c = 0; c < chunks; ++c) {
        float a = 0.0f, b = 0.0f;
        if ((e = cudaEventElapsedTime(&a, evs[3 * c], evs[3 * c + 1])) != cudaSuccess) return cuda_status(e);
        if ((e = cudaEventElapsedTime(&b, evs[3 * c + 1], evs[3 * c + 2])) != cudaSuccess) return cuda_status(e);
        ms_s += a;
        ms_t += b;
    }
    if (ms_small_dilations) *ms_small_dilations = ms_s;
    if (ms_large_dilations) *ms_large_dilations = ms_t;
    return ROCKET_OK;
}

int64_t rocket_kernel_launch_count(void) { return g_launch_count.load(std::memory_order_relaxed); }

int64_t rocket_device_alloc_count(void) { return g_alloc_count.load(std::memory_order_relaxed); }

int rocket_params_reserve(rocket_params_t* p, int max_N, int passes) {
    if (!p || max_N < 1 || passes < 1 || passes > 15) return ROCKET_EINVAL;
    if ((int64_t)max_N * p->host.K > 0x7fffffffll) return ROCKET_EUNSUPPORTED;
    int st = ensure_device(p);
    if (st != ROCKET_OK) return st;
    DeviceGuard g(p->device);
    if (!g.ok) return ROCKET_ECUDA;
    const bool soft = (passes & ROCKET_PASS_SOFT) != 0, backward = (passes & ROCKET_PASS_BACKWARD) != 0;
    const bool u8 = (passes & ROCKET_PASS_U8_INPUT) != 0;
    const int64_t nW = n_weights_of(p);
    if (p->fast->host.enabled) {
        cudaError_t e = fast::reserve_fast_state(*p->fast, p->dp, max_N, soft, backward, u8, nW);
        if (e != cudaSuccess) return cuda_status(e);
    }
    std::lock_guard<std::mutex> lk(p->mu);
    // kernels outside the fused path: the backward's per-example partial sums; 8-bit input: its fp32 copy
    const bool some_generic = !p->fast->host.enabled || !p->fast->host.generic_list.empty() || p->path == 1;
    if (backward && some_generic) {
        cudaError_t e = p->scratch.reserve(generic_backward_scratch_floats(max_N, nW, p->host.K) * sizeof(float));
        if (e != cudaSuccess) return cuda_status(e);
    }
    if (u8 && (some_generic || p->host.C > fast::kNormMaxChannels)) {
        cudaError_t e = p->u8_x.reserve((size_t)max_N * p->host.C * p->host.L * sizeof(float));
        if (e == cudaSuccess) e = p->u8_norm.reserve((size_t)2 * p->host.C * sizeof(float));
        if (e != cudaSuccess) return cuda_status(e);
    }
    return ROCKET_OK;
}

int rocket_transform(const rocket_params_t* p, const float* X_dev, int N, int C, int L, float* feat_dev,
                     void* cuda_stream) {
    int st = check_call(p, X_dev, N, C, L);
    if (st != ROCKET_OK) return st;
    if (N == 0) return ROCKET_OK;
    if (!feat_dev) return ROCKET_EINVAL;
    if ((st = ensure_device(p)) != ROCKET_OK) return st;
    DeviceGuard g(p->device);
    if (!g.ok) return ROCKET_ECUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const bool aligned = (reinterpret_cast<uintptr_t>(X_dev) & 3u) == 0;
    if (p->path == 0 && p->fast->host.enabled && aligned) {
        cudaError_t e = fast::launch_fast_forward(*p->fast, p->dp, X_dev, N, feat_dev, stream);
        if (e != cudaSuccess) return cuda_status(e);
        if (p->fast->dev.n_generic == 0) return ROCKET_OK;
        return cuda_status(launch_generic_forward(p->dp, X_dev, N, false, 0.0f, 0.0f, feat_dev, nullptr, stream,
                                                  p->fast->dev.generic_list, p->fast->dev.n_generic));
    }
    return cuda_status(launch_generic_forward(p->dp, X_dev, N, false, 0.0f, 0.0f, feat_dev, nullptr, stream));
}

// Half-precision form of the hard transform (Section 5, "FP16 compute"): fused kernels only.
int rocket_transform_f16(const rocket_params_t* p, const float* X_dev, int N, int C, int L, float* feat_dev,
                         void* cuda_stream) {
    int st = check_call(p, X_dev, N, C, L);
    if (st != ROCKET_OK) return st;
    if (N == 0) return ROCKET_OK;
    if (!feat_dev) return ROCKET_EINVAL;
    if ((st = ensure_device(p)) != ROCKET_OK) return st;
    if (!p->fast->host.enabled || p->fast->dev.n_generic != 0) return ROCKET_EUNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(X_dev) & 3u) != 0) return ROCKET_EINVAL;
    DeviceGuard g(p->device);
    if (!g.ok) return ROCKET_ECUDA;
    return cuda_status(fast::launch_fast_forward(*p->fast, p->dp, X_dev, N, feat_dev, static_cast<cudaStream_t>(cuda_stream),
                                                 false, 0.0f, 0.0f, nullptr, nullptr, nullptr, true));
}

int rocket_transform_soft(const rocket_params_t* p, const float* X_dev, int N, int C, int L, float lambda,
                          float shift, float* feat_dev, int32_t* argmax_dev, void* cuda_stream) {
    int st = check_call(p, X_dev, N, C, L);
    if (st != ROCKET_OK) return st;
    if (!(lambda == lambda) || !(shift == shift)) return ROCKET_EINVAL;
    if (N == 0) return ROCKET_OK;
    if (!feat_dev) return ROCKET_EINVAL;
    if ((st = ensure_device(p)) != ROCKET_OK) return st;
    DeviceGuard g(p->device);
    if (!g.ok) return ROCKET_ECUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const bool aligned = (reinterpret_cast<uintptr_t>(X_dev) & 3u) == 0;
    if (p->path == 0 && p->fast->host.enabled && aligned) {
        cudaError_t e = fast::launch_fast_forward(*p->fast, p->dp, X_dev, N, feat_dev, stream, true, lambda, shift, argmax_dev);
        if (e != cudaSuccess) return cuda_status(e);
        if (p->fast->dev.n_generic == 0) return ROCKET_OK;
        return cuda_status(launch_generic_forward(p->dp, X_dev, N, true, lambda, shift, feat_dev, argmax_dev, stream,
                                                  p->fast->dev.generic_list, p->fast->dev.n_generic));
    }
    return cuda_status(launch_generic_forward(p->dp, X_dev, N, true, lambda, shift, feat_dev, argmax_dev, stream));
}

// 8-bit input (Sections 4.1, 4.3): x = (v - mean[c]) * inv_std[c], then the transform of x.
static int transform_u8(const rocket_params_t* p, const uint8_t* X_u8_dev, int N, int C, int L, const float* mean,
                        const float* inv_std, bool soft, float lambda, float shift, float* feat_dev,
                        int32_t* argmax_dev, void* cuda_stream) {
    int st = check_call(p, X_u8_dev, N, C, L);
    if (st != ROCKET_OK) return st;
    if (!mean || !inv_std) return ROCKET_EINVAL;
    for (int c = 0; c < C; ++c)
        if (!(mean[c] == mean[c]) || !(inv_std[c] == inv_std[c])) return ROCKET_EINVAL;
    if (soft && (!(lambda == lambda) || !(shift == shift))) return ROCKET_EINVAL;
    if (N == 0) return ROCKET_OK;
    if (!feat_dev) return ROCKET_EINVAL;
    if ((st = ensure_device(p)) != ROCKET_OK) return st;
    DeviceGuard g(p->device);
    if (!g.ok) return ROCKET_ECUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const bool aligned = (reinterpret_cast<uintptr_t>(X_u8_dev) & 3u) == 0 && L % 4 == 0;
    if (p->path == 0 && p->fast->host.enabled && p->fast->dev.n_generic == 0 && aligned && C <= fast::kNormMaxChannels) {
        // every kernel is served by the fused kernels: the scaling happens while their staging copy is written
        fast::NormArgs norm;
        for (int c = 0; c < fast::kNormMaxChannels; ++c) {
            norm.mean[c] = c < C ? mean[c] : 0.0f;
            norm.inv_std[c] = c < C ? inv_std[c] : 0.0f;
        }
        return cuda_status(fast::launch_fast_forward(*p->fast, p->dp, nullptr, N, feat_dev, stream, soft, lambda, shift,
                                                     argmax_dev, X_u8_dev, &norm));
    }
    // otherwise: a scaled fp32 copy of the batch in a buffer of the handle, then the fp32 route
    const float* Xf = nullptr;
    {
        std::lock_guard<std::mutex> lock(p->mu);
        cudaError_t e = p->u8_x.reserve((size_t)N * C * L * sizeof(float));
        if (e == cudaSuccess) e = p->u8_norm.reserve((size_t)2 * C * sizeof(float));
        if (e != cudaSuccess) return cuda_status(e);
        float* nb = static_cast<float*>(p->u8_norm.ptr);
        // from pageable memory of the handle: the values are taken before the copy call returns
        p->u8_norm_host.assign(mean, mean + C);
        p->u8_norm_host.insert(p->u8_norm_host.end(), inv_std, inv_std + C);
        e = cudaMemcpyAsync(nb, p->u8_norm_host.data(), (size_t)2 * C * sizeof(float), cudaMemcpyHostToDevice, stream);
        if (e == cudaSuccess)
            e = launch_normalise_u8(X_u8_dev, (int64_t)N * C, L, C, nb, nb + C, static_cast<float*>(p->u8_x.ptr), stream);
        if (e != cudaSuccess) return cuda_status(e);
        Xf = static_cast<const float*>(p->u8_x.ptr);
    }
    return soft ? rocket_transform_soft(p, Xf, N, C, L, lambda, shift, feat_dev, argmax_dev, cuda_stream)
                : rocket_transform(p, Xf, N, C, L, feat_dev, cuda_stream);
}

int rocket_transform_u8(const rocket_params_t* p, const uint8_t* X_u8_dev, int N, int C, int L, const float* mean,
                        const float* inv_std, float* feat_dev, void* cuda_stream) {
    return transform_u8(p, X_u8_dev, N, C, L, mean, inv_std, false, 0.0f, 0.0f, feat_dev, nullptr, cuda_stream);
}

int rocket_transform_soft_u8(const rocket_params_t* p, const uint8_t* X_u8_dev, int N, int C, int L, const float* mean,
                             const float* inv_std, float lambda, float shift, float* feat_dev, int32_t* argmax_dev,
                             void* cuda_stream) {
    return transform_u8(p, X_u8_dev, N, C, L, mean, inv_std, true, lambda, shift, feat_dev, argmax_dev, cuda_stream);
}

int rocket_transform_soft_backward(const rocket_params_t* p, const float* X_dev, int N, int C, int L, float lambda,
                                   float shift, const float* dfeat_dev, const int32_t* argmax_dev, float* dW_dev,
                                   float* db_dev, void* cuda_stream) {
    int st = check_call(p, X_dev, N, C, L);
    if (st != ROCKET_OK) return st;
    if (!(lambda == lambda) || !(shift == shift)) return ROCKET_EINVAL;
    if (!dW_dev || !db_dev) return ROCKET_EINVAL;
    if (N > 0 && (!dfeat_dev || !argmax_dev)) return ROCKET_EINVAL;
    if ((st = ensure_device(p)) != ROCKET_OK) return st;
    DeviceGuard g(p->device);
    if (!g.ok) return ROCKET_ECUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int64_t nW = n_weights_of(p);
    const bool aligned = (reinterpret_cast<uintptr_t>(X_dev) & 3u) == 0;
    const bool use_fast = p->path == 0 && p->fast->host.enabled && (aligned || N == 0);
    const int n_generic = use_fast ? (int)p->fast->host.generic_list.size() : p->host.K;
    if (use_fast) {   // the fused kernels assign dW / db of the kernels they serve
        cudaError_t e = fast::launch_fast_backward(*p->fast, p->dp, nW, X_dev, N, lambda, shift, dfeat_dev, argmax_dev,
                                                   dW_dev, db_dev, stream);
        if (e != cudaSuccess) return cuda_status(e);
        if (n_generic == 0) return ROCKET_OK;
    }
    float* scratch = nullptr;
    if (N > 0) {
        std::lock_guard<std::mutex> lk(p->mu);
        cudaError_t e = p->scratch.reserve(generic_backward_scratch_floats(N, nW, p->host.K) * sizeof(float));
        if (e != cudaSuccess) return cuda_status(e);
        scratch = static_cast<float*>(p->scratch.ptr);
    }
    return cuda_status(launch_generic_backward(p->dp, nW, X_dev, N, lambda, shift, dfeat_dev, argmax_dev, scratch,
                                               dW_dev, db_dev, stream, use_fast ? p->fast->dev.generic_list : nullptr,
                                               use_fast ? n_generic : 0));
}

// ---- host-buffer forms ----------------------------------------------------------------------

static int host_stream_of(rocket_params_t* p, cudaStream_t* s) {
    if (!p->host_stream && cudaStreamCreateWithFlags(&p->host_stream, cudaStreamNonBlocking) != cudaSuccess) {
        cudaGetLastError();
        p->host_stream = nullptr;
        return ROCKET_ECUDA;
    }
    *s = p->host_stream;
    return ROCKET_OK;
}

#define ROCKET_TRY_CUDA(expr)                                  \
    do {                                                       \
        cudaError_t e__ = (expr);                              \
        if (e__ != cudaSuccess) return cuda_status(e__);       \
    } while (0)

// Host form of a forward transform, pipelined: the batch is uploaded on a second stream in chunks of
// the size the fused kernels work through, and the transform of a chunk starts as soon as its bytes
// have arrived, so all but the first upload hide behind the kernels.  run(n0, nc, stream) enqueues the
// device transform of examples [n0, n0 + nc).
static int host_pipeline(rocket_params_t* p, const void* X_host, size_t bytes_per_example, DeviceBuffer& stage, int N,
                         float* feat_host, cudaStream_t s, const std::function<int(int, int, cudaStream_t)>& run) {
    if (!p->copy_stream && cudaStreamCreateWithFlags(&p->copy_stream, cudaStreamNonBlocking) != cudaSuccess) {
        cudaGetLastError();
        p->copy_stream = nullptr;
        return ROCKET_ECUDA;
    }
    const int chunk = fast::kChunkExamples, n_chunks = (N + chunk - 1) / chunk;
    while ((int)p->copy_events.size() < n_chunks) {
        cudaEvent_t ev = nullptr;
        ROCKET_TRY_CUDA(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
        p->copy_events.push_back(ev);
    }
    const size_t fb = (size_t)N * 2 * p->host.K * sizeof(float);
    ROCKET_TRY_CUDA(stage.reserve((size_t)N * bytes_per_example));
    ROCKET_TRY_CUDA(p->stage_feat.reserve(fb));
    for (int c = 0; c < n_chunks; ++c) {
        const int n0 = c * chunk, nc = std::min(chunk, N - n0);
        const size_t off = (size_t)n0 * bytes_per_example;
        ROCKET_TRY_CUDA(cudaMemcpyAsync(static_cast<char*>(stage.ptr) + off, static_cast<const char*>(X_host) + off,
                                        (size_t)nc * bytes_per_example, cudaMemcpyHostToDevice, p->copy_stream));
        ROCKET_TRY_CUDA(cudaEventRecord(p->copy_events[c], p->copy_stream));
    }
    int st = ROCKET_OK;
    for (int c = 0; c < n_chunks && st == ROCKET_OK; ++c) {
        const int n0 = c * chunk, nc = std::min(chunk, N - n0);
        ROCKET_TRY_CUDA(cudaStreamWaitEvent(s, p->copy_events[c], 0));
        st = run(n0, nc, s);
    }
    if (st != ROCKET_OK) {   // nothing of this call may still be in flight when it returns
        cudaStreamSynchronize(p->copy_stream);
        cudaStreamSynchronize(s);
        return st;
    }
    ROCKET_TRY_CUDA(cudaMemcpyAsync(feat_host, p->stage_feat.ptr, fb, cudaMemcpyDeviceToHost, s));
    ROCKET_TRY_CUDA(cudaStreamSynchronize(s));
    return ROCKET_OK;
}

int rocket_transform_host(rocket_params_t* p, const float* X_host, int N, int C, int L, float* feat_host) {
    int st = check_call(p, X_host, N, C, L);
    if (st != ROCKET_OK) return st;
    if (N == 0) return ROCKET_OK;
    if (!feat_host) return ROCKET_EINVAL;
    if ((st = ensure_device(p)) != ROCKET_OK) return st;
    DeviceGuard g(p->device);
    if (!g.ok) return ROCKET_ECUDA;
    cudaStream_t s;
    if ((st = host_stream_of(p, &s)) != ROCKET_OK) return st;
    const size_t per_example = (size_t)C * L, K2 = (size_t)2 * p->host.K;
    return host_pipeline(p, X_host, per_example * sizeof(float), p->stage_x, N, feat_host, s,
                         [&](int n0, int nc, cudaStream_t stream) {
                             return rocket_transform(p, static_cast<const float*>(p->stage_x.ptr) + n0 * per_example, nc, C, L,
                                                     static_cast<float*>(p->stage_feat.ptr) + n0 * K2, stream);
                         });
}

int rocket_transform_u8_host(rocket_params_t* p, const uint8_t* X_u8_host, int N, int C, int L, const float* mean,
                             const float* inv_std, float* feat_host) {
    int st = check_call(p, X_u8_host, N, C, L);
    if (st != ROCKET_OK) return st;
    if (N == 0) return ROCKET_OK;
    if (!feat_host) return ROCKET_EINVAL;
    if ((st = ensure_device(p)) != ROCKET_OK) return st;
    DeviceGuard g(p->device);
    if (!g.ok) return ROCKET_ECUDA;
    cudaStream_t s;
    if ((st = host_stream_of(p, &s)) != ROCKET_OK) return st;
    const size_t per_example = (size_t)C * L, K2 = (size_t)2 * p->host.K;
    return host_pipeline(p, X_u8_host, per_example, p->stage_u8, N, feat_host, s,
                         [&](int n0, int nc, cudaStream_t stream) {
                             return rocket_transform_u8(p, static_cast<const uint8_t*>(p->stage_u8.ptr) + n0 * per_example, nc, C,
                                                        L, mean, inv_std, static_cast<float*>(p->stage_feat.ptr) + n0 * K2, stream);
                         });
}

int rocket_transform_soft_host(rocket_params_t* p, const float* X_host, int N, int C, int L, float lambda,
                               float shift, float* feat_host, int32_t* argmax_host) {
    int st = check_call(p, X_host, N, C, L);
    if (st != ROCKET_OK) return st;
    if (N == 0) return ROCKET_OK;
    if (!feat_host) return ROCKET_EINVAL;
    if ((st = ensure_device(p)) != ROCKET_OK) return st;
    DeviceGuard g(p->device);
    if (!g.ok) return ROCKET_ECUDA;
    cudaStream_t s;
    if ((st = host_stream_of(p, &s)) != ROCKET_OK) return st;
    const size_t xb = (size_t)N * C * L * sizeof(float), fb = (size_t)N * 2 * p->host.K * sizeof(float);
    const size_t ab = (size_t)N * p->host.K * sizeof(int32_t);
    ROCKET_TRY_CUDA(p->stage_x.reserve(xb));
    ROCKET_TRY_CUDA(p->stage_feat.reserve(fb));
    if (argmax_host) ROCKET_TRY_CUDA(p->stage_arg.reserve(ab));
    ROCKET_TRY_CUDA(cudaMemcpyAsync(p->stage_x.ptr, X_host, xb, cudaMemcpyHostToDevice, s));
    st = rocket_transform_soft(p, static_cast<const float*>(p->stage_x.ptr), N, C, L, lambda, shift,
                               static_cast<float*>(p->stage_feat.ptr),
                               argmax_host ? static_cast<int32_t*>(p->stage_arg.ptr) : nullptr, s);
    if (st != ROCKET_OK) return st;
    ROCKET_TRY_CUDA(cudaMemcpyAsync(feat_host, p->stage_feat.ptr, fb, cudaMemcpyDeviceToHost, s));
    if (argmax_host) ROCKET_TRY_CUDA(cudaMemcpyAsync(argmax_host, p->stage_arg.ptr, ab, cudaMemcpyDeviceToHost, s));
    ROCKET_TRY_CUDA(cudaStreamSynchronize(s));
    return ROCKET_OK;
}

int rocket_transform_soft_backward_host(rocket_params_t* p, const float* X_host, int N, int C, int L, float lambda,
                                        float shift, const float* dfeat_host, const int32_t* argmax_host,
                                        float* dW_host, float* db_host) {
    int st = check_call(p, X_host, N, C, L);
    if (st != ROCKET_OK) return st;
    if (!dW_host || !db_host) return ROCKET_EINVAL;
    if (N > 0 && (!dfeat_host || !argmax_host)) return ROCKET_EINVAL;
    if ((st = ensure_device(p)) != ROCKET_OK) return st;
    DeviceGuard g(p->device);
    if (!g.ok) return ROCKET_ECUDA;
    cudaStream_t s;
    if ((st = host_stream_of(p, &s)) != ROCKET_OK) return st;
    const int64_t nW = n_weights_of(p);
    const size_t xb = (size_t)N * C * L * sizeof(float), fb = (size_t)N * 2 * p->host.K * sizeof(float);
    const size_t ab = (size_t)N * p->host.K * sizeof(int32_t);
    const size_t wb = (size_t)(nW + p->host.K) * sizeof(float);
    ROCKET_TRY_CUDA(p->stage_x.reserve(std::max<size_t>(xb, 256)));
    ROCKET_TRY_CUDA(p->stage_g.reserve(std::max<size_t>(fb, 256)));
    ROCKET_TRY_CUDA(p->stage_arg.reserve(std::max<size_t>(ab, 256)));
    ROCKET_TRY_CUDA(p->stage_dw.reserve(wb));
    if (N > 0) {
        ROCKET_TRY_CUDA(cudaMemcpyAsync(p->stage_x.ptr, X_host, xb, cudaMemcpyHostToDevice, s));
        ROCKET_TRY_CUDA(cudaMemcpyAsync(p->stage_g.ptr, dfeat_host, fb, cudaMemcpyHostToDevice, s));
        ROCKET_TRY_CUDA(cudaMemcpyAsync(p->stage_arg.ptr, argmax_host, ab, cudaMemcpyHostToDevice, s));
    }
    float* dW = static_cast<float*>(p->stage_dw.ptr);
    st = rocket_transform_soft_backward(p, static_cast<const float*>(p->stage_x.ptr), N, C, L, lambda, shift,
                                        static_cast<const float*>(p->stage_g.ptr),
                                        static_cast<const int32_t*>(p->stage_arg.ptr), dW, dW + nW, s);
    if (st != ROCKET_OK) return st;
    ROCKET_TRY_CUDA(cudaMemcpyAsync(dW_host, dW, (size_t)nW * sizeof(float), cudaMemcpyDeviceToHost, s));
    ROCKET_TRY_CUDA(cudaMemcpyAsync(db_host, dW + nW, (size_t)p->host.K * sizeof(float), cudaMemcpyDeviceToHost, s));
    ROCKET_TRY_CUDA(cudaStreamSynchronize(s));
    return ROCKET_OK;
}

}  // extern "C"
