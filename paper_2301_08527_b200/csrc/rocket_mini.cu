// MINIROCKET on the device (the extension the paper names in Section 6: "the PyTorch GPU implementation could
// be extended to the MINIROCKET model"; Section 2 describes the model: two-valued kernels from a fixed set,
// biases sampled from the input data, PPV as the only pooled feature).
//
//   parameters   built on the host from one seed (rocket_mini_create): 84 kernels of length 9 with three taps
//                of weight 2 and six of weight -1, dilations floor(2^x) spread up to (L - 1) / 8, padding 4 d on
//                every other (dilation, kernel) combination, a random channel subset per combination
//   fit          rocket_mini_fit, on the host (a one-off over one training example per combination): the bias of
//                a feature is a quantile of the combination's convolution output on that example
//   transform    rocket_mini_transform, one fused kernel: per (example, combination) the channels are summed, the
//                nine-tap dilated convolution runs on a register window that slides down a column of the
//                dilated view, and every output is compared with the combination's biases on the fly, so the
//                convolution outputs never reach memory; feature = count / number of outputs (Eq. 1-2 against
//                the bias)
//
// The kernel weights take two values, so every product is one fused multiply-add with -1 or 2: on this
// hardware an addition and a fused multiply-add take the same issue slot, and the additions-only form that
// speeds the method up on a CPU brings nothing here.  The bound of the kernel is the traffic from L2: every
// combination reads its channels once.
#include <algorithm>
#include <cmath>
#include <mutex>
#include <new>
#include <numeric>
#include <thread>
#include <vector>

#include "rocket_internal.h"

namespace {

constexpr int kKernels = 84, kLen = 9;
constexpr int kMaxFeaturesPerItem = 16;
constexpr int kThreads = 256;
constexpr int kSmallDilation = 32;     // below: consecutive outputs from a staged run of samples; from here on: column walks
constexpr int kChunk = 4096;           // outputs per staged run
constexpr uint64_t kGolden = 0x9E3779B97F4A7C15ull;
constexpr uint64_t kStreamBase = 1ull << 32;
constexpr double kInvGoldenRatio = 0.6180339887498949;

inline uint64_t mix(uint64_t z) {   // splitmix64 finaliser
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
inline uint64_t draw_u64(uint64_t seed, uint64_t stream, uint64_t slot) {
    return mix(mix(seed + kGolden * (stream + 1)) + kGolden * (slot + 1));
}
inline double draw_uniform(uint64_t seed, uint64_t stream, uint64_t slot) {
    return static_cast<double>(draw_u64(seed, stream, slot) >> 11) * 0x1.0p-53;
}

// One unit of device work: a combination, or a slice of at most 16 of its features.
struct MiniItem {
    int32_t d, padded, m, f0, nf;
    int32_t tap[3];
    int32_t ch[kLen];
    int32_t pad_[3];
};
static_assert(sizeof(MiniItem) == 80, "MiniItem layout");

__global__ void __launch_bounds__(kThreads)
mini_transform_kernel(const float* __restrict__ X, int C, int L, const MiniItem* __restrict__ items, int n_items,
                      const float* __restrict__ bias, float* __restrict__ feat, int F) {
    __shared__ int s_cnt[kMaxFeaturesPerItem];
    __shared__ float s_x[kChunk + 8 * kSmallDilation];
    const int n = blockIdx.x / n_items;
    const MiniItem it = items[blockIdx.x - n * n_items];
    const float* __restrict__ Xn = X + (size_t)n * C * L;
    if (threadIdx.x < kMaxFeaturesPerItem) s_cnt[threadIdx.x] = 0;
    __syncthreads();
    const int d = it.d, m = it.m;
    const int first = it.padded ? 0 : 4 * d, last = it.padded ? L : L - 4 * d;
    float w[kLen];
#pragma unroll
    for (int j = 0; j < kLen; ++j) w[j] = (j == it.tap[0] || j == it.tap[1] || j == it.tap[2]) ? 2.0f : -1.0f;
    float b[kMaxFeaturesPerItem];
#pragma unroll
    for (int f = 0; f < kMaxFeaturesPerItem; ++f) b[f] = f < it.nf ? __ldg(bias + it.f0 + f) : __int_as_float(0x7f800000);
    int cnt[kMaxFeaturesPerItem];
#pragma unroll
    for (int f = 0; f < kMaxFeaturesPerItem; ++f) cnt[f] = 0;

    // the series seen as rows of d samples: a thread walks down one column over a run of rows
    const int T = (L + d - 1) / d;
    const int nseg = max(1, min(T, (1024 + d - 1) / d));
    const int rows_per_seg = (T + nseg - 1) / nseg;
    const int n_units = d * nseg;
    // channel rows of this example (unused entries repeat the first: their loads are predicated off)
    const float* __restrict__ chan[kLen];
#pragma unroll
    for (int q = 0; q < kLen; ++q) chan[q] = Xn + (size_t)it.ch[q < m ? q : 0] * L;
    // sum of the chosen channels at sample pos; zero outside the series (the nesting keeps the number of
    // executed loads at the number of channels: m is the same for the whole block)
    auto sample_at = [&](int pos) -> float {
        if ((unsigned)pos >= (unsigned)L) return 0.0f;
        float v = __ldg(chan[0] + pos);
        if (m > 1) { v += __ldg(chan[1] + pos);
        if (m > 2) { v += __ldg(chan[2] + pos);
        if (m > 3) { v += __ldg(chan[3] + pos);
        if (m > 4) { v += __ldg(chan[4] + pos);
        if (m > 5) { v += __ldg(chan[5] + pos);
        if (m > 6) { v += __ldg(chan[6] + pos);
        if (m > 7) { v += __ldg(chan[7] + pos);
        if (m > 8) { v += __ldg(chan[8] + pos); } } } } } } } }
        return v;
    };
    const int nf = it.nf;
    auto pool = [&](const float (&win)[kLen]) {   // one output: nine products, then Eq. 1 against every bias
        float z = 0.0f;
#pragma unroll
        for (int j = 0; j < kLen; ++j) z = fmaf(w[j], win[j], z);
#pragma unroll
        for (int g = 0; g < kMaxFeaturesPerItem; g += 4)
            if (g < nf) {
#pragma unroll
                for (int f = g; f < g + 4; ++f) cnt[f] += z > b[f] ? 1 : 0;
            }
    };
    if (d < kSmallDilation) {
        // Small dilations: adjacent threads of a column walk would sit in far-apart rows and every load would
        // touch its own memory sector.  Instead the block stages the channel sum of a run of consecutive
        // samples (with 4 d more on either side) in shared memory and every thread takes consecutive outputs.
        for (int p0 = first; p0 < last; p0 += kChunk) {
            const int lo = p0 - 4 * d, n_stage = min(kChunk, last - p0) + 8 * d;
            __syncthreads();
            for (int e = threadIdx.x; e < n_stage; e += kThreads) s_x[e] = sample_at(lo + e);
            __syncthreads();
            const int n_out = min(kChunk, last - p0);
            for (int e = threadIdx.x; e < n_out; e += kThreads) {
                float win[kLen];
#pragma unroll
                for (int j = 0; j < kLen; ++j) win[j] = s_x[e + j * d];
                pool(win);
            }
        }
    } else {
    constexpr int kStep = 4;   // rows fetched ahead of their use: their loads are in flight together
    for (int u = threadIdx.x; u < n_units; u += kThreads) {
        const int seg = u / d, r = u - seg * d;
        const int t_a = seg * rows_per_seg, t_b = min(T, t_a + rows_per_seg);
        // every position of the walk fits 32 bits: (T + 8) d <= L + 9 d
        float win[kLen];
        int pos = (t_a - 4) * d + r;                 // the sample the next window entry comes from
#pragma unroll
        for (int j = 0; j < kLen - 1; ++j) { win[j + 1] = sample_at(pos); pos += d; }
        int i = t_a * d + r;                         // the output the window is centred on next
        for (int t0 = t_a; t0 < t_b; t0 += kStep) {
            float nxt[kStep];
#pragma unroll
            for (int k = 0; k < kStep; ++k) { nxt[k] = sample_at(pos); pos += d; }
#pragma unroll
            for (int k = 0; k < kStep; ++k) {
#pragma unroll
                for (int j = 0; j < kLen - 1; ++j) win[j] = win[j + 1];
                win[kLen - 1] = nxt[k];
                if (t0 + k < t_b && i >= first && i < last) pool(win);
                i += d;
            }
        }
    }
    }
#pragma unroll
    for (int f = 0; f < kMaxFeaturesPerItem; ++f) {
        const int v = __reduce_add_sync(0xffffffffu, cnt[f]);
        if ((threadIdx.x & 31) == 0 && v) atomicAdd(&s_cnt[f], v);
    }
    __syncthreads();
    if (threadIdx.x < it.nf)
        feat[(size_t)n * F + it.f0 + threadIdx.x] = (float)s_cnt[threadIdx.x] / (float)(last - first);   // Eq. 2
}

}  // namespace

struct rocket_mini {
    int C = 0, L = 0, F = 0, n_combos = 0;
    std::vector<int32_t> taps, dilation, kernel_index, padded, num_channels, channel_idx, channel_offset, feature_offset;
    std::vector<double> example_draw, quantile;
    std::vector<float> bias;
    bool fitted = false;
    std::vector<MiniItem> items;
    mutable std::mutex mu;
    mutable int device = -1;
    mutable void* blob = nullptr;          // items, then biases
    mutable const MiniItem* d_items = nullptr;
    mutable float* d_bias = nullptr;
    mutable bool bias_uploaded = false;
};

namespace {

void build_items(rocket_mini& p) {
    p.items.clear();
    for (int c = 0; c < p.n_combos; ++c)
        for (int f0 = p.feature_offset[c]; f0 < p.feature_offset[c + 1]; f0 += kMaxFeaturesPerItem) {
            MiniItem it{};
            it.d = p.dilation[c]; it.padded = p.padded[c]; it.m = p.num_channels[c];
            it.f0 = f0; it.nf = std::min(kMaxFeaturesPerItem, p.feature_offset[c + 1] - f0);
            for (int k = 0; k < 3; ++k) it.tap[k] = p.taps[3 * p.kernel_index[c] + k];
            for (int q = 0; q < it.m; ++q) it.ch[q] = p.channel_idx[p.channel_offset[c] + q];
            p.items.push_back(it);
        }
}

int ensure_mini_device(const rocket_mini* p) {
    std::lock_guard<std::mutex> lk(p->mu);
    if (p->device < 0) {
        int dev = -1;
        if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return ROCKET_ECUDA; }
        const size_t ib = (p->items.size() * sizeof(MiniItem) + 255) / 256 * 256, bb = (size_t)p->F * sizeof(float);
        cudaError_t e = rocket::device_malloc(&p->blob, ib + bb + 256);
        if (e != cudaSuccess) { cudaGetLastError(); p->blob = nullptr; return e == cudaErrorMemoryAllocation ? ROCKET_ENOMEM : ROCKET_ECUDA; }
        if (cudaMemcpy(p->blob, p->items.data(), p->items.size() * sizeof(MiniItem), cudaMemcpyHostToDevice) != cudaSuccess) {
            cudaGetLastError(); cudaFree(p->blob); p->blob = nullptr; return ROCKET_ECUDA;
        }
        p->d_items = static_cast<const MiniItem*>(p->blob);
        p->d_bias = reinterpret_cast<float*>(static_cast<char*>(p->blob) + ib);
        p->device = dev;
        p->bias_uploaded = false;
    }
    if (!p->bias_uploaded) {
        int prev = -1;
        cudaGetDevice(&prev);
        if (prev != p->device) cudaSetDevice(p->device);
        const cudaError_t e = cudaMemcpy(p->d_bias, p->bias.data(), (size_t)p->F * sizeof(float), cudaMemcpyHostToDevice);
        if (prev != p->device) cudaSetDevice(prev);
        if (e != cudaSuccess) { cudaGetLastError(); return ROCKET_ECUDA; }
        p->bias_uploaded = true;
    }
    return ROCKET_OK;
}

}  // namespace

extern "C" {

int rocket_mini_create(uint64_t seed, int C, int L, int num_features, rocket_mini_t** out) {
    if (!out || C < 1 || L < kLen || num_features < kKernels) return ROCKET_EINVAL;
    rocket_mini* p = new (std::nothrow) rocket_mini();
    if (!p) return ROCKET_ENOMEM;
    try {
        p->C = C; p->L = L; p->F = (num_features / kKernels) * kKernels;
        for (int a = 0; a < kLen; ++a)
            for (int b = a + 1; b < kLen; ++b)
                for (int c = b + 1; c < kLen; ++c) { p->taps.push_back(a); p->taps.push_back(b); p->taps.push_back(c); }
        // dilations and the share of every kernel's features each of them holds
        const int fpk = p->F / kKernels, n = std::min(fpk, 32);
        const double E = std::log2((L - 1.0) / 8.0);
        std::vector<int64_t> dil;
        std::vector<int64_t> count;
        for (int k = 0; k < n; ++k) {
            const double x = n > 1 ? k * E / (n - 1) : 0.0;
            const int64_t d = (int64_t)std::floor(std::exp2(x));
            if (!dil.empty() && dil.back() == d) ++count.back();
            else { dil.push_back(d); count.push_back(1); }
        }
        std::vector<int> share(dil.size());
        int left = fpk;
        for (size_t i = 0; i < dil.size(); ++i) { share[i] = (int)std::floor(count[i] * ((double)fpk / n)); left -= share[i]; }
        for (size_t i = 0; left > 0; i = (i + 1) % dil.size()) { ++share[i]; --left; }
        p->n_combos = (int)dil.size() * kKernels;
        p->channel_offset.assign(1, 0);
        p->feature_offset.assign(1, 0);
        const int cap = std::min(C, kLen);
        std::vector<uint64_t> keys(C);
        std::vector<int> order(C);
        for (int c = 0; c < p->n_combos; ++c) {
            const int i_d = c / kKernels, kappa = c % kKernels;
            const uint64_t stream = (uint64_t)c + kStreamBase;
            int m = (int)std::floor(std::exp2(draw_uniform(seed, stream, 0) * std::log2(cap + 1.0)));
            m = std::max(1, std::min(m, cap));
            for (int ch = 0; ch < C; ++ch) keys[ch] = draw_u64(seed, stream, 1024 + (uint64_t)ch);
            std::iota(order.begin(), order.end(), 0);
            std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return keys[a] < keys[b]; });
            std::vector<int> chosen(order.begin(), order.begin() + m);
            std::sort(chosen.begin(), chosen.end());
            for (int ch : chosen) p->channel_idx.push_back(ch);
            p->dilation.push_back((int32_t)dil[i_d]); p->kernel_index.push_back(kappa);
            p->padded.push_back((i_d + kappa) % 2 == 0 ? 1 : 0); p->num_channels.push_back(m);
            p->channel_offset.push_back((int32_t)p->channel_idx.size());
            p->feature_offset.push_back(p->feature_offset.back() + share[i_d]);
            p->example_draw.push_back(draw_uniform(seed, stream, 1));
        }
        p->quantile.resize(p->F);
        for (int f = 0; f < p->F; ++f) p->quantile[f] = std::fmod((f + 1.0) * kInvGoldenRatio, 1.0);
        p->bias.assign(p->F, 0.0f);
        build_items(*p);
    } catch (const std::bad_alloc&) {
        delete p;
        return ROCKET_ENOMEM;
    }
    *out = p;
    return ROCKET_OK;
}

int rocket_mini_counts(const rocket_mini_t* p, int* C, int* L, int* n_features, int* n_combinations, int64_t* n_channel_idx) {
    if (!p) return ROCKET_EINVAL;
    if (C) *C = p->C;
    if (L) *L = p->L;
    if (n_features) *n_features = p->F;
    if (n_combinations) *n_combinations = p->n_combos;
    if (n_channel_idx) *n_channel_idx = (int64_t)p->channel_idx.size();
    return ROCKET_OK;
}

int rocket_mini_host_view(const rocket_mini_t* p, const int32_t** taps, const int32_t** dilation, const int32_t** kernel_index,
                          const int32_t** padded, const int32_t** num_channels, const int32_t** channel_idx,
                          const int32_t** feature_offset, const double** example_draw, const double** quantile,
                          const float** bias) {
    if (!p) return ROCKET_EINVAL;
    if (taps) *taps = p->taps.data();
    if (dilation) *dilation = p->dilation.data();
    if (kernel_index) *kernel_index = p->kernel_index.data();
    if (padded) *padded = p->padded.data();
    if (num_channels) *num_channels = p->num_channels.data();
    if (channel_idx) *channel_idx = p->channel_idx.data();
    if (feature_offset) *feature_offset = p->feature_offset.data();
    if (example_draw) *example_draw = p->example_draw.data();
    if (quantile) *quantile = p->quantile.data();
    if (bias) *bias = p->bias.data();
    return ROCKET_OK;
}

int rocket_mini_fit(rocket_mini_t* p, const float* X_host, int N) {
    if (!p || !X_host || N < 1) return ROCKET_EINVAL;
    const int L = p->L, C = p->C;
    std::vector<float> bias(p->F);
    const unsigned hw = std::max(1u, std::min(32u, std::thread::hardware_concurrency()));
    std::vector<std::thread> pool;
    std::atomic<int> next{0};
    std::atomic<bool> failed{false};
    auto worker = [&]() {
        try {
            std::vector<double> xs(L), z;
            for (int c = next.fetch_add(1); c < p->n_combos; c = next.fetch_add(1)) {
                const int n = std::min((int)(p->example_draw[c] * N), N - 1);
                const float* Xn = X_host + (size_t)n * C * L;
                const int d = p->dilation[c];
                std::fill(xs.begin(), xs.end(), 0.0);
                for (int q = p->channel_offset[c]; q < p->channel_offset[c + 1]; ++q) {
                    const float* x = Xn + (size_t)p->channel_idx[q] * L;
                    for (int i = 0; i < L; ++i) xs[i] += (double)x[i];
                }
                const int32_t* tap = p->taps.data() + 3 * p->kernel_index[c];
                const int first = p->padded[c] ? 0 : 4 * d, last = p->padded[c] ? L : L - 4 * d;
                z.resize(last - first);
                for (int i = first; i < last; ++i) {
                    double v = 0.0;
                    for (int j = 0; j < kLen; ++j) {
                        const long long t = (long long)i + (long long)(j - 4) * d;
                        if (t >= 0 && t < L) v += ((j == tap[0] || j == tap[1] || j == tap[2]) ? 2.0 : -1.0) * xs[t];
                    }
                    z[i - first] = v;
                }
                std::sort(z.begin(), z.end());
                const long long nz = (long long)z.size();
                for (int f = p->feature_offset[c]; f < p->feature_offset[c + 1]; ++f) {
                    const double pos = p->quantile[f] * (double)(nz - 1);
                    const long long lo = (long long)std::floor(pos), hi = std::min(lo + 1, nz - 1);
                    bias[f] = (float)(z[lo] + (pos - (double)lo) * (z[hi] - z[lo]));
                }
            }
        } catch (...) {
            failed = true;
        }
    };
    try {
        for (unsigned t = 0; t < hw; ++t) pool.emplace_back(worker);
    } catch (...) {
        failed = failed || pool.empty();
    }
    for (auto& t : pool) t.join();
    if (failed) return ROCKET_ENOMEM;
    std::lock_guard<std::mutex> lk(p->mu);
    p->bias.swap(bias);
    p->fitted = true;
    p->bias_uploaded = false;
    return ROCKET_OK;
}

int rocket_mini_set_biases(rocket_mini_t* p, const float* bias) {
    if (!p || !bias) return ROCKET_EINVAL;
    for (int f = 0; f < p->F; ++f)
        if (!(bias[f] - bias[f] == 0.0f)) return ROCKET_EINVAL;
    std::lock_guard<std::mutex> lk(p->mu);
    p->bias.assign(bias, bias + p->F);
    p->fitted = true;
    p->bias_uploaded = false;
    return ROCKET_OK;
}

int rocket_mini_transform(const rocket_mini_t* p, const float* X_dev, int N, int C, int L, float* feat_dev, void* cuda_stream) {
    if (!p || N < 0) return ROCKET_EINVAL;
    if (C != p->C || L != p->L) return ROCKET_ESHAPE;
    if (!p->fitted) return ROCKET_EINVAL;
    if (N == 0) return ROCKET_OK;
    if (!X_dev || !feat_dev) return ROCKET_EINVAL;
    const long long blocks = (long long)N * (long long)p->items.size();
    if (blocks > 0x7fffffffll) return ROCKET_EUNSUPPORTED;
    const int st = ensure_mini_device(p);
    if (st != ROCKET_OK) return st;
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) { cudaGetLastError(); return ROCKET_ECUDA; }
    if (prev != p->device && cudaSetDevice(p->device) != cudaSuccess) { cudaGetLastError(); return ROCKET_ECUDA; }
    mini_transform_kernel<<<(unsigned)blocks, kThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        X_dev, C, L, p->d_items, (int)p->items.size(), p->d_bias, feat_dev, p->F);
    rocket::count_launch();
    const cudaError_t e = cudaGetLastError();
    if (prev != p->device) cudaSetDevice(prev);
    if (e != cudaSuccess) { cudaGetLastError(); return ROCKET_ECUDA; }
    return ROCKET_OK;
}

void rocket_mini_destroy(rocket_mini_t* p) {
    if (!p) return;
    if (p->device >= 0 && p->blob) {
        int prev = -1;
        cudaGetDevice(&prev);
        if (prev != p->device) cudaSetDevice(p->device);
        cudaFree(p->blob);
        if (prev >= 0 && prev != p->device) cudaSetDevice(prev);
        cudaGetLastError();
    }
    delete p;
}

}  // extern "C"
