// MINIROCKET on the device (the extension the paper names in Section 6: "the PyTorch GPU implementation could
// be extended to the MINIROCKET model"; Section 2 describes the model: two-valued kernels from a fixed set,
// biases sampled from the input data, PPV as the only pooled feature).
//
//   parameters   built on the host from one seed (rocket_mini_create): 84 kernels of length 9 with three taps
//                of weight 2 and six of weight -1, dilations floor(2^x) spread up to (L - 1) / 8, padding 4 d on
//                every other (dilation, kernel) combination, a random channel subset per combination
//   fit          rocket_mini_fit, on the host (a one-off over one training example per combination): the bias of
//                a feature is a quantile of the combination's convolution output on that example
//   transform    rocket_mini_transform, one fused kernel: per (example, combination) the channels are summed into
//                a shared-memory tile of the dilated view, the nine-tap dilated convolution runs on a register
//                window that slides down a column of the tile, and every output is compared with the
//                combination's biases on the fly, so the convolution outputs never reach memory; feature =
//                count / number of outputs (Eq. 1-2 against the bias)
//
// The kernel weights take two values, so every product is one fused multiply-add with -1 or 2: on this
// hardware an addition and a fused multiply-add take the same issue slot, and the additions-only form that
// speeds the method up on a CPU brings nothing here.  The bound of the kernel is the traffic from L2: every
// combination reads its channels once.
#include <algorithm>
#include <array>
#include <cmath>
#include <map>
#include <mutex>
#include <new>
#include <numeric>
#include <thread>
#include <type_traits>
#include <vector>

#include "rocket_internal.h"

namespace {

constexpr int kKernels = 84, kLen = 9;
constexpr int kMaxFeaturesPerItem = 8;      // a combination with more features becomes several items
constexpr int kThreads = 256;
#ifndef ROCKET_MINI_TILE
#define ROCKET_MINI_TILE (16 * 1024)
#endif
constexpr int kTileSamples = ROCKET_MINI_TILE;
#ifndef ROCKET_MINI_BLOCKS
#define ROCKET_MINI_BLOCKS 3
#endif   // channel-summed samples a block stages at a time (64 KB of shared memory)
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

// One unit of device work: a combination, or a slice of at most 8 of its features, with the tiling of the
// dilated view the kernel uses for its dilation (chosen on the host, choose_tiling).
struct MiniItem {
    int32_t d, padded, m, f0, nf;
    int32_t tap[3];
    int32_t ch[kLen];
    int32_t width, seg_rows, segs;   // columns of a tile (= its pitch), rows a thread walks, such runs per tile
};
static_assert(sizeof(MiniItem) == 80, "MiniItem layout");

// Sample k of a channel row through the read-only path: at a constant byte offset from the row's first sample
// (STRIDE samples apart), or, with a run-time stride, at an address formed by one widening multiply-add.
template <int STRIDE>
__device__ __forceinline__ float load_at(const float* __restrict__ x0, int k, int stride) {
    float v;
    if constexpr (STRIDE != 0) {
        switch (k) {   // k is a constant after unrolling; the offset must be an immediate
            case 0: asm("ld.global.nc.f32 %0, [%1];" : "=f"(v) : "l"(x0)); break;
            case 1: asm("ld.global.nc.f32 %0, [%1+%2];" : "=f"(v) : "l"(x0), "n"(4 * STRIDE)); break;
            case 2: asm("ld.global.nc.f32 %0, [%1+%2];" : "=f"(v) : "l"(x0), "n"(8 * STRIDE)); break;
            case 3: asm("ld.global.nc.f32 %0, [%1+%2];" : "=f"(v) : "l"(x0), "n"(12 * STRIDE)); break;
            case 4: asm("ld.global.nc.f32 %0, [%1+%2];" : "=f"(v) : "l"(x0), "n"(16 * STRIDE)); break;
            case 5: asm("ld.global.nc.f32 %0, [%1+%2];" : "=f"(v) : "l"(x0), "n"(20 * STRIDE)); break;
            case 6: asm("ld.global.nc.f32 %0, [%1+%2];" : "=f"(v) : "l"(x0), "n"(24 * STRIDE)); break;
            default: asm("ld.global.nc.f32 %0, [%1+%2];" : "=f"(v) : "l"(x0), "n"(28 * STRIDE)); break;
        }
    } else {
        const float* p;
        asm("mad.wide.s32 %0, %1, 4, %2;" : "=l"(p) : "r"(k * stride), "l"(x0));
        asm("ld.global.nc.f32 %0, [%1];" : "=f"(v) : "l"(p));
    }
    return v;
}

// One output of the convolution from the nine window entries (the oldest sits in slot S0; taps are taken in
// the order 0..8 whatever the slot), compared with the first 4 NG biases of the item (Eq. 1 against the bias).
template <int S0, int NG>
__device__ __forceinline__ void mini_pool(const float (&win)[kLen], const float (&w)[kLen],
                                          const float (&b)[kMaxFeaturesPerItem], int (&cnt)[kMaxFeaturesPerItem]) {
    float z = 0.0f;
#pragma unroll
    for (int j = 0; j < kLen; ++j) z = fmaf(w[j], win[(S0 + j) % kLen], z);
    // Eq. 1 against every bias: one compare and one predicated add each
#pragma unroll
    for (int f = 0; f < 4 * NG; ++f)
        asm("{ .reg .pred p; setp.gt.f32 p, %1, %2; @p add.s32 %0, %0, 1; }" : "+r"(cnt[f]) : "f"(z), "f"(b[f]));
}

// Steps K .. 8 of a group of nine outputs: the next row's sample enters the slot the oldest one leaves, so
// the window never moves between registers.  GUARD: the run may end inside the group.
template <int K, bool GUARD, int NG>
__device__ __forceinline__ void mini_steps(const float*& p, int pitch, int left, float (&win)[kLen], const float (&w)[kLen],
                                           const float (&b)[kMaxFeaturesPerItem], int (&cnt)[kMaxFeaturesPerItem]) {
    if constexpr (K < kLen) {
        if (!GUARD || K < left) {
            win[(K + kLen - 1) % kLen] = *p;
            p += pitch;
            mini_pool<K, NG>(win, w, b, cnt);
        }
        mini_steps<K + 1, GUARD, NG>(p, pitch, left, win, w, b, cnt);
    }
}

// The walks over one staged tile: thread u of cols * segs takes column u % cols over run u / cols.  Outputs of
// column c are the rows t_min <= t < t_full + (c < c_more): t d + c < last with last = t_full d + c_more.
template <int NG>
__device__ __forceinline__ void mini_walk_tile(const float* s_x, int P, int cols, int rows, int seg_rows, int ta, int ca,
                                               int t_min, int t_full, int c_more, const float (&w)[kLen],
                                               const float (&b)[kMaxFeaturesPerItem], int (&cnt)[kMaxFeaturesPerItem]) {
    const int segs = (rows + seg_rows - 1) / seg_rows;
    // (run, column) of thread u, stepped without divisions: u advances by the block's threads
    const int dq = kThreads / cols, dr = kThreads - dq * cols;
    int seg = threadIdx.x / cols, c = threadIdx.x - seg * cols;
    for (int u = threadIdx.x; u < cols * segs; u += kThreads) {
        const int t_end = t_full + (ca + c < c_more ? 1 : 0);
        const int t_lo = max(ta + seg * seg_rows, t_min);
        const int t_hi = min(min(ta + rows, ta + (seg + 1) * seg_rows), t_end);
        int left = t_hi - t_lo;
        if (left > 0) {
            // the window of output row t holds rows t - 4 .. t + 4; staged row 0 is row ta - 4
            const float* p = s_x + (t_lo - ta) * P + c;
            float win[kLen];
#pragma unroll
            for (int j = 0; j < kLen - 1; ++j) { win[j] = *p; p += P; }
            for (; left >= kLen; left -= kLen) mini_steps<0, false, NG>(p, P, left, win, w, b, cnt);
            if (left > 0) mini_steps<0, true, NG>(p, P, left, win, w, b, cnt);
        }
        seg += dq; c += dr;
        if (c >= cols) { c -= cols; ++seg; }
    }
}

// One block per (example, item).  The series is seen as rows of d samples (A[t][c] = x[t d + c]); a tile of it -
// rows [ta - 4, ta + rows + 4) of `width` columns, channels already summed, zeros outside the series - is
// staged in shared memory, then every thread walks down one column over a run of seg_rows rows with the nine
// taps in registers: one shared-memory load, nine multiply-adds and the bias compares per output.
__global__ void __launch_bounds__(kThreads, ROCKET_MINI_BLOCKS)
mini_transform_kernel(const float* __restrict__ X, int C, int L, const MiniItem* __restrict__ items, int n_items,
                      const float* __restrict__ bias, float* __restrict__ feat, int F) {
    extern __shared__ float s_x[];
    __shared__ int s_cnt[kMaxFeaturesPerItem];
    __shared__ int s_choff[kLen];
    const int n = blockIdx.x / n_items;
    const MiniItem* __restrict__ item = items + (blockIdx.x - n * n_items);
    const MiniItem it = *item;
    const float* __restrict__ Xn = X + (size_t)n * C * L;
    const int tid = threadIdx.x;
    if (tid < kMaxFeaturesPerItem) s_cnt[tid] = 0;
    if (tid < kLen) s_choff[tid] = __ldg(item->ch + (tid < it.m ? tid : 0)) * L;     // C L < 2^31 (checked at creation)
    const int d = it.d, m = it.m, nf = it.nf;
    const int first = it.padded ? 0 : 4 * d, last = it.padded ? L : L - 4 * d;
    float w[kLen];
#pragma unroll
    for (int j = 0; j < kLen; ++j) w[j] = (j == it.tap[0] || j == it.tap[1] || j == it.tap[2]) ? 2.0f : -1.0f;
    float b[kMaxFeaturesPerItem];
#pragma unroll
    for (int f = 0; f < kMaxFeaturesPerItem; ++f) b[f] = f < nf ? __ldg(bias + it.f0 + f) : __int_as_float(0x7f800000);
    int cnt[kMaxFeaturesPerItem];
#pragma unroll
    for (int f = 0; f < kMaxFeaturesPerItem; ++f) cnt[f] = 0;

    const int T = (L + d - 1) / d;                       // rows of the dilated view
    const int P = it.width, seg_rows = it.seg_rows;      // P: columns of a tile and its pitch in shared memory
    const int tile_rows = seg_rows * it.segs;
    const bool whole_rows = P == d;                      // a tile spans whole rows: its samples are one contiguous run
    const int t_min = it.padded ? 0 : 4;                 // rows below hold no output of an unpadded combination
    const int t_full = last / d, c_more = last - t_full * d;   // column c has outputs in rows t < t_full + (c < c_more)
    const int groups = (nf + 3) / 4;

    // NK staged samples per thread at a time: position base + k * stride goes to slot + k * slot_stride.  The
    // channels are taken two at a time, so that 2 NK loads are in flight per thread.  CHECK: a sample may lie
    // beyond the series (then it is zero).  STRIDE = 0: the stride is a run-time value.
    auto stage = [&](auto nk_tag, auto stride_tag, auto check_tag, int base, int stride_rt, int slot, int slot_stride) {
        constexpr int NK = decltype(nk_tag)::value;
        constexpr int STRIDE = decltype(stride_tag)::value;
        constexpr bool CHECK = decltype(check_tag)::value;
        const int stride = STRIDE ? STRIDE : stride_rt;
        float acc[NK];
        bool ok[NK];
#pragma unroll
        for (int k = 0; k < NK; ++k) {
            acc[k] = 0.0f;
            ok[k] = !CHECK || (unsigned)(base + k * stride) < (unsigned)L;
        }
        int q = 0;
        for (; q + 2 <= m; q += 2) {
            const float* __restrict__ x0 = Xn + s_choff[q] + base;
            const float* __restrict__ x1 = Xn + s_choff[q + 1] + base;
            float v0[NK], v1[NK];
#pragma unroll
            for (int k = 0; k < NK; ++k) {
                v0[k] = ok[k] ? load_at<STRIDE>(x0, k, stride) : 0.0f;
                v1[k] = ok[k] ? load_at<STRIDE>(x1, k, stride) : 0.0f;
            }
#pragma unroll
            for (int k = 0; k < NK; ++k) acc[k] = (acc[k] + v0[k]) + v1[k];
        }
        if (q < m) {
            const float* __restrict__ x0 = Xn + s_choff[q] + base;
#pragma unroll
            for (int k = 0; k < NK; ++k)
                if (ok[k]) acc[k] += load_at<STRIDE>(x0, k, stride);
        }
#pragma unroll
        for (int k = 0; k < NK; ++k) s_x[slot + k * slot_stride] = acc[k];
    };
    using Strided = std::integral_constant<int, 0>;
    using Dense = std::integral_constant<int, kThreads>;
    using N8 = std::integral_constant<int, 8>;
    using N4 = std::integral_constant<int, 4>;
    using N2 = std::integral_constant<int, 2>;
    using N1 = std::integral_constant<int, 1>;
    using Checked = std::true_type;
    using Inside = std::false_type;

    for (int ta = 0; ta < T; ta += tile_rows) {
        const int rows = min(tile_rows, T - ta);
        for (int ca = 0; ca < d; ca += P) {
            const int cols = min(P, d - ca);
            __syncthreads();                             // the previous tile's walks are over (and s_choff is written)
            if (whole_rows) {
                // slots [0, count) hold positions g0 .. g0 + count: zeros before the series, the samples in
                // rounds of 8 x 256 and of 256 without any test, one last partial round, zeros after the series
                const int count = (rows + 8) * d, g0 = (ta - 4) * d;
                const int z0 = min(max(-g0, 0), count), z1 = min(max(L - g0, 0), count);
                for (int e = tid; e < z0; e += kThreads) s_x[e] = 0.0f;
                for (int e = z1 + tid; e < count; e += kThreads) s_x[e] = 0.0f;
                int e0 = z0;
                for (; e0 + 8 * kThreads <= z1; e0 += 8 * kThreads) stage(N8{}, Dense{}, Inside{}, g0 + e0 + tid, 0, e0 + tid, kThreads);
                for (; e0 + kThreads <= z1; e0 += kThreads) stage(N1{}, Dense{}, Inside{}, g0 + e0 + tid, 0, e0 + tid, kThreads);
                if (e0 + tid < z1) stage(N1{}, Dense{}, Inside{}, g0 + e0 + tid, 0, e0 + tid, kThreads);
            } else {
                for (int cb = 0; cb < cols; cb += kThreads) {
                    if (cb + tid >= cols) continue;
                    // staged row r is row ta - 4 + r of the view: zeros above the series, rows that lie inside it
                    // for every column of this block without any test, the rows the series ends in, zeros below
                    const int w = min(kThreads, cols - cb), c_lo = ca + cb;
                    const int n_rows = rows + 8;
                    const int r_a = min(max(4 - ta, 0), n_rows);
                    const int t_full = L >= c_lo + w ? (L - c_lo - w) / d + 1 : 0;     // rows t < t_full hold all w columns
                    const int t_some = L > c_lo ? (L - c_lo - 1) / d + 1 : 0;          // rows t < t_some hold at least one
                    const int r_b = min(max(t_full - (ta - 4), r_a), n_rows), r_c = min(max(t_some - (ta - 4), r_b), n_rows);
                    const int pos0 = (ta - 4) * d + c_lo + tid, slot0 = cb + tid;
                    for (int r = 0; r < r_a; ++r) s_x[slot0 + r * P] = 0.0f;
                    int r = r_a;
                    for (; r + 8 <= r_b; r += 8) stage(N8{}, Strided{}, Inside{}, pos0 + r * d, d, slot0 + r * P, P);
                    if (r + 4 <= r_b) { stage(N4{}, Strided{}, Inside{}, pos0 + r * d, d, slot0 + r * P, P); r += 4; }
                    if (r + 2 <= r_b) { stage(N2{}, Strided{}, Inside{}, pos0 + r * d, d, slot0 + r * P, P); r += 2; }
                    if (r + 1 <= r_b) { stage(N1{}, Strided{}, Inside{}, pos0 + r * d, d, slot0 + r * P, P); r += 1; }
                    for (; r < r_c; ++r) stage(N1{}, Strided{}, Checked{}, pos0 + r * d, d, slot0 + r * P, P);
                    for (; r < n_rows; ++r) s_x[slot0 + r * P] = 0.0f;
                }
            }
            __syncthreads();
            static_assert(kMaxFeaturesPerItem == 8, "two groups of four features");
            if (groups == 1) mini_walk_tile<1>(s_x, P, cols, rows, seg_rows, ta, ca, t_min, t_full, c_more, w, b, cnt);
            else mini_walk_tile<2>(s_x, P, cols, rows, seg_rows, ta, ca, t_min, t_full, c_more, w, b, cnt);
        }
    }
#pragma unroll
    for (int f = 0; f < kMaxFeaturesPerItem; ++f) {
        const int v = __reduce_add_sync(0xffffffffu, cnt[f]);
        if ((tid & 31) == 0 && v) atomicAdd(&s_cnt[f], v);
    }
    __syncthreads();
    if (tid < nf) feat[(size_t)n * F + it.f0 + tid] = (float)s_cnt[tid] / (float)(last - first);   // Eq. 2
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

// Tiling of the dilated view for dilation d: the cheapest of the candidates under a simple cost model (staged
// samples, and thread slots of the walks including the ones that idle in a partly filled round of the block).
// Tiles either span whole rows (width = d) or 256-column multiples; runs are multiples of the window length;
// below 32 columns only run lengths that keep the lanes of a warp on different shared-memory banks.
void choose_tiling(int d, int L, int& width, int& seg_rows, int& segs) {
    const int T = (L + d - 1) / d;
    const double c_stage = 17.0, c_walk = 21.0, c_fill = 16.0;
    double best = 1e300;
    width = 0;
    auto consider = [&](int w, int sr, int sg) {
        if ((int64_t)(sg * sr + 8) * w > kTileSamples) return;
        const int tile_rows = sr * sg;
        double cost = 0.0;
        for (int ta = 0; ta < T; ta += tile_rows) {
            const int rows = std::min(tile_rows, T - ta), sgt = (rows + sr - 1) / sr;
            for (int ca = 0; ca < d; ca += w) {
                const int cols = std::min(w, d - ca);
                const double rounds = std::ceil((double)cols * sgt / kThreads);
                cost += (double)(rows + 8) * cols * c_stage + rounds * kThreads * (std::min(sr, rows) * c_walk + c_fill);
            }
        }
        if (cost < best) { best = cost; width = w; seg_rows = sr; segs = sg; }
    };
    for (int sr = kLen; sr <= 7 * kLen; sr += kLen) {
        if (d < 32 && sr != 3 * kLen && sr != 7 * kLen) continue;
        const int max_segs = std::max(1, (T + sr - 1) / sr);
        for (int sg = 1; sg <= max_segs; sg = sg < 8 ? sg + 1 : sg * 2) consider(d, sr, sg);
        consider(d, sr, max_segs);
        if (kTileSamples / d - 8 >= sr) consider(d, sr, std::min(max_segs, (kTileSamples / d - 8) / sr));
        for (int w = kThreads; w < d; w += kThreads)
            for (int sg = 1; sg <= std::min(max_segs, 4); ++sg) consider(w, sr, sg);
    }
}

// false when a dilation has no tiling that fits the shared-memory tile (cannot happen for L >= 9; checked all the same)
bool build_items(rocket_mini& p) {
    p.items.clear();
    std::map<int, std::array<int, 3>> tiling;           // by dilation
    for (int c = 0; c < p.n_combos; ++c)
        for (int f0 = p.feature_offset[c]; f0 < p.feature_offset[c + 1]; f0 += kMaxFeaturesPerItem) {
            MiniItem it{};
            it.d = p.dilation[c]; it.padded = p.padded[c]; it.m = p.num_channels[c];
            it.f0 = f0; it.nf = std::min(kMaxFeaturesPerItem, p.feature_offset[c + 1] - f0);
            for (int k = 0; k < 3; ++k) it.tap[k] = p.taps[3 * p.kernel_index[c] + k];
            for (int q = 0; q < it.m; ++q) it.ch[q] = p.channel_idx[p.channel_offset[c] + q];
            auto found = tiling.find(it.d);
            if (found == tiling.end()) {
                std::array<int, 3> t{};
                choose_tiling(it.d, p.L, t[0], t[1], t[2]);
                if (t[0] < 1 || t[1] < kLen || t[2] < 1 || (int64_t)(t[1] * t[2] + 8) * t[0] > kTileSamples) return false;
                found = tiling.emplace(it.d, t).first;
            }
            it.width = found->second[0]; it.seg_rows = found->second[1]; it.segs = found->second[2];
            p.items.push_back(it);
        }
    return true;
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
        if (cudaFuncSetAttribute(mini_transform_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)(kTileSamples * sizeof(float))) != cudaSuccess) {
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
    if ((int64_t)C * L > 0x7fffffffll) return ROCKET_EUNSUPPORTED;     // positions within an example are 32-bit
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
            // a power that is an integer (the last one is (L - 1) / 8) must not fall below it by exp2's rounding
            const int64_t d = (int64_t)std::floor(std::exp2(x) * (1.0 + 0x1.0p-40));
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
        if (!build_items(*p)) {
            delete p;
            return ROCKET_EUNSUPPORTED;
        }
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
    mini_transform_kernel<<<(unsigned)blocks, kThreads, kTileSamples * sizeof(float), static_cast<cudaStream_t>(cuda_stream)>>>(
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
