// Random kernel initialisation (Section 3.1) on the host: a counter-based generator so that
// kernel k is a pure function of (seed, k, C, L).
#include <algorithm>
#include <cmath>
#include <numeric>

#include "rocket_internal.h"

namespace rocket {
namespace {

constexpr uint64_t kGolden = 0x9E3779B97F4A7C15ull;

// splitmix64 finaliser
inline uint64_t mix(uint64_t z) {
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

enum : uint64_t { kSlotLength = 0, kSlotDilation = 1, kSlotPadding = 2, kSlotChannels = 3, kSlotBias = 4,
                  kSlotWeights = 64, kSlotChannelKeys = 1024 };

}  // namespace

void generate_host_params(uint64_t seed, int K, int C, int L, HostParams& hp) {
    hp = HostParams();
    hp.K = K; hp.C = C; hp.L = L;
    hp.length.resize(K); hp.dilation.resize(K); hp.padding.resize(K); hp.num_channels.resize(K);
    hp.bias.resize(K);
    const double kTwoPi = 6.283185307179586476925286766559;
    std::vector<uint64_t> keys(C);
    std::vector<int> order(C);
    for (int k = 0; k < K; ++k) {
        const uint64_t s = static_cast<uint64_t>(k);
        const int len = 7 + 2 * std::min(static_cast<int>(draw_uniform(seed, s, kSlotLength) * 3.0), 2);
        const double hi = std::log2((L - 1.0) / (len - 1.0));
        long long d = static_cast<long long>(std::floor(std::exp2(draw_uniform(seed, s, kSlotDilation) * hi)));
        d = std::max(1ll, std::min<long long>(d, (L - 1) / (len - 1)));
        const int pad = draw_uniform(seed, s, kSlotPadding) < 0.5 ? static_cast<int>(((len - 1) * d) / 2) : 0;
        const int cap = std::min(C, len);
        int m = static_cast<int>(std::floor(std::exp2(draw_uniform(seed, s, kSlotChannels) * std::log2(cap + 1.0))));
        m = std::max(1, std::min(m, cap));
        hp.length[k] = len; hp.dilation[k] = static_cast<int32_t>(d); hp.padding[k] = pad; hp.num_channels[k] = m;
        hp.bias[k] = static_cast<float>(2.0 * draw_uniform(seed, s, kSlotBias) - 1.0);

        // channel subset: the m smallest of C random keys, reported in ascending channel order
        for (int c = 0; c < C; ++c) keys[c] = draw_u64(seed, s, kSlotChannelKeys + c);
        std::iota(order.begin(), order.end(), 0);
        std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return keys[a] < keys[b]; });
        std::vector<int> chosen(order.begin(), order.begin() + m);
        std::sort(chosen.begin(), chosen.end());
        for (int c : chosen) hp.channel_idx.push_back(c);

        // weights: Box-Muller in fp64, mean-centred per channel row, rounded once to fp32
        for (int q = 0; q < m; ++q) {
            double row[ROCKET_MAX_LENGTH];
            double sum = 0.0;
            for (int j = 0; j < len; ++j) {
                const uint64_t slot = kSlotWeights + 2ull * (static_cast<uint64_t>(q) * ROCKET_MAX_LENGTH + j);
                const double u1 = (static_cast<double>(draw_u64(seed, s, slot) >> 11) + 1.0) * 0x1.0p-53;
                const double u2 = draw_uniform(seed, s, slot + 1);
                row[j] = std::sqrt(-2.0 * std::log(u1)) * std::cos(kTwoPi * u2);
                sum += row[j];
            }
            const double mean = sum / len;
            for (int j = 0; j < len; ++j) hp.weights.push_back(static_cast<float>(row[j] - mean));
        }
    }
}

}  // namespace rocket
