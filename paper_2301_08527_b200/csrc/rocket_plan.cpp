// Host-side launch plan of the fast path: buckets kernels by dilation, lays out band rasters,
// cuts them into tiles and orders the tiles by cost (largest first) for the persistent kernels.
#include <algorithm>
#include <map>

#include "rocket_fast.h"

namespace rocket {
namespace fast {
namespace {

inline int64_t floor_div(int64_t a, int64_t b) { return (a >= 0) ? a / b : -((-a + b - 1) / b); }

}  // namespace

void build_plan(const HostParams& hp, int split, PlanHost& out) {
    out = PlanHost();
    if (split < 64) split = 64;  // T tiles need d >= 64 so that a 128-column tile spans at most 3 bands
    out.split = split;
    const int K = hp.K;
    // The fast kernels want 16-byte aligned channel rows (bulk copies) and at most
    // kSMaxChannels channels in an S tile.
    const bool shape_ok = (hp.L % 4 == 0) && hp.C <= kSMaxChannels && hp.L >= 16;
    std::vector<int> s_kernels, t_kernels;
    for (int k = 0; k < K; ++k) {
        const int len = hp.length[k], d = hp.dilation[k];
        const bool fast_len = (len == 7 || len == 9 || len == 11);
        if (!shape_ok || !fast_len) out.generic_list.push_back(k);
        else if (d < split) s_kernels.push_back(k);
        else t_kernels.push_back(k);
    }
    out.enabled = !(s_kernels.empty() && t_kernels.empty());
    if (!out.enabled) return;

    auto add_kernel = [&](int k) {
        FastKernel f{};
        f.len = hp.length[k]; f.d = hp.dilation[k]; f.p = hp.padding[k]; f.m = hp.num_channels[k];
        f.nout = (int32_t)((int64_t)hp.L + 2 * (int64_t)f.p - (int64_t)(f.len - 1) * f.d);
        f.woff = (int32_t)out.negw.size();
        f.k = k; f.lo_u = -f.p; f.hi_u = f.nout - f.p;
        f.negb = 0.0f - hp.bias[k];
        const int32_t* S = hp.channel_idx.data() + hp.channel_offset[k];
        const float* W = hp.weights.data() + hp.weight_offset[k];
        // weights of fast kernel i live at negw[i * kWeightsPerKernel], rows padded to kWeightRow
        out.negw.resize(out.negw.size() + kWeightsPerKernel, 0.0f);
        for (int q = 0; q < f.m; ++q) {
            f.ch[q] = S[q];
            for (int j = 0; j < f.len; ++j) out.negw[f.woff + q * kWeightRow + j] = 0.0f - W[q * f.len + j];
        }
        out.fk.push_back(f);
    };

    // ---- S regime: one bucket per dilation, kernels inside ordered by cost (largest first)
    std::map<int, std::vector<int>> by_d;
    for (int k : s_kernels) by_d[hp.dilation[k]].push_back(k);
    struct Cost { double c; int idx; };
    std::vector<Cost> s_cost;
    for (auto& kv : by_d) {
        const int d = kv.first;
        auto& ks = kv.second;
        std::stable_sort(ks.begin(), ks.end(), [&](int a, int b) {
            return hp.length[a] * hp.num_channels[a] > hp.length[b] * hp.num_channels[b];
        });
        SBucket b{};
        b.d = d; b.kbeg = (int32_t)out.fk.size();
        int64_t tmin = INT64_MAX, tmax = INT64_MIN;
        int maxlen = 0;
        double work = 0.0;
        for (int k : ks) {
            add_kernel(k);
            const FastKernel& f = out.fk.back();
            tmin = std::min(tmin, floor_div(f.lo_u, d));
            tmax = std::max(tmax, floor_div((int64_t)f.hi_u - 1, d));
            maxlen = std::max(maxlen, f.len);
            work += (double)f.len * f.m;
        }
        b.kend = (int32_t)out.fk.size();
        b.tmin = (int32_t)tmin;
        b.nbands = (int32_t)((tmax - tmin + 1 + kBandRows - 1) / kBandRows);
        b.raster_len = b.nbands * d;
        b.rows = kBandRows + maxlen - 1;
        const int bi = (int)out.sb.size();
        out.sb.push_back(b);
        for (int c0 = 0; c0 < b.raster_len; c0 += kSCols) {
            s_cost.push_back({work + 0.02 * hp.C * b.rows, (int)out.sitems.size()});
            out.sitems.push_back({bi, c0});
        }
    }
    {
        std::stable_sort(s_cost.begin(), s_cost.end(), [](const Cost& a, const Cost& b) { return a.c > b.c; });
        std::vector<SItem> sorted;
        sorted.reserve(out.sitems.size());
        for (auto& c : s_cost) sorted.push_back(out.sitems[c.idx]);
        out.sitems.swap(sorted);
    }

    // ---- T regime: per kernel, full bands of 32 rows and one tail band of 8/16/24/32 rows
    std::vector<Cost> t_cost;
    for (int k : t_kernels) {
        const int fi = (int)out.fk.size();
        add_kernel(k);
        const FastKernel f = out.fk.back();
        const int64_t tmin = floor_div(f.lo_u, f.d), tmax = floor_div((int64_t)f.hi_u - 1, f.d);
        const int64_t rows = tmax - tmin + 1;
        const int64_t nb = rows / kBandRows, rem = rows % kBandRows;
        auto add_group = [&](int64_t t0, int R, int64_t raster_len) {
            for (int64_t c0 = 0; c0 < raster_len; c0 += kTCols) {
                TItem it{};
                it.fk = fi; it.t0 = (int32_t)t0; it.R = R; it.c0 = (int32_t)c0; it.raster_len = (int32_t)raster_len;
                t_cost.push_back({(double)f.len * f.m * (R + 3.0) + 40.0, (int)out.titems.size()});
                out.titems.push_back(it);
            }
        };
        if (nb > 0) add_group(tmin, kBandRows, nb * f.d);
        if (rem > 0) add_group(tmin + nb * kBandRows, (int)((rem + 7) / 8 * 8), f.d);
    }
    {
        std::stable_sort(t_cost.begin(), t_cost.end(), [](const Cost& a, const Cost& b) { return a.c > b.c; });
        std::vector<TItem> sorted;
        sorted.reserve(out.titems.size());
        for (auto& c : t_cost) sorted.push_back(out.titems[c.idx]);
        out.titems.swap(sorted);
    }
}

}  // namespace fast
}  // namespace rocket
