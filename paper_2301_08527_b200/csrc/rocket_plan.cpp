// Host-side launch plan of the fast path: buckets kernels by dilation, lays out band rasters,
// cuts them into tiles and orders the tiles by cost (largest first).
#include <algorithm>
#include <map>
#include <tuple>

#include "rocket_fast.h"
#include "rocket_fast_geom.h"

namespace rocket {
namespace fast {
namespace {

inline int64_t floor_div(int64_t a, int64_t b) { return (a >= 0) ? a / b : -((-a + b - 1) / b); }

}  // namespace

void fill_record_weights(const HostParams& hp, KRec& f) {
    const float* W = hp.weights.data() + hp.weight_offset[f.k];
    f.negb = 0.0f - hp.bias[f.k];
    for (int q = 0; q < f.m; ++q)
        for (int j = 0; j < f.len; ++j) f.w2[q][2 * j] = f.w2[q][2 * j + 1] = 0.0f - W[q * f.len + j];
}

void build_plan(const HostParams& hp, int split, PlanHost& out) {
    out = PlanHost();
    out.flops_s = out.flops_t = 0.0;
    if (split < kTMinDilation) split = kTMinDilation;
    out.split = split;
    const int K = hp.K;
    // The fast kernels stage at most kSMaxChannels channels in an S tile.  Any series length will do: the
    // small-dilation kernel copies single floats and the large-dilation kernel reads the zero-margined
    // copies, whose pitch does not depend on L.
    const bool shape_ok = hp.C <= kSMaxChannels && hp.L >= 16;
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
        KRec f{};
        f.len = hp.length[k]; f.d = hp.dilation[k]; f.p = hp.padding[k]; f.m = hp.num_channels[k];
        f.nout = (int32_t)((int64_t)hp.L + 2 * (int64_t)f.p - (int64_t)(f.len - 1) * f.d);
        f.k = k; f.lo_u = -f.p; f.hi_u = f.nout - f.p;
        f.woff = hp.weight_offset[k];
        f.tl = (int32_t)floor_div(f.lo_u, f.d); f.rl = f.lo_u - f.tl * f.d;
        f.th = (int32_t)floor_div(f.hi_u, f.d); f.rh = f.hi_u - f.th * f.d;
        const int32_t* S = hp.channel_idx.data() + hp.channel_offset[k];
        for (int q = 0; q < f.m; ++q) f.ch[q] = S[q];
        fill_record_weights(hp, f);
        out.krec.push_back(f);
    };

    // ---- S regime: one bucket per dilation, kernels inside ordered by cost (largest first: the warps of a
    // block pull them one by one, so the cheap ones fill the end of a tile evenly).  Buckets with many
    // kernels per warp are ordered by length first: warps that run side by side then share one instance of
    // the inner loops, which the instruction caches reward (backward 5 % faster, hard transform unchanged;
    // for the small buckets the balance at the end of a tile is worth more).
    std::map<int, std::vector<int>> by_d;
    for (int k : s_kernels) by_d[hp.dilation[k]].push_back(k);
    struct Cost { double c; int idx; };
    std::vector<Cost> s_cost;
    for (auto& kv : by_d) {
        const int d = kv.first;
        auto& ks = kv.second;
        std::stable_sort(ks.begin(), ks.end(), [&](int a, int b) {
            if ((int)ks.size() >= kSLengthOrderMin && hp.length[a] != hp.length[b]) return hp.length[a] > hp.length[b];
            return hp.length[a] * hp.num_channels[a] > hp.length[b] * hp.num_channels[b];
        });
        SBucket b{};
        b.d = d; b.kbeg = (int32_t)out.krec.size();
        int64_t tmin = INT64_MAX, tmax = INT64_MIN;
        int maxlen = 0;
        double work = 0.0;
        for (int k : ks) {
            add_kernel(k);
            const KRec& f = out.krec.back();
            out.flops_s += 2.0 * f.len * f.m * (double)f.nout;
            tmin = std::min(tmin, floor_div(f.lo_u, d));
            tmax = std::max(tmax, floor_div((int64_t)f.hi_u - 1, d));
            maxlen = std::max(maxlen, f.len);
            work += (double)f.m * (f.len + 2) + 6.0;
        }
        b.kend = (int32_t)out.krec.size();
        b.tmin = (int32_t)tmin;
        b.nbands = (int32_t)((tmax - tmin + 1 + kRS - 1) / kRS);
        b.raster_len = b.nbands * d;
        b.rows = kRS + maxlen - 1;
        const int bi = (int)out.sb.size();
        out.sb.push_back(b);
        // a tile is interior when its 64 raster positions exist and the u of every (row, column) lies inside
        // the output range of every kernel of the bucket
        int64_t lo_max = INT64_MIN, hi_min = INT64_MAX;
        for (int f = b.kbeg; f < b.kend; ++f) {
            lo_max = std::max<int64_t>(lo_max, out.krec[f].lo_u);
            hi_min = std::min<int64_t>(hi_min, out.krec[f].hi_u);
        }
        for (int c0 = 0; c0 < b.raster_len; c0 += kWarpCols) {
            bool interior = c0 + kWarpCols <= b.raster_len;
            for (int c = c0; interior && c < c0 + kWarpCols; ++c) {
                const int64_t u0 = s_column_u0(b, c);
                interior = u0 >= lo_max && u0 + (int64_t)(kRS - 1) * d < hi_min;
            }
            s_cost.push_back({work + 0.3 * hp.C * b.rows, (int)out.sitems.size()});
            out.sitems.push_back({bi, c0, interior ? 1 : 0, 0});
        }
    }
    {
        std::stable_sort(s_cost.begin(), s_cost.end(), [](const Cost& a, const Cost& b) { return a.c > b.c; });
        std::vector<SItem> sorted;
        sorted.reserve(out.sitems.size());
        for (auto& c : s_cost) sorted.push_back(out.sitems[c.idx]);
        out.sitems.swap(sorted);
    }

    // ---- T regime: per kernel, the grid of 16-row x 64-column warp tiles is cut into block tiles of
    // rg x cg warp tiles (rg * cg <= the consumer warps of a block); the column-group width that needs the
    // fewest block tiles wins
    int d_max = 0;
    std::map<std::tuple<int, int, int>, int> map_index;
    // kernels of one length follow one another, so that the blocks running at any one time execute the same
    // instance of the inner loops (instruction caches: backward 3.5 % faster, forward 0.1-1 %)
    std::stable_sort(t_kernels.begin(), t_kernels.end(), [&](int a, int b) { return hp.length[a] > hp.length[b]; });
    for (int k : t_kernels) {
        const int ki = (int)out.krec.size();
        add_kernel(k);
        const KRec f = out.krec.back();
        out.flops_t += 2.0 * f.len * f.m * (double)f.nout;
        d_max = std::max(d_max, f.d);
        const int64_t tmin = floor_div(f.lo_u, f.d);
        const int64_t tmax = floor_div((int64_t)f.hi_u - 1, f.d);
        const int R16 = (int)((tmax - tmin + 1 + kR - 1) / kR), C64 = (f.d + kWarpCols - 1) / kWarpCols;
        // column chunks for a main width cg: C64 / cg chunks of cg, the rest in chunks of 2 and 1
        auto chunks_of = [&](int cg, std::vector<int>& widths) {
            widths.assign(C64 / cg, cg);
            int rest = C64 % cg;
            if (rest >= 2) { widths.push_back(2); rest -= 2; }
            if (rest >= 1) widths.push_back(1);
        };
        constexpr int W = kTConsumerWarps;
        // A single row group under tiles narrower than the block has warps would leave warps idle: it can be cut
        // into wide tiles instead (all consumer warps side by side, only the rows that hold samples), as long
        // as the halves fit a stage.
        auto wide_fits = [&](int r16) {
            const TWindow win = t_window((int)(tmin + (int64_t)kR * r16), kR + f.len - 1, f.d, hp.L);
            return C64 > W / 2 && kTWideHalves * t_wide_half_floats(win.g_hi - win.g_lo) <= kTStageFloats;
        };
        // widths of the tiles of a wide band: W column groups each, the rest in ordinary tiles of one row group
        std::vector<int> wide_widths(C64 / W, W);
        {
            int rest = C64 % W;
            if (rest > W / 2) { wide_widths.push_back(W); rest = 0; }
            if (W > 4 && rest >= 3) { wide_widths.push_back(4); rest = 0; }
            if (rest >= 2) { wide_widths.push_back(2); rest -= 2; }
            if (rest >= 1) wide_widths.push_back(1);
        }
        // candidates: main width 2, 4 or 1 over all row groups, or the widest main width over all row groups
        // but the last and wide tiles over that one; the fewest block tiles win
        int best_cg = 2;
        bool last_wide = false;
        int64_t best_tiles = INT64_MAX;
        for (int cg : {2, 4, 1}) {
            if (cg > kTMaxCg) continue;
            std::vector<int> widths;
            chunks_of(cg, widths);
            int64_t tiles = 0;
            for (int w : widths) tiles += (R16 + W / w - 1) / (W / w);
            if (tiles < best_tiles) { best_tiles = tiles; best_cg = cg; }
        }
        if (R16 % 2 == 1 && wide_fits(R16 - 1)) {
            std::vector<int> widths;
            chunks_of(kTMaxCg, widths);
            int64_t tiles = (int64_t)wide_widths.size();
            for (int w : widths) tiles += (R16 - 1 + W / w - 1) / (W / w);
            if (tiles < best_tiles) { best_tiles = tiles; best_cg = kTMaxCg; last_wide = true; }
        }
        struct Band { int r16, nrg; std::vector<int> widths; bool wide_band; };
        std::vector<Band> bands;
        std::vector<int> main_widths;
        chunks_of(best_cg, main_widths);
        const int main_rows = last_wide ? R16 - 1 : R16;
        if (main_rows > 0) bands.push_back({0, main_rows, main_widths, false});
        if (last_wide) bands.push_back({R16 - 1, 1, wide_widths, true});
        for (const Band& band : bands) {
            int c64 = 0;
            for (int w : band.widths) {
                const bool wide_tile = band.wide_band && w == W;
                const int rg_full = wide_tile ? 1 : W / w;
                for (int r16 = band.r16; r16 < band.r16 + band.nrg; r16 += rg_full) {
                    TItem it{};
                    it.rg = std::min(rg_full, band.r16 + band.nrg - r16);
                    it.wide = wide_tile ? 1 : 0;
                    it.cg = it.wide ? 4 : w;
                    it.t0 = (int32_t)(tmin + (int64_t)kR * r16); it.r0 = c64 * kWarpCols;
                    // a tile none of whose (row, column) pairs is an output of the kernel is left out
                    bool any_output = false;
                    for (int t = it.t0; t < it.t0 + kR * it.rg && !any_output; ++t) {
                        const int64_t c_lo = std::max<int64_t>(it.r0, (int64_t)f.lo_u - (int64_t)t * f.d);
                        const int64_t c_hi = std::min<int64_t>(std::min(it.r0 + kWarpCols * w, f.d), (int64_t)f.hi_u - (int64_t)t * f.d);
                        any_output = c_lo < c_hi;
                    }
                    if (!any_output) continue;
                    it.d = f.d; it.len = f.len; it.m = f.m;
                    const TWindow win = t_window(it.t0, kR + f.len - 1, f.d, hp.L);
                    it.g_lo = it.wide ? win.g_lo : 0;
                    it.g_hi = it.wide ? win.g_hi : t_box_rows(it.rg, f.len);
                    it.box_rows = it.g_hi - it.g_lo;
                    for (int q = 0; q < f.m; ++q) it.ch[q] = (uint8_t)f.ch[q];
                    it.krec = ki;
                    const auto key = std::make_tuple(f.d, t_box_cols(it.cg), it.box_rows);
                    auto found = map_index.find(key);
                    if (found == map_index.end()) {
                        found = map_index.emplace(key, (int)out.tmaps.size()).first;
                        out.tmaps.push_back({f.d, t_box_cols(it.cg), it.box_rows});
                    }
                    it.map = found->second;
                    // per consumer warp: does every / any (row, column) of its warp tile hold an output?
                    for (int w8 = 0; w8 < kTConsumerWarps; ++w8) {
                        const int wr = it.wide ? 0 : w8 / it.cg, wc = it.wide ? w8 : w8 % it.cg;
                        if (wr >= it.rg) continue;
                        const int64_t ta = (int64_t)it.t0 + kR * wr, ca = (int64_t)it.r0 + kWarpCols * wc;
                        const int64_t cb = std::min<int64_t>(ca + kWarpCols, f.d);
                        if (cb <= ca) continue;
                        bool any = false;
                        for (int64_t t = ta; t < ta + kR && !any; ++t)
                            any = std::max<int64_t>(t * f.d + ca, f.lo_u) < std::min<int64_t>(t * f.d + cb, f.hi_u);
                        if (any) it.warp_active |= 1 << w8;
                        if (cb == ca + kWarpCols && ta * f.d + ca >= f.lo_u && (ta + kR - 1) * f.d + cb - 1 < f.hi_u)
                            it.warp_interior |= 1 << w8;
                    }
                    for (int ph = 0; ph < 4; ++ph) {
                        const TPhase tp = t_phase(it.t0, it.r0, it.d, ph);
                        it.x[ph] = tp.x; it.y[ph] = tp.y + it.g_lo; it.j[ph] = tp.j;
                    }
                    out.titems.push_back(it);
                }
                c64 += w;
            }
        }
    }
    // every channel row of the zero-margined copy: front zeros, L samples, zeros for the run a box may
    // read past the last sample; rounded to 128 bytes
    const int64_t pitch = (int64_t)kTPadFront + hp.L + 4ll * d_max + kTXExtra + t_box_cols(4);
    out.pad_pitch = (pitch + 31) / 32 * 32;
}

}  // namespace fast
}  // namespace rocket
