// Host-side checker of the fast path's launch plan and index arithmetic (no GPU needed).
// For a set of (seed, K, C, L) it builds the plan and replays, with the same integer functions
// the kernels use, which outputs every thread of every tile owns and which boxes every T tile
// loads.  It fails (exit 1) unless every output of every fast kernel is owned exactly once, every
// box obeys the TMA rules (16-byte aligned x, 128-byte aligned destination inside the stage,
// reads inside the channel row of the zero-margined copy) and every shared-memory word a
// consumer thread reads holds the sample it expects (or a zero outside the series).
#include <cstdio>
#include <cstdlib>
#include <vector>

#include "rocket_fast.h"
#include "rocket_fast_geom.h"

using namespace rocket;
using namespace rocket::fast;

namespace rocket { std::atomic<int64_t> g_launch_count{0}; }

#define REQUIRE(cond, ...)                                        \
    do {                                                          \
        if (!(cond)) {                                            \
            std::fprintf(stderr, "FAIL %s:%d: ", __FILE__, __LINE__); \
            std::fprintf(stderr, __VA_ARGS__);                    \
            std::fprintf(stderr, "\n");                           \
            return 1;                                             \
        }                                                         \
    } while (0)

static int check(uint64_t seed, int K, int C, int L, int split, const HostParams* given = nullptr) {
    HostParams hp;
    if (given) hp = *given;
    else generate_host_params(seed, K, C, L, hp);
    hp.channel_offset.assign(hp.K + 1, 0);
    hp.weight_offset.assign(hp.K + 1, 0);
    for (int k = 0; k < hp.K; ++k) {
        hp.channel_offset[k + 1] = hp.channel_offset[k] + hp.num_channels[k];
        hp.weight_offset[k + 1] = hp.weight_offset[k] + hp.num_channels[k] * hp.length[k];
    }
    PlanHost plan;
    build_plan(hp, split, plan);
    std::vector<std::vector<uint8_t>> cover(plan.krec.size());
    for (size_t f = 0; f < plan.krec.size(); ++f) cover[f].assign(plan.krec[f].nout, 0);
    std::vector<char> is_generic(hp.K, 0);
    for (int k : plan.generic_list) is_generic[k] = 1;
    REQUIRE(plan.krec.size() + plan.generic_list.size() == (size_t)hp.K, "kernel partition");
    for (auto& f : plan.krec) {
        REQUIRE(!is_generic[f.k], "kernel %d in both lists", f.k);
        const float* W = hp.weights.data() + hp.weight_offset[f.k];
        for (int q = 0; q < f.m; ++q)
            for (int j = 0; j < kPairRow / 2; ++j) {
                const float want = j < f.len ? 0.0f - W[q * f.len + j] : 0.0f;
                REQUIRE(f.w2[q][2 * j] == want && f.w2[q][2 * j + 1] == want, "weight pair");
            }
    }

    for (const SItem& it : plan.sitems) {
        const SBucket& b = plan.sb[it.bucket];
        REQUIRE(b.rows <= kSRowsMax && b.d < plan.split && it.c0 % kWarpCols == 0, "S bucket shape");
        bool all_full = true;
        for (int col = 0; col < kWarpCols; ++col) {
            const int cg = it.c0 + col;
            const bool col_ok = cg < b.raster_len;
            const int u0 = s_column_u0(b, cg);
            for (int kk = b.kbeg; kk < b.kend; ++kk) {
                const KRec& f = plan.krec[kk];
                REQUIRE(f.d == b.d && kRS + f.len - 1 <= b.rows, "S kernel in wrong bucket");
                int o_lo, o_hi, q_lo, q_hi;
                valid_rows(u0, b.d, f.lo_u, f.hi_u, kRS, col_ok, q_lo, q_hi);
                const int band = cg / b.d;
                valid_rows_tc(b.tmin + band * kRS, cg - band * b.d, f.tl, f.rl, f.th, f.rh, kRS, col_ok, o_lo, o_hi);
                REQUIRE((o_lo >= o_hi && q_lo >= q_hi) || (o_lo == q_lo && o_hi == q_hi), "S row range: the two forms disagree");
                all_full = all_full && o_lo == 0 && o_hi == kRS;
                for (int o = o_lo; o < o_hi; ++o) {
                    const int64_t i = (int64_t)u0 + (int64_t)o * b.d + f.p;
                    REQUIRE(i >= 0 && i < f.nout, "S output out of range");
                    cover[kk][i]++;
                }
            }
        }
        // the kernels skip every range test on a tile flagged interior
        REQUIRE((it.interior != 0) == all_full, "S interior flag %d, replay says %d", it.interior, (int)all_full);
    }

    const int64_t pitch = plan.pad_pitch;
    REQUIRE(plan.titems.empty() || (pitch % 32 == 0 && pitch >= kTPadFront + L), "pad pitch");
    for (const TItem& it : plan.titems) {
        const KRec& f = plan.krec[it.krec];
        REQUIRE(it.map >= 0 && it.map < (int)plan.tmaps.size(), "T map index");
        const TMapSpec& sp = plan.tmaps[it.map];
        REQUIRE(f.d >= kTMinDilation && f.d == it.d && f.len == it.len && f.m == it.m, "T item fields");
        REQUIRE((it.cg == 1 || it.cg == 2 || it.cg == 4) && (it.cg <= kTMaxCg || it.wide) && it.rg >= 1 && it.rg * it.cg <= kTConsumerWarps, "T shape");
        REQUIRE(it.r0 % kWarpCols == 0 && it.r0 < f.d, "T column origin");
        for (int q = 0; q < f.m; ++q) REQUIRE(it.ch[q] == f.ch[q], "T channel list");
        const bool wide = it.wide != 0;
        const int rows_out = kR * it.rg, boxw = t_box_cols(it.cg);
        const int tile_cols = wide ? kTWideHalves * kTWideCols : boxw;
        const int rows = rows_out + f.len - 1;
        if (wide) {
            const TWindow win = t_window(it.t0, rows, f.d, L);
            REQUIRE(it.rg == 1 && it.cg == 4 && boxw == kTWideCols, "wide tile shape");
            REQUIRE(it.g_lo == win.g_lo && it.g_hi == win.g_hi && win.g_lo >= 0 && win.g_lo < win.g_hi && 4 * win.g_hi < rows + 4,
                    "wide tile window");
            REQUIRE(kTWideHalves * t_wide_half_floats(it.box_rows) <= kTStageFloats, "wide stage size");
        } else {
            REQUIRE(it.g_lo == 0 && it.g_hi == t_box_rows(it.rg, f.len) && 4 * it.g_hi >= rows, "T box rows");
        }
        REQUIRE(it.box_rows == it.g_hi - it.g_lo, "T box rows and window");
        REQUIRE(sp.d == f.d && sp.box_cols == boxw && sp.box_rows == it.box_rows && boxw <= 256 && it.box_rows <= 256, "T map spec");
        REQUIRE(4 * t_phase_floats(it.cg, it.box_rows) <= kTStageFloats, "stage size");
        const long long run = 4ll * f.d, ny = (kTPadFront + (long long)L + run - 1) / run;
        // the boxes the producer issues: four phases, twice for a wide tile
        TPhase ph[4 * (kTWideHalves > 1 ? kTWideHalves : 1)];
        for (int k = 0; k < (wide ? 4 * kTWideHalves : 4); ++k) {
            if (k < 4) {
                ph[k] = t_phase(it.t0, it.r0, f.d, k);
                ph[k].y += it.g_lo;
                REQUIRE(it.x[k] == ph[k].x && it.y[k] == ph[k].y && it.j[k] == ph[k].j, "stored box coordinates");
            } else {
                ph[k] = t_phase_right(ph[k - 4], kTWideCols, f.d);
            }
            REQUIRE(ph[k].x % 4 == 0 && ph[k].x >= 0 && ph[k].x < run && ph[k].j >= 0 && ph[k].j < 4, "box x");
            REQUIRE(ph[k].x + boxw <= run + kTXExtra, "box leaves the tensor row");
            const int dst = t_box_offset(it.cg, k, it.box_rows);
            REQUIRE(dst % 32 == 0 && dst + it.box_rows * boxw <= kTStageFloats, "box destination");
            for (int j = 0; j < it.box_rows; ++j) {
                const long long y = ph[k].y + j;
                if (y < 0 || y >= ny) continue;  // zero-filled by the copy engine
                // copy j holds the layout moved down by j floats: the box row reads layout[first + j .. last + j]
                const long long first = y * run + ph[k].x + ph[k].j, last = first + boxw - 1;
                REQUIRE(first >= 0 && last < pitch, "box row reads outside its channel row: %lld..%lld of %lld", first,
                        last, (long long)pitch);
            }
        }
        // what every consumer thread owns and reads
        bool w_full[kTConsumerWarps], w_any[kTConsumerWarps];
        for (int w8 = 0; w8 < kTConsumerWarps; ++w8) { w_full[w8] = true; w_any[w8] = false; }
        for (int lc = 0; lc < tile_cols; ++lc) {
            const bool col_ok = it.r0 + lc < f.d;
            for (int wr = 0; wr < it.rg; ++wr) {
                const int u0 = (it.t0 + kR * wr) * f.d + it.r0 + lc;
                int o_lo, o_hi, q_lo, q_hi;
                valid_rows(u0, f.d, f.lo_u, f.hi_u, kR, col_ok, q_lo, q_hi);
                valid_rows_tc(it.t0 + kR * wr, it.r0 + lc, f.tl, f.rl, f.th, f.rh, kR, col_ok, o_lo, o_hi);
                REQUIRE((o_lo >= o_hi && q_lo >= q_hi) || (o_lo == q_lo && o_hi == q_hi), "T row range: the two forms disagree");
                const int w8 = wide ? lc / kWarpCols : wr * it.cg + lc / kWarpCols;
                w_full[w8] = w_full[w8] && o_lo == 0 && o_hi == kR;
                w_any[w8] = w_any[w8] || o_lo < o_hi;
                for (int o = o_lo; o < o_hi; ++o) {
                    const int64_t i = (int64_t)u0 + (int64_t)o * f.d + f.p;
                    REQUIRE(i >= 0 && i < f.nout, "T output out of range");
                    cover[it.krec][i]++;
                }
                if (o_lo >= o_hi) continue;
                for (int s2 = 0; s2 < kR + f.len - 1; ++s2) {
                    const int s = kR * wr + s2;
                    const long long want = (long long)kTPadFront + (long long)(it.t0 + s) * f.d + it.r0 + lc;
                    const bool in_series = want >= kTPadFront && want < kTPadFront + L;
                    if ((s >> 2) < it.g_lo || (s >> 2) >= it.g_hi) {
                        // a row the consumer skips: it must hold no sample
                        REQUIRE(wide && !in_series, "a skipped row holds a sample");
                        continue;
                    }
                    const int k = (s & 3) + (wide ? 4 * (lc / kTWideCols) : 0);
                    const int pos = wide ? t_wide_elem_offset(s, lc, it.box_rows, it.g_lo) : t_elem_offset(it.cg, s, lc, it.box_rows);
                    REQUIRE(pos >= 0 && pos < kTStageFloats, "read outside the stage");
                    if ((lc & 1) == 0) REQUIRE(pos % 2 == 0, "pair not 8-byte aligned");
                    // which sample the copy engine put there
                    const int rel = pos - t_box_offset(it.cg, k, it.box_rows);
                    const int j = rel / boxw, i = rel % boxw;
                    REQUIRE(rel >= 0 && j < it.box_rows, "read outside the box");
                    const long long y = ph[k].y + j;
                    const long long flat = y * run + ph[k].x + i + ph[k].j;
                    REQUIRE(flat == want, "wrong sample: got flat %lld, want %lld", flat, want);
                    if (y < 0 || y >= ny) REQUIRE(!in_series, "zero fill where a sample is expected");
                }
            }
        }
        // the per-warp flags the consumers trust instead of range tests
        const int n_tiles_w = wide ? kTConsumerWarps : it.rg * it.cg;
        for (int w8 = 0; w8 < kTConsumerWarps; ++w8) {
            const bool in_tile = w8 < n_tiles_w;
            const bool full = in_tile && w_full[w8], any = in_tile && w_any[w8];
            REQUIRE(((it.warp_interior >> w8) & 1) == (int)full, "T interior flag of warp %d", w8);
            REQUIRE(((it.warp_active >> w8) & 1) == (int)any, "T active flag of warp %d", w8);
        }
    }
    // (the flag check of the T tiles sits at the end of the tile loop above)
    for (size_t fidx = 0; fidx < plan.krec.size(); ++fidx)
        for (int i = 0; i < plan.krec[fidx].nout; ++i)
            REQUIRE(cover[fidx][i] == 1, "kernel %d (len %d d %d p %d) output %d owned %d times", plan.krec[fidx].k,
                    plan.krec[fidx].len, plan.krec[fidx].d, plan.krec[fidx].p, i, (int)cover[fidx][i]);
    size_t n_wide = 0;
    for (const TItem& it : plan.titems) n_wide += it.wide != 0;
    std::printf("ok seed=%llu K=%d C=%d L=%d split=%d: %zu fast kernels, %zu generic, %zu S items, %zu T items (%zu wide)\n",
                (unsigned long long)seed, hp.K, hp.C, hp.L, plan.split, plan.krec.size(), plan.generic_list.size(),
                plan.sitems.size(), plan.titems.size(), n_wide);
    return 0;
}

int main() {
    int rc = 0;
    rc |= check(8527, 1000, 1, 512, 64);
    rc |= check(8527, 3000, 20, 5000, 64);
    rc |= check(11, 600, 20, 50000, 64);
    rc |= check(12, 400, 7, 10000, 128);
    rc |= check(13, 300, 3, 1000, 64);
    rc |= check(14, 200, 2, 16, 64);
    rc |= check(21, 300, 20, 200000, 64);
    rc |= check(22, 300, 5, 4099, 64);      // series lengths that are no multiple of four floats
    rc |= check(23, 200, 20, 50001, 64);
    // hand-made kernels: padding that is not a multiple of the dilation, extreme dilations, tiny outputs
    HostParams hp;
    hp.K = 0; hp.C = 2; hp.L = 1000;
    auto add = [&](int len, int d, int p) {
        hp.length.push_back(len); hp.dilation.push_back(d); hp.padding.push_back(p); hp.num_channels.push_back(1);
        hp.channel_idx.push_back(0); hp.bias.push_back(0.5f);
        for (int j = 0; j < len; ++j) hp.weights.push_back(1.0f);
        hp.K++;
    };
    add(7, 166, 0); add(7, 166, 498); add(11, 99, 495); add(9, 7, 40); add(7, 64, 5); add(9, 65, 300); add(11, 100, 1);
    add(7, 1, 0); add(7, 1, 3); add(9, 63, 17); add(7, 127, 381); add(7, 128, 0); add(9, 124, 0); add(3, 5, 0); add(5, 70, 3);
    add(7, 129, 5); add(9, 77, 308); add(11, 91, 2);
    add(7, 330, 990); add(7, 340, 1000); add(7, 512, 1536); add(11, 345, 1725);   // at most 16 rows of outputs: wide tiles
    rc |= check(0, hp.K, hp.C, hp.L, 64, &hp);
    return rc;
}
