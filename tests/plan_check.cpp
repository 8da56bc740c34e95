// Host-side checker of the fast path's launch plan and index arithmetic (no GPU needed).
// For a set of (seed, K, C, L) it builds the plan and replays, with the same integer functions
// the kernels use, which outputs every thread of every tile owns and which bulk copies every
// tile issues.  It fails (exit 1) unless every output of every fast kernel is owned exactly once
// and every copy stays inside its source row and its shared-memory slot with 16-byte alignment.
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
    std::vector<std::vector<uint8_t>> cover(plan.fk.size());
    for (size_t f = 0; f < plan.fk.size(); ++f) cover[f].assign(plan.fk[f].nout, 0);
    std::vector<char> is_generic(hp.K, 0);
    for (int k : plan.generic_list) is_generic[k] = 1;
    REQUIRE(plan.fk.size() + plan.generic_list.size() == (size_t)hp.K, "kernel partition");
    for (auto& f : plan.fk) REQUIRE(!is_generic[f.k], "kernel %d in both lists", f.k);

    for (const SItem& it : plan.sitems) {
        const SBucket& b = plan.sb[it.bucket];
        REQUIRE(b.rows <= kRowsMax && b.d < plan.split, "S bucket shape");
        for (int lane = 0; lane < kSCols; ++lane) {
            const int cg = it.c0 + lane;
            const bool lane_ok = cg < b.raster_len;
            const int u0 = s_column_u0(b, cg);
            for (int kk = b.kbeg; kk < b.kend; ++kk) {
                const FastKernel& f = plan.fk[kk];
                REQUIRE(f.d == b.d && kBandRows + f.len - 1 <= b.rows, "S kernel in wrong bucket");
                int o_lo, o_hi;
                valid_rows(u0, b.d, f.lo_u, f.hi_u, kBandRows, lane_ok, o_lo, o_hi);
                for (int o = o_lo; o < o_hi; ++o) {
                    const int64_t i = (int64_t)u0 + (int64_t)o * b.d + f.p;
                    REQUIRE(i >= 0 && i < f.nout, "S output out of range");
                    cover[kk][i]++;
                }
            }
        }
    }
    for (const TItem& it : plan.titems) {
        const FastKernel& f = plan.fk[it.fk];
        REQUIRE(f.d >= 64 && (it.R == 8 || it.R == 16 || it.R == 24 || it.R == 32), "T item shape");
        const int rows = it.R + f.len - 1;
        REQUIRE(rows <= kRowsMax, "T rows");
        TChunk chunks[kTMaxChunks];
        int ncols;
        const int nch = t_make_chunks(it, f.d, chunks, ncols);
        REQUIRE(nch >= 1 && nch <= kTMaxChunks && ncols >= 1, "T chunks");
        for (int c = 0; c < nch; ++c) {
            const int slot_end = (c + 1 < nch) ? chunks[c + 1].off : kTPitch;
            REQUIRE(chunks[c].off % 4 == 0 && chunks[c].off + ((chunks[c].w + 3) & ~3) + 4 <= slot_end, "chunk slot");
        }
        for (int task = 0; task < nch * rows; ++task) {
            const TCopy cp = t_copy_of(task, chunks, rows, f.d, L);
            REQUIRE(cp.tot_bytes % 16 == 0 && cp.in_bytes % 16 == 0 && cp.in_bytes > 0 && cp.in_bytes <= cp.tot_bytes, "copy size");
            REQUIRE(cp.dst_bytes % 16 == 0 && cp.dst_bytes + cp.tot_bytes <= (uint32_t)kTStageFloats * 4, "copy dst");
            REQUIRE(cp.tot_bytes - cp.in_bytes <= (uint32_t)kZeroFloats * 4 && cp.tot_bytes <= (uint32_t)kZeroFloats * 4, "zero page");
            if (cp.src_elem >= 0)
                REQUIRE(cp.src_elem % 4 == 0 && (int64_t)cp.src_elem + cp.in_bytes / 4 <= L, "copy src %d + %u > %d", cp.src_elem, cp.in_bytes / 4, L);
        }
        for (int lc = 0; lc < kTCols; ++lc) {
            const TColumn tc = t_column(chunks, nch, ncols, f.d, lc);
            int o_lo, o_hi;
            valid_rows(tc.u0, f.d, f.lo_u, f.hi_u, it.R, tc.ok, o_lo, o_hi);
            for (int o = o_lo; o < o_hi; ++o) {
                const int64_t i = (int64_t)tc.u0 + (int64_t)o * f.d + f.p;
                REQUIRE(i >= 0 && i < f.nout, "T output out of range");
                cover[it.fk][i]++;
            }
            // every row the thread reads lies inside a copied region and holds the element it expects
            int sel = 0, start = 0, within = lc;
            for (int c = 0; c < nch; ++c) { if (lc >= start && lc < start + chunks[c].w) { sel = c; within = lc - start; } start += chunks[c].w; }
            if (!tc.ok) { sel = 0; within = 0; }
            for (int s = 0; s < rows; ++s) {
                const int pos = tc.col[s & 3] + s * kTPitch;
                REQUIRE(pos >= 0 && pos < kTStageFloats, "column read outside the stage");
                const TCopy cp = t_copy_of(sel * rows + s, chunks, rows, f.d, L);
                const int rel = pos * 4 - (int)cp.dst_bytes;
                REQUIRE(rel >= 0 && rel + 4 <= (int)cp.tot_bytes, "column read outside the copied row");
                const int64_t want = (int64_t)(chunks[sel].tb + s) * f.d + chunks[sel].ra + within;  // x index
                if (cp.src_elem >= 0 && rel < (int)cp.in_bytes) REQUIRE(cp.src_elem + rel / 4 == want, "wrong element");
                else REQUIRE(want < 0 || want >= L || cp.src_elem < 0, "zero page where data is expected");
                if (cp.src_elem < 0) REQUIRE(want < 0 || want >= L || (chunks[sel].tb + s) < 0 ||
                                             (int64_t)(chunks[sel].tb + s) * f.d + chunks[sel].ra >= L, "zero row misplaced");
            }
        }
    }
    for (size_t fidx = 0; fidx < plan.fk.size(); ++fidx)
        for (int i = 0; i < plan.fk[fidx].nout; ++i)
            REQUIRE(cover[fidx][i] == 1, "kernel %d (len %d d %d p %d) output %d owned %d times", plan.fk[fidx].k,
                    plan.fk[fidx].len, plan.fk[fidx].d, plan.fk[fidx].p, i, (int)cover[fidx][i]);
    std::printf("ok seed=%llu K=%d C=%d L=%d split=%d: %zu fast kernels, %zu generic, %zu S items, %zu T items\n",
                (unsigned long long)seed, hp.K, hp.C, hp.L, plan.split, plan.fk.size(), plan.generic_list.size(),
                plan.sitems.size(), plan.titems.size());
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
    rc |= check(0, hp.K, hp.C, hp.L, 64, &hp);
    return rc;
}
