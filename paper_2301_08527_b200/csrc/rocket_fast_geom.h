// Index arithmetic of the fast path, shared by the device kernels and the host-side plan checker
// (plain integer code, compiled for both).
#pragma once

#include <cstdint>

#include "rocket_fast.h"

#ifdef __CUDACC__
#define ROCKET_HD __host__ __device__ __forceinline__
#else
#define ROCKET_HD inline
#endif

namespace rocket {
namespace fast {

ROCKET_HD int imin(int a, int b) { return a < b ? a : b; }

// Rows of a thread's band that are real outputs: u0 + o*d must lie in [lo_u, hi_u).
ROCKET_HD void valid_rows(int u0, int d, int lo_u, int hi_u, int R, bool lane_ok, int& o_lo, int& o_hi) {
    const int a_lo = lo_u - u0, a_hi = hi_u - u0;
    o_lo = a_lo > 0 ? (a_lo + d - 1) / d : 0;
    o_hi = a_hi > 0 ? imin(R, (a_hi + d - 1) / d) : 0;
    if (!lane_ok) o_hi = 0;
}

// S regime: the u of the first output row of raster column cg of a bucket.
ROCKET_HD int s_column_u0(const SBucket& b, int cg) {
    const int band = cg / b.d, r = cg - band * b.d;
    return (b.tmin + band * kBandRows) * b.d + r;
}

// T regime: a tile is cut into chunks, runs of consecutive residues, one per band it touches.
struct TChunk { int tb, ra, w, off; };  // first A-row, first residue, width, column offset in the stage row

ROCKET_HD int t_make_chunks(const TItem& item, int d, TChunk (&chunks)[kTMaxChunks], int& ncols) {
    const int band0 = item.c0 / d, rs = item.c0 - band0 * d;
    ncols = imin(kTCols, item.raster_len - item.c0);
    int remaining = ncols, ra = rs, band = band0, off = 0, nch = 0;
    while (remaining > 0 && nch < kTMaxChunks) {
        const int w = imin(d - ra, remaining);
        chunks[nch].tb = item.t0 + band * item.R; chunks[nch].ra = ra; chunks[nch].w = w; chunks[nch].off = off;
        off += ((w + 3) & ~3) + 4;
        remaining -= w; ra = 0; ++band; ++nch;
    }
    return remaining > 0 ? -1 : nch;  // -1: the tile would need more chunks than the stage row holds
}

// Column lc of a T tile: its chunk, residue, first output's u, and the four shared-memory column
// offsets (index = row & 3) that absorb the 16-byte alignment shift of each bulk-copied row.
struct TColumn { int u0; int col[4]; bool ok; };

ROCKET_HD TColumn t_column(const TChunk* chunks, int nch, int ncols, int d, int lc) {
    TColumn c;
    c.ok = lc < ncols;
    int start = 0, sel = 0;
    for (int i = 0; i < nch; ++i) {
        if (lc >= start && lc < start + chunks[i].w) sel = i;
        start += chunks[i].w;
    }
    const TChunk ch = chunks[sel];
    int within = lc;
    for (int i = 0; i < sel; ++i) within -= chunks[i].w;
    if (!c.ok) within = 0;
    c.u0 = ch.tb * d + ch.ra + within;
    for (int j = 0; j < 4; ++j) c.col[j] = ch.off + within + ((ch.tb * d + ch.ra + j * d) & 3);
    return c;
}

// One bulk copy of the fill: row s of chunk c.  Bytes [0, in_bytes) come from the series at
// element offset src_elem of the channel row (or from the zero page when src_elem < 0), bytes
// [in_bytes, tot_bytes) from the zero page.  dst_bytes is relative to the stage slot.
struct TCopy { int src_elem; uint32_t dst_bytes, in_bytes, tot_bytes; };

ROCKET_HD TCopy t_copy_of(int task, const TChunk* chunks, int rows, int d, int L) {
    const int c = task / rows, s = task - c * rows;
    const TChunk ch = chunks[c];
    const int t = ch.tb + s;
    const int xs = t * d + ch.ra;
    const int al = xs & 3;
    TCopy cp;
    cp.tot_bytes = (uint32_t)((al + ch.w + 3) & ~3) * 4u;
    cp.dst_bytes = (uint32_t)(s * kTPitch + ch.off) * 4u;
    if (t < 0 || xs >= L) {
        cp.src_elem = -1; cp.in_bytes = cp.tot_bytes;
    } else {
        const int as = xs - al;
        const int end = imin(xs + ch.w, L);
        cp.src_elem = as;
        const uint32_t in = (uint32_t)((end - as + 3) & ~3) * 4u;
        cp.in_bytes = in < cp.tot_bytes ? in : cp.tot_bytes;
    }
    return cp;
}

}  // namespace fast
}  // namespace rocket
