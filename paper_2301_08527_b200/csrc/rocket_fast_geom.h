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

// T regime.  Column lc (0..127) of a tile owns residue r0 + lc.  Row s of the tile (A-row t0 + s)
// arrives with the box of phase s & 3; the box starts at a 16-byte aligned element, so the
// wanted element sits `shift` floats into the box row, shift = (t0*d + r0 + (s & 3)*d) & 3
// (rows 4 apart differ by 4d floats, which keeps the shift).
struct TColumn { int u0; int col[4]; bool ok; };

ROCKET_HD TColumn t_column(int t0, int r0, int d, int lc) {
    TColumn c;
    c.ok = r0 + lc < d;
    const int within = c.ok ? lc : 0;
    c.u0 = t0 * d + r0 + within;
    for (int j = 0; j < 4; ++j) c.col[j] = within + ((t0 * d + r0 + j * d) & 3);
    return c;
}

// Offset (floats) of row s inside a stage: phase block (s & 3), box row (s >> 2).
ROCKET_HD constexpr int t_row_offset(int s) { return (s & 3) * kTPhaseFloats + (s >> 2) * kTBoxCols; }

// One tiled TMA load of the fill: phase k of a stage.  e0 is the flat float index, in the padded
// buffer, of the tile's row 0 / column 0 element for the stage's channel.  The buffer is seen
// through one of two tensor views with rows of 4d floats: view 0 starts at float 0, view 1 at
// float t_view_shift(d).  The box is kTBoxCols wide and starts at the 16-byte aligned coordinate
// (x, y); the view is chosen so that the box does not cross the end of a tensor row.
ROCKET_HD int t_view_shift(int d) { return (2 * d + 3) & ~3; }
struct TBox { int view, x, y; };

ROCKET_HD TBox t_box_of(uint32_t kappa0, uint32_t rho0, int k, int d) {
    const uint32_t w = 4u * (uint32_t)d;
    uint32_t kappa = kappa0 + (uint32_t)k * (uint32_t)d, rho = rho0;
    if (kappa >= w) { kappa -= w; rho += 1; }
    TBox b;
    if ((kappa & ~3u) + (uint32_t)kTBoxCols <= w) {
        b.view = 0; b.x = (int)(kappa & ~3u); b.y = (int)rho;
    } else {
        b.view = 1; b.x = (int)((kappa - (uint32_t)t_view_shift(d)) & ~3u); b.y = (int)rho;
    }
    return b;
}

}  // namespace fast
}  // namespace rocket
