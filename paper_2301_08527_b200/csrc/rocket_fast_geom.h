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

// Rows of a thread's column that are real outputs: u0 + o*d must lie in [lo_u, hi_u).
ROCKET_HD void valid_rows(int u0, int d, int lo_u, int hi_u, int R, bool col_ok, int& o_lo, int& o_hi) {
    const int a_lo = lo_u - u0, a_hi = hi_u - u0;
    o_lo = a_lo > 0 ? (a_lo + d - 1) / d : 0;
    o_hi = a_hi > 0 ? imin(R, (a_hi + d - 1) / d) : 0;
    if (!col_ok) o_hi = 0;
}

// The same without a division, for a column given as (first A-row t_row0, residue c in [0, d)):
// u = t*d + c >= lo_u = tl*d + rl  <=>  t >= tl + (c < rl), and likewise for the upper end.
ROCKET_HD void valid_rows_tc(int t_row0, int c, int tl, int rl, int th, int rh, int R, bool col_ok, int& o_lo, int& o_hi) {
    const int t_lo = tl + (c < rl ? 1 : 0) - t_row0, t_hi = th + (c < rh ? 1 : 0) - t_row0;
    o_lo = t_lo < 0 ? 0 : (t_lo > R ? R : t_lo);
    o_hi = t_hi < 0 ? 0 : (t_hi > R ? R : t_hi);
    if (!col_ok) o_hi = 0;
}

// S regime: the u of the first output row of raster column cg of a bucket.
ROCKET_HD int s_column_u0(const SBucket& b, int cg) {
    const int band = cg / b.d, r = cg - band * b.d;
    return (b.tmin + band * kRS) * b.d + r;
}

// T regime.  A tile starts at A-row t0 and residue r0 (a multiple of 64).  Row s of the tile
// (A-row t0 + s) arrives with the box of phase s & 3, as that box's row s >> 2.  In the
// zero-margined copy the element (A-row t, residue r) of a channel row sits at float
// front + t*d + r of that row; copy j holds the same data moved down by j floats, so the element
// is 16-byte aligned in copy j = position & 3.  Every copy is seen as runs of 4d floats (tensor
// coordinate y = which run, x = position in the run).
struct TPhase { int x, y, j; };

ROCKET_HD TPhase t_phase(int t0, int r0, int d, int k) {
    const long long flat = (long long)kTPadFront + (long long)(t0 + k) * d + r0;
    TPhase p;
    p.j = (int)(flat & 3);
    const long long pos = flat - p.j, run = 4ll * d;
    long long y = pos / run;
    if (pos - y * run < 0) --y;  // floor for negative positions
    p.x = (int)(pos - y * run);
    p.y = (int)y;
    return p;
}

// The box `cols` floats to the right of box p in the same row of A (same shifted copy when cols
// is a multiple of 4).
ROCKET_HD TPhase t_phase_right(TPhase p, int cols, int d) {
    p.x += cols;
    if (p.x >= 4 * d) { p.x -= 4 * d; p.y += 1; }
    return p;
}

// Rows of A that hold samples are [0, ceil(L / d)): every other row is zero.  A wide tile loads
// and multiplies only the groups of four tile rows [g_lo, g_hi) that hold samples (at least one
// group, so that a box is never empty).
struct TWindow { int g_lo, g_hi; };

ROCKET_HD TWindow t_window(int t0, int rows, int d, int L) {
    const int t_data = (L + d - 1) / d;
    const int s_lo = -t0 > 0 ? -t0 : 0;
    const int s_hi = imin(rows, t_data - t0);
    TWindow w;
    if (s_hi <= s_lo) { w.g_lo = 0; w.g_hi = 1; return w; }
    w.g_lo = s_lo >> 2;
    w.g_hi = (s_hi + 3) >> 2;
    return w;
}

// Float offset, inside a stage, of the box of phase k.
ROCKET_HD int t_box_offset(int cg, int k, int box_rows) { return k * t_phase_floats(cg, box_rows); }

// Float offset, inside a stage, of tile row s / tile column lc as the consumer reads it.
ROCKET_HD int t_elem_offset(int cg, int s, int lc, int box_rows) {
    return t_box_offset(cg, s & 3, box_rows) + (s >> 2) * t_box_cols(cg) + lc;
}

// The same for a wide tile: column lc in [0, 512) lies in half lc / 256; row s must belong to a
// loaded group (g_lo <= s / 4 < g_lo + box_rows).
ROCKET_HD int t_wide_half_floats(int box_rows) { return 4 * t_phase_floats(4, box_rows); }
ROCKET_HD int t_wide_elem_offset(int s, int lc, int box_rows, int g_lo) {
    return (lc / kTWideCols) * t_wide_half_floats(box_rows) + t_box_offset(4, s & 3, box_rows) +
           ((s >> 2) - g_lo) * kTWideCols + (lc % kTWideCols);
}

}  // namespace fast
}  // namespace rocket
