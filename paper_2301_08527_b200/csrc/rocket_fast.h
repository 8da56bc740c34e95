// Fast path of the forward transform: data structures shared by the host planner and the
// fused kernels.
//
// Geometry.  A kernel with dilation d reads x[u + j*d] for output u = i - p (i the output
// index, p the padding).  Writing u = t*d + r with 0 <= r < d turns the series into a 2-D array
// A[t][r] = x[t*d + r], and the dilated convolution into a dense length-len filter down the
// columns of A: output (t, r) needs A[t .. t+len-1][r].  A thread owns two adjacent columns
// and 16 consecutive rows, keeps the 32 accumulators in registers as 16 packed pairs and
// streams 16+len-1 input pairs per channel past them with packed two-wide FMAs
// (fma.rn.f32x2), so every input is loaded once and used len times.  Lanes of a warp own
// adjacent column pairs: a warp tile is 16 rows x 64 columns.
//
// Two regimes share the arithmetic core:
//   S (d < split): kernels of one dilation form a bucket.  Columns of successive bands of kRS rows
//     are strung together into one "raster" (band-major, r-minor) and a tile is 64 consecutive
//     raster positions, so lanes stay busy even when d < 64.  A block stages one tile of ALL
//     channels in shared memory, then its warps pull kernels of the bucket from a shared
//     counter, so one staged tile serves dozens to hundreds of kernels.
//   T (d >= split): few kernels share a dilation, so a block of eight consumer warps takes one
//     kernel and one tile of up to eight warp tiles (128 x 64, 64 x 128, 32 x 256, or 16 x 512 for
//     kernels whose outputs span at most 16 rows of A) and streams the kernel's channels through a
//     ring of shared-memory stages.  A producer warp fills the
//     ring with tiled TMA loads from a zero-margined copy of the batch, viewed as a 3-D tensor
//     (x within a run of 4d floats, y = which run, z = channel row): rows s, s+4, s+8, .. of
//     a tile are then one box, and four boxes (one per s mod 4) bring a whole stage without
//     spending issue slots of the consumer warps.
#pragma once

#include <cstdint>
#include <mutex>
#include <vector>

#include "rocket_internal.h"

#ifdef __CUDACC__
#define ROCKET_CX __host__ __device__ constexpr
#else
#define ROCKET_CX constexpr
#endif

namespace rocket {
namespace fast {

constexpr int kR = 16;                                             // output rows of a warp tile
constexpr int kWarpCols = 64;                                      // columns of a warp tile (2 per lane)
constexpr int kRowsMax = kR + ROCKET_MAX_LENGTH - 1;               // staged rows a warp tile reads
#ifndef ROCKET_SPLIT
#define ROCKET_SPLIT 64
#endif
constexpr int kSplitDefault = ROCKET_SPLIT;                        // S below, T at or above
constexpr int kTMinDilation = 64;                                  // a T tile needs 64 residues in one band

// ---- kernel record: one fast kernel as the device reads it (header + duplicated weights) ----
constexpr int kPairRow = 24;                                       // floats of one channel's weight row
struct alignas(16) KRec {
    int32_t len, d, p, m;
    int32_t nout, k, lo_u, hi_u;   // k: original kernel index; lo_u = -p; hi_u = nout - p (exclusive)
    float negb;                    // 0 - bias (never -0.0)
    int32_t ch[ROCKET_MAX_CHANNELS_PER_KERNEL];
    int32_t tl, rl, th, rh;        // lo_u = tl * d + rl and hi_u = th * d + rh with 0 <= rl, rh < d
    int32_t woff;                  // offset of the kernel's weights in the caller's ragged weight array
    int32_t pad_[7];
    // w2[q][2j] = w2[q][2j+1] = 0 - W[q][j]: each weight twice, ready as a packed pair
    float w2[ROCKET_MAX_CHANNELS_PER_KERNEL][kPairRow];
};
static_assert(sizeof(KRec) == 128 + 4 * ROCKET_MAX_CHANNELS_PER_KERNEL * kPairRow, "KRec layout");
static_assert(sizeof(KRec) % 16 == 0, "KRec must be copyable in 16-byte pieces");

// ---- S regime --------------------------------------------------------------------------------
// Per-channel feature scaling of 8-bit input (Section 4.3): x = (v - mean[c]) * inv_std[c].
constexpr int kNormMaxChannels = 20;
struct NormArgs { float mean[kNormMaxChannels], inv_std[kNormMaxChannels]; };

constexpr int kSMaxChannels = 20;                                  // channels the S tile can stage
// Output rows of a warp tile in the S regime (the band height of its rasters).  More rows per thread than in
// the T regime: the work per (kernel, tile) grows while the per-kernel bookkeeping and the rows staged per
// output shrink.  Measured at 60 x 20 x 50,000 (hard): 16 rows 25.7 ms, 20 rows 24.9, 22 rows 24.6, 24 to 26
// rows 24.1 (16 warps each; 12 warps are slower at every height), 28 rows need 14 warps for the tile to fit.
#ifndef ROCKET_S_ROWS
#define ROCKET_S_ROWS 24
#endif
#ifndef ROCKET_S_THREADS
#define ROCKET_S_THREADS 512
#endif
constexpr int kRS = ROCKET_S_ROWS;
static_assert(kRS >= 8 && kRS <= 32, "the row masks of the pooling hold at most 32 rows");
constexpr int kSRowsMax = kRS + ROCKET_MAX_LENGTH - 1;             // staged rows an S warp tile reads
constexpr int kSThreads = ROCKET_S_THREADS, kSWarps = kSThreads / 32;   // one block per SM
constexpr int kSPlaneFloats = kSRowsMax * kWarpCols;               // one channel of an S tile
constexpr int kSLengthOrderMin = 100;                              // buckets from this many kernels up are ordered by length

struct SBucket {
    int32_t d, tmin, nbands, raster_len;  // raster_len = nbands * d
    int32_t kbeg, kend, rows, pad_;       // kernels [kbeg, kend) of krec; rows = kRS + max len - 1
};
// One S tile: 64 raster positions from c0 of a bucket.  interior = 1 when every (row, column) of the
// tile is an output of every kernel of the bucket (then the kernels need no range tests).
struct SItem { int32_t bucket, c0, interior, pad_; };

// ---- T regime --------------------------------------------------------------------------------
// Consumer warps per block, blocks per SM and ring depth of the T kernel.  A block's consumer warps move
// through a stage in step, so the number of independent blocks per SM decides how often the FMA pipes
// find a warp that is ready.
#ifndef ROCKET_T_WARPS
#define ROCKET_T_WARPS 8
#endif
#ifndef ROCKET_T_BLOCKS
#define ROCKET_T_BLOCKS 2
#endif
#ifndef ROCKET_T_STAGES
#define ROCKET_T_STAGES 2
#endif
constexpr int kTConsumerWarps = ROCKET_T_WARPS;
static_assert(kTConsumerWarps == 4 || kTConsumerWarps == 8, "tile shapes are laid out for 4 or 8 consumer warps");
constexpr int kTBlocksPerSM = ROCKET_T_BLOCKS;
constexpr int kTThreads = 32 * (kTConsumerWarps + 1);              // one group: consumer warps + one producer warp
// Groups per block: every group is a producer with its consumers, its own ring and its own stream of tiles.
// Two groups in one block instead of two blocks of one group leave more registers to every thread (the
// register file is handed out per pair of warps, and a group has an odd number of warps).
#ifndef ROCKET_T_GROUPS
#define ROCKET_T_GROUPS 1
#endif
constexpr int kTGroups = ROCKET_T_GROUPS;
constexpr int kTBlockThreads = kTGroups * kTThreads;
constexpr int kTStages = ROCKET_T_STAGES;
constexpr int kTParamSlots = kTStages + 2;
// A T tile is rg row groups x cg column groups of warp tiles, rg * cg <= the consumer warps, cg in {1, 2, 4}
// (cg = 4 only with 8 consumer warps: a 16 x 256 tile would load 26 rows for 16 rows of outputs).
// One box per phase brings all column groups (64 * cg floats wide).  The zero-margined copy is kept
// four times, shifted by 0, 1, 2 and 3 floats, so that every row start is 16-byte aligned in one
// of them: a box needs no alignment slack and every pair a consumer reads is 8-byte aligned.
constexpr int kTMaxCg = kTConsumerWarps >= 8 ? 4 : 2;
ROCKET_CX int t_box_cols(int cg) { return kWarpCols * cg; }
// Box rows of one phase (rows s, s+4, ..), and the floats of one phase box (a multiple of 64
// floats, so every box destination stays 128-byte aligned).
ROCKET_CX int t_box_rows(int rg, int len) { return (kR * rg + len - 1 + 3) / 4; }
ROCKET_CX int t_phase_floats(int cg, int box_rows) { return box_rows * t_box_cols(cg); }
ROCKET_CX int t_stage_floats(int rg, int cg, int len) { return 4 * t_phase_floats(cg, t_box_rows(rg, len)); }
ROCKET_CX int imax_cx(int a, int b) { return a > b ? a : b; }
constexpr int kTStageFloats =
    imax_cx(imax_cx(t_stage_floats(kTConsumerWarps, 1, ROCKET_MAX_LENGTH), t_stage_floats(kTConsumerWarps / 2, 2, ROCKET_MAX_LENGTH)),
            kTMaxCg >= 4 ? t_stage_floats(kTConsumerWarps / 4, 4, ROCKET_MAX_LENGTH) : 0);
constexpr int kTChunkTiles = 4;                                    // consecutive tiles a block draws at a time
constexpr int kTWideCols = 256;                                    // columns of one half of a wide tile
constexpr int kTWideHalves = kTConsumerWarps / 4;                  // a wide tile is one row of all consumer warps' tiles
constexpr int kChunkExamples = 12;                                // examples per pass through the fused kernels
constexpr int kTPadFront = 128;                                    // zero floats before every channel row
constexpr int kTXExtra = 256;                                      // floats a box may run past a 4d run

// One T tile with everything the producer warp needs (32 words).
struct alignas(16) TItem {
    int32_t map, t0, r0, rg;              // map: index of the tile's tensor map; tile origin (t0, r0)
    int32_t d, len, m, box_rows;
    uint8_t ch[12];
    int32_t krec;                         // index into the kernel records
    int32_t cg, wide, g_lo, g_hi;         // wide tile: one row of warp tiles in halves of 256 columns, of which only
                                          // the groups of four rows [g_lo, g_hi) are loaded (box_rows = g_hi - g_lo)
    int32_t x[4], y[4];                   // tensor coordinates of the four phase boxes (first half; y of group g_lo)
    int32_t j[4];                         // which shifted copy each phase reads
    // bit w: every output of consumer warp w's warp tile exists (no range tests needed) / at least one does
    int32_t warp_interior, warp_active;
    int32_t pad1_[2];
};
static_assert(sizeof(TItem) == 128, "TItem must be 32 words");
// One tensor map: boxes of box_cols x box_rows floats over runs of 4 * d floats.
struct TMapSpec { int32_t d, box_cols, box_rows; };

struct PlanHost {
    bool enabled = false;
    int split = kSplitDefault;
    std::vector<KRec> krec;
    std::vector<SBucket> sb;
    std::vector<SItem> sitems;
    std::vector<TItem> titems;            // kernel by kernel, in the order the blocks walk them
    std::vector<TMapSpec> tmaps;          // tensor maps the T tiles refer to
    std::vector<int32_t> generic_list;    // kernels the fast path does not take
    int64_t pad_pitch = 0;                // floats per channel row of the zero-margined copy
    double flops_s = 0.0, flops_t = 0.0;  // conv flop of one example in either regime
};

struct PlanDevice {
    const KRec* krec = nullptr;
    const SBucket* sb = nullptr;
    const SItem* sitems = nullptr;
    const TItem* titems = nullptr;
    const int32_t* generic_list = nullptr;
    unsigned* counters = nullptr;         // [0] S work counter, [1] T work counter
    int* error_flag = nullptr;            // set when a bounded wait gave up
    const void* tmaps = nullptr;          // CUtensorMap[n_tmaps], 128 bytes each
    float* xpad = nullptr;                // zero-margined copy of the batch
    int64_t pad_pitch = 0;
    int n_krec = 0, n_sitems = 0, n_titems = 0, n_generic = 0, n_tmaps = 0;
};

// Writes kernel f.k's bias and weights (negated, every weight twice) into its record.
void fill_record_weights(const HostParams& hp, KRec& f);
// Copies the records of the host plan to the device again (after their weights changed).
cudaError_t upload_records(FastState& fs);

// Builds the launch plan for the kernels in hp (host side, once per handle).
void build_plan(const HostParams& hp, int split, PlanHost& out);

// Device-side state of the fast path owned by a handle.
struct FastState {
    std::mutex mu;                        // guards the grow-only buffers below and the launch sequence of a call
    PlanHost host;
    PlanDevice dev;
    void* plan_blob = nullptr;            // records, buckets, items, counters, error flag
    void* maps_blob = nullptr;            // tensor maps
    float* xpad = nullptr;                // the four shifted zero-margined copies, capacity pad_examples
    int pad_examples = 0;
    int64_t copy_floats = 0;              // floats of one copy
    void* soft_ws = nullptr;              // soft mode: 16 bytes per (example, kernel), grows with N
    size_t soft_ws_bytes = 0;
    void* bwd_ws = nullptr;               // backward: fixed-point sums [n_weights + K], scales [K], max |x|
    bool profile = false;                 // record events around the S and T launches
    std::vector<cudaEvent_t> evs;         // three per chunk: before S, between S and T, after T
    int ev_chunks = 0;                    // chunks of the last profiled call
};

// Uploads the plan (once per handle, at binding).
cudaError_t upload_plan(FastState& fs);
// Frees everything upload_plan / ensure_pad_capacity allocated.
void release_fast_state(FastState& fs);
// Makes the padded copy hold N examples and (re-)encodes the tensor maps over it.
cudaError_t ensure_pad_capacity(FastState& fs, int N, int C, int L, bool without_maps = false);

// Allocates, once, everything the fused kernels need for calls of up to max_N examples (the zero-margined
// copies and their tensor maps, the soft transform's and the backward's workspaces) and opts the kernels
// into their shared-memory sizes; later calls within that size allocate nothing.
cudaError_t reserve_fast_state(FastState& fs, const DeviceParams& dp, int max_N, bool soft, bool backward, bool u8,
                               int64_t n_weights);

// Backward of the soft transform through the fast path (every kernel must be a fast-path kernel):
// dW (ragged like the weights, n_weights floats) and db [K] are assigned.
cudaError_t launch_fast_backward(FastState& fs, const DeviceParams& dp, int64_t n_weights, const float* X, int N,
                                 float lambda, float shift, const float* dfeat, const int32_t* argmax, float* dW,
                                 float* db, cudaStream_t stream);

// Forward through the fast path: init, pad copy, S kernel, T kernel, finalise.  soft = false:
// PPV + max; soft = true: softPPV + max (+ argmax when argmax != nullptr).
// With X_u8 (raw 8-bit intensities [N][C][L], 4-byte aligned) the samples are normalised per channel
// with *norm while the zero-margined copies are written, and X is not read.  half (hard transform only): samples,
// weights and biases are rounded to binary16 and every multiply-add of the convolution rounds once to binary16.
cudaError_t launch_fast_forward(FastState& fs, const DeviceParams& dp, const float* X, int N, float* feat,
                                cudaStream_t stream, bool soft = false, float lambda = 0.0f, float shift = 0.0f,
                                int32_t* argmax = nullptr, const uint8_t* X_u8 = nullptr, const NormArgs* norm = nullptr,
                                bool half = false);

}  // namespace fast
}  // namespace rocket
