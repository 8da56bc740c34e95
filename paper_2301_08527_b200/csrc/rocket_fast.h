// Fast path of the forward transform: data structures shared by the host planner and the
// fused kernels.
//
// Geometry.  A kernel with dilation d reads x[u + j*d] for output u = i - p (i the output
// index, p the padding).  Writing u = t*d + r with 0 <= r < d turns the series into a 2-D array
// A[t][r] = x[t*d + r], and the dilated convolution into a dense length-len filter down the
// columns of A: output (t, r) needs A[t .. t+len-1][r].  A thread owns one column r and R
// consecutive rows ("a band"), keeps R accumulators in registers and streams R+len-1 inputs
// per channel past them, so every input is loaded once and used len times.  Lanes of a warp own
// adjacent columns.
//
// Two regimes share the arithmetic core:
//   S (d < split): kernels of one dilation form a bucket.  Columns of successive bands are
//     strung together into one "raster" (band-major, r-minor) and a tile is 32 consecutive raster
//     positions, so lanes stay busy even when d < 32.  A block stages one tile of ALL channels
//     in shared memory (threads copy and zero-pad), then its warps pull kernels of the bucket
//     from a shared counter, so one staged tile serves dozens to hundreds of kernels.
//   T (d >= split): few kernels share a dilation, so a block takes one kernel, one band and 128
//     adjacent residues, and streams the kernel's channels through a ring of shared-memory
//     stages.  A producer warp fills the ring with tiled TMA loads: the zero-padded copy of the
//     batch is viewed as a 2-D tensor with rows of 4d floats (row pitch 16d bytes, a legal TMA
//     stride for every d), in which the rows s, s+4, s+8, .. of a tile's column block form one
//     box; four boxes (one per s mod 4) bring a whole stage.  Consumer warps do nothing but
//     shared-memory loads, FMAs and pooling.
#pragma once

#include <cstdint>
#include <vector>

#include "rocket_internal.h"

namespace rocket {
namespace fast {

constexpr int kBandRows = 32;                                      // R of a full band
constexpr int kWeightRow = 12;                                     // weights of one channel, padded
constexpr int kWeightsPerKernel = kWeightRow * ROCKET_MAX_CHANNELS_PER_KERNEL;  // fixed stride in negw
constexpr int kRowsMax = kBandRows + ROCKET_MAX_LENGTH - 1;        // staged rows per band
constexpr int kSplitDefault = 72;                                  // S below, T at or above
constexpr int kSMaxChannels = 20;                                  // channels the S tile can stage

constexpr int kSThreads = 256, kSWarps = kSThreads / 32, kSCols = 32;
constexpr int kSPlaneFloats = kRowsMax * kSCols;                   // one channel of an S tile

constexpr int kTConsumerWarps = 4, kTThreads = 32 * (kTConsumerWarps + 1), kTCols = 32 * kTConsumerWarps;
constexpr int kTBoxCols = kTCols + 4;                              // 4 floats of 16-byte alignment slack
constexpr int kTBoxRowsMax = (kRowsMax + 3) / 4;                   // rows of one phase (s mod 4)
constexpr int kTPhaseFloats = (kTBoxCols * kTBoxRowsMax + 31) / 32 * 32;  // 128-byte aligned phases
constexpr int kTStageFloats = 4 * kTPhaseFloats;
constexpr int kTStages = 3;
constexpr int kTParamBufs = kTStages + 1;
// Smallest dilation of the T regime: with two tensor views whose bases differ by about 2d floats,
// one of them always holds a 132-wide box without crossing the end of a 4d-wide tensor row.
constexpr int kTMinDilation = 72;

// One kernel as the fast kernels read it (32 words).
struct alignas(16) FastKernel {
    int32_t len, d, p, m;
    int32_t nout, woff, k, lo_u;   // woff: offset into negw; k: original kernel index; lo_u = -p
    int32_t hi_u;                  // nout - p (exclusive bound on u)
    float negb;                    // 0 - bias (never -0.0)
    int32_t ch[ROCKET_MAX_CHANNELS_PER_KERNEL];
    int32_t pad_[11];
};
static_assert(sizeof(FastKernel) == 128, "FastKernel must be 32 words");

struct SBucket {
    int32_t d, tmin, nbands, raster_len;  // raster_len = nbands * d
    int32_t kbeg, kend, rows, pad_;       // kernels [kbeg, kend) of fk; rows = 32 + max len - 1
};
struct SItem { int32_t bucket, c0; };

// One T tile, with everything the producer warp needs (16 words).
struct alignas(16) TItem {
    int32_t fk, t0, R, r0;                // band starts at A-row t0, R rows, residues [r0, r0+128)
    int32_t map, len, d, m;               // map: index of the tile's pair of tensor views
    int32_t box_rows;                     // rows per phase box = ceil((R + len - 1) / 4)
    uint8_t ch[12];
    int32_t pad_[4];
};
static_assert(sizeof(TItem) == 64, "TItem must be 16 words");
struct TMapSpec { int32_t d, box_rows; };  // one pair of tensor views (bases 0 and ~2d floats)

// Zero-padded copy of the batch the T regime reads: row (n, c) starts at float
// front + (n*C + c) * pitch and is followed by at least `margin` zeros.
struct PadLayout { int64_t front = 0, pitch = 0, margin = 0; };

struct PlanHost {
    bool enabled = false;
    int split = kSplitDefault;
    std::vector<FastKernel> fk;
    std::vector<float> negw;
    std::vector<SBucket> sb;
    std::vector<SItem> sitems;
    std::vector<TItem> titems;
    std::vector<TMapSpec> tspecs;
    std::vector<int32_t> generic_list;    // kernels the fast path does not take
    PadLayout pad;
};

struct PlanDevice {
    const FastKernel* fk = nullptr;
    const float* negw = nullptr;
    const SBucket* sb = nullptr;
    const SItem* sitems = nullptr;
    const TItem* titems = nullptr;
    const int32_t* generic_list = nullptr;
    unsigned* counters = nullptr;         // [0] S work counter, [1] T work counter
    int* error_flag = nullptr;            // set when a bounded wait gave up
    const void* tmaps = nullptr;          // CUtensorMap[2 * n_tspecs], 128 bytes each
    float* xpad = nullptr;                // zero-padded copy of the batch
    int64_t pad_front = 0, pad_pitch = 0;
    int n_fk = 0, n_sitems = 0, n_titems = 0, n_generic = 0, n_tspecs = 0;
};

// Builds the launch plan for the kernels in hp (host side, once per handle).
void build_plan(const HostParams& hp, int split, PlanHost& out);

// Floats the padded copy needs for N examples.
int64_t pad_buffer_floats(const PlanHost& plan, int N, int C);

// Encodes the tensor views of every TMapSpec over a padded buffer of total_floats floats at
// xpad (device address) into maps_host (2 * n_tspecs * 128 bytes).  Needs the CUDA driver.
cudaError_t encode_tensor_maps(const PlanHost& plan, float* xpad, int64_t total_floats, void* maps_host);

// Hard forward through the fast path: pad copy, init, S kernel, T kernel, finalise.
cudaError_t launch_fast_forward(const PlanDevice& pd, const DeviceParams& dp, const float* X, int N, float* feat,
                                cudaStream_t stream);

}  // namespace fast
}  // namespace rocket
