// Fast path of the forward transform: data structures shared by the host planner and the
// fused kernels.
//
// Geometry.  A kernel with dilation d reads x[u + j*d] for output u = i - p (i the output
// index, p the padding).  Writing u = t*d + r with 0 <= r < d turns the series into a 2-D array
// A[t][r] = x[t*d + r], and the dilated convolution into a dense length-len filter down the
// columns of A: output (t, r) needs A[t .. t+len-1][r].  A thread owns one column r and R
// consecutive rows ("a band"), keeps R accumulators in registers and streams R+len-1 inputs
// per channel past them, so every input is loaded once and used len times.  Lanes of a warp own
// adjacent columns.  Columns of successive bands are strung together into one "raster"
// (band-major, r-minor) and tiles are runs of consecutive raster positions, so lanes stay busy
// even when d is smaller than a tile.
//
// Two regimes share the arithmetic core:
//   S (d < split): kernels of one dilation form a bucket; a block stages one 32-column tile of
//     ALL channels in shared memory (threads copy and zero-pad), then its warps pull kernels of
//     the bucket from a shared counter, so one staged tile serves dozens to hundreds of kernels.
//   T (d >= split): few kernels share a dilation, so a block takes one kernel and a 128-column
//     tile and streams the kernel's channels through a two-slot ring filled by bulk TMA row
//     copies (no issue slots spent on the fill), overlapped with the FMAs of the previous channel.
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
constexpr int kSplitDefault = 64;                                  // S below, T at or above
constexpr int kSMaxChannels = 20;                                  // channels the S tile can stage

constexpr int kSThreads = 256, kSWarps = kSThreads / 32, kSCols = 32;
constexpr int kSPlaneFloats = kRowsMax * kSCols;                   // one channel of an S tile

constexpr int kTThreads = 128, kTCols = 128, kTMaxChunks = 3;
constexpr int kTPitch = 152;                                       // 128 + 3 * (3 + 4) rounded up to 8
constexpr int kTStageFloats = kRowsMax * kTPitch;
constexpr int kTStages = 2;
constexpr int kZeroFloats = 256;                                   // zero page for out-of-range rows

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
struct TItem {
    int32_t fk, t0, R, c0;                // t0: A-row of band 0 of the item's band group
    int32_t raster_len, pad_[3];
};

struct PlanHost {
    bool enabled = false;
    int split = kSplitDefault;
    std::vector<FastKernel> fk;
    std::vector<float> negw;
    std::vector<SBucket> sb;
    std::vector<SItem> sitems;
    std::vector<TItem> titems;
    std::vector<int32_t> generic_list;    // kernels the fast path does not take
};

struct PlanDevice {
    const FastKernel* fk = nullptr;
    const float* negw = nullptr;
    const SBucket* sb = nullptr;
    const SItem* sitems = nullptr;
    const TItem* titems = nullptr;
    const int32_t* generic_list = nullptr;
    const float* zeros = nullptr;
    unsigned* counters = nullptr;         // [0] S work counter, [1] T work counter
    int* error_flag = nullptr;            // set when a bounded wait gave up
    int n_fk = 0, n_sitems = 0, n_titems = 0, n_generic = 0;
};

// Builds the launch plan for the kernels in hp (host side, once per handle).
void build_plan(const HostParams& hp, int split, PlanHost& out);

// Hard forward through the fast path: init, S kernel, T kernel, finalise.  feat is [N][2K].
cudaError_t launch_fast_forward(const PlanDevice& pd, const DeviceParams& dp, const float* X, int N, float* feat,
                                cudaStream_t stream);

}  // namespace fast
}  // namespace rocket
