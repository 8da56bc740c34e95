// Fused forward kernels of the fast path (hard PPV + max): see rocket_fast.h for the geometry.
//
// Arithmetic conventions shared by both kernels
//   - Accumulators hold -z: weights and bias are stored negated (acc = (0 - b) + sum (-w) x).  Then
//     z > 0  <=>  the sign bit of acc is set, exactly: a zero accumulator is always +0 (it starts
//     at +0 when b == 0, exact cancellation rounds to +0, and +0 plus a -0 product stays +0), so
//     the PPV count is one shift-and-add per output and MAX = -min(acc) one min per output.
//   - Outputs outside the kernel's range are replaced by +inf before pooling (sign bit clear,
//     neutral for the min).
//   - Per (example, kernel) the count is combined with integer atomic adds and the max with an
//     integer atomic max on an order-preserving key, both exact and order-independent, so the
//     result is run-to-run identical.  The feature buffer itself holds these integers until the
//     finalise kernel turns them into (count / L_out, max).
#include <cfloat>
#include <climits>

#include "rocket_fast.h"
#include "rocket_fast_geom.h"

namespace rocket {
namespace fast {
namespace {

constexpr unsigned kFull = 0xffffffffu;

extern __shared__ __align__(128) float smem[];

// Order-preserving map float -> signed int (for atomicMax) and back.
__device__ __forceinline__ int float_key(float v) {
    const int b = __float_as_int(v);
    return b >= 0 ? b : b ^ 0x7fffffff;
}
__device__ __forceinline__ float key_float(int k) { return __int_as_float(k >= 0 ? k : k ^ 0x7fffffff); }

// One channel of one band: R outputs down a column, R+ELL-1 inputs streamed past them.
// Row s of the column sits at sm[col[s & 3] + s * PITCH]; the four column offsets absorb the
// per-row 16-byte alignment shift of bulk-copied rows (all four are equal in the S regime).
template <int ELL, int R, int PITCH>
__device__ __forceinline__ void conv_channel(const float* __restrict__ sm, const int (&col)[4],
                                             const float* __restrict__ w, float (&acc)[R]) {
    const float4 w0 = *reinterpret_cast<const float4*>(w);
    const float4 w1 = *reinterpret_cast<const float4*>(w + 4);
    const float4 w2 = *reinterpret_cast<const float4*>(w + 8);
    const float wall[12] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w, w2.x, w2.y, w2.z, w2.w};
    float wr[ELL];
#pragma unroll
    for (int j = 0; j < ELL; ++j) wr[j] = wall[j];
#pragma unroll
    for (int s = 0; s < R + ELL - 1; ++s) {
        const float x = sm[col[s & 3] + s * PITCH];
#pragma unroll
        for (int j = 0; j < ELL; ++j) {
            const int o = s - j;
            if (o >= 0 && o < R) acc[o] = fmaf(wr[j], x, acc[o]);
        }
    }
}

// PPV count and min(-z) over the thread's R outputs; rows outside [o_lo, o_hi) are neutralised.
template <int R>
__device__ __forceinline__ void pool_hard(const float (&acc)[R], bool interior, int o_lo, int o_hi, int& cnt,
                                          float& mn) {
    if (interior) {
#pragma unroll
        for (int o = 0; o < R; ++o) {
            cnt += (int)(__float_as_uint(acc[o]) >> 31);
            mn = fminf(mn, acc[o]);
        }
    } else {
#pragma unroll
        for (int o = 0; o < R; ++o) {
            const float a = (o >= o_lo && o < o_hi) ? acc[o] : __int_as_float(0x7f800000);
            cnt += (int)(__float_as_uint(a) >> 31);
            mn = fminf(mn, a);
        }
    }
}

__device__ __forceinline__ void publish(int* __restrict__ feat_i, int64_t pair, int cnt, float mn, int lane) {
    cnt = __reduce_add_sync(kFull, cnt);
    const int key = __reduce_max_sync(kFull, float_key(-mn));
    if (lane == 0) {
        if (cnt) atomicAdd(feat_i + pair * 2, cnt);
        atomicMax(feat_i + pair * 2 + 1, key);
    }
}

struct FwdArgs {
    PlanDevice plan;
    const float* X;
    int* feat_i;
    int N, C, L, K;
};

// ------------------------------------------------------------------------------------------------
// S regime
// ------------------------------------------------------------------------------------------------
template <int ELL>
__device__ __forceinline__ void s_kernel_tile(const float* planes, const float* wb, const int* kb, int lane,
                                              bool interior, int o_lo, int o_hi, int& cnt, float& mn) {
    float acc[kBandRows];
    const float negb = __int_as_float(kb[9]);
#pragma unroll
    for (int o = 0; o < kBandRows; ++o) acc[o] = negb;
    const int m = kb[3];
    for (int q = 0; q < m; ++q) {
        const int base = kb[10 + q] * kSPlaneFloats + lane;
        const int col[4] = {base, base, base, base};
        conv_channel<ELL, kBandRows, kSCols>(planes, col, wb + q * kWeightRow, acc);
    }
    pool_hard<kBandRows>(acc, interior, o_lo, o_hi, cnt, mn);
}

__global__ void __launch_bounds__(kSThreads, 2) fast_s_forward(FwdArgs a) {
    float* planes = smem;                                        // [C][kRowsMax][32]
    float* wbuf = planes + a.C * kSPlaneFloats;                  // [warps][11 * 12]
    int* kbuf = reinterpret_cast<int*>(wbuf + kSWarps * ROCKET_MAX_CHANNELS_PER_KERNEL * kWeightRow);  // [warps][32]
    __shared__ unsigned s_item;
    __shared__ int s_next;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned n_items = (unsigned)a.plan.n_sitems;
    const unsigned long long total = (unsigned long long)a.N * n_items;
    float* wb = wbuf + warp * (ROCKET_MAX_CHANNELS_PER_KERNEL * kWeightRow);
    int* kb = kbuf + warp * 32;

    for (;;) {
        __syncthreads();  // the previous tile is fully consumed
        if (threadIdx.x == 0) s_item = atomicAdd(a.plan.counters + 0, 1u);
        __syncthreads();
        const unsigned g = s_item;
        if (g >= total) break;
        const int n = (int)(g / n_items);
        const SItem item = a.plan.sitems[g - (unsigned)n * n_items];
        const SBucket b = a.plan.sb[item.bucket];
        const int d = b.d;
        const int cg = item.c0 + lane;
        const bool lane_ok = cg < b.raster_len;
        const int u0 = s_column_u0(b, cg);  // u of the thread's first output row
        const float* __restrict__ Xn = a.X + (size_t)n * a.C * a.L;

        // stage the tile: every channel, rows 0..rows-1 of every column, zero outside the series
        for (int s = warp; s < b.rows; s += kSWarps) {
            const int xi = u0 + s * d;
            const bool ok = lane_ok && (unsigned)xi < (unsigned)a.L;
            const float* __restrict__ src = Xn + (ok ? xi : 0);
            float* dst = planes + s * kSCols + lane;
#pragma unroll 4
            for (int c = 0; c < a.C; ++c) {
                float v = 0.0f;
                if (ok) v = __ldg(src + (size_t)c * a.L);
                dst[c * kSPlaneFloats] = v;
            }
        }
        if (threadIdx.x == 0) s_next = b.kbeg;
        __syncthreads();

        // kernels of the bucket, pulled from the shared counter; the parameters of the next kernel
        // are fetched into registers while the current one computes
        int kk = 0;
        if (lane == 0) kk = atomicAdd(&s_next, 1);
        kk = __shfl_sync(kFull, kk, 0);
        int kb_next = 0;
        float w_next[5] = {0.f, 0.f, 0.f, 0.f, 0.f};
        auto prefetch = [&](int k) {
            if (k < b.kend) {
                kb_next = __ldg(reinterpret_cast<const int*>(a.plan.fk + k) + lane);
                const float* wsrc = a.plan.negw + (size_t)k * kWeightsPerKernel;
#pragma unroll
                for (int i = 0; i < 5; ++i)
                    if (lane + 32 * i < kWeightsPerKernel) w_next[i] = __ldg(wsrc + lane + 32 * i);
            }
        };
        prefetch(kk);
        while (kk < b.kend) {
            __syncwarp();
            kb[lane] = kb_next;
#pragma unroll
            for (int i = 0; i < 5; ++i)
                if (lane + 32 * i < kWeightsPerKernel) wb[lane + 32 * i] = w_next[i];
            int kk_next = 0;
            if (lane == 0) kk_next = atomicAdd(&s_next, 1);
            kk_next = __shfl_sync(kFull, kk_next, 0);
            prefetch(kk_next);
            __syncwarp();
            const int len = kb[0], korig = kb[6], lo_u = kb[7], hi_u = kb[8];
            const bool mine = lane_ok && u0 >= lo_u && (u0 + (kBandRows - 1) * d) < hi_u;
            const bool interior = __all_sync(kFull, mine);
            int o_lo = 0, o_hi = kBandRows;
            if (!interior) valid_rows(u0, d, lo_u, hi_u, kBandRows, lane_ok, o_lo, o_hi);
            int cnt = 0;
            float mn = __int_as_float(0x7f800000);
            if (len == 7) s_kernel_tile<7>(planes, wb, kb, lane, interior, o_lo, o_hi, cnt, mn);
            else if (len == 9) s_kernel_tile<9>(planes, wb, kb, lane, interior, o_lo, o_hi, cnt, mn);
            else s_kernel_tile<11>(planes, wb, kb, lane, interior, o_lo, o_hi, cnt, mn);
            publish(a.feat_i, (int64_t)n * a.K + korig, cnt, mn, lane);
            kk = kk_next;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// T regime
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait on a phase parity: returns false when the limit is reached (the caller records it).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (int it = 0; it < (1 << 20); ++it) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}
// Bulk copy global -> shared (16-byte aligned addresses, size a multiple of 16), completion on bar.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// Warp 0 fills one ring slot with one channel of the tile: one bulk copy per (chunk, row), the
// source rounded down to 16 bytes; rows or tails outside the series come from the zero page.
__device__ __noinline__ void t_issue_stage(const float* __restrict__ xrow, const float* __restrict__ zeros,
                                           const TChunk* chunks, int nch, int rows, int d, int L, uint32_t stage,
                                           uint32_t bar, int lane) {
    const int tasks = nch * rows;
    uint32_t mine = 0;
    for (int task = lane; task < tasks; task += 32) mine += t_copy_of(task, chunks, rows, d, L).tot_bytes;
    const uint32_t total = __reduce_add_sync(kFull, mine);
    if (lane == 0) mbar_arrive_expect_tx(bar, total);
    __syncwarp();
    for (int task = lane; task < tasks; task += 32) {
        const TCopy cp = t_copy_of(task, chunks, rows, d, L);
        const uint32_t dst = stage + cp.dst_bytes;
        bulk_g2s(dst, cp.src_elem >= 0 ? xrow + cp.src_elem : zeros, cp.in_bytes, bar);
        if (cp.in_bytes < cp.tot_bytes) bulk_g2s(dst + cp.in_bytes, zeros, cp.tot_bytes - cp.in_bytes, bar);
    }
}

template <int ELL, int R>
__device__ __forceinline__ void t_kernel_tile(const FwdArgs& a, const float* stages, const float* wbuf,
                                              const int* kb, const TChunk* chunks, int nch, const float* Xn,
                                              const int (&col)[4], uint32_t bar0, uint32_t (&phase)[kTStages],
                                              bool interior, int o_lo, int o_hi, int& cnt, float& mn) {
    float acc[R];
    const float negb = __int_as_float(kb[9]);
#pragma unroll
    for (int o = 0; o < R; ++o) acc[o] = negb;
    const int m = kb[3], d = kb[1];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int rows = R + ELL - 1;
    for (int q = 0; q < m; ++q) {
        const int slot = q & 1;
        if (warp == 0 && q + 1 < m)
            t_issue_stage(Xn + (size_t)kb[10 + q + 1] * a.L, a.plan.zeros, chunks, nch, rows, d, a.L,
                          smem_u32(stages + (slot ^ 1) * kTStageFloats), bar0 + 8u * (slot ^ 1), lane);
        if (!mbar_wait(bar0 + 8u * slot, phase[slot])) atomicExch(a.plan.error_flag, 1);
        phase[slot] ^= 1u;
        conv_channel<ELL, R, kTPitch>(stages + slot * kTStageFloats, col, wbuf + q * kWeightRow, acc);
        __syncthreads();  // every warp is done with this slot before it is refilled
    }
    pool_hard<R>(acc, interior, o_lo, o_hi, cnt, mn);
}

__global__ void __launch_bounds__(kTThreads, 4) fast_t_forward(FwdArgs a) {
    float* stages = smem;                                   // [2][kRowsMax][kTPitch]
    float* wbuf = stages + kTStages * kTStageFloats;        // [11 * 12]
    int* kb = reinterpret_cast<int*>(wbuf + ROCKET_MAX_CHANNELS_PER_KERNEL * kWeightRow);  // [32]
    __shared__ __align__(8) unsigned long long bars[kTStages];
    __shared__ TChunk chunks[kTMaxChunks];
    __shared__ unsigned s_item;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t bar0 = smem_u32(bars);
    if (threadIdx.x == 0) {
        for (int i = 0; i < kTStages; ++i) mbar_init(bar0 + 8u * i, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    uint32_t phase[kTStages] = {0u, 0u};
    const unsigned n_items = (unsigned)a.plan.n_titems;
    const unsigned long long total = (unsigned long long)a.N * n_items;

    for (;;) {
        __syncthreads();
        if (threadIdx.x == 0) {
            // a wait that gave up anywhere ends the whole launch early (results are flagged invalid)
            const bool failed = *reinterpret_cast<volatile int*>(a.plan.error_flag) != 0;
            s_item = failed ? 0xffffffffu : atomicAdd(a.plan.counters + 1, 1u);
        }
        __syncthreads();
        const unsigned g = s_item;
        if (g >= total) break;
        const int n = (int)(g / n_items);
        const TItem item = a.plan.titems[g - (unsigned)n * n_items];
        if (warp == 0) kb[lane] = __ldg(reinterpret_cast<const int*>(a.plan.fk + item.fk) + lane);
        __syncthreads();
        const int len = kb[0], d = kb[1], m = kb[3], woff = kb[5], korig = kb[6], lo_u = kb[7], hi_u = kb[8];
        for (int i = threadIdx.x; i < m * kWeightRow; i += kTThreads) wbuf[i] = __ldg(a.plan.negw + woff + i);
        const int R = item.R;
        // chunks of the tile (every thread computes them; thread 0 publishes them for the fill)
        TChunk my_chunks[kTMaxChunks];
        int ncols;
        const int nch = t_make_chunks(item, d, my_chunks, ncols);
        if (threadIdx.x == 0)
            for (int i = 0; i < nch; ++i) chunks[i] = my_chunks[i];
        const TColumn tc = t_column(my_chunks, nch, ncols, d, threadIdx.x);
        const bool lane_ok = tc.ok;
        const int u0 = tc.u0;
        const int col[4] = {tc.col[0], tc.col[1], tc.col[2], tc.col[3]};
        const bool mine = lane_ok && u0 >= lo_u && (u0 + (R - 1) * d) < hi_u;
        const bool interior = __all_sync(kFull, mine);
        int o_lo = 0, o_hi = R;
        if (!interior) valid_rows(u0, d, lo_u, hi_u, R, lane_ok, o_lo, o_hi);
        __syncthreads();  // kb, wbuf, chunks visible to everyone
        const float* __restrict__ Xn = a.X + (size_t)n * a.C * a.L;
        if (warp == 0)
            t_issue_stage(Xn + (size_t)kb[10] * a.L, a.plan.zeros, chunks, nch, R + len - 1, d, a.L,
                          smem_u32(stages), bar0, lane);
        int cnt = 0;
        float mn = __int_as_float(0x7f800000);
#define ROCKET_T_CASE(ELL_, R_)                                                                               \
    t_kernel_tile<ELL_, R_>(a, stages, wbuf, kb, chunks, nch, Xn, col, bar0, phase, interior, o_lo, o_hi, cnt, mn)
#define ROCKET_T_LEN(R_)                                                          \
    do {                                                                          \
        if (len == 7) ROCKET_T_CASE(7, R_);                                       \
        else if (len == 9) ROCKET_T_CASE(9, R_);                                  \
        else ROCKET_T_CASE(11, R_);                                               \
    } while (0)
        if (R == 32) ROCKET_T_LEN(32);
        else if (R == 24) ROCKET_T_LEN(24);
        else if (R == 16) ROCKET_T_LEN(16);
        else ROCKET_T_LEN(8);
#undef ROCKET_T_LEN
#undef ROCKET_T_CASE
        publish(a.feat_i, (int64_t)n * a.K + korig, cnt, mn, lane);
    }
}

// ------------------------------------------------------------------------------------------------
// init / finalise
// ------------------------------------------------------------------------------------------------
__global__ void fast_init_kernel(int* __restrict__ feat_i, int64_t pairs, unsigned* counters) {
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e == 0) { counters[0] = 0u; counters[1] = 0u; }
    if (e < pairs) { feat_i[2 * e] = 0; feat_i[2 * e + 1] = INT_MIN; }
}

__global__ void fast_finalize_kernel(float* __restrict__ feat, const FastKernel* __restrict__ fk, int n_fk, int N,
                                     int K) {
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= (int64_t)N * n_fk) return;
    const int n = (int)(e / n_fk), f = (int)(e - (int64_t)n * n_fk);
    const int k = fk[f].k, nout = fk[f].nout;
    int* fi = reinterpret_cast<int*>(feat) + ((int64_t)n * K + k) * 2;
    const int cnt = fi[0], key = fi[1];
    feat[((int64_t)n * K + k) * 2] = (float)cnt / (float)nout;   // Eq. 2
    feat[((int64_t)n * K + k) * 2 + 1] = key_float(key);
}

}  // namespace

size_t s_smem_bytes(int C) {
    return (size_t)(C * kSPlaneFloats + kSWarps * ROCKET_MAX_CHANNELS_PER_KERNEL * kWeightRow + kSWarps * 32) * 4;
}
size_t t_smem_bytes() {
    return (size_t)(kTStages * kTStageFloats + ROCKET_MAX_CHANNELS_PER_KERNEL * kWeightRow + 32) * 4;
}

cudaError_t launch_fast_forward(const PlanDevice& pd, const DeviceParams& dp, const float* X, int N, float* feat,
                                cudaStream_t stream) {
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    static bool attr_done = false;
    const size_t s_bytes = s_smem_bytes(dp.C), t_bytes = t_smem_bytes();
    if (!attr_done) {
        e = cudaFuncSetAttribute(fast_s_forward, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)s_smem_bytes(kSMaxChannels));
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(fast_t_forward, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)t_bytes);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    FwdArgs a;
    a.plan = pd; a.X = X; a.feat_i = reinterpret_cast<int*>(feat);
    a.N = N; a.C = dp.C; a.L = dp.L; a.K = dp.K;
    const int64_t pairs = (int64_t)N * dp.K;
    fast_init_kernel<<<(unsigned)((pairs + 255) / 256), 256, 0, stream>>>(a.feat_i, pairs, pd.counters);
    count_launch();
    if (pd.n_sitems > 0) {
        const unsigned long long total = (unsigned long long)N * pd.n_sitems;
        const unsigned grid = (unsigned)std::min<unsigned long long>(total, (unsigned long long)sms * 2);
        fast_s_forward<<<grid, kSThreads, s_bytes, stream>>>(a);
        count_launch();
    }
    if (pd.n_titems > 0) {
        const unsigned long long total = (unsigned long long)N * pd.n_titems;
        const unsigned grid = (unsigned)std::min<unsigned long long>(total, (unsigned long long)sms * 4);
        fast_t_forward<<<grid, kTThreads, t_bytes, stream>>>(a);
        count_launch();
    }
    const int64_t fin = (int64_t)N * pd.n_fk;
    if (fin > 0) {
        fast_finalize_kernel<<<(unsigned)((fin + 255) / 256), 256, 0, stream>>>(feat, pd.fk, pd.n_fk, N, dp.K);
        count_launch();
    }
    return cudaGetLastError();
}

}  // namespace fast
}  // namespace rocket
