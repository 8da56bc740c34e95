// Fused forward kernels of the fast path (hard PPV + max, soft PPV + max + argmax): see rocket_fast.h
// for the geometry.
//
// Arithmetic conventions shared by both kernels
//   - Accumulators hold -z: weights and bias are stored negated (acc = (0 - b) + sum (-w) x).  Then
//     z > 0  <=>  the sign bit of acc is set, exactly: a zero accumulator is always +0 (it starts
//     at +0 when b == 0, exact cancellation rounds to +0, and +0 plus a -0 product stays +0), so
//     the PPV count is one shift-and-add per output and MAX = -min(acc).
//   - A thread's two columns travel together as one packed pair (fma.rn.f32x2 gives each half the
//     result of a separate fused multiply-add).
//   - Outputs outside the kernel's range are replaced by +inf before pooling (sign bit clear,
//     neutral for the min).
//   - Per (example, kernel) the count is combined with integer atomic adds and the max with an
//     integer atomic max on an order-preserving key, both exact and order-independent, so the
//     result is run-to-run identical.  The feature buffer itself holds these integers until the
//     finalise kernel turns them into (count / L_out, max).
#include <cuda.h>

#include <algorithm>
#include <cfloat>
#include <climits>
#include <cstring>
#include <mutex>

#include "rocket_fast.h"
#include "rocket_fast_geom.h"

namespace rocket {
namespace fast {
namespace {

typedef unsigned long long u64;
constexpr unsigned kFull = 0xffffffffu;
constexpr long long kWaitLimitClocks = 1ll << 31;  // about a second: no wait inside a kernel lasts longer

extern __shared__ __align__(128) unsigned char smem_raw[];

__device__ __forceinline__ u64 pack2(float lo, float hi) {
    u64 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(u64 v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ void fma2(u64& acc, u64 a, u64 b) {
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(acc) : "l"(a), "l"(b));
}
__device__ __forceinline__ u64 fma2_to(u64 a, u64 b, u64 c) {
    u64 r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ float min3(float a, float b, float c) {
    float d;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// Order-preserving map float -> signed int (for atomicMax) and back.
__device__ __forceinline__ int float_key(float v) {
    const int b = __float_as_int(v);
    return b >= 0 ? b : b ^ 0x7fffffff;
}
__device__ __forceinline__ float key_float(int k) { return __int_as_float(k >= 0 ? k : k ^ 0x7fffffff); }

// One channel of one warp tile: 16 output rows of the thread's column pair, 16+ELL-1 input pairs
// streamed past them.  Row s of the tile sits at st[off[s & 3] + (s >> 2) * STEP]; w2 holds the
// channel's negated weights, each twice.  With WIN, only the groups of four rows [gl, gh) are read
// and multiplied (the others hold no sample and are not in shared memory); gl and gh are the same
// for the whole warp.  With FIRST the accumulators come in undefined and every one of them starts as
// init + w[0] * x (its first product), which is bit for bit what starting at init and adding gives.
template <int ELL, int STEP, bool WIN, bool FIRST = false, int R = kR>
__device__ __forceinline__ void conv_channel(const float* __restrict__ st, const int (&off)[4],
                                             const float* __restrict__ w2, u64 (&acc)[R], int gl = 0, int gh = 0,
                                             u64 init = 0ull) {
    static_assert(!(WIN && FIRST), "a windowed pass may skip an accumulator's first product");
    u64 wp[ELL + 1];
#pragma unroll
    for (int j = 0; j < ELL; j += 2) {
        const ulonglong2 v = *reinterpret_cast<const ulonglong2*>(w2 + 2 * j);
        wp[j] = v.x;
        wp[j + 1] = v.y;
    }
#pragma unroll
    for (int g = 0; g < (R + ELL - 1 + 3) / 4; ++g) {
        if (!WIN || (g >= gl && g < gh)) {
#pragma unroll
            for (int s = 4 * g; s < 4 * g + 4 && s < R + ELL - 1; ++s) {
                const float* p = st + off[s & 3] + (s >> 2) * STEP;
                const u64 x = *reinterpret_cast<const u64*>(p);
#pragma unroll
                for (int j = 0; j < ELL; ++j) {
                    const int o = s - j;
                    if (o >= 0 && o < R) {
                        if (FIRST && j == 0) acc[o] = fma2_to(wp[0], x, init);
                        else fma2(acc[o], wp[j], x);
                    }
                }
            }
        }
    }
}

// ---- half precision (mode 3): binary16 samples, weights and bias, every multiply-add rounded once to binary16 ----
typedef uint32_t h2;   // two binary16 numbers: the thread's column pair
__device__ __forceinline__ h2 to_h2(float lo, float hi) {   // round to nearest even, both halves
    h2 r;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ void hfma2(h2& acc, h2 a, h2 b) {
    asm("fma.rn.f16x2 %0, %1, %2, %0;" : "+r"(acc) : "r"(a), "r"(b));
}
// The pair as two floats (exact); a negative zero (a tiny negative result rounded to zero) becomes +0, so that
// the sign bit means "below zero" as it does for the FP32 accumulators.
__device__ __forceinline__ u64 h2_to_pair(h2 v) {
    asm("add.rn.f16x2 %0, %0, %1;" : "+r"(v) : "r"(0u));
    unsigned short lo, hi;
    asm("mov.b32 {%0, %1}, %2;" : "=h"(lo), "=h"(hi) : "r"(v));
    float a, b;
    asm("cvt.f32.f16 %0, %1;" : "=f"(a) : "h"(lo));
    asm("cvt.f32.f16 %0, %1;" : "=f"(b) : "h"(hi));
    return pack2(a, b);
}
// conv_channel in half precision: the FP32 samples of the staged tile and the FP32 weights of the record are
// rounded to binary16 on the way (the same value every time it is used), the accumulators hold 0 - z as binary16.
template <int ELL, int STEP, bool WIN, int R>
__device__ __forceinline__ void conv_channel_h(const float* __restrict__ st, const int (&off)[4],
                                               const float* __restrict__ w2, h2 (&acc)[R], int gl = 0, int gh = 0) {
    h2 wp[ELL];
#pragma unroll
    for (int j = 0; j < ELL; ++j) {
        const float2 v = *reinterpret_cast<const float2*>(w2 + 2 * j);
        wp[j] = to_h2(v.x, v.y);
    }
#pragma unroll
    for (int g = 0; g < (R + ELL - 1 + 3) / 4; ++g) {
        if (!WIN || (g >= gl && g < gh)) {
#pragma unroll
            for (int s = 4 * g; s < 4 * g + 4 && s < R + ELL - 1; ++s) {
                const float2 xf = *reinterpret_cast<const float2*>(st + off[s & 3] + (s >> 2) * STEP);
                const h2 x = to_h2(xf.x, xf.y);
#pragma unroll
                for (int j = 0; j < ELL; ++j) {
                    const int o = s - j;
                    if (o >= 0 && o < R) hfma2(acc[o], wp[j], x);
                }
            }
        }
    }
}
// The accumulators of a tile in half precision start at 0 - bias (rounded to binary16; +0 when it rounds to zero).
template <int R>
__device__ __forceinline__ void init_acc_h(h2 (&acc)[R], float negb) {
    h2 v = to_h2(negb, negb);
    if ((v & 0x7fff7fffu) == 0u) v = 0u;
#pragma unroll
    for (int o = 0; o < R; ++o) acc[o] = v;
}
template <int R>
__device__ __forceinline__ void widen_acc(const h2 (&acch)[R], u64 (&acc)[R]) {
#pragma unroll
    for (int o = 0; o < R; ++o) acc[o] = h2_to_pair(acch[o]);
}

// Adds the PPV count of the thread's 2 x 16 outputs to cnt and folds their min(-z) into mn.  Outputs outside the kernel's range
// never need a test here: their accumulators start at +inf and stay there (sign bit clear,
// neutral for the min).
template <int R>
__device__ __forceinline__ void pool_hard(const u64 (&acc)[R], int& cnt, float& mn) {
    unsigned signs = 0;  // one sign bit per output, shifted in from the right (counted every 16 rows)
#pragma unroll
    for (int o = 0; o < R; ++o) {
        float a, b;
        unpack2(acc[o], a, b);
        signs = __funnelshift_l(__float_as_uint(a), signs, 1);
        signs = __funnelshift_l(__float_as_uint(b), signs, 1);
        mn = min3(mn, a, b);
        if ((o & 15) == 15 && o + 1 < R) { cnt += __popc(signs); signs = 0; }
    }
    cnt += __popc(signs);
}

// The same for a warp tile with outputs that do not exist: m0 / m1 hold one bit per row of the thread's two
// columns (bit o set: row o is an output); the others are replaced by +inf on the way (sign bit clear, neutral
// for the min), so the accumulators may hold anything there.
template <int R>
__device__ __forceinline__ void pool_hard_masked(const u64 (&acc)[R], unsigned m0, unsigned m1, int& cnt, float& mn) {
    const float inf = __int_as_float(0x7f800000);
    unsigned signs = 0;
#pragma unroll
    for (int o = 0; o < R; ++o) {
        float a, b;
        unpack2(acc[o], a, b);
        a = (m0 & (1u << o)) ? a : inf;
        b = (m1 & (1u << o)) ? b : inf;
        signs = __funnelshift_l(__float_as_uint(a), signs, 1);
        signs = __funnelshift_l(__float_as_uint(b), signs, 1);
        mn = min3(mn, a, b);
        if ((o & 15) == 15 && o + 1 < R) { cnt += __popc(signs); signs = 0; }
    }
    cnt += __popc(signs);
}
// Bit o set for lo <= o < hi (0 <= lo, hi <= 31).
__device__ __forceinline__ unsigned row_mask(int lo, int hi) { return hi > lo ? ((1u << hi) - 1u) & ~((1u << lo) - 1u) : 0u; }

// Accumulators of a tile: 0 - bias where the output exists, +inf elsewhere.
template <int R>
__device__ __forceinline__ void init_acc(u64 (&acc)[R], float negb, bool interior, int lo0, int hi0, int lo1, int hi1) {
    if (interior) {
        const u64 v = pack2(negb, negb);
#pragma unroll
        for (int o = 0; o < R; ++o) acc[o] = v;
    } else {
        const float inf = __int_as_float(0x7f800000);
#pragma unroll
        for (int o = 0; o < R; ++o) acc[o] = pack2((o >= lo0 && o < hi0) ? negb : inf, (o >= lo1 && o < hi1) ? negb : inf);
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

__device__ __forceinline__ u64 add2(u64 a, u64 b) {
    u64 r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ float ex2_approx(float v) {
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(v));
    return r;
}
__device__ __forceinline__ float rcp_approx(float v) {
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(v));
    return r;
}

constexpr float kSoftFixedScale = 1073741824.0f;  // 2^30: soft sums travel as fixed-point integers

// Soft pooling of a warp tile (Eq. 3-4): sum of h = 1 / (1 + 2^(c1 * acc + c0)) over the valid
// outputs (acc = -z, c1 = lambda * log2 e, c0 = -shift * log2 e), the max and the lowest output
// index attaining it.  base0 / base1 are the output indices of row 0 of the thread's two columns,
// step the index distance between rows.  The warp's sum is added to ws[2 * pair] as a fixed-point
// integer and (max key, INT_MAX - index) is folded into ws[2 * pair + 1] with one 64-bit atomic max:
// both are exact and order-free, so results are run-to-run identical.
template <int R>
__device__ __forceinline__ void pool_publish_soft(unsigned long long* __restrict__ ws, int64_t pair, const u64 (&acc)[R],
                                                  float c1, float c0, bool interior, int lo0, int hi0, int lo1, int hi1,
                                                  int base0, int base1, int step, int lane) {
    const u64 c1p = pack2(c1, c1), c0p = pack2(c0, c0), one = pack2(1.0f, 1.0f);
    u64 hs = pack2(0.0f, 0.0f);
    float mn = __int_as_float(0x7f800000);
#pragma unroll
    for (int o = 0; o < R; ++o) {
        u64 t = c0p;
        fma2(t, acc[o], c1p);
        float ta, tb, a, b;
        unpack2(t, ta, tb);
        const u64 den = add2(pack2(ex2_approx(ta), ex2_approx(tb)), one);
        unpack2(den, ta, tb);
        float ha = rcp_approx(ta), hb = rcp_approx(tb);
        if (!interior) {
            if (o < lo0 || o >= hi0) ha = 0.0f;
            if (o < lo1 || o >= hi1) hb = 0.0f;
        }
        hs = add2(hs, pack2(ha, hb));
        unpack2(acc[o], a, b);
        mn = min3(mn, a, b);
    }
    float h0, h1;
    unpack2(hs, h0, h1);
    float hsum = h0 + h1;
#pragma unroll
    for (int sh = 16; sh > 0; sh >>= 1) hsum += __shfl_xor_sync(kFull, hsum, sh);
    const int key = float_key(-mn);
    const int wkey = __reduce_max_sync(kFull, key);
    int idx = INT_MAX;
    if (key == wkey) {
#pragma unroll
        for (int o = R - 1; o >= 0; --o) {
            float a, b;
            unpack2(acc[o], a, b);
            if (b == mn) idx = min(idx, base1 + o * step);
            if (a == mn) idx = min(idx, base0 + o * step);
        }
    }
    idx = __reduce_min_sync(kFull, idx);
    if (lane == 0) {
        atomicAdd(ws + 2 * pair, __float2ull_rn(hsum * kSoftFixedScale));
        const unsigned long long k64 = ((unsigned long long)((unsigned)wkey ^ 0x80000000u) << 32) |
                                       (unsigned long long)(unsigned)(INT_MAX - idx);
        atomicMax(ws + 2 * pair + 1, k64);
    }
}

__device__ __forceinline__ u64 mul2(u64 a, u64 b) {
    u64 r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

// Backward, first half: turns the accumulators (acc = -z) of a warp tile into
//   gz = gPs * h (1 - h) + gM [output index == argmax],  h = 1 / (1 + 2^(c1 * acc + c0)),
// zero where the output does not exist, and returns the thread's sum of gz (its share of db).
// oA0 / oA1: the row of the thread's first / second column that is the argmax, or -1.
template <int R>
__device__ __forceinline__ float make_gz(u64 (&acc)[R], float c1, float c0, float gPs, float gM, bool interior, int lo0,
                                         int hi0, int lo1, int hi1, int oA0, int oA1) {
    const u64 c1p = pack2(c1, c1), c0p = pack2(c0, c0), one = pack2(1.0f, 1.0f), neg1 = pack2(-1.0f, -1.0f);
    const u64 gp = pack2(gPs, gPs);
    u64 sum = pack2(0.0f, 0.0f);
#pragma unroll
    for (int o = 0; o < R; ++o) {
        u64 t = c0p;
        fma2(t, acc[o], c1p);
        float ta, tb;
        unpack2(t, ta, tb);
        const u64 den = add2(pack2(ex2_approx(ta), ex2_approx(tb)), one);
        unpack2(den, ta, tb);
        const u64 hh = pack2(rcp_approx(ta), rcp_approx(tb));
        u64 omh = one;
        fma2(omh, hh, neg1);                      // 1 - h
        u64 g = mul2(mul2(hh, omh), gp);
        float ga, gb;
        unpack2(g, ga, gb);
        if (!interior) {
            if (o < lo0 || o >= hi0) ga = 0.0f;
            if (o < lo1 || o >= hi1) gb = 0.0f;
        }
        if (o == oA0) ga += gM;
        if (o == oA1) gb += gM;
        g = pack2(ga, gb);
        acc[o] = g;
        sum = add2(sum, g);
    }
    float s0, s1;
    unpack2(sum, s0, s1);
    return s0 + s1;
}

// Backward, second half, one channel of one warp tile: dw[j] += gz[o] * x[o + j] for the thread's
// column pair (same traversal as conv_channel with the roles of weights and accumulators swapped).
template <int ELL, int STEP, bool WIN, int R = kR>
__device__ __forceinline__ void grad_channel(const float* __restrict__ st, const int (&off)[4], const u64 (&gz)[R],
                                             u64 (&dw)[ELL], int gl = 0, int gh = 0) {
#pragma unroll
    for (int g = 0; g < (R + ELL - 1 + 3) / 4; ++g) {
        if (!WIN || (g >= gl && g < gh)) {
#pragma unroll
            for (int s = 4 * g; s < 4 * g + 4 && s < R + ELL - 1; ++s) {
                const float* p = st + off[s & 3] + (s >> 2) * STEP;
                const u64 x = *reinterpret_cast<const u64*>(p);
#pragma unroll
                for (int j = 0; j < ELL; ++j) {
                    const int o = s - j;
                    if (o >= 0 && o < R) fma2(dw[j], gz[o], x);
                }
            }
        }
    }
}

// Adds a float to a fixed-point accumulator (value * scale as a 64-bit integer): exact and order-free.
__device__ __forceinline__ void add_fixed(long long* dst, float v, double scale) {
    atomicAdd(reinterpret_cast<unsigned long long*>(dst), (unsigned long long)__double2ll_rn((double)v * scale));
}

// Sums dw[j] (both halves) over the warp and adds the ELL totals to dst[0..ELL).  A butterfly that
// halves the number of live values at every step leaves total j on the lanes with (lane >> 1) == j.
template <int ELL>
__device__ __forceinline__ void reduce_publish_dw(const u64 (&dw)[ELL], long long* dst, double scale, int lane) {
    float v[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        if (j < ELL) {
            float a, b;
            unpack2(dw[j], a, b);
            v[j] = a + b;
        } else {
            v[j] = 0.0f;
        }
    }
#pragma unroll
    for (int half = 8; half >= 1; half >>= 1) {
        const int mask = half * 2;
        const bool up = (lane & mask) != 0;
#pragma unroll
        for (int i = 0; i < half; ++i) {
            const float send = up ? v[i] : v[i + half];
            const float keep = up ? v[i + half] : v[i];
            v[i] = keep + __shfl_xor_sync(kFull, send, mask);
        }
    }
    const float total = v[0] + __shfl_xor_sync(kFull, v[0], 1);
    const int j = lane >> 1;
    if ((lane & 1) == 0 && j < ELL) add_fixed(dst + j, total, scale);
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

struct FwdArgs {
    PlanDevice plan;
    const float* X;
    int* feat_i;
    unsigned long long* ws;  // soft mode: (fixed-point sum, max key and index) per (example, kernel)
    float c1, c0;            // soft mode: lambda * log2 e, -shift * log2 e
    int N, C, L, K;
    // backward
    const float* dfeat;      // [N][2K]
    const int32_t* argmax;   // [N][K]
    long long* accfix;       // fixed-point sums: dW ragged [n_weights], then db [K]
    const double* scale;     // [K] fixed-point scale of every kernel's sums
    long long n_weights;
    float lambda;
    long long x_row_stride;  // floats between the channel rows of X (L, or the pitch of the zero-margined copy)
};

// ------------------------------------------------------------------------------------------------
// S regime
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void cp_async4_zfill(uint32_t dst, const void* src, bool ok) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(ok ? 4 : 0) : "memory");
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Backward second half for one kernel on an S tile: per channel, dW sums of the warp tile.
template <int ELL>
__device__ __forceinline__ void s_grad_tile(const float* planes, const KRec* rec, int lane, const u64 (&gz)[kRS],
                                            long long* accfix, double scale) {
    const int m = rec->m;
    const int off[4] = {2 * lane, kWarpCols + 2 * lane, 2 * kWarpCols + 2 * lane, 3 * kWarpCols + 2 * lane};
    for (int q = 0; q < m; ++q) {
        u64 dw[ELL];
#pragma unroll
        for (int j = 0; j < ELL; ++j) dw[j] = 0ull;
        grad_channel<ELL, 4 * kWarpCols, false, kRS>(planes + rec->ch[q] * kSPlaneFloats, off, gz, dw);
        reduce_publish_dw<ELL>(dw, accfix + rec->woff + q * ELL, scale, lane);
    }
}

// The channels of one kernel on an S tile.  fold: the accumulators come in undefined and start at the
// kernel's 0 - bias inside the first channel's pass (every output of the warp tile exists).
template <int ELL, bool FOLD>
__device__ __forceinline__ void s_kernel_tile(const float* planes, const KRec* rec, int lane, u64 (&acc)[kRS]) {
    const int m = rec->m;
    const int off[4] = {2 * lane, kWarpCols + 2 * lane, 2 * kWarpCols + 2 * lane, 3 * kWarpCols + 2 * lane};
    int q = 0;
    if constexpr (FOLD) {
        const float nb = rec->negb;
        conv_channel<ELL, 4 * kWarpCols, false, true, kRS>(planes + rec->ch[0] * kSPlaneFloats, off, rec->w2[0], acc, 0, 0, pack2(nb, nb));
        q = 1;
    }
    for (; q < m; ++q)
        conv_channel<ELL, 4 * kWarpCols, false, false, kRS>(planes + rec->ch[q] * kSPlaneFloats, off, rec->w2[q], acc);
}

// The same in half precision (mode 3).
template <int ELL>
__device__ __forceinline__ void s_kernel_tile_h(const float* planes, const KRec* rec, int lane, h2 (&acc)[kRS]) {
    const int m = rec->m;
    const int off[4] = {2 * lane, kWarpCols + 2 * lane, 2 * kWarpCols + 2 * lane, 3 * kWarpCols + 2 * lane};
    for (int q = 0; q < m; ++q)
        conv_channel_h<ELL, 4 * kWarpCols, false, kRS>(planes + rec->ch[q] * kSPlaneFloats, off, rec->w2[q], acc);
}

template <int MODE>  // 0 = hard, 1 = soft, 2 = backward of soft, 3 = hard in half precision
__global__ void __launch_bounds__(kSThreads, 1) fast_s_forward(FwdArgs a) {
    float* planes = reinterpret_cast<float*>(smem_raw);                               // [C][kRowsMax][64]
    KRec* recs = reinterpret_cast<KRec*>(planes + a.C * kSPlaneFloats);                // [warps][2]
    __shared__ unsigned s_item;
    __shared__ int s_next;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned n_items = (unsigned)a.plan.n_sitems;
    const unsigned long long total = (unsigned long long)a.N * n_items;
    KRec* myrec = recs + warp * 2;

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
        const bool tile_interior = item.interior != 0;
        const float* __restrict__ Xn = a.X + (size_t)n * a.C * a.x_row_stride;

        // stage the tile: every channel, rows 0..rows-1 of every column, zero outside the series
        {
            const int col = threadIdx.x & (kWarpCols - 1), rg = threadIdx.x / kWarpCols;
            const int cg = item.c0 + col;
            const bool col_ok = cg < b.raster_len;
            const int fu0 = s_column_u0(b, cg);
            for (int s = rg; s < b.rows; s += kSThreads / kWarpCols) {
                const int xi = fu0 + s * d;
                const bool ok = col_ok && (unsigned)xi < (unsigned)a.L;
                const float* __restrict__ src = Xn + (ok ? xi : 0);
                uint32_t dst = smem_u32(planes + s * kWarpCols + col);
#pragma unroll 4
                for (int c = 0; c < a.C; ++c) {
                    cp_async4_zfill(dst, src, ok);
                    src += a.x_row_stride;
                    dst += kSPlaneFloats * 4;
                }
            }
            cp_async_commit();
        }
        // the thread's two columns
        const int cg0 = item.c0 + 2 * lane;
        const bool ok0 = cg0 < b.raster_len, ok1 = cg0 + 1 < b.raster_len;
        const int band0 = cg0 / d, c0 = cg0 - band0 * d;          // (first A-row, residue) of the two columns
        const int band1 = c0 + 1 < d ? band0 : band0 + 1, c1 = c0 + 1 < d ? c0 + 1 : 0;
        const int trow0 = b.tmin + band0 * kRS, trow1 = b.tmin + band1 * kRS;
        if (threadIdx.x == 0) s_next = b.kbeg;
        cp_async_wait<0>();
        __syncthreads();

        // kernels of the bucket, pulled from the shared counter; the record of the next kernel is
        // copied into the warp's other slot while the current one computes
        auto fetch = [&](int k, int slot) {
            if (k < b.kend) {
                const char* src = reinterpret_cast<const char*>(a.plan.krec + k);
                const uint32_t dst = smem_u32(myrec + slot);
                for (int i = lane; i < (int)(sizeof(KRec) / 16); i += 32) cp_async16(dst + 16 * i, src + 16 * i);
            }
            cp_async_commit();
        };
        int kk = 0;
        if (lane == 0) kk = atomicAdd(&s_next, 1);
        kk = __shfl_sync(kFull, kk, 0);
        int cur = 0;
        fetch(kk, cur);
        while (kk < b.kend) {
            int kk_next = 0;
            if (lane == 0) kk_next = atomicAdd(&s_next, 1);
            kk_next = __shfl_sync(kFull, kk_next, 0);
            fetch(kk_next, cur ^ 1);
            cp_async_wait<1>();
            __syncwarp();
            const KRec* rec = myrec + cur;
            const int len = rec->len, korig = rec->k;
            // on an interior tile (the plan's flag) every output exists for every kernel of the bucket
            int lo0 = 0, hi0 = kRS, lo1 = 0, hi1 = kRS;
            bool interior = tile_interior;
            if (!tile_interior) {
                valid_rows_tc(trow0, c0, rec->tl, rec->rl, rec->th, rec->rh, kRS, ok0, lo0, hi0);
                valid_rows_tc(trow1, c1, rec->tl, rec->rl, rec->th, rec->rh, kRS, ok1, lo1, hi1);
                interior = __all_sync(kFull, lo0 == 0 && lo1 == 0 && hi0 == kRS && hi1 == kRS);
            }
            u64 acc[kRS];
            // hard mode: the pooling masks the outputs that do not exist, so the accumulators always start inside
            // the first channel's pass; the other modes start them at 0 - bias, or +inf where there is no output
            constexpr bool kFold = MODE == 0;
            if constexpr (MODE == 3) {
                h2 acch[kRS];
                init_acc_h(acch, rec->negb);
                if (len == 7) s_kernel_tile_h<7>(planes, rec, lane, acch);
                else if (len == 9) s_kernel_tile_h<9>(planes, rec, lane, acch);
                else s_kernel_tile_h<11>(planes, rec, lane, acch);
                widen_acc(acch, acc);
            } else {
                if (!kFold) init_acc(acc, rec->negb, interior, lo0, hi0, lo1, hi1);
                if (len == 7) s_kernel_tile<7, kFold>(planes, rec, lane, acc);
                else if (len == 9) s_kernel_tile<9, kFold>(planes, rec, lane, acc);
                else s_kernel_tile<11, kFold>(planes, rec, lane, acc);
            }
            if (MODE == 2) {
                const int64_t pair = (int64_t)n * a.K + korig;
                const float gP = __ldg(a.dfeat + 2 * pair), gM = __ldg(a.dfeat + 2 * pair + 1);
                const int uA = __ldg(a.argmax + pair) - rec->p;
                int tA = uA / d, cA = uA - tA * d;                        // floor division: uA >= -p may be negative
                if (cA < 0) { cA += d; --tA; }
                const int oA0 = (ok0 && c0 == cA && tA >= trow0 && tA < trow0 + kRS) ? tA - trow0 : -1;
                const int oA1 = (ok1 && c1 == cA && tA >= trow1 && tA < trow1 + kRS) ? tA - trow1 : -1;
                float dbs = make_gz(acc, a.c1, a.c0, gP * a.lambda / (float)rec->nout, gM, interior, lo0, hi0, lo1, hi1, oA0, oA1);
#pragma unroll
                for (int sh = 16; sh > 0; sh >>= 1) dbs += __shfl_xor_sync(kFull, dbs, sh);
                const double scale = __ldg(a.scale + korig);
                if (lane == 0) add_fixed(a.accfix + a.n_weights + korig, dbs, scale);
                if (len == 7) s_grad_tile<7>(planes, rec, lane, acc, a.accfix, scale);
                else if (len == 9) s_grad_tile<9>(planes, rec, lane, acc, a.accfix, scale);
                else s_grad_tile<11>(planes, rec, lane, acc, a.accfix, scale);
            } else if (MODE == 1) {
                const int p = rec->p;
                pool_publish_soft(a.ws, (int64_t)n * a.K + korig, acc, a.c1, a.c0, interior, lo0, hi0, lo1, hi1,
                                  trow0 * d + c0 + p, trow1 * d + c1 + p, d, lane);
            } else {
                int cnt = 0;
                float mn = __int_as_float(0x7f800000);
                if (interior) pool_hard(acc, cnt, mn);
                else pool_hard_masked(acc, row_mask(lo0, hi0), row_mask(lo1, hi1), cnt, mn);
                publish(a.feat_i, (int64_t)n * a.K + korig, cnt, mn, lane);
            }
            __syncwarp();  // every lane is done with the record before its slot is refilled
            kk = kk_next;
            cur ^= 1;
        }
        cp_async_wait<0>();
    }
}

// ------------------------------------------------------------------------------------------------
// T regime
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done != 0;
}
// Wait on a phase parity, bounded in time: returns false when the limit is reached (the caller
// records it and the block winds down).  Between polls the warp sleeps, so a waiting warp does
// not take issue slots from the warps that compute.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        __nanosleep(64);
        if (mbar_try(bar, parity)) return true;
        if (clock64() - t0 > kWaitLimitClocks) return false;
    }
}
// Bulk copy global -> shared (16-byte aligned addresses, size a multiple of 16), completion on bar.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// Tiled TMA load of one 4-D box (x a multiple of 4 floats), completion on bar.
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const void* tmap, int x, int y, int z, int w, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
        ::"r"(dst), "l"(tmap), "r"(x), "r"(y), "r"(z), "r"(w), "r"(bar) : "memory");
}

// What the producer tells the consumers about a tile (written with plain stores before its
// arrive on the stage's barrier, which releases them).
struct TSlotItem {
    int32_t t0, r0, rg, cg, box_rows, rec_slot, wide, g_lo;
    int32_t g_hi, n, stop, flags;         // n: example of the tile; stop: no tile, the block is done;
                                          // flags: the plan's warp_interior | warp_active << 8
};

// Dynamic shared memory of one group: the stages of its ring, then its kernel-record slots (a multiple of 128 bytes).
constexpr size_t kTGroupSmemBytes = ((size_t)kTStages * kTStageFloats * 4 + (size_t)kTParamSlots * sizeof(KRec) + 127) / 128 * 128;

struct TShared {
    unsigned long long full[kTStages];
    unsigned long long empty[kTStages];
    TSlotItem items[kTParamSlots];
    int abort;
};

// The channels of one tile for one consumer warp; returns false when a wait gave up.  A warp
// without a valid output (active == false) only keeps the ring moving.
template <int ELL, int STEP, bool WIN>
__device__ __forceinline__ bool t_channels(const float* stages, const KRec* rec, const int (&off)[4], uint32_t full0,
                                           uint32_t empty0, uint32_t& st, int lane, bool active, u64 (&acc)[kR], int gl,
                                           int gh) {
    const int m = rec->m;
    for (int q = 0; q < m; ++q) {
        const uint32_t slot = st % kTStages;
        if (q > 0 && !mbar_wait(full0 + 8u * slot, (st / kTStages) & 1u)) return false;
        if (active) conv_channel<ELL, STEP, WIN>(stages + slot * kTStageFloats, off, rec->w2[q], acc, gl, gh);
        __syncwarp();
        if (lane == 0) mbar_arrive(empty0 + 8u * slot);
        ++st;
    }
    return true;
}

// Backward second half on a T tile: the kernel's channels stream through the ring once more.
template <int ELL, int STEP, bool WIN>
__device__ __forceinline__ bool t_grad_channels(const float* stages, const KRec* rec, const int (&off)[4], uint32_t full0,
                                                uint32_t empty0, uint32_t& st, int lane, bool active, const u64 (&gz)[kR],
                                                long long* accfix, double scale, int gl, int gh) {
    const int m = rec->m;
    for (int q = 0; q < m; ++q) {
        const uint32_t slot = st % kTStages;
        if (!mbar_wait(full0 + 8u * slot, (st / kTStages) & 1u)) return false;
        if (active) {
            u64 dw[ELL];
#pragma unroll
            for (int j = 0; j < ELL; ++j) dw[j] = 0ull;
            grad_channel<ELL, STEP, WIN>(stages + slot * kTStageFloats, off, gz, dw, gl, gh);
            __syncwarp();
            if (lane == 0) mbar_arrive(empty0 + 8u * slot);
            reduce_publish_dw<ELL>(dw, accfix + rec->woff + q * ELL, scale, lane);
        } else {
            __syncwarp();
            if (lane == 0) mbar_arrive(empty0 + 8u * slot);
        }
        ++st;
    }
    return true;
}

template <int STEP, bool WIN>
__device__ __forceinline__ bool t_grad_dispatch(int len, const float* stages, const KRec* rec, const int (&off)[4],
                                                uint32_t full0, uint32_t empty0, uint32_t& st, int lane, bool active,
                                                const u64 (&gz)[kR], long long* accfix, double scale, int gl, int gh) {
    if (len == 7) return t_grad_channels<7, STEP, WIN>(stages, rec, off, full0, empty0, st, lane, active, gz, accfix, scale, gl, gh);
    if (len == 9) return t_grad_channels<9, STEP, WIN>(stages, rec, off, full0, empty0, st, lane, active, gz, accfix, scale, gl, gh);
    return t_grad_channels<11, STEP, WIN>(stages, rec, off, full0, empty0, st, lane, active, gz, accfix, scale, gl, gh);
}

template <int STEP, bool WIN>
__device__ __forceinline__ bool t_dispatch(int len, const float* stages, const KRec* rec, const int (&off)[4],
                                           uint32_t full0, uint32_t empty0, uint32_t& st, int lane, bool active,
                                           u64 (&acc)[kR], int gl, int gh) {
    if (len == 7) return t_channels<7, STEP, WIN>(stages, rec, off, full0, empty0, st, lane, active, acc, gl, gh);
    if (len == 9) return t_channels<9, STEP, WIN>(stages, rec, off, full0, empty0, st, lane, active, acc, gl, gh);
    return t_channels<11, STEP, WIN>(stages, rec, off, full0, empty0, st, lane, active, acc, gl, gh);
}

// The channels of one tile in half precision (mode 3).
template <int ELL, int STEP, bool WIN>
__device__ __forceinline__ bool t_channels_h(const float* stages, const KRec* rec, const int (&off)[4], uint32_t full0,
                                             uint32_t empty0, uint32_t& st, int lane, bool active, h2 (&acc)[kR], int gl,
                                             int gh) {
    const int m = rec->m;
    for (int q = 0; q < m; ++q) {
        const uint32_t slot = st % kTStages;
        if (q > 0 && !mbar_wait(full0 + 8u * slot, (st / kTStages) & 1u)) return false;
        if (active) conv_channel_h<ELL, STEP, WIN, kR>(stages + slot * kTStageFloats, off, rec->w2[q], acc, gl, gh);
        __syncwarp();
        if (lane == 0) mbar_arrive(empty0 + 8u * slot);
        ++st;
    }
    return true;
}
template <int STEP, bool WIN>
__device__ __forceinline__ bool t_dispatch_h(int len, const float* stages, const KRec* rec, const int (&off)[4],
                                             uint32_t full0, uint32_t empty0, uint32_t& st, int lane, bool active,
                                             h2 (&acc)[kR], int gl, int gh) {
    if (len == 7) return t_channels_h<7, STEP, WIN>(stages, rec, off, full0, empty0, st, lane, active, acc, gl, gh);
    if (len == 9) return t_channels_h<9, STEP, WIN>(stages, rec, off, full0, empty0, st, lane, active, acc, gl, gh);
    return t_channels_h<11, STEP, WIN>(stages, rec, off, full0, empty0, st, lane, active, acc, gl, gh);
}

template <int MODE>  // 0 = hard, 1 = soft, 2 = backward of soft, 3 = hard in half precision
__global__ void __launch_bounds__(kTBlockThreads, kTBlocksPerSM) fast_t_forward(FwdArgs a) {
    __shared__ __align__(16) TShared shs[kTGroups];
    // the block's groups work independently of one another: each has its part of the shared memory
    const int group = threadIdx.x / kTThreads, tid = threadIdx.x - group * kTThreads;
    TShared& sh = shs[group];
    // dynamic shared memory, aligned to 128 bytes by hand: per group its stages, then its kernel-record slots
    const uint32_t raw = smem_u32(smem_raw);
    unsigned char* base = smem_raw + (((raw + 127u) & ~127u) - raw) + (size_t)group * kTGroupSmemBytes;
    float* stages = reinterpret_cast<float*>(base);
    KRec* recs = reinterpret_cast<KRec*>(base + (size_t)kTStages * kTStageFloats * 4);
    const int lane = tid & 31, warp = tid >> 5;
    const uint32_t full0 = smem_u32(sh.full), empty0 = smem_u32(sh.empty);
    if (tid == 0) {
        for (int i = 0; i < kTStages; ++i) {
            mbar_init(full0 + 8u * i, 1);
            mbar_init(empty0 + 8u * i, kTConsumerWarps);
        }
        sh.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // Work is handed out in units of kTChunkTiles consecutive tiles of one example, example after
    // example (all blocks read one example at a time, so it stays in L2; consecutive tiles mostly
    // share a kernel).  The producer draws the units from a global counter and tells the consumers
    // what to do through the ring, a stop item last.
    const unsigned n_chunks = ((unsigned)a.plan.n_titems + kTChunkTiles - 1u) / kTChunkTiles;
    const unsigned total_units = (unsigned)a.N * n_chunks;
    volatile int* abort_flag = &sh.abort;

    if (warp == kTConsumerWarps) {
        // ---- producer: one lane issues every copy of the block
        if (lane == 0) {
            uint32_t st = 0, it = 0, nrec = 0;
            int cur_krec = -1;
            bool ok = true;
            unsigned u = atomicAdd(a.plan.counters + 1, 1u);
            while (ok && u < total_units) {
                const unsigned u_next = atomicAdd(a.plan.counters + 1, 1u);   // on its way while this unit is issued
                const int n = (int)(u / n_chunks);
                const int i_beg = (int)((u - (unsigned)n * n_chunks) * kTChunkTiles);
                const int i_end = min(i_beg + (int)kTChunkTiles, a.plan.n_titems);
                const int4* tp = reinterpret_cast<const int4*>(a.plan.titems + i_beg);
                int4 w0 = __ldg(tp), w1 = __ldg(tp + 1), w2 = __ldg(tp + 2), w3 = __ldg(tp + 3), w4 = __ldg(tp + 4),
                     w5 = __ldg(tp + 5), w6 = __ldg(tp + 6), w7 = __ldg(tp + 7);
                for (int i = i_beg; ok && i < i_end; ++i) {
                    if (*abort_flag) { ok = false; break; }
                    const int map = w0.x, t0 = w0.y, r0 = w0.z, rg = w0.w;
                    const int m = w1.z, box_rows = w1.w, krec = w2.w, cg = w3.x, wide = w3.y, g_lo = w3.z, g_hi = w3.w;
                    const unsigned chw[3] = {(unsigned)w2.x, (unsigned)w2.y, (unsigned)w2.z};
                    const int px[4] = {w4.x, w4.y, w4.z, w4.w}, py[4] = {w5.x, w5.y, w5.z, w5.w}, pj[4] = {w6.x, w6.y, w6.z, w6.w};
                    const int run = 4 * w1.x;
                    const int flags = (w7.x & 0xff) | ((w7.y & 0xff) << 8);
                    {   // the next tile's description is on its way while this one is issued
                        const int inext = min(i + 1, i_end - 1);
                        tp = reinterpret_cast<const int4*>(a.plan.titems + inext);
                        w0 = __ldg(tp); w1 = __ldg(tp + 1); w2 = __ldg(tp + 2); w3 = __ldg(tp + 3); w4 = __ldg(tp + 4);
                        w5 = __ldg(tp + 5); w6 = __ldg(tp + 6); w7 = __ldg(tp + 7);
                    }
                    const uint32_t box_bytes = (uint32_t)box_rows * (uint32_t)t_box_cols(cg) * 4u;
                    const uint32_t phase_bytes = (uint32_t)t_phase_floats(cg, box_rows) * 4u;
                    const char* tmap = reinterpret_cast<const char*>(a.plan.tmaps) + (size_t)map * 128;
                    const bool new_rec = krec != cur_krec;
                    if (new_rec) { cur_krec = krec; ++nrec; }
                    const uint32_t rslot = (nrec - 1u) % kTParamSlots;
                    const int n_stages = MODE == 2 ? 2 * m : m;   // the backward streams the channels twice
                    for (int q2 = 0; q2 < n_stages; ++q2) {
                        const int q = q2 < m ? q2 : q2 - m;
                        const uint32_t slot = st % kTStages;
                        if (st >= (uint32_t)kTStages && !mbar_wait(empty0 + 8u * slot, ((st / kTStages) - 1u) & 1u)) {
                            ok = false;
                            break;
                        }
                        const uint32_t bar = full0 + 8u * slot;
                        uint32_t tx = (wide ? 4u * (uint32_t)kTWideHalves : 4u) * box_bytes;
                        if (q2 == 0) {
                            TSlotItem& si = sh.items[it % kTParamSlots];
                            si.t0 = t0; si.r0 = r0; si.rg = rg; si.cg = cg; si.box_rows = box_rows; si.rec_slot = (int)rslot;
                            si.wide = wide; si.g_lo = g_lo; si.g_hi = g_hi; si.n = n; si.stop = 0; si.flags = flags;
                            if (new_rec) tx += (uint32_t)sizeof(KRec);
                        }
                        mbar_arrive_expect_tx(bar, tx);
                        if (q2 == 0 && new_rec) bulk_g2s(smem_u32(recs + rslot), a.plan.krec + krec, (uint32_t)sizeof(KRec), bar);
                        const int ch = (int)((chw[q >> 2] >> (8 * (q & 3))) & 0xffu);
                        const int z = n * a.C + ch;
                        const uint32_t dst0 = smem_u32(stages + slot * kTStageFloats);
#pragma unroll
                        for (int k = 0; k < 4; ++k) tma_load_4d(dst0 + (uint32_t)k * phase_bytes, tmap, px[k], py[k], z, pj[k], bar);
                        if (wide) {   // the further halves: the boxes 256 columns further right each
                            for (int h = 1; h < kTWideHalves; ++h) {
#pragma unroll
                                for (int k = 0; k < 4; ++k) {
                                    int x2 = px[k] + h * kTWideCols, y2 = py[k];
                                    while (x2 >= run) { x2 -= run; ++y2; }
                                    tma_load_4d(dst0 + (uint32_t)(4 * h + k) * phase_bytes, tmap, x2, y2, z, pj[k], bar);
                                }
                            }
                        }
                        ++st;
                    }
                    ++it;
                }
                u = u_next;
            }
            if (ok) {   // the stop item takes a stage of its own (no copy)
                const uint32_t slot = st % kTStages;
                if (st >= (uint32_t)kTStages && !mbar_wait(empty0 + 8u * slot, ((st / kTStages) - 1u) & 1u)) {
                    ok = false;
                } else {
                    sh.items[it % kTParamSlots].stop = 1;
                    mbar_arrive(full0 + 8u * slot);
                    ++st;
                }
            }
            if (!ok) {
                *abort_flag = 1;
                atomicExch(a.plan.error_flag, 1);
            }
            // nothing of this block may still be in flight when it exits: every issued stage has
            // either been consumed or is waited for here (bounded)
            for (uint32_t back = 1; back <= (uint32_t)kTStages && back <= st; ++back) {
                const uint32_t s2 = st - back;
                mbar_wait(full0 + 8u * (s2 % kTStages), (s2 / kTStages) & 1u);
            }
        }
    } else {
        // ---- consumers
        uint32_t st = 0, it = 0;
        bool ok = true;
        // hard mode: the count and the min(-z) of the (example, kernel) pair the warp is working on travel from
        // tile to tile (consecutive tiles mostly share a kernel) and are published when the pair changes
        int64_t cur_pair = -1;
        int cnt = 0;
        float mn = __int_as_float(0x7f800000);
        for (;;) {
            if (*abort_flag) { ok = false; break; }
            const uint32_t slot = st % kTStages;
            if (!mbar_wait(full0 + 8u * slot, (st / kTStages) & 1u)) {
                ok = false;
                break;
            }
            const TSlotItem si = sh.items[it % kTParamSlots];
            if (si.stop) break;
            const int n = si.n;
            const KRec* rec = recs + si.rec_slot;
            const int t0 = si.t0, r0 = si.r0, cg = si.cg, box_rows = si.box_rows;
            const int len = rec->len, d = rec->d, korig = rec->k;
            const bool wide = si.wide != 0;
            // warp tile (wr, wc) of the tile; a wide tile is one row of all consumer warps' tiles
            const int wr = wide ? 0 : (cg == 1 ? warp : (cg == 2 ? warp >> 1 : warp >> 2));
            const int wc = wide ? warp : (warp & (cg - 1));
            const int lc = kWarpCols * wc + 2 * lane;
            // the plan says per warp whether every / any output of its warp tile exists
            bool interior = ((si.flags >> warp) & 1) != 0;
            const bool active = ((si.flags >> (8 + warp)) & 1) != 0;
            const bool ok0 = active && r0 + lc < d, ok1 = active && r0 + lc + 1 < d;
            int lo0 = 0, hi0 = kR, lo1 = 0, hi1 = kR;
            if (active && !interior) {
                valid_rows_tc(t0 + kR * wr, r0 + lc, rec->tl, rec->rl, rec->th, rec->rh, kR, ok0, lo0, hi0);
                valid_rows_tc(t0 + kR * wr, r0 + lc + 1, rec->tl, rec->rl, rec->th, rec->rh, kR, ok1, lo1, hi1);
            }
            // where rows 0..3 of the warp tile sit in a stage: the box of phase k starts k * phase floats in; an
            // ordinary tile's warp tile starts 4 wr box rows down, a wide tile's in half lc / 256, g_lo box rows up
            // (t_elem_offset / t_wide_elem_offset for tile rows 0..3)
            const int boxw = wide ? kTWideCols : t_box_cols(cg);
            const int phase = box_rows * boxw;
            const int base = wide ? (lc >> 8) * (4 * phase) - si.g_lo * kTWideCols + (lc & (kTWideCols - 1)) : 4 * wr * boxw + lc;
            const int off[4] = {base, base + phase, base + 2 * phase, base + 3 * phase};
            const int gl = si.g_lo, gh = si.g_hi;
            u64 acc[kR];
            // Hard mode: every accumulator starts at 0 - bias and the pooling masks the outputs that do not exist.
            // The other modes start at +inf where there is no output.  (Starting the accumulators inside the first
            // channel's pass, as the small-dilation kernel does, doubles the inner-loop instances here: measured
            // slower, the kernel then waits for instructions.)
            if constexpr (MODE == 3) {
                h2 acch[kR];
                init_acc_h(acch, rec->negb);
                if (wide) ok = t_dispatch_h<kTWideCols, true>(len, stages, rec, off, full0, empty0, st, lane, active, acch, gl, gh);
                else if (cg == 1) ok = t_dispatch_h<kWarpCols, false>(len, stages, rec, off, full0, empty0, st, lane, active, acch, 0, 0);
                else if (cg == 2) ok = t_dispatch_h<2 * kWarpCols, false>(len, stages, rec, off, full0, empty0, st, lane, active, acch, 0, 0);
                else ok = t_dispatch_h<4 * kWarpCols, false>(len, stages, rec, off, full0, empty0, st, lane, active, acch, 0, 0);
                widen_acc(acch, acc);
            } else {
                if (active) init_acc(acc, rec->negb, interior || MODE == 0, lo0, hi0, lo1, hi1);
                if (wide) ok = t_dispatch<kTWideCols, true>(len, stages, rec, off, full0, empty0, st, lane, active, acc, gl, gh);
                else if (cg == 1) ok = t_dispatch<kWarpCols, false>(len, stages, rec, off, full0, empty0, st, lane, active, acc, 0, 0);
                else if (cg == 2) ok = t_dispatch<2 * kWarpCols, false>(len, stages, rec, off, full0, empty0, st, lane, active, acc, 0, 0);
                else ok = t_dispatch<4 * kWarpCols, false>(len, stages, rec, off, full0, empty0, st, lane, active, acc, 0, 0);
            }
            if (!ok) break;
            const int64_t pair = (int64_t)n * a.K + korig;
            if (MODE == 2) {
                double scale = 0.0;
                if (active) {
                    const float gP = __ldg(a.dfeat + 2 * pair), gM = __ldg(a.dfeat + 2 * pair + 1);
                    const int uA = __ldg(a.argmax + pair) - rec->p;
                    int tA = uA / d, cA = uA - tA * d;                        // floor division: uA >= -p may be negative
                    if (cA < 0) { cA += d; --tA; }
                    const int trow = t0 + kR * wr, c0 = r0 + lc;
                    const bool rowhit = tA >= trow && tA < trow + kR;
                    const int oA0 = (ok0 && rowhit && c0 == cA) ? tA - trow : -1;
                    const int oA1 = (ok1 && rowhit && c0 + 1 == cA) ? tA - trow : -1;
                    float dbs = make_gz(acc, a.c1, a.c0, gP * a.lambda / (float)rec->nout, gM, interior, lo0, hi0, lo1, hi1, oA0,
                                        oA1);
#pragma unroll
                    for (int sh = 16; sh > 0; sh >>= 1) dbs += __shfl_xor_sync(kFull, dbs, sh);
                    scale = __ldg(a.scale + korig);
                    if (lane == 0) add_fixed(a.accfix + a.n_weights + korig, dbs, scale);
                }
                if (wide) ok = t_grad_dispatch<kTWideCols, true>(len, stages, rec, off, full0, empty0, st, lane, active, acc, a.accfix, scale, gl, gh);
                else if (cg == 1) ok = t_grad_dispatch<kWarpCols, false>(len, stages, rec, off, full0, empty0, st, lane, active, acc, a.accfix, scale, 0, 0);
                else if (cg == 2) ok = t_grad_dispatch<2 * kWarpCols, false>(len, stages, rec, off, full0, empty0, st, lane, active, acc, a.accfix, scale, 0, 0);
                else ok = t_grad_dispatch<4 * kWarpCols, false>(len, stages, rec, off, full0, empty0, st, lane, active, acc, a.accfix, scale, 0, 0);
                if (!ok) break;
            } else if (active) {
                if (MODE == 1) {
                    const int base = (t0 + kR * wr) * d + r0 + lc + rec->p;
                    pool_publish_soft(a.ws, pair, acc, a.c1, a.c0, interior, lo0, hi0, lo1, hi1, base, base + 1, d, lane);
                } else {
                    if (pair != cur_pair) {
                        if (cur_pair >= 0) publish(a.feat_i, cur_pair, cnt, mn, lane);
                        cur_pair = pair;
                        cnt = 0;
                        mn = __int_as_float(0x7f800000);
                    }
                    if (interior) pool_hard(acc, cnt, mn);
                    else pool_hard_masked(acc, row_mask(lo0, hi0), row_mask(lo1, hi1), cnt, mn);
                }
            }
            ++it;
        }
        // what the warp still carries is published even when a wait gave up: counts and maxima are only
        // ever combined with commutative atomics, and the error flag marks the result as incomplete
        if ((MODE == 0 || MODE == 3) && cur_pair >= 0) publish(a.feat_i, cur_pair, cnt, mn, lane);
        if (!ok) {
            *abort_flag = 1;
            if (lane == 0) atomicExch(a.plan.error_flag, 1);
        }
    }
    __syncthreads();  // every wait above is bounded, so every warp gets here
}

// ------------------------------------------------------------------------------------------------
// pad copy / init / finalise
// ------------------------------------------------------------------------------------------------
// Writes the samples of the batch into the four shifted copies: copy j holds the zero-margined
// layout moved down by j floats (copy_j[i] = layout[i + j]); margins are never written and stay zero.
__global__ void fast_pad_copy_kernel(const float4* __restrict__ X, float* __restrict__ xpad, int64_t rows, int L4,
                                     int64_t pitch, int front, int64_t copy_floats) {
    const int64_t total = rows * L4;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t rho = e / L4;
        const int i = (int)(e - rho * L4);
        const float4 v = __ldg(X + e);
        float* dst = xpad + rho * pitch + front + 4 * (int64_t)i;
        *reinterpret_cast<float4*>(dst) = v;
#pragma unroll
        for (int j = 1; j < 4; ++j) {
            float* dj = dst + j * copy_floats - j;
            dj[0] = v.x; dj[1] = v.y; dj[2] = v.z; dj[3] = v.w;
        }
    }
}

// The same for series whose length is not a multiple of four floats, or whose base is not 16-byte aligned:
// one float per thread and step.
__global__ void fast_pad_copy_scalar_kernel(const float* __restrict__ X, float* __restrict__ xpad, int64_t rows, int L,
                                            int64_t pitch, int front, int64_t copy_floats) {
    const int64_t total = rows * L;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t rho = e / L;
        const int i = (int)(e - rho * L);
        const float v = __ldg(X + e);
        float* dst = xpad + rho * pitch + front + i;
#pragma unroll
        for (int j = 0; j < 4; ++j) dst[j * copy_floats - j] = v;
    }
}

// The same from raw 8-bit intensities (Section 4.1): every sample becomes (v - mean[c]) * inv_std[c]
// (per-channel feature scaling, Section 4.3) on its way into the four copies.
__global__ void fast_pad_copy_u8_kernel(const uchar4* __restrict__ X, float* __restrict__ xpad, int64_t rows, int L4,
                                        int C, int64_t pitch, int front, int64_t copy_floats, NormArgs norm) {
    const int64_t total = rows * L4;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t rho = e / L4;
        const int i = (int)(e - rho * L4);
        const int c = (int)(rho % C);
        const uchar4 u = __ldg(X + e);
        const float mu = norm.mean[c], is = norm.inv_std[c];
        float4 v;
        v.x = ((float)u.x - mu) * is; v.y = ((float)u.y - mu) * is;
        v.z = ((float)u.z - mu) * is; v.w = ((float)u.w - mu) * is;
        float* dst = xpad + rho * pitch + front + 4 * (int64_t)i;
        *reinterpret_cast<float4*>(dst) = v;
#pragma unroll
        for (int j = 1; j < 4; ++j) {
            float* dj = dst + j * copy_floats - j;
            dj[0] = v.x; dj[1] = v.y; dj[2] = v.z; dj[3] = v.w;
        }
    }
}

__global__ void fast_init_kernel(int* __restrict__ feat_i, int64_t pairs, unsigned* counters) {
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e == 0) { counters[0] = 0u; counters[1] = 0u; }
    if (e < pairs) { feat_i[2 * e] = 0; feat_i[2 * e + 1] = INT_MIN; }
}

__global__ void fast_finalize_kernel(float* __restrict__ feat, const KRec* __restrict__ krec, int n_krec, int N,
                                     int K) {
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= (int64_t)N * n_krec) return;
    const int n = (int)(e / n_krec), f = (int)(e - (int64_t)n * n_krec);
    const int k = krec[f].k, nout = krec[f].nout;
    int* fi = reinterpret_cast<int*>(feat) + ((int64_t)n * K + k) * 2;
    const int cnt = fi[0], key = fi[1];
    feat[((int64_t)n * K + k) * 2] = (float)cnt / (float)nout;   // Eq. 2
    feat[((int64_t)n * K + k) * 2 + 1] = key_float(key);
}

__global__ void fast_init_soft_kernel(unsigned long long* __restrict__ ws, int64_t pairs, unsigned* counters) {
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e == 0) { counters[0] = 0u; counters[1] = 0u; }
    if (e < pairs) { ws[2 * e] = 0ull; ws[2 * e + 1] = 0ull; }
}

__global__ void fast_finalize_soft_kernel(float* __restrict__ feat, int32_t* __restrict__ argmax,
                                          const unsigned long long* __restrict__ ws, const KRec* __restrict__ krec,
                                          int n_krec, int N, int K) {
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= (int64_t)N * n_krec) return;
    const int n = (int)(e / n_krec), f = (int)(e - (int64_t)n * n_krec);
    const int k = krec[f].k, nout = krec[f].nout;
    const int64_t pair = (int64_t)n * K + k;
    const unsigned long long sum = ws[2 * pair], k64 = ws[2 * pair + 1];
    feat[pair * 2] = (float)((double)sum / (double)kSoftFixedScale / (double)nout);   // Eq. 4
    feat[pair * 2 + 1] = key_float((int)((unsigned)(k64 >> 32) ^ 0x80000000u));
    if (argmax) argmax[pair] = INT_MAX - (int)(unsigned)(k64 & 0xffffffffull);
}

size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

size_t s_smem_bytes(int C) { return (size_t)C * kSPlaneFloats * 4 + (size_t)kSWarps * 2 * sizeof(KRec); }
size_t t_smem_bytes() { return (size_t)kTGroups * kTGroupSmemBytes + 128; }

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// Opts every fused kernel into its dynamic shared memory size, once per device.
cudaError_t set_kernel_attributes(int dev) {
    cudaError_t e = cudaSuccess;
    static std::mutex attr_mu;
    std::lock_guard<std::mutex> attr_lock(attr_mu);
    static bool attr_done_for[64] = {};
    bool& attr_done = attr_done_for[dev & 63];
    const size_t t_bytes = t_smem_bytes();
    if (!attr_done) {
        e = cudaFuncSetAttribute(fast_s_forward<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)s_smem_bytes(kSMaxChannels));
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(fast_s_forward<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)s_smem_bytes(kSMaxChannels));
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(fast_t_forward<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)t_bytes);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(fast_t_forward<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)t_bytes);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(fast_s_forward<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)s_smem_bytes(kSMaxChannels));
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(fast_t_forward<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)t_bytes);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(fast_s_forward<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)s_smem_bytes(kSMaxChannels));
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(fast_t_forward<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)t_bytes);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    return cudaSuccess;
}

// ---- backward helpers ----------------------------------------------------------------------------
// Largest |x| of the batch, as the bit pattern of a non-negative float (integer order = float order).
__global__ void fast_absmax_scalar_kernel(const float* __restrict__ X, int64_t n, unsigned* __restrict__ out) {
    float m = 0.0f;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (int64_t)gridDim.x * blockDim.x)
        m = fmaxf(m, fabsf(__ldg(X + e)));
    unsigned b = __float_as_uint(m);
    b = __reduce_max_sync(kFull, b);
    if ((threadIdx.x & 31) == 0) atomicMax(out, b);
}

__global__ void fast_absmax_kernel(const float4* __restrict__ X, int64_t n4, unsigned* __restrict__ out) {
    float m = 0.0f;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < n4; e += (int64_t)gridDim.x * blockDim.x) {
        const float4 v = __ldg(X + e);
        m = fmaxf(fmaxf(m, fabsf(v.x)), fmaxf(fabsf(v.y), fmaxf(fabsf(v.z), fabsf(v.w))));
    }
    unsigned b = __float_as_uint(m);
    b = __reduce_max_sync(kFull, b);
    if ((threadIdx.x & 31) == 0) atomicMax(out, b);
}

// Per kernel: a bound on sum |gz| |x| over the batch gives the fixed-point scale of its sums
// (|sum_i gz_i| <= |gP| lambda / 4 + |gM| per example since h (1 - h) <= 1/4), and its sums are cleared.
__global__ void fast_bwd_prepare_kernel(const float* __restrict__ dfeat, const KRec* __restrict__ krec, int n_krec, int N,
                                        int K, float lambda, const unsigned* __restrict__ absmax_bits,
                                        double* __restrict__ scale, long long* __restrict__ accfix, long long n_weights) {
    const int f = blockIdx.x * blockDim.x + threadIdx.x;
    if (f >= n_krec) return;
    const int k = krec[f].k;
    double bound = 0.0;
    for (int n = 0; n < N; ++n) {
        const float gP = dfeat[((int64_t)n * K + k) * 2], gM = dfeat[((int64_t)n * K + k) * 2 + 1];
        bound += (double)fabsf(gP) * (double)fabsf(lambda) * 0.25 + (double)fabsf(gM);
    }
    const double xmax = fmax((double)__uint_as_float(*absmax_bits), 1.0);
    bound *= xmax * 1.01;
    scale[k] = (bound > 0.0 && bound < 1e300) ? 1152921504606846976.0 / bound : 0.0;  // 2^60 / bound
    const int taps = krec[f].m * krec[f].len;
    for (int t = 0; t < taps; ++t) accfix[krec[f].woff + t] = 0;
    accfix[n_weights + k] = 0;
}

__global__ void fast_bwd_finalize_kernel(const long long* __restrict__ accfix, const double* __restrict__ scale,
                                         const KRec* __restrict__ krec, int n_krec, long long n_weights,
                                         float* __restrict__ dW, float* __restrict__ db) {
    const int f = blockIdx.x * blockDim.x + threadIdx.x;
    if (f >= n_krec) return;
    const int k = krec[f].k;
    const double sc = scale[k], inv = sc > 0.0 ? 1.0 / sc : 0.0;
    const int taps = krec[f].m * krec[f].len;
    for (int t = 0; t < taps; ++t) dW[krec[f].woff + t] = (float)((double)accfix[krec[f].woff + t] * inv);
    db[k] = (float)((double)accfix[n_weights + k] * inv);
}

}  // namespace

// Blocks of the T kernel: as many as are resident at a time, never more than there are work units.
static unsigned t_grid(int n_examples, int n_titems, int sms) {
    const unsigned long long units = (unsigned long long)n_examples * ((n_titems + kTChunkTiles - 1) / kTChunkTiles);
    return (unsigned)std::min<unsigned long long>((units + kTGroups - 1) / kTGroups, (unsigned long long)kTBlocksPerSM * (unsigned long long)sms);
}

cudaError_t upload_plan(FastState& fs) {
    const PlanHost& h = fs.host;
    PlanDevice& d = fs.dev;
    d = PlanDevice();
    struct Part { const void* src; size_t bytes; size_t off; };
    Part parts[7] = {
        {h.krec.data(), h.krec.size() * sizeof(KRec), 0},   {h.sb.data(), h.sb.size() * sizeof(SBucket), 0},
        {h.sitems.data(), h.sitems.size() * sizeof(SItem), 0}, {h.titems.data(), h.titems.size() * sizeof(TItem), 0},
        {h.generic_list.data(), h.generic_list.size() * 4, 0}, {nullptr, 256, 0}, {nullptr, 256, 0}};
    size_t total = 0;
    for (auto& pt : parts) { pt.off = total; total += align256(pt.bytes); }
    cudaError_t e = device_malloc(&fs.plan_blob, std::max<size_t>(total, 256));
    if (e != cudaSuccess) { fs.plan_blob = nullptr; return e; }
    char* base = static_cast<char*>(fs.plan_blob);
    e = cudaMemset(base, 0, std::max<size_t>(total, 256));
    for (auto& pt : parts)
        if (e == cudaSuccess && pt.src && pt.bytes) e = cudaMemcpy(base + pt.off, pt.src, pt.bytes, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) { cudaFree(fs.plan_blob); fs.plan_blob = nullptr; return e; }
    d.krec = reinterpret_cast<const KRec*>(base + parts[0].off);
    d.sb = reinterpret_cast<const SBucket*>(base + parts[1].off);
    d.sitems = reinterpret_cast<const SItem*>(base + parts[2].off);
    d.titems = reinterpret_cast<const TItem*>(base + parts[3].off);
    d.generic_list = reinterpret_cast<const int32_t*>(base + parts[4].off);
    d.counters = reinterpret_cast<unsigned*>(base + parts[5].off);
    d.error_flag = reinterpret_cast<int*>(base + parts[6].off);
    d.n_krec = (int)h.krec.size(); d.n_sitems = (int)h.sitems.size(); d.n_titems = (int)h.titems.size();
    d.n_generic = (int)h.generic_list.size(); d.n_tmaps = (int)h.tmaps.size();
    d.pad_pitch = h.pad_pitch;
    return cudaSuccess;
}

cudaError_t upload_records(FastState& fs) {
    if (!fs.plan_blob || fs.host.krec.empty()) return cudaSuccess;
    return cudaMemcpy(const_cast<KRec*>(fs.dev.krec), fs.host.krec.data(), fs.host.krec.size() * sizeof(KRec),
                      cudaMemcpyHostToDevice);
}

void release_fast_state(FastState& fs) {
    if (fs.plan_blob) cudaFree(fs.plan_blob);
    if (fs.maps_blob) cudaFree(fs.maps_blob);
    if (fs.xpad) cudaFree(fs.xpad);
    if (fs.soft_ws) cudaFree(fs.soft_ws);
    if (fs.bwd_ws) cudaFree(fs.bwd_ws);
    fs.bwd_ws = nullptr;
    fs.soft_ws = nullptr;
    fs.soft_ws_bytes = 0;
    for (cudaEvent_t ev : fs.evs) cudaEventDestroy(ev);
    fs.evs.clear();
    fs.ev_chunks = 0;
    fs.plan_blob = fs.maps_blob = nullptr;
    fs.xpad = nullptr;
    fs.pad_examples = 0;
}

cudaError_t ensure_pad_capacity(FastState& fs, int N, int C, int L, bool without_maps) {
    if ((fs.host.tmaps.empty() && !without_maps) || N <= fs.pad_examples) return cudaSuccess;
    EncodeTiledFn encode = fs.host.tmaps.empty() ? nullptr : encode_tiled_fn();
    if (!encode && !fs.host.tmaps.empty()) return cudaErrorNotSupported;
    const int64_t pitch = fs.host.pad_pitch, rows = (int64_t)N * C;
    const int64_t copy_floats = (rows + 1) * pitch;   // pitch is a multiple of 32 floats
    const size_t bytes = (size_t)copy_floats * 4 * 4;
    if (fs.xpad) cudaFree(fs.xpad);  // waits for work that still reads it
    fs.xpad = nullptr;
    fs.pad_examples = 0;
    cudaError_t e = device_malloc(reinterpret_cast<void**>(&fs.xpad), bytes);
    if (e != cudaSuccess) { fs.xpad = nullptr; return e; }
    e = cudaMemset(fs.xpad, 0, bytes);  // the margins stay zero from here on: the pad copy writes samples only
    if (e != cudaSuccess) return e;
    const size_t n_maps = fs.host.tmaps.size();
    std::vector<CUtensorMap> maps(n_maps);
    for (size_t i = 0; i < n_maps; ++i) {
        const TMapSpec& sp = fs.host.tmaps[i];
        const cuuint64_t run = 4ull * (cuuint64_t)sp.d;
        const cuuint64_t dims[4] = {run + kTXExtra, ((cuuint64_t)kTPadFront + (cuuint64_t)L + run - 1) / run, (cuuint64_t)rows, 4ull};
        const cuuint64_t strides[3] = {run * 4ull, (cuuint64_t)pitch * 4ull, (cuuint64_t)copy_floats * 4ull};
        const cuuint32_t box[4] = {(cuuint32_t)sp.box_cols, (cuuint32_t)sp.box_rows, 1u, 1u};
        const cuuint32_t elem[4] = {1u, 1u, 1u, 1u};
        const CUresult r = encode(&maps[i], CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, fs.xpad, dims, strides, box, elem,
                                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                                  CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    }
    static_assert(sizeof(CUtensorMap) == 128, "tensor maps are addressed in 128-byte steps");
    if (n_maps > 0) {
        if (!fs.maps_blob) {
            e = device_malloc(&fs.maps_blob, n_maps * sizeof(CUtensorMap));
            if (e != cudaSuccess) { fs.maps_blob = nullptr; return e; }
        }
        e = cudaMemcpy(fs.maps_blob, maps.data(), n_maps * sizeof(CUtensorMap), cudaMemcpyHostToDevice);
        if (e != cudaSuccess) return e;
    }
    fs.pad_examples = N;
    fs.copy_floats = copy_floats;
    fs.dev.tmaps = fs.maps_blob;
    fs.dev.xpad = fs.xpad;
    return cudaSuccess;
}

// Writes `rows` channel rows of X into the four shifted zero-margined copies (16-byte pieces when the rows allow).
static void launch_pad_copy(FastState& fs, const float* X, int64_t rows, int L, int sms, cudaStream_t stream) {
    if (L % 4 == 0 && (reinterpret_cast<uintptr_t>(X) & 15u) == 0)
        fast_pad_copy_kernel<<<sms * 8, 256, 0, stream>>>(reinterpret_cast<const float4*>(X), fs.xpad, rows, L / 4, fs.host.pad_pitch,
                                                          kTPadFront, fs.copy_floats);
    else
        fast_pad_copy_scalar_kernel<<<sms * 8, 256, 0, stream>>>(X, fs.xpad, rows, L, fs.host.pad_pitch, kTPadFront, fs.copy_floats);
    count_launch();
}

// Soft transform: 16 bytes per (example, kernel), grow-only.
static cudaError_t ensure_soft_ws(FastState& fs, int64_t pairs) {
    if ((size_t)pairs * 16 <= fs.soft_ws_bytes) return cudaSuccess;
    if (fs.soft_ws) cudaFree(fs.soft_ws);  // waits for work that still uses it
    fs.soft_ws = nullptr;
    fs.soft_ws_bytes = 0;
    cudaError_t e = device_malloc(&fs.soft_ws, (size_t)pairs * 16);
    if (e != cudaSuccess) { fs.soft_ws = nullptr; return e; }
    fs.soft_ws_bytes = (size_t)pairs * 16;
    return cudaSuccess;
}

// Backward: fixed-point sums [n_weights + K], scales [K], max |x| (fixed size per handle).
static cudaError_t ensure_bwd_ws(FastState& fs, const DeviceParams& dp, int64_t n_weights) {
    if (fs.bwd_ws) return cudaSuccess;
    const size_t acc_bytes = align256((size_t)(n_weights + dp.K) * 8), scale_bytes = align256((size_t)dp.K * 8);
    cudaError_t e = device_malloc(&fs.bwd_ws, acc_bytes + scale_bytes + 256);
    if (e != cudaSuccess) fs.bwd_ws = nullptr;
    return e;
}

cudaError_t reserve_fast_state(FastState& fs, const DeviceParams& dp, int max_N, bool soft, bool backward, bool u8,
                               int64_t n_weights) {
    std::lock_guard<std::mutex> lk(fs.mu);
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if ((e = set_kernel_attributes(dev)) != cudaSuccess) return e;
    if (fs.dev.n_titems > 0 || u8) {
        e = ensure_pad_capacity(fs, std::min(max_N, kChunkExamples), dp.C, dp.L, u8 && fs.dev.n_titems == 0);
        if (e != cudaSuccess) return e;
    }
    if (soft && (e = ensure_soft_ws(fs, (int64_t)max_N * dp.K)) != cudaSuccess) return e;
    if (backward && (e = ensure_bwd_ws(fs, dp, n_weights)) != cudaSuccess) return e;
    return cudaSuccess;
}

cudaError_t launch_fast_forward(FastState& fs, const DeviceParams& dp, const float* X, int N, float* feat,
                                cudaStream_t stream, bool soft, float lambda, float shift, int32_t* argmax,
                                const uint8_t* X_u8, const NormArgs* norm, bool half) {
    if (half && soft) return cudaErrorInvalidValue;
    std::lock_guard<std::mutex> lk(fs.mu);
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    e = set_kernel_attributes(dev);
    if (e != cudaSuccess) return e;
    const size_t s_bytes = s_smem_bytes(dp.C), t_bytes = t_smem_bytes();
    const PlanDevice& pd = fs.dev;
    if (pd.n_titems > 0 || X_u8) {
        e = ensure_pad_capacity(fs, std::min(N, kChunkExamples), dp.C, dp.L, X_u8 != nullptr);
        if (e != cudaSuccess) return e;
    }
    const int64_t pairs = (int64_t)N * dp.K;
    if (soft && (e = ensure_soft_ws(fs, pairs)) != cudaSuccess) return e;
    FwdArgs a;
    a.plan = fs.dev;
    a.c1 = lambda * 1.4426950408889634f; a.c0 = -shift * 1.4426950408889634f;
    a.C = dp.C; a.L = dp.L; a.K = dp.K;
    a.dfeat = nullptr; a.argmax = nullptr; a.accfix = nullptr; a.scale = nullptr; a.n_weights = 0; a.lambda = lambda;
    int* feat_i = reinterpret_cast<int*>(feat);
    unsigned long long* ws = static_cast<unsigned long long*>(fs.soft_ws);
    if (soft) fast_init_soft_kernel<<<(unsigned)((pairs + 255) / 256), 256, 0, stream>>>(ws, pairs, pd.counters);
    else fast_init_kernel<<<(unsigned)((pairs + 255) / 256), 256, 0, stream>>>(feat_i, pairs, pd.counters);
    count_launch();
    // the batch goes through in chunks of a few examples: the shifted copies of a chunk are read while
    // they are still in L2, and they stay small
    const int n_chunks = (N + kChunkExamples - 1) / kChunkExamples;
    if (fs.profile) {
        while ((int)fs.evs.size() < 3 * n_chunks) {
            cudaEvent_t ev = nullptr;
            if ((e = cudaEventCreate(&ev)) != cudaSuccess) return e;
            fs.evs.push_back(ev);
        }
        fs.ev_chunks = 0;
    }
    for (int c = 0; c < n_chunks; ++c) {
        const int n0 = c * kChunkExamples, nc = std::min(kChunkExamples, N - n0);
        if (X_u8) {   // the kernels read the normalised samples from the unshifted zero-margined copy
            a.X = fs.xpad + kTPadFront;
            a.x_row_stride = fs.host.pad_pitch;
        } else {
            a.X = X + (size_t)n0 * dp.C * dp.L;
            a.x_row_stride = dp.L;
        }
        a.feat_i = feat_i + (size_t)n0 * 2 * dp.K;
        a.ws = ws ? ws + (size_t)n0 * 2 * dp.K : nullptr;
        a.N = nc;
        if (c > 0) {
            e = cudaMemsetAsync(pd.counters, 0, 8, stream);
            if (e != cudaSuccess) return e;
        }
        if (X_u8) {
            fast_pad_copy_u8_kernel<<<sms * 8, 256, 0, stream>>>(
                reinterpret_cast<const uchar4*>(X_u8 + (size_t)n0 * dp.C * dp.L), fs.xpad, (int64_t)nc * dp.C, dp.L / 4, dp.C,
                fs.host.pad_pitch, kTPadFront, fs.copy_floats, *norm);
            count_launch();
        } else if (pd.n_titems > 0) {
            launch_pad_copy(fs, a.X, (int64_t)nc * dp.C, dp.L, sms, stream);
        }
        if (fs.profile) cudaEventRecord(fs.evs[3 * c], stream);
        if (pd.n_sitems > 0) {
            const unsigned long long total = (unsigned long long)nc * pd.n_sitems;
            const unsigned grid = (unsigned)std::min<unsigned long long>(total, (unsigned long long)sms);
            if (soft) fast_s_forward<1><<<grid, kSThreads, s_bytes, stream>>>(a);
            else if (half) fast_s_forward<3><<<grid, kSThreads, s_bytes, stream>>>(a);
            else fast_s_forward<0><<<grid, kSThreads, s_bytes, stream>>>(a);
            count_launch();
        }
        if (fs.profile) cudaEventRecord(fs.evs[3 * c + 1], stream);
        if (pd.n_titems > 0) {
            const unsigned grid = t_grid(nc, pd.n_titems, sms);
            if (soft) fast_t_forward<1><<<grid, kTBlockThreads, t_bytes, stream>>>(a);
            else if (half) fast_t_forward<3><<<grid, kTBlockThreads, t_bytes, stream>>>(a);
            else fast_t_forward<0><<<grid, kTBlockThreads, t_bytes, stream>>>(a);
            count_launch();
        }
        if (fs.profile) {
            cudaEventRecord(fs.evs[3 * c + 2], stream);
            fs.ev_chunks = c + 1;
        }
    }
    const int64_t fin = (int64_t)N * pd.n_krec;
    if (fin > 0) {
        if (soft) fast_finalize_soft_kernel<<<(unsigned)((fin + 255) / 256), 256, 0, stream>>>(feat, argmax, ws, pd.krec, pd.n_krec, N, dp.K);
        else fast_finalize_kernel<<<(unsigned)((fin + 255) / 256), 256, 0, stream>>>(feat, pd.krec, pd.n_krec, N, dp.K);
        count_launch();
    }
    return cudaGetLastError();
}

cudaError_t launch_fast_backward(FastState& fs, const DeviceParams& dp, int64_t n_weights, const float* X, int N,
                                 float lambda, float shift, const float* dfeat, const int32_t* argmax, float* dW,
                                 float* db, cudaStream_t stream) {
    std::lock_guard<std::mutex> lk(fs.mu);
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    e = set_kernel_attributes(dev);
    if (e != cudaSuccess) return e;
    const size_t s_bytes = s_smem_bytes(dp.C), t_bytes = t_smem_bytes();
    const PlanDevice& pd = fs.dev;
    // workspace: fixed-point sums [n_weights + K], scales [K], max |x| (fixed size per handle)
    const size_t acc_bytes = align256((size_t)(n_weights + dp.K) * 8), scale_bytes = align256((size_t)dp.K * 8);
    if ((e = ensure_bwd_ws(fs, dp, n_weights)) != cudaSuccess) return e;
    long long* accfix = static_cast<long long*>(fs.bwd_ws);
    double* scale = reinterpret_cast<double*>(static_cast<char*>(fs.bwd_ws) + acc_bytes);
    unsigned* absmax = reinterpret_cast<unsigned*>(static_cast<char*>(fs.bwd_ws) + acc_bytes + scale_bytes);
    if (pd.n_titems > 0 && N > 0) {
        e = ensure_pad_capacity(fs, std::min(N, kChunkExamples), dp.C, dp.L);
        if (e != cudaSuccess) return e;
    }
    e = cudaMemsetAsync(absmax, 0, 256, stream);
    if (e != cudaSuccess) return e;
    const int64_t n_x = (int64_t)N * dp.C * dp.L;
    if (n_x > 0) {
        if (dp.L % 4 == 0 && (reinterpret_cast<uintptr_t>(X) & 15u) == 0)
            fast_absmax_kernel<<<sms * 8, 256, 0, stream>>>(reinterpret_cast<const float4*>(X), n_x / 4, absmax);
        else fast_absmax_scalar_kernel<<<sms * 8, 256, 0, stream>>>(X, n_x, absmax);
        count_launch();
    }
    fast_bwd_prepare_kernel<<<(pd.n_krec + 127) / 128, 128, 0, stream>>>(dfeat, pd.krec, pd.n_krec, N, dp.K, lambda, absmax, scale,
                                                                         accfix, n_weights);
    count_launch();
    FwdArgs a;
    a.plan = fs.dev; a.feat_i = nullptr; a.ws = nullptr;
    a.c1 = lambda * 1.4426950408889634f; a.c0 = -shift * 1.4426950408889634f;
    a.C = dp.C; a.L = dp.L; a.K = dp.K;
    a.accfix = accfix; a.scale = scale; a.n_weights = n_weights; a.lambda = lambda;
    a.x_row_stride = dp.L;
    for (int n0 = 0; n0 < N; n0 += kChunkExamples) {
        const int nc = std::min(kChunkExamples, N - n0);
        a.X = X + (size_t)n0 * dp.C * dp.L;
        a.dfeat = dfeat + (size_t)n0 * 2 * dp.K;
        a.argmax = argmax + (size_t)n0 * dp.K;
        a.N = nc;
        e = cudaMemsetAsync(pd.counters, 0, 8, stream);
        if (e != cudaSuccess) return e;
        if (pd.n_titems > 0) launch_pad_copy(fs, a.X, (int64_t)nc * dp.C, dp.L, sms, stream);
        if (pd.n_sitems > 0) {
            const unsigned long long total = (unsigned long long)nc * pd.n_sitems;
            const unsigned grid = (unsigned)std::min<unsigned long long>(total, (unsigned long long)sms);
            fast_s_forward<2><<<grid, kSThreads, s_bytes, stream>>>(a);
            count_launch();
        }
        if (pd.n_titems > 0) {
            fast_t_forward<2><<<t_grid(nc, pd.n_titems, sms), kTBlockThreads, t_bytes, stream>>>(a);
            count_launch();
        }
    }
    fast_bwd_finalize_kernel<<<(pd.n_krec + 127) / 128, 128, 0, stream>>>(accfix, scale, pd.krec, pd.n_krec, n_weights, dW, db);
    count_launch();
    return cudaGetLastError();
}

}  // namespace fast
}  // namespace rocket
