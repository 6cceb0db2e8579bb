// Pieces shared by the two tensor-core attention kernels (one CTA per SM, and CTA pairs): tile constants, the
// tensor-memory column map, the base-2 exponential helpers of the softmax and the walk over a call's key tiles.
#pragma once
#include "ff_internal.h"
#include "attn_schedule.h"
#include "sm100_ptx.cuh"

namespace ffk {

constexpr int kThreads = 384;  // warps 0-7 softmax, 8 producer, 9-10 MMA issuers, 11 idle (fills the warpgroup)
constexpr uint32_t kTmemCols = 512;
constexpr int kHalf = 64;   // keys per score buffer: 64 = a 128-key tile is consumed as two halves, 128 = whole tiles
constexpr int kNB = kTile / kHalf;  // score buffers per query tile
// S_t[b] / P_t[b]: scores of query tile t against half b of the current key tile
__host__ __device__ constexpr uint32_t col_s(int t, int b) { return static_cast<uint32_t>(t) * 128u + static_cast<uint32_t>(b) * kHalf; }
__host__ __device__ constexpr uint32_t col_o(int t) { return 256u + static_cast<uint32_t>(t) * 128u; }  // O_t
constexpr float kRescaleThreshold = 8.0f;  // in log2 units
// Registers per thread after setmaxnreg: the two softmax warpgroups take what the third one gives up.
// setmaxnreg.inc blocks until the registers exist, and no bounded wait can rescue a CTA stuck there, so the
// total must stay clear of the 64K-register file (a request for exactly 65536 never returned).
// The split also steers the compiler's register allocation in the softmax loop, and more is not better: measured
// per 480p layer-call on the one-CTA kernel, softmax/other = 160..216: 200/96 0.402 ms, 216/64 0.408, 208/80 0.413,
// 192/112 0.408, 184/128 0.398, 176/144 0.403, 168/160 0.404; on the CTA-pair kernel at 720p 200/96 2.090 ms,
// 184/128 2.114, 176/144 2.082.
template <int kSoftmax, int kOther>
struct RegSplit {
    static constexpr int softmax = kSoftmax, other = kOther;
    static_assert(2 * 128 * kSoftmax + 128 * kOther <= 64 * 1024 - 2048, "setmaxnreg budget exceeds the register file");
};
using RegsOneCta = RegSplit<184, 128>;
using RegsCtaPair = RegSplit<176, 144>;
constexpr float kLog2e = 1.4426950408889634f;

template <int D>
struct SmemLayout {
    static constexpr int kBoxBytes = 128 * 64 * 2;           // one 128-row x 64-column bf16 box
    static constexpr int kTileBytes = kBoxBytes * (D / 64);  // 128 x D
    static constexpr int kQ = 0;                             // two query tiles
    static constexpr int kK = 2 * kTileBytes;                // two stages
    static constexpr int kV = 4 * kTileBytes;                // two stages
    static constexpr int kTotal = 6 * kTileBytes;
    // requested size: above half of an SM's shared memory, so that exactly one CTA (which takes all 512
    // tensor-memory columns) is resident per SM
    static constexpr int kDynamic = (kTotal + 1024) > 120 * 1024 ? (kTotal + 1024) : 120 * 1024;
};

// Every kPolyEvery-th pair of exponentials is evaluated by exp2_poly2 on the FMA and integer pipes instead of the
// MUFU unit (0 = none).  The two softmax warps that share a scheduler collide on its MUFU unit (64 exponentials
// per row and half tile, 4 lanes per clock), so moving a quarter of them away shortens their exp phase; the step
// runs on the GPU's power cap, where the extra FMA work costs clock: measured on the 480p shape over 20-step runs,
// 0: 53.4 ms per step, 4: 52.5, 3: 52.8, 2: 53.2.
#ifndef FF_POLY_EVERY
#define FF_POLY_EVERY 4
#endif
constexpr int kPolyEvery = FF_POLY_EVERY;

__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// 2^x for two values on the FMA and integer pipes (no MUFU): x = n + f with n = floor(x) obtained by adding
// 1.5 * 2^23 with rounding toward -inf, 2^f by a cubic on [0,1) (relative error < 1e-4, far below the bf16
// rounding the result gets), and n added into the exponent field.  Inputs below -126 give (almost) zero.
__device__ __forceinline__ float2 exp2_poly2(float2 x) {
    const float kMagic = 12582912.f;  // 1.5 * 2^23
    x.x = fmaxf(x.x, -126.f);
    x.y = fmaxf(x.y, -126.f);
    const float2 xr = __fadd2_rd(x, make_float2(kMagic, kMagic));
    const float2 n = __fadd2_rn(xr, make_float2(-kMagic, -kMagic));
    const float2 f = __fadd2_rn(x, make_float2(-n.x, -n.y));
    float2 p = __ffma2_rn(make_float2(0.0771190f, 0.0771190f), f, make_float2(0.2275643f, 0.2275643f));
    p = __ffma2_rn(p, f, make_float2(0.6951461f, 0.6951461f));
    p = __ffma2_rn(p, f, make_float2(1.f, 1.f));
    float2 r;
    r.x = __uint_as_float(__float_as_uint(p.x) + (__float_as_uint(xr.x) << 23));
    r.y = __uint_as_float(__float_as_uint(p.y) + (__float_as_uint(xr.y) << 23));
    return r;
}

// One half step of the online softmax for one query row (one thread owns the row): the 64 scores of the row against
// the current half of a key tile have been read from tensor memory into sr.  Masks the keys beyond n_here, raises
// the running reference maximum m_used lazily (only when some row of the warp outgrew it by kRescaleThreshold in
// log2 units; the accumulator row at o_addr is then rescaled in tensor memory, after the product that is still
// adding to it - awaited on bar_pv_done with parity pv_parity unless this is the first half of the piece - has
// finished), turns the scores into p = 2^(c*s - c*m_used), adds them to the row sum l and stores them as bf16 pairs
// over the scores at s_addr.  The stores are left in flight: the caller waits for them (tmem_st_wait) before it
// signals the issuer.  Shared by both tensor-core kernels; the code is inlined into each softmax loop.
template <int D>
__device__ __forceinline__ void softmax_half_step(uint32_t (&sr)[kHalf / 32][32], int n_here, float c, bool first_half,
                                                  uint32_t s_addr, uint32_t o_addr, uint64_t* bar_pv_done,
                                                  uint32_t pv_parity, uint32_t* status, uint32_t err, float& m_used,
                                                  float& l) {
    if (n_here < kHalf) {
#pragma unroll
        for (int q2 = 0; q2 < kHalf / 32; ++q2)
#pragma unroll
            for (int i = 0; i < 32; ++i)
                if (q2 * 32 + i >= n_here) sr[q2][i] = 0xff800000u;  // -inf
    }
    float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
    for (int q2 = 0; q2 < kHalf / 32; ++q2)
#pragma unroll
        for (int i = 0; i < 32; i += 2)
            mx[(i >> 1) & 3] = fmax3(mx[(i >> 1) & 3], __uint_as_float(sr[q2][i]), __uint_as_float(sr[q2][i + 1]));
    const float tmax = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));

    // raise the reference maximum only when some row of this warp outgrew it by the threshold
    const bool grow = (tmax - m_used) * c > kRescaleThreshold;  // true on the first half (m_used = -inf)
    if (__any_sync(0xffffffffu, grow)) {
        const float m_new = fmaxf(m_used, tmax);
        if (!first_half) {
            // O_t may only be touched once the product fed by the previous half tile has finished
            mbar_wait(bar_pv_done, pv_parity, status, err);
            tc_fence_after_sync();
            const float alpha = ex2_approx((m_used - m_new) * c);
            l *= alpha;
#pragma unroll
            for (int q4 = 0; q4 < D / 32; ++q4) {
                uint32_t o[32];
                tmem_ld_32x32b_x32(o_addr + q4 * 32, o);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                tmem_st_32x32b_x32(o_addr + q4 * 32, o);
            }
            tmem_st_wait();
        }
        m_used = m_new;
    }
    const float2 c2 = make_float2(c, c);
    const float2 nmc2 = make_float2(-m_used * c, -m_used * c);
    float2 sum2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
    for (int q2 = 0; q2 < kHalf / 32; ++q2) {
        uint32_t pk[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const float2 x =
                __ffma2_rn(make_float2(__uint_as_float(sr[q2][2 * i]), __uint_as_float(sr[q2][2 * i + 1])), c2, nmc2);
            float2 pr;
            if (kPolyEvery > 0 && (i % (kPolyEvery > 0 ? kPolyEvery : 1)) == 0) {
                pr = exp2_poly2(x);   // a fraction of the exponentials on the FMA pipe
            } else {
                pr.x = ex2_approx(x.x);
                pr.y = ex2_approx(x.y);
            }
            sum2[i & 1] = __fadd2_rn(sum2[i & 1], pr);
            pk[i] = pack_bf16x2(pr.x, pr.y);
        }
        tmem_st_32x32b_x16(s_addr + q2 * 16, pk);
    }
    l += (sum2[0].x + sum2[0].y) + (sum2[1].x + sum2[1].y);
}

// Position in the list of key tiles: segment and token offset inside it.
struct TileWalker {
    int seg, t0;
    __device__ __forceinline__ void seek(const KvSegs& s, int j) {
        seg = 0;
        while (seg < s.n) {
            const int nt = (s.tokens[seg] + kTile - 1) / kTile;
            if (j < nt) break;
            j -= nt;
            ++seg;
        }
        t0 = j * kTile;
    }
    __device__ __forceinline__ void next(const KvSegs& s) {
        t0 += kTile;
        if (t0 >= s.tokens[seg]) { ++seg; t0 = 0; }
    }
    __device__ __forceinline__ int row(const KvSegs& s, int h) const { return s.row0[seg] + h * s.head_stride[seg] + t0; }
    __device__ __forceinline__ int n_valid(const KvSegs& s) const { return min(kTile, s.tokens[seg] - t0); }
};

}  // namespace ffk
