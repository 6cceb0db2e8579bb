// Rotary embedding of the chunk's Q and K and the in-place publish of (K', V) into a cache slot
// (Eq. 2: B_k <- Append(B_k, (i, K, V)); Alg. 1 Phase B "Write in place").  Also serves the anchor publish
// (Alg. 1 Phase A, last line) with q == nullptr.
//
// HBM-bound: every input element is read once and every output element written once with 16-byte accesses.
// Consecutive threads take consecutive 16-byte pieces of the [token, head, dim] inputs, so loads are fully
// coalesced; a (token, head) row is 16 (bf16, d=128) consecutive pieces, so stores into the head-major cache
// are contiguous runs of 256 bytes.
//
// Rotation arithmetic (must round exactly like the definition the tests check bit for bit): cos and sin come
// from tables the host evaluated in double and rounded to float; each product and each sum is rounded
// separately (no fused multiply-add), then the result is rounded to nearest-even bf16.
#include <cuda_bf16.h>
#include <atomic>
#include "ff_internal.h"

namespace ffk {

constexpr int kMaxDevices = 64;

__device__ __forceinline__ void rotate(float a, float b, float2 cs, float& r0, float& r1) {
    float t1 = __fmul_rn(a, cs.x);
    float t2 = __fmul_rn(b, cs.y);
    float t3 = __fmul_rn(a, cs.y);
    float t4 = __fmul_rn(b, cs.x);
    r0 = __fsub_rn(t1, t2);
    r1 = __fadd_rn(t3, t4);
}

// A piece is 16 bytes of a (token, head) row: 8 bf16 or 4 fp32 elements, i.e. 4 or 2 rotary pairs.
template <bool kBf16>
__device__ __forceinline__ void unpack_piece(uint4 in, float (&x)[kBf16 ? 8 : 4]) {
    const uint32_t w[4] = {in.x, in.y, in.z, in.w};
    if constexpr (kBf16) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            x[2 * i] = __uint_as_float(w[i] << 16);          // bf16 -> fp32 is exact
            x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) x[i] = __uint_as_float(w[i]);
    }
}

template <bool kBf16>
__device__ __forceinline__ uint4 rotate_pack_piece(const float (&x)[kBf16 ? 8 : 4], const float2 (&cs)[4]) {
    uint32_t w[4];
    if constexpr (kBf16) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float r0, r1;
            rotate(x[2 * i], x[2 * i + 1], cs[i], r0, r1);
            const __nv_bfloat162 o = __floats2bfloat162_rn(r0, r1);  // one conversion for the pair, each half RNE
            w[i] = *reinterpret_cast<const uint32_t*>(&o);
        }
    } else {
        float r0, r1, r2, r3;
        rotate(x[0], x[1], cs[0], r0, r1);
        rotate(x[2], x[3], cs[1], r2, r3);
        w[0] = __float_as_uint(r0); w[1] = __float_as_uint(r1); w[2] = __float_as_uint(r2); w[3] = __float_as_uint(r3);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// Optional RMS normalisation of a (token, head) row before the rotation: x * 1/sqrt(mean(x^2) + eps).
// The order of every rounding is fixed so that the published cache can be compared bit for bit: squares and
// their running sum inside a piece in element order (product and sum rounded separately), then a balanced
// tree over the row's pieces (xor-butterfly: every lane ends with the same value), mean by an exact power of
// two, correctly rounded sqrt and division, then per element one rounded product with the inverse and one
// with the channel's gain.
// The normalisation is split in three so that the expensive part runs once per row instead of once per lane:
// row_sum_squares leaves the row's sum of squares in every lane of the row; then ONE lane per row and tensor
// evaluates 1/sqrt(mean + eps) (inv_rms_shared: the up to four sums a lane holds - two rows in flight, K and Q -
// are dealt out to the row's first four lanes, each evaluates one, and the results are handed back by shuffle);
// scale_row applies it.  The values are the same as if every lane had evaluated its own.
template <int E>
__device__ __forceinline__ float row_sum_squares(const float (&x)[E], int ppr) {
    float acc = __fmul_rn(x[0], x[0]);
#pragma unroll
    for (int e = 1; e < E; ++e) acc = __fadd_rn(acc, __fmul_rn(x[e], x[e]));
    for (int off = 1; off < ppr; off <<= 1) acc = __fadd_rn(acc, __shfl_xor_sync(0xffffffffu, acc, off));
    return acc;
}
__device__ __forceinline__ void inv_rms_shared(float (&acc)[4], int ppr, float inv_d, float eps) {
    const int lane = threadIdx.x & 31, row_lane0 = lane & ~(ppr - 1);
    const int j = lane & 3;
    const float mine = j == 0 ? acc[0] : (j == 1 ? acc[1] : (j == 2 ? acc[2] : acc[3]));
    const float inv = __fdiv_rn(1.0f, __fsqrt_rn(__fadd_rn(__fmul_rn(mine, inv_d), eps)));
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[i] = __shfl_sync(0xffffffffu, inv, row_lane0 + i);
}
template <int E>
__device__ __forceinline__ void scale_row(float (&x)[E], const float* __restrict__ gain, float inv) {
    // the thread's E channel gains are read where they are used (two 16-byte loads that hit L1): holding them in
    // registers for the whole kernel cost a resident block per SM
#pragma unroll
    for (int e = 0; e < E; e += 4) {
        const float4 g = __ldg(reinterpret_cast<const float4*>(gain + e));
        x[e] = __fmul_rn(__fmul_rn(x[e], inv), g.x);
        x[e + 1] = __fmul_rn(__fmul_rn(x[e + 1], inv), g.y);
        x[e + 2] = __fmul_rn(__fmul_rn(x[e + 2], inv), g.z);
        x[e + 3] = __fmul_rn(__fmul_rn(x[e + 3], inv), g.w);
    }
}

// Where a (token, head) row sits: token t = (f, py, px) on the chunk's grid, head h.  A thread's rows advance by a
// fixed number of rows per iteration, so the position is carried along (one set of divisions per thread at the
// start) instead of being recomputed with four integer divisions per row.
struct RowPos {
    int row, t, h, f, py, px;
    __device__ __forceinline__ void init(int row_, int n_heads, int grid_w, int tf) {
        row = row_;
        t = row / n_heads;
        h = row - t * n_heads;
        f = t / tf;
        const int r = t - f * tf;
        py = r / grid_w;
        px = r - py * grid_w;
    }
    // row += step, with step = dt * n_heads + dh, 0 <= dh < n_heads
    __device__ __forceinline__ void advance(int step, int dt, int dh, int n_heads, int grid_h, int grid_w) {
        row += step;
        h += dh;
        int inc = dt;
        if (h >= n_heads) { h -= n_heads; ++inc; }
        t += inc;
        px += inc;
        while (px >= grid_w) { px -= grid_w; ++py; }
        while (py >= grid_h) { py -= grid_h; ++f; }
    }
};

// Thread layout: a thread keeps one 16-byte piece position of the (token, head) row for the whole kernel, so the
// rotary pairs it handles - and with them the table and axis each pair reads - are fixed; it walks over the
// rows of its block's contiguous share with 32-bit index arithmetic.  Q and K share the cos/sin values.
template <bool kBf16, bool kNorm>
__global__ void __launch_bounds__(256, kNorm ? 2 : 0) rope_publish_kernel(const __grid_constant__ PublishBatch batch) {
    const PublishArgs& a = batch.items[blockIdx.y];
    constexpr int kElemsPerPiece = kBf16 ? 8 : 4;
    constexpr int kPairs = kElemsPerPiece / 2;
    grid_dependency_wait();  // inputs may come from, and the slot may still be read by, the kernel before this one
    const int ppr = a.head_dim / kElemsPerPiece;       // pieces per (token, head) row: 8, 16 or 32
    const int rows_per_pass = 256 / ppr;
    const int piece = threadIdx.x % ppr;
    const int rowslot = threadIdx.x / ppr;
    const int tf = a.grid_h * a.grid_w;
    const int n_rows = a.n_tok * a.n_heads;            // rows that carry data
    const int n_rows_pad = a.n_tok_pad * a.n_heads;    // plus the zero rows up to the tile boundary
    const int rows_per_block = (n_rows_pad + gridDim.x - 1) / gridDim.x;
    const int row_begin = blockIdx.x * rows_per_block;
    const int row_end = min(row_begin + rows_per_block, n_rows_pad);
    const float inv_d = 1.0f / static_cast<float>(a.head_dim);

    // which table (axis) and which column of it each of this thread's pairs reads
    const float2* tab[kPairs];
    int tab_stride[kPairs], axis[kPairs];
#pragma unroll
    for (int i = 0; i < kPairs; ++i) {
        int pair = piece * kPairs + i;
        if (pair < a.tab.pairs_f) {
            tab[i] = a.tab.frame + pair; tab_stride[i] = a.tab.pairs_f; axis[i] = 0;
        } else if (pair < a.tab.pairs_f + a.tab.pairs_h) {
            tab[i] = a.tab.row + (pair - a.tab.pairs_f); tab_stride[i] = a.tab.pairs_h; axis[i] = 1;
        } else {
            tab[i] = a.tab.col + (pair - a.tab.pairs_f - a.tab.pairs_h); tab_stride[i] = a.tab.pairs_w; axis[i] = 2;
        }
    }
    // the gains of this thread's channels (its piece position never changes)
    const float* gain_q = kNorm ? a.gain_q + piece * kElemsPerPiece : nullptr;
    const float* gain_k = kNorm ? a.gain_k + piece * kElemsPerPiece : nullptr;
    const uint4* __restrict__ qin = reinterpret_cast<const uint4*>(a.q);
    const uint4* __restrict__ kin = reinterpret_cast<const uint4*>(a.k);
    const uint4* __restrict__ vin = reinterpret_cast<const uint4*>(a.v);
    uint4* __restrict__ qout = reinterpret_cast<uint4*>(a.q_rot);
    uint4* __restrict__ kout = reinterpret_cast<uint4*>(a.kmat);
    uint4* __restrict__ vout = reinterpret_cast<uint4*>(a.vmat);

    // two rows per iteration: all six loads are issued before the first rotation, to keep more bytes in flight.
    // The loop bound is the same for all threads of a warp (the normalisation shuffles across a row's threads).
    const int first_row = row_begin + rowslot;
    const int n_iter = (row_end - row_begin + 2 * rows_per_pass - 1) / (2 * rows_per_pass);
    // With the normalisation the loads of iteration it+1 are issued before the arithmetic of iteration it (all
    // blocks start together and walk in step: without that the memory system idles while everybody reduces).
    uint4 nk[kNorm ? 2 : 1], nv[kNorm ? 2 : 1], nq[kNorm ? 2 : 1];
    auto fetch_ahead = [&](int it) {
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int row = first_row + (2 * it + u) * rows_per_pass;
            nk[u] = nv[u] = nq[u] = make_uint4(0, 0, 0, 0);
            if (row < n_rows && row < row_end) {
                const long long src = (long long)row * ppr + piece;
                nk[u] = __ldg(kin + src);
                nv[u] = __ldg(vin + src);
                if (qin) nq[u] = __ldg(qin + src);
            }
        }
    };
    if constexpr (kNorm) {
        if (n_iter > 0) fetch_ahead(0);
    }
    RowPos next_row;   // the first of the two rows of the coming iteration
    next_row.init(first_row, a.n_heads, a.grid_w, tf);
    const int half_dt = rows_per_pass / a.n_heads, half_dh = rows_per_pass - half_dt * a.n_heads;
    for (int it = 0; it < n_iter; ++it) {
        RowPos at[2];
        at[0] = next_row;
        next_row.advance(rows_per_pass, half_dt, half_dh, a.n_heads, a.grid_h, a.grid_w);
        at[1] = next_row;
        next_row.advance(rows_per_pass, half_dt, half_dh, a.n_heads, a.grid_h, a.grid_w);
        uint4 kv[2], vv[2], qv[2];
        bool live[2], data[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int row = at[u].row;
            live[u] = row < row_end;
            data[u] = row < n_rows && live[u];
            if constexpr (kNorm) {
                kv[u] = nk[u]; vv[u] = nv[u]; qv[u] = nq[u];
            } else {
                kv[u] = vv[u] = qv[u] = make_uint4(0, 0, 0, 0);
                if (data[u]) {
                    const long long src = (long long)row * ppr + piece;
                    kv[u] = __ldg(kin + src);
                    vv[u] = __ldg(vin + src);
                    if (qin) qv[u] = __ldg(qin + src);
                }
            }
        }
        // with the normalisation both rows are unpacked and normalised first (their inverse RMS values are evaluated
        // together); without it each row is unpacked where it is rotated, which keeps fewer registers live
        float kxs[kNorm ? 2 : 1][kElemsPerPiece], qxs[kNorm ? 2 : 1][kElemsPerPiece];
        if constexpr (kNorm) {   // executed by every lane: rows without data carry zeros
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                unpack_piece<kBf16>(kv[u], kxs[u]);
                unpack_piece<kBf16>(qv[u], qxs[u]);
            }
            if (it + 1 < n_iter) fetch_ahead(it + 1);
            float acc[4];
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                acc[2 * u] = row_sum_squares<kElemsPerPiece>(kxs[u], ppr);
                acc[2 * u + 1] = qin ? row_sum_squares<kElemsPerPiece>(qxs[u], ppr) : 0.f;
            }
            inv_rms_shared(acc, ppr, inv_d, a.qk_norm_eps);
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                scale_row<kElemsPerPiece>(kxs[u], gain_k, acc[2 * u]);
                if (qin) scale_row<kElemsPerPiece>(qxs[u], gain_q, acc[2 * u + 1]);
            }
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            float (&kx)[kElemsPerPiece] = kxs[kNorm ? u : 0];
            float (&qx)[kElemsPerPiece] = qxs[kNorm ? u : 0];
            if constexpr (!kNorm) {
                unpack_piece<kBf16>(kv[u], kx);
                unpack_piece<kBf16>(qv[u], qx);
            }
            const RowPos& here = at[u];
            if (!live[u]) continue;
            const int t = here.t, h = here.h;
            const long long dst = ((long long)a.dst_row0 + (long long)h * a.dst_head_stride + t) * ppr + piece;
            const long long qdst = ((long long)h * a.q_rows_per_head + t) * ppr + piece;
            if (data[u]) {
                const int pos[3] = {a.first_frame_pos + here.f * a.frame_pos_stride, here.py, here.px};
                float2 cs[4];
#pragma unroll
                for (int i = 0; i < kPairs; ++i) cs[i] = __ldg(tab[i] + pos[axis[i]] * tab_stride[i]);
                kout[dst] = rotate_pack_piece<kBf16>(kx, cs);
                vout[dst] = vv[u];
                if (qin) qout[qdst] = rotate_pack_piece<kBf16>(qx, cs);
            } else {
                // rows between the token count and the next tile boundary: zero, so that a key tile that hangs
                // over the end of the slot multiplies zero probabilities with zeros, never with stale bits
                const uint4 z = make_uint4(0, 0, 0, 0);
                kout[dst] = z;
                vout[dst] = z;
                if (qin) qout[qdst] = z;
            }
        }
    }
}

namespace {

// One launch = exactly one wave: as many blocks as are resident at once (what the kernel's register count allows
// per SM, asked of the runtime once per variant), shared equally by the items of the batch; each block walks a
// contiguous share of its item's rows.  A grid sized for more blocks per SM than fit leaves a partly filled last
// wave, which shows in a kernel this short.
template <bool kBf16, bool kNorm>
cudaError_t launch_variant(const PublishBatch& b, int sm_count, cudaStream_t s) {
    // resident blocks per SM of this variant on the current device, asked once per device
    static std::atomic<int> per_sm_of[kMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) dev = 0;
    int per_sm = per_sm_of[dev].load(std::memory_order_relaxed);
    if (per_sm == 0) {
        int n = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, rope_publish_kernel<kBf16, kNorm>, 256, 0) != cudaSuccess || n < 1)
            n = 1;
        per_sm = n;
        per_sm_of[dev].store(n, std::memory_order_relaxed);
    }
    const int elems = kBf16 ? 8 : 4;
    long long blocks = 1;  // per item: at least one pass of rows per block, for the largest item
    for (int i = 0; i < b.n; ++i) {
        const int rows_per_pass = 256 / (b.items[i].head_dim / elems);
        const long long rows = static_cast<long long>(b.items[i].n_tok_pad) * b.items[i].n_heads;
        const long long want = (rows + rows_per_pass - 1) / rows_per_pass;
        if (want > blocks) blocks = want;
    }
    const long long cap = static_cast<long long>(sm_count) * per_sm / b.n;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return launch_overlapped(rope_publish_kernel<kBf16, kNorm>, dim3(static_cast<unsigned>(blocks), static_cast<unsigned>(b.n)),
                             dim3(256), 0, s, b);
}

}  // namespace

cudaError_t launch_rope_publish_batch(const PublishBatch& b, int dtype, int sm_count, cudaStream_t s) {
    if (b.n < 1 || b.n > kMaxInline) return cudaErrorInvalidValue;
    const bool norm = b.items[0].qk_norm != 0;
    if (dtype == 0) return norm ? launch_variant<true, true>(b, sm_count, s) : launch_variant<true, false>(b, sm_count, s);
    return norm ? launch_variant<false, true>(b, sm_count, s) : launch_variant<false, false>(b, sm_count, s);
}

cudaError_t launch_rope_publish(const PublishArgs& a, int dtype, int sm_count, cudaStream_t s) {
    PublishBatch b{};
    b.n = 1;
    b.items[0] = a;
    return launch_rope_publish_batch(b, dtype, sm_count, s);
}

}  // namespace ffk
