// Flash attention of one chunk's queries over the visible cache segments, for B200 (sm_100a):
// TMA-staged Q/K/V tiles, tcgen05 matrix multiplies accumulating in tensor memory, online softmax with one
// query row per thread, and a persistent schedule that gives every SM the same number of tile iterations.
//
// Work.  A launch serves one layer-call or several independent ones (the nodes of a wavefront round, or
// consecutive chunks of a clip).  A work item is a PAIR of 128-row query tiles of one head of one call; it needs
// every key tile (128 keys) visible to that call.  One CTA per SM; every CTA first takes the same number of
// whole pairs, then an equal share of the (pair, key tile) iterations of the remaining pairs (attn_schedule.h).
// A pair handled by one CTA alone is normalised and stored as bf16 directly; a piece of a split pair stores its
// unnormalised fp32 accumulator, row maximum and row sum to scratch, and a small second kernel merges the
// pieces.
//
// Roles inside a CTA (384 threads = 3 warpgroups; the third gives most of its registers to the first two):
//   warps 0-3   softmax + epilogue of query tile 0: thread r owns row r (TMEM lane r)
//   warps 4-7   the same for query tile 1
//   warp  8     TMA producer (one lane): Q pair, then K and V tiles through two 2-stage rings
//   warps 9,10  tcgen05.mma issue (warp 9 for query tile 0, warp 10 for query tile 1; the whole warp walks the
//               loop in uniform control flow, one elected lane issues); warp 9 also allocates tensor memory
// Tensor memory (512 columns): every query tile t has two 64-column score buffers S_t[0] at column 128t and
// S_t[1] at 128t+64, one per half (64 keys) of a key tile; a buffer's first 32 columns are overwritten with
// P_t[b] in bf16, which the second product reads straight from tensor memory; O0 [256,256+D) and
// O1 [384,384+D) accumulate P_t V.
// A 128-key tile is consumed as two halves so that the scores of the next half are always computed while a
// softmax group is still busy with the current one: as soon as P_t[b] has been multiplied into O_t, the same
// buffer is refilled with Q_t K^T for half b of the NEXT key tile.  Pipe order per key tile j:
//   P0[0]V | Q0K(j+1)[0] | P1[0]V | Q1K(j+1)[0] | P0[1]V | Q0K(j+1)[1] | P1[1]V | Q1K(j+1)[1].
//
// Softmax in base 2 with a lazily raised reference maximum: p = 2^(c*s - c*m); m is only raised when a row's
// tile maximum exceeds it by more than 2^8 (then O and the row sum are rescaled by the owning thread); a quarter
// of the exponentials are evaluated by a cubic on the FMA pipe, the rest by the MUFU unit.  Key
// columns beyond a segment's token count get probability zero; the cache rows they map to were zero-filled
// by the publish kernel.
//
// Every wait is bounded (mbar_wait): on expiry an error code goes to the status word and the CTA runs on to
// its end, frees its tensor memory and returns.
#include "attn_common.cuh"

namespace ffk {

// S[128 x 64] = Q_t . (64 keys)^T : D/16 products, both operands K-major in 128-byte-swizzled boxes of 64 columns.
template <int D>
__device__ __forceinline__ void issue_qk_half(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi,
                                              uint32_t idesc, uint32_t leader) {
#pragma unroll
    for (int kk = 0; kk < D / 16; ++kk) {
        const uint32_t off = ((kk / 4) * (128 * 64 * 2) + (kk % 4) * 32) >> 4;
        mma_ss_lohi_p(d_tmem, a_lo + off, b_lo + off, hi, idesc, kk > 0 ? 1u : 0u, leader);
    }
}
// O[128 x D] (+)= P[128 x 64] (bf16 in tensor memory) . V(64 keys, MN-major): four products of 16 keys.
__device__ __forceinline__ void issue_pv_half(uint32_t d_tmem, uint32_t p_tmem, uint32_t b_lo, uint32_t hi,
                                              uint32_t idesc, uint32_t accumulate, uint32_t leader) {
    mma_ts_lohi_p(d_tmem, p_tmem, b_lo, hi, idesc, accumulate, leader);
#pragma unroll
    for (int kk = 1; kk < kHalf / 16; ++kk)
        mma_ts_lohi_p(d_tmem, p_tmem + kk * 8, b_lo + ((kk * 2048) >> 4), hi, idesc, 1u, leader);
}

// Event trace (CTA 0 only): one thread per role appends (event id, SM clock).  Compiled in only for the kernel
// variant that is launched while a trace buffer is set: even a predicated-off mark costs a clock read, a store
// and counter arithmetic, several per 64-key half in the loops that pace the kernel.
template <bool kOn>
struct Tracer {
    unsigned long long* base;
    int cap, n;
    __device__ __forceinline__ void init(const AttnArgs& a, int role, bool on) {
        if constexpr (kOn) {
            base = (on && a.trace) ? a.trace + static_cast<size_t>(role) * a.trace_cap : nullptr;
            cap = a.trace_cap;
            n = 0;
        }
    }
    __device__ __forceinline__ void mark(unsigned id) {
        if constexpr (kOn) {
            if (base && n < cap) base[n++] = (static_cast<unsigned long long>(id) << 48) | (clock64() & 0xFFFFFFFFFFFFull);
        }
    }
};

template <int D, bool kTrace, bool kTable>
__global__ void __launch_bounds__(kThreads, 1)
attn_tcgen05_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ AttnArgs a) {
    using L = SmemLayout<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ uint64_t bar_q_full, bar_q_empty, bar_k_full[2], bar_k_empty[2], bar_v_full[2], bar_v_empty[2],
        bar_s_full[2][2], bar_p_full[2][2], bar_pv_done[2], bar_o_full[2];
    __shared__ uint32_t tmem_base_slot;

    // warp index and (below) the tensor-memory base are broadcast from lane 0, which tells the compiler that they
    // are the same in all lanes: role branches become uniform branches and addresses built from them can live in
    // uniform registers
    const int warp = __shfl_sync(0xffffffffu, static_cast<int>(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    const int cta = blockIdx.x;

    if (threadIdx.x == 0) {
        mbar_init(&bar_q_full, 1);
        mbar_init(&bar_q_empty, 2);  // both issuers hand Q, K and V back
        for (int i = 0; i < 2; ++i) {
            mbar_init(&bar_k_full[i], 1);
            mbar_init(&bar_k_empty[i], 2);
            mbar_init(&bar_v_full[i], 1);
            mbar_init(&bar_v_empty[i], 2);
            for (int b = 0; b < kNB; ++b) {
                mbar_init(&bar_s_full[i][b], 1);
                mbar_init(&bar_p_full[i][b], 4);
            }
            mbar_init(&bar_pv_done[i], 1);
            mbar_init(&bar_o_full[i], 1);
        }
        fence_mbar_init();
    }
    if (warp == 9) {
        tmem_alloc<kTmemCols>(&tmem_base_slot);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = __shfl_sync(0xffffffffu, tmem_base_slot, 0);
    // everything above needed no global memory; the publish kernel before this launch may still have been draining
    grid_dependency_wait();

    if (warp >= 8) {
      asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(RegsOneCta::other));
      if (warp == 8) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            prefetch_tensormap(&tm_q);
            prefetch_tensormap(&tm_k);
            prefetch_tensormap(&tm_v);
            uint32_t kiter = 0, viter = 0, n_piece = 0;
            TileWalker w;
            PieceIter<kTable> pit;
            pit.init(a, cta);
            Piece p;
            for (; pit.next(a, p); ++n_piece) {
                if (n_piece > 0) mbar_wait(&bar_q_empty, (n_piece - 1) & 1, a.status, a.launch_tag | kErrWaitQ);
                mbar_expect_tx(&bar_q_full, (p.two ? 2 : 1) * L::kTileBytes);
                for (int t = 0; t < (p.two ? 2 : 1); ++t)
#pragma unroll
                    for (int b = 0; b < D / 64; ++b)
                        tma_load_2d(smem + L::kQ + t * L::kTileBytes + b * L::kBoxBytes, &tm_q, b * 64,
                                    item_at<kTable>(a, p.item).q_row0 + p.h * a.q_rows_per_head + (2 * p.pr + t) * kTile,
                                    &bar_q_full);
                const KvSegs& segs = item_at<kTable>(a, p.item).segs;
                w.seek(segs, p.j0);
                for (int j = p.j0; j < p.j1; ++j) {
                    const int row = w.row(segs, p.h);
                    uint32_t st = kiter & 1;
                    if (kiter >= 2) mbar_wait(&bar_k_empty[st], ((kiter >> 1) - 1) & 1, a.status, a.launch_tag | kErrWaitKEmpty);
                    mbar_expect_tx(&bar_k_full[st], L::kTileBytes);
#pragma unroll
                    for (int b = 0; b < D / 64; ++b)
                        tma_load_2d(smem + L::kK + st * L::kTileBytes + b * L::kBoxBytes, &tm_k, b * 64, row,
                                    &bar_k_full[st]);
                    ++kiter;
                    st = viter & 1;
                    if (viter >= 2) mbar_wait(&bar_v_empty[st], ((viter >> 1) - 1) & 1, a.status, a.launch_tag | kErrWaitVEmpty);
                    mbar_expect_tx(&bar_v_full[st], L::kTileBytes);
#pragma unroll
                    for (int b = 0; b < D / 64; ++b)
                        tma_load_2d(smem + L::kV + st * L::kTileBytes + b * L::kBoxBytes, &tm_v, b * 64, row,
                                    &bar_v_full[st]);
                    ++viter;
                    w.next(segs);
                }
            }
            // After an expired wait the roles stop consuming, so copies may still be on their way into shared
            // memory: give the last ones a bounded time to land before the CTA ends and the memory is handed on.
            if (*reinterpret_cast<volatile uint32_t*>(a.status) != 0u) {
                constexpr unsigned long long kDrainNs = 5000000ull;
                if (n_piece > 0) mbar_wait(&bar_q_full, (n_piece - 1) & 1, nullptr, 0, kDrainNs);
                for (uint32_t back = 1; back <= 2; ++back) {
                    if (kiter >= back) mbar_wait(&bar_k_full[(kiter - back) & 1], ((kiter - back) >> 1) & 1, nullptr, 0, kDrainNs);
                    if (viter >= back) mbar_wait(&bar_v_full[(viter - back) & 1], ((viter - back) >> 1) & 1, nullptr, 0, kDrainNs);
                }
            }
        }
      } else if (warp == 9 || warp == 10) {
        // ------------------------------------------------------------------ MMA issuers: warp 9 serves query
        // tile 0, warp 10 query tile 1.  Two issuing threads because one thread's own instruction latency
        // (descriptor arithmetic, barrier polls, commits) cannot keep the pipe fed with 64-key products.
        // The whole warp runs the loop with identical values (the warp index is taken through a shuffle so that
        // the compiler can see it is uniform); one elected lane issues the products and the commits.
        {
            const int t = warp - 9;
            const uint32_t leader = elect_one_sync();
            constexpr uint32_t idesc_s = make_idesc_bf16(128, kHalf, false);  // S[128 x 64] = Q . K half (both K-major)
            constexpr uint32_t idesc_o = make_idesc_bf16(128, D, true);       // O[128 x D] += P (TMEM) . V half (MN-major)
            // descriptor halves: low = start address (+ leading offset for V), high = stride / version / swizzle
            constexpr uint32_t kHi = desc_hi_sw128(1024);
            const uint32_t q_lo = desc_lo_sw128(smem_u32(smem + L::kQ + t * L::kTileBytes), 16);
            const uint32_t k_lo0 = desc_lo_sw128(smem_u32(smem + L::kK), 16);
            const uint32_t v_lo0 = desc_lo_sw128(smem_u32(smem + L::kV), L::kBoxBytes);
            const uint32_t s_col[2] = {tmem + col_s(t, 0), tmem + col_s(t, kNB - 1)};
            const uint32_t o_col = tmem + col_o(t);
            uint32_t kiter = 0, viter = 0, n_piece = 0, sp = 0;  // sp: key tiles this stream has consumed
            Tracer<kTrace> tr;
            tr.init(a, 2, cta == 0 && t == 0 && leader != 0);

            PieceIter<kTable> pit;
            pit.init(a, cta);
            Piece p;
            for (; pit.next(a, p); ++n_piece) {
                const bool active = (t == 0) || p.two;  // an idle stream still takes part in the K/V/Q hand-back
                mbar_wait(&bar_q_full, n_piece & 1, a.status, a.launch_tag | kErrWaitQ);
                uint32_t k_cur = k_lo0 + (kiter & 1) * (L::kTileBytes >> 4);
                mbar_wait(&bar_k_full[kiter & 1], (kiter >> 1) & 1, a.status, a.launch_tag | kErrWaitK);
                tc_fence_after_sync();
                if (active) {
#pragma unroll
                    for (int b = 0; b < kNB; ++b) {
                        issue_qk_half<D>(s_col[b], q_lo, k_cur + ((b * kHalf * 128) >> 4), kHi, idesc_s, leader);
                        mma_commit_p(&bar_s_full[t][b], leader);
                    }
                }
                mma_commit_p(&bar_k_empty[kiter & 1], leader);
                ++kiter;
                if (p.j1 - p.j0 == 1) mma_commit_p(&bar_q_empty, leader);  // a one-tile piece has issued all its scores
                // The V tile of a key tile and the K tile of the next one are waited for one key tile ahead, while
                // this thread would otherwise just wait for the first probabilities: a barrier wait costs it
                // more than a hundred cycles even when the barrier is ready, and that would delay the products.
                mbar_wait(&bar_v_full[viter & 1], (viter >> 1) & 1, a.status, a.launch_tag | kErrWaitV);
                if (p.j1 - p.j0 > 1) mbar_wait(&bar_k_full[kiter & 1], (kiter >> 1) & 1, a.status, a.launch_tag | kErrWaitK);
                for (int j = p.j0; j < p.j1; ++j) {
                    const bool last = (j == p.j1 - 1);
                    const uint32_t vst = viter & 1, kst = kiter & 1;
                    const uint32_t v_cur = v_lo0 + vst * (L::kTileBytes >> 4);
                    k_cur = k_lo0 + kst * (L::kTileBytes >> 4);
                    if (active) {
#pragma unroll
                        for (int b = 0; b < kNB; ++b) {
                            tr.mark(10 + b);
                            mbar_wait(&bar_p_full[t][b], sp & 1, a.status, a.launch_tag | kErrWaitP);
                            tr.mark(20 + b);
                            tc_fence_after_sync();
                            // O_t += P_t[b] . V(keys 64b..64b+63): 16 keys per product = two groups of 8 rows of
                            // 128 bytes (stride 1024); the second 64 head-dim columns live in the next box
                            issue_pv_half(o_col, s_col[b], v_cur + ((b * (kHalf / 16) * 2048) >> 4), kHi, idesc_o,
                                          (j > p.j0 || b > 0) ? 1u : 0u, leader);
                            mma_commit_p(&bar_pv_done[t], leader);
                            if (!last) {
                                // refill the score buffer just consumed with the same half of the next key tile
                                issue_qk_half<D>(s_col[b], q_lo, k_cur + ((b * kHalf * 128) >> 4), kHi, idesc_s, leader);
                                mma_commit_p(&bar_s_full[t][b], leader);
                            } else if (b == kNB - 1) {
                                mma_commit_p(&bar_o_full[t], leader);
                            }
                            tr.mark(30 + b);
                        }
                        ++sp;
                    }
                    mma_commit_p(&bar_v_empty[vst], leader);
                    ++viter;
                    if (!last) {
                        mma_commit_p(&bar_k_empty[kst], leader);
                        ++kiter;
                        // the scores of the piece's last key tile have just been issued: Q is no longer needed and
                        // the producer may fetch the next piece's query tiles while this piece finishes
                        if (j + 2 == p.j1) mma_commit_p(&bar_q_empty, leader);
                        mbar_wait(&bar_v_full[viter & 1], (viter >> 1) & 1, a.status, a.launch_tag | kErrWaitV);
                        if (j + 2 < p.j1) mbar_wait(&bar_k_full[kiter & 1], (kiter >> 1) & 1, a.status, a.launch_tag | kErrWaitK);
                    }
                }
            }
        }
      }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(RegsOneCta::softmax));
        // ------------------------------------------------------------------ softmax + epilogue (one row per thread)
        const int t = warp >> 2;                                   // query tile of the pair this group serves
        const int r = threadIdx.x & 127;                           // row inside the tile
        const uint32_t lane_addr = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const float c = a.scale * kLog2e;                          // scores are used in base 2
        uint32_t sp = 0, op = 0, halves = 0;                       // key tiles, pieces, half tiles this group has done
        Tracer<kTrace> tr;
        tr.init(a, t, cta == 0 && r == 0);
        TileWalker w;
        PieceIter<kTable> pit;
        pit.init(a, cta);
        Piece p;
        while (pit.next(a, p)) {
            if (t == 1 && !p.two) continue;
            float m_used = -INFINITY;  // raw-score maximum the exponents are taken against
            float l = 0.f;
            const AttnItem& item = item_at<kTable>(a, p.item);
            w.seek(item.segs, p.j0);
            for (int j = p.j0; j < p.j1; ++j, ++sp) {
                const int n_valid = w.n_valid(item.segs);
                w.next(item.segs);
#pragma unroll
                for (int b = 0; b < kNB; ++b, ++halves) {
                    const int n_here = n_valid - b * kHalf;  // valid key columns of this half (may be <= 0)
                    tr.mark(1);
                    mbar_wait(&bar_s_full[t][b], sp & 1, a.status, a.launch_tag | kErrWaitS);
                    tr.mark(2);
                    tc_fence_after_sync();
                    uint32_t sr[kHalf / 32][32];
#pragma unroll
                    for (int q2 = 0; q2 < kHalf / 32; ++q2) tmem_ld_32x32b_x32(tmem + lane_addr + col_s(t, b) + q2 * 32, sr[q2]);
                    tmem_ld_wait();
                    tr.mark(3);
                    softmax_half_step<D>(sr, n_here, c, j == p.j0 && b == 0, tmem + lane_addr + col_s(t, b),
                                         tmem + lane_addr + col_o(t), &bar_pv_done[t], (halves - 1) & 1, a.status,
                                         a.launch_tag | kErrWaitO, m_used, l);
                    tr.mark(4);
                    tmem_st_wait();
                    tr.mark(5);
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bar_p_full[t][b]);  // one arrival per warp
                }
            }
            // epilogue of the piece
            mbar_wait(&bar_o_full[t], op & 1, a.status, a.launch_tag | kErrWaitO);
            ++op;
            tc_fence_after_sync();
            const int row = (2 * p.pr + t) * kTile + r;
            if (p.slot < 0) {
                const float inv = 1.f / l;
                __nv_bfloat16* out =
                    reinterpret_cast<__nv_bfloat16*>(item.out) + (static_cast<size_t>(row) * a.n_heads + p.h) * D;
                const bool row_ok = row < item.n_q;
#pragma unroll
                for (int q4 = 0; q4 < D / 32; ++q4) {
                    uint32_t o[32];
                    tmem_ld_32x32b_x32(tmem + lane_addr + col_o(t) + q4 * 32, o);
                    tmem_ld_wait();
                    if (row_ok) {
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            uint4 v;
                            v.x = pack_bf16x2(__uint_as_float(o[8 * i + 0]) * inv, __uint_as_float(o[8 * i + 1]) * inv);
                            v.y = pack_bf16x2(__uint_as_float(o[8 * i + 2]) * inv, __uint_as_float(o[8 * i + 3]) * inv);
                            v.z = pack_bf16x2(__uint_as_float(o[8 * i + 4]) * inv, __uint_as_float(o[8 * i + 5]) * inv);
                            v.w = pack_bf16x2(__uint_as_float(o[8 * i + 6]) * inv, __uint_as_float(o[8 * i + 7]) * inv);
                            *reinterpret_cast<uint4*>(out + q4 * 32 + i * 8) = v;
                        }
                    }
                }
            } else {
                const size_t prow = (static_cast<size_t>(p.slot) * 2 + t) * kTile + r;
                float* po = a.part_o + prow * D;
#pragma unroll
                for (int q4 = 0; q4 < D / 32; ++q4) {
                    uint32_t o[32];
                    tmem_ld_32x32b_x32(tmem + lane_addr + col_o(t) + q4 * 32, o);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        *reinterpret_cast<uint4*>(po + q4 * 32 + i * 4) =
                            make_uint4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
                }
                a.part_ml[prow] = make_float2(m_used * c, l);
            }
            tc_fence_before_sync();  // the O reads above are ordered before the next piece's first P arrival
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 9) tmem_dealloc<kTmemCols>(tmem);
}

// Merges the pieces of every remainder pair whose key range was split over several CTAs:
// out = sum_i 2^(m_i - m*) O_i / sum_i 2^(m_i - m*) l_i.  One warp per query row (a lane owns D/32 columns),
// 8 rows per block, so that enough rows are in flight to hide the latency of the scattered reads.  The grid
// covers the remainder pairs only (whole pairs store their final result themselves).
template <int D, bool kTable>
__global__ void __launch_bounds__(256) attn_combine_kernel(const __grid_constant__ AttnArgs a) {
    constexpr int kPerLane = D / 32;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    grid_dependency_wait();  // the partial results come from the attention kernel before this launch
    // row index over the remainder units: unit_pairs pairs of 2 x 128 rows each
    // (32-bit arithmetic throughout: the launcher only starts this kernel when the row count and the iteration
    // count of the remainder fit, and a 64-bit division costs a warp this short a third of its instructions)
    const int up = a.unit_pairs;
    const uint32_t gr = blockIdx.x * 8u + static_cast<uint32_t>(warp);
    const uint32_t pair_of_row = gr / (2 * kTile);                  // 2 * kTile is a power of two
    const int g = a.n_full * a.n_ctas + static_cast<int>(up == 2 ? pair_of_row >> 1 : pair_of_row);
    if (g >= a.n_pairs) return;
    const int which = up == 2 ? static_cast<int>(pair_of_row & 1u) : 0;   // which pair of the unit (the CTA of a CTA pair that owned it)
    const int rr = static_cast<int>(gr % (2 * kTile));
    const uint32_t cz = static_cast<uint32_t>(a.iters_per_cta);
    int it_i;
    const uint32_t s_g = static_cast<uint32_t>(rem_iter_start<kTable>(a, g, &it_i));
    const AttnItem& item = item_at<kTable>(a, it_i);
    const uint32_t e_g = s_g + static_cast<uint32_t>(item.n_kv_tiles);
    const int first = static_cast<int>(s_g / cz);
    const int last = static_cast<int>((e_g - 1) / cz);
    if (first == last) return;  // the unit was handled by one schedule slot, which stored the final result itself
    const int local = g - item.pair0;
    const int h = local / item.n_up, pr = (local - h * item.n_up) * up + which;
    const int t = rr / kTile, r = rr - t * kTile;
    const int row = (2 * pr + t) * kTile + r;
    if (pr >= item.n_qp || 2 * pr + t >= item.n_qt || row >= item.n_q) return;
    float acc[kPerLane];
#pragma unroll
    for (int e = 0; e < kPerLane; ++e) acc[e] = 0.f;
    float mstar = -INFINITY, lsum = 0.f;
    for (int cta = first; cta <= last; ++cta) {
        // a CTA's piece of this pair sits in scratch slot 2*cta when the CTA's share begins inside the pair
        // (then it was the CTA's first piece), else in slot 2*cta + 1
        const uint32_t c0 = static_cast<uint32_t>(cta) * cz;
        const int slot = 2 * (cta * up + which) + ((c0 >= s_g && c0 < e_g) ? 0 : 1);
        const size_t prow = (static_cast<size_t>(slot) * 2 + t) * kTile + r;
        const float2 ml = a.part_ml[prow];
        const float* po = a.part_o + prow * D + lane * kPerLane;
        float o[kPerLane];
        if (kPerLane == 4) {
            const float4 v = *reinterpret_cast<const float4*>(po);
            o[0] = v.x; o[1] = v.y; o[2 % kPerLane] = v.z; o[3 % kPerLane] = v.w;
        } else {
            const float2 v = *reinterpret_cast<const float2*>(po);
            o[0] = v.x; o[1] = v.y;
        }
        const float m_new = fmaxf(mstar, ml.x);
        const float w_old = exp2f(mstar - m_new), w_new = exp2f(ml.x - m_new);  // exp2(-inf) = 0 on the first piece
        lsum = lsum * w_old + ml.y * w_new;
#pragma unroll
        for (int e = 0; e < kPerLane; ++e) acc[e] = acc[e] * w_old + o[e] * w_new;
        mstar = m_new;
    }
    const float inv = 1.f / lsum;
    __nv_bfloat16* out =
        reinterpret_cast<__nv_bfloat16*>(item.out) + (static_cast<size_t>(row) * a.n_heads + h) * D + lane * kPerLane;
#pragma unroll
    for (int e = 0; e < kPerLane; e += 2)
        *reinterpret_cast<uint32_t*>(out + e) = pack_bf16x2(acc[e] * inv, acc[e + 1] * inv);
}

template <int D>
static cudaError_t set_smem() {
    const int bytes = SmemLayout<D>::kDynamic;
    cudaError_t e = cudaFuncSetAttribute(attn_tcgen05_kernel<D, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(attn_tcgen05_kernel<D, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(attn_tcgen05_kernel<D, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    return e;
}

cudaError_t attn_tcgen05_prepare(int head_dim) {
    if (head_dim == 128)
        return set_smem<128>();
    if (head_dim == 64)
        return set_smem<64>();
    return cudaErrorInvalidValue;
}

// Fills the schedule fields of `a` and of its n_items descriptors `items` (host memory: the array inside `a`, or
// the host copy of the table) for at most `n_ctas_max` resident CTAs; returns the number of remainder pairs if
// some of them are cut (their pieces need merging), else 0.
template <bool kTable>
static int plan_impl(AttnArgs& a, AttnItem* items, int n_ctas_max) {
    long long n_pairs = 0, work = 0;
    for (int i = 0; i < a.n_items; ++i) {
        AttnItem& I = items[i];
        I.n_qt = (I.n_q + kTile - 1) / kTile;
        I.n_qp = (I.n_qt + 1) / 2;
        I.n_up = (I.n_qp + a.unit_pairs - 1) / a.unit_pairs;
        int tiles = 0;
        for (int s = 0; s < I.segs.n; ++s) tiles += (I.segs.tokens[s] + kTile - 1) / kTile;
        I.n_kv_tiles = tiles;
        I.pair0 = static_cast<int>(n_pairs);
        n_pairs += static_cast<long long>(a.n_heads) * I.n_up;
        work += static_cast<long long>(a.n_heads) * I.n_up * tiles;
    }
    a.n_pairs = static_cast<int>(n_pairs);
    long long n_cta = work / 4;  // at least four key tiles per CTA
    if (n_cta < 1) n_cta = 1;
    if (n_cta > n_ctas_max) n_cta = n_ctas_max;
    a.n_ctas = static_cast<int>(n_cta);
    a.n_full = static_cast<int>(n_pairs / n_cta);  // whole pairs per CTA
    const long long g0 = static_cast<long long>(a.n_full) * n_cta;  // first pair shared out by key-tile ranges
    long long iters = 0;
    for (int i = 0; i < a.n_items; ++i) {
        AttnItem& I = items[i];
        const long long pairs = static_cast<long long>(a.n_heads) * I.n_up;
        long long first_rem = g0 - I.pair0;
        if (first_rem < 0) first_rem = 0;
        if (first_rem > pairs) first_rem = pairs;
        I.rem_pair0 = static_cast<int>(first_rem);
        I.rem_iter0 = iters;
        iters += (pairs - first_rem) * I.n_kv_tiles;
    }
    a.total_iters = iters;
    a.iters_per_cta = static_cast<int>((iters + n_cta - 1) / n_cta);
    bool cut = false;
    for (long long g = g0; g < n_pairs && !cut; ++g) {
        int it_i;
        const long long s_g = rem_iter_start<kTable>(a, static_cast<int>(g), &it_i);
        cut = s_g / a.iters_per_cta != (s_g + items[it_i].n_kv_tiles - 1) / a.iters_per_cta;
    }
    return cut ? static_cast<int>(n_pairs - g0) : 0;
}

int attn_tcgen05_plan(AttnArgs& a, AttnItem* items, int n_ctas_max) {
    if (a.unit_pairs < 1) a.unit_pairs = 1;
    if (items == a.items) {
        a.items_tab = nullptr;
        return plan_impl<false>(a, items, n_ctas_max);
    }
    a.items_tab = items;
    return plan_impl<true>(a, items, n_ctas_max);
}

// `a` has been planned (attn_tcgen05_plan returned merge_pairs); with more than kMaxInline items a.items_tab must
// point to the device copy of the planned descriptors.
template <int D>
static cudaError_t launch_impl(const AttnArgs& a, int merge_pairs, const CUtensorMap& tm_q, const CUtensorMap& tm_k,
                               const CUtensorMap& tm_v, cudaStream_t s) {
    const bool table = a.items_tab != nullptr, trace = a.trace != nullptr && !table;
    const dim3 grid(a.n_ctas), block(kThreads), mgrid(merge_pairs * a.unit_pairs * (2 * kTile / 8)), mblock(256);
    const size_t smem = SmemLayout<D>::kDynamic;
    if (merge_pairs && a.total_iters >= (1ll << 31)) return cudaErrorInvalidValue;  // the merge kernel indexes in 32 bits
    cudaError_t e;
    if (a.unit_pairs == 2) e = launch_attn_pair(a, tm_q, tm_k, tm_v, s);   // tm_k: the map with 32-row boxes
    else if (table) e = launch_overlapped(attn_tcgen05_kernel<D, false, true>, grid, block, smem, s, tm_q, tm_k, tm_v, a);
    else if (trace) e = launch_overlapped(attn_tcgen05_kernel<D, true, false>, grid, block, smem, s, tm_q, tm_k, tm_v, a);
    else e = launch_overlapped(attn_tcgen05_kernel<D, false, false>, grid, block, smem, s, tm_q, tm_k, tm_v, a);
    if (e == cudaSuccess && merge_pairs)
        e = table ? launch_overlapped(attn_combine_kernel<D, true>, mgrid, mblock, 0, s, a)
                  : launch_overlapped(attn_combine_kernel<D, false>, mgrid, mblock, 0, s, a);
    return e;
}

cudaError_t launch_attn_tcgen05(const AttnArgs& a, int merge_pairs, const CUtensorMap& tm_q, const CUtensorMap& tm_k,
                                const CUtensorMap& tm_v, cudaStream_t s, int* n_launches) {
    *n_launches = merge_pairs ? 2 : 1;
    if (a.n_items > kMaxInline && !a.items_tab) return cudaErrorInvalidValue;
    if (a.head_dim == 128) return launch_impl<128>(a, merge_pairs, tm_q, tm_k, tm_v, s);
    if (a.head_dim == 64) return launch_impl<64>(a, merge_pairs, tm_q, tm_k, tm_v, s);
    return cudaErrorInvalidValue;
}

// A one-thread kernel that waits on a barrier nothing arrives on, with a short limit: exercises the bounded
// wait and the status word without hanging anything.
__global__ void wait_probe_kernel(uint32_t* status, unsigned long long limit_ns) {
    __shared__ uint64_t bar;
    mbar_init(&bar, 1);
    fence_mbar_init();
    mbar_wait(&bar, 0, status, kErrProbe, limit_ns);
}

cudaError_t launch_wait_probe(uint32_t* status, unsigned long long limit_ns, cudaStream_t s) {
    wait_probe_kernel<<<1, 1, 0, s>>>(status, limit_ns);
    return cudaGetLastError();
}

}  // namespace ffk
