// Flash attention of one chunk's queries on CTA PAIRS (a cluster of two CTAs on the two SMs of a TPC working as
// one through tcgen05 cta_group::2), head_dim 128.  Same arithmetic, tile sizes, tensor-memory map and roles as
// the one-CTA-per-SM kernel (attn_sm100.cu); what changes is who stages what:
//
//   * a work unit is TWO consecutive pairs of query tiles of one head: CTA 0 of the pair owns query tiles 4u and
//     4u+1, CTA 1 owns 4u+2 and 4u+3; both walk the same key tiles;
//   * every product is issued once, by CTA 0, for 256 query rows: rows 0-127 come from CTA 0's shared / tensor
//     memory, rows 128-255 from CTA 1's, and each CTA's half of the result lands in its own tensor memory;
//   * the B operand of a product is split between the two CTAs' shared memories: of the 64 keys of a score half
//     each CTA stages 32 (QK^T), and of the 128 value columns each CTA stages 64 (PV).  Per key tile a CTA fetches
//     16 KB of K and 16 KB of V instead of 32 + 32: half the L2 -> shared-memory traffic per query row, and the
//     64-key QK^T products no longer saturate one SM's shared-memory port;
//   * every copy is a plain TMA tile load into the issuing CTA's own shared memory (no multicast); its completion
//     bytes are signalled on CTA 0's barrier, where the issuing threads wait.
//
// Barriers: "full" barriers of Q, K and V and the "probabilities ready" barriers live in CTA 0 (the only CTA that
// issues products); "empty", "scores ready", "product done" and "output ready" barriers exist in both CTAs and
// are signalled by commits that arrive in both.  Every wait is bounded, as in the single-CTA kernel.
#include "attn_common.cuh"

namespace ffk {

namespace {

// K/V tiles in flight per CTA (the halved tiles leave room for more stages than the single-CTA kernel has).
#ifndef FF_PAIR_STAGES
#define FF_PAIR_STAGES 4
#endif
constexpr uint32_t kS = FF_PAIR_STAGES;

struct PairSmem {
    static constexpr int kTileBytes = 128 * 128 * 2;     // one 128-row query tile, head_dim 128
    static constexpr int kQBox = 128 * 64 * 2;           // 128 rows x 64 columns
    static constexpr int kKStage = 64 * 128 * 2;         // this CTA's 64 of a tile's 128 keys, all 128 columns
    static constexpr int kKBox = 32 * 64 * 2;            // 32 keys x 64 columns
    static constexpr int kKColBox = 64 * 64 * 2;         // both score halves' 32 keys x 64 columns
    static constexpr int kVStage = 128 * 64 * 2;         // all 128 keys, this CTA's 64 of the 128 value columns
    static constexpr int kQ = 0;
    static constexpr int kK = 2 * kTileBytes;
    static constexpr int kV = kK + static_cast<int>(kS) * kKStage;
    static constexpr int kTotal = kV + static_cast<int>(kS) * kVStage;
    static constexpr int kDynamic = kTotal + 1024;       // above half an SM's shared memory: one CTA per SM
};
static_assert(PairSmem::kDynamic > 114 * 1024, "two CTAs of this kernel must not share an SM (512 tensor-memory columns each)");

constexpr int D = 128;

__device__ __forceinline__ void issue_qk_half_pair(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc,
                                                   uint32_t leader) {
#pragma unroll
    for (int kk = 0; kk < D / 16; ++kk) {
        const uint32_t off_a = ((kk / 4) * PairSmem::kQBox + (kk % 4) * 32) >> 4;
        const uint32_t off_b = ((kk / 4) * PairSmem::kKColBox + (kk % 4) * 32) >> 4;
        mma2_ss_lohi_p(d_tmem, a_lo + off_a, b_lo + off_b, hi, idesc, kk > 0 ? 1u : 0u, leader);
    }
}
__device__ __forceinline__ void issue_pv_half_pair(uint32_t d_tmem, uint32_t p_tmem, uint32_t b_lo, uint32_t hi, uint32_t idesc,
                                                   uint32_t accumulate, uint32_t leader) {
    mma2_ts_lohi_p(d_tmem, p_tmem, b_lo, hi, idesc, accumulate, leader);
#pragma unroll
    for (int kk = 1; kk < kHalf / 16; ++kk)
        mma2_ts_lohi_p(d_tmem, p_tmem + kk * 8, b_lo + ((kk * 2048) >> 4), hi, idesc, 1u, leader);
}

}  // namespace

template <bool kTable>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
attn_pair_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k32,
                 const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ AttnArgs a) {
    using L = PairSmem;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ uint64_t bar_q_full, bar_q_empty, bar_k_full[kS], bar_k_empty[kS], bar_v_full[kS], bar_v_empty[kS],
        bar_s_full[2][2], bar_p_full[2][2], bar_pv_done[2], bar_o_full[2];
    __shared__ uint32_t tmem_base_slot;

    const int warp = __shfl_sync(0xffffffffu, static_cast<int>(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();        // 0: the CTA that issues the pair's products
    const int cl = blockIdx.x >> 1;                 // the pair's index: its slot in the schedule

    if (threadIdx.x == 0) {
        mbar_init(&bar_q_full, 1);
        mbar_init(&bar_q_empty, 2);
        for (uint32_t i = 0; i < kS; ++i) {
            mbar_init(&bar_k_full[i], 1);
            mbar_init(&bar_k_empty[i], 2);
            mbar_init(&bar_v_full[i], 1);
            mbar_init(&bar_v_empty[i], 2);
        }
        for (int i = 0; i < 2; ++i) {
            for (int b = 0; b < kNB; ++b) {
                mbar_init(&bar_s_full[i][b], 1);
                mbar_init(&bar_p_full[i][b], 8);   // four softmax warps of each CTA
            }
            mbar_init(&bar_pv_done[i], 1);
            mbar_init(&bar_o_full[i], 1);
        }
        fence_mbar_init();
    }
    if (warp == 9) {
        tmem_alloc_pair<kTmemCols>(&tmem_base_slot);
        tmem_relinquish_pair();
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();   // both CTAs' barriers exist before either signals the other's
    tc_fence_after_sync();
    const uint32_t tmem = __shfl_sync(0xffffffffu, tmem_base_slot, 0);
    grid_dependency_wait();

    if (warp >= 8) {
      asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(RegsCtaPair::other));
      if (warp == 8) {
        // ------------------------------------------------------------------ TMA producer (one lane, in each CTA)
        if (lane == 0) {
            prefetch_tensormap(&tm_q);
            prefetch_tensormap(&tm_k32);
            prefetch_tensormap(&tm_v);
            const uint32_t lead_q_full = mapa_u32(smem_u32(&bar_q_full), 0);
            const uint32_t lead_k_full0 = mapa_u32(smem_u32(&bar_k_full[0]), 0), lead_v_full0 = mapa_u32(smem_u32(&bar_v_full[0]), 0);
            uint32_t kiter = 0, viter = 0, n_piece = 0;
            TileWalker w;
            PieceIter<kTable> pit;
            pit.init(a, cl);
            Piece p;
            for (; pit.next(a, p); ++n_piece) {
                const AttnItem& item = item_at<kTable>(a, p.item);
                const int tile0 = (2 * p.pr + static_cast<int>(rank)) * 2;   // this CTA's first query tile of the unit
                if (n_piece > 0) mbar_wait(&bar_q_empty, (n_piece - 1) & 1, a.status, a.launch_tag | kErrWaitQ);
                // both CTAs always fetch two query tiles (tiles past the head's last one read rows nobody uses)
                if (rank == 0) mbar_expect_tx(&bar_q_full, 4 * L::kTileBytes);
                for (int t = 0; t < 2; ++t)
#pragma unroll
                    for (int b = 0; b < 2; ++b)
                        tma_load_2d_pair(smem + L::kQ + t * L::kTileBytes + b * L::kQBox, &tm_q, b * 64,
                                         item.q_row0 + p.h * a.q_rows_per_head + (tile0 + t) * kTile, lead_q_full);
                const KvSegs& segs = item.segs;
                w.seek(segs, p.j0);
                for (int j = p.j0; j < p.j1; ++j) {
                    const int row = w.row(segs, p.h);
                    uint32_t st = kiter % kS;
                    if (kiter >= kS) mbar_wait(&bar_k_empty[st], ((kiter / kS) - 1) & 1, a.status, a.launch_tag | kErrWaitKEmpty);
                    if (rank == 0) mbar_expect_tx(&bar_k_full[st], 2 * L::kKStage);
                    // of each score half's 64 keys this CTA stages 32: keys [64 half + 32 rank, +32)
#pragma unroll
                    for (int cb = 0; cb < 2; ++cb)
#pragma unroll
                        for (int hb = 0; hb < kNB; ++hb)
                            tma_load_2d_pair(smem + L::kK + st * L::kKStage + cb * L::kKColBox + hb * L::kKBox, &tm_k32, cb * 64,
                                             row + hb * kHalf + static_cast<int>(rank) * 32, lead_k_full0 + st * 8);
                    ++kiter;
                    st = viter % kS;
                    if (viter >= kS) mbar_wait(&bar_v_empty[st], ((viter / kS) - 1) & 1, a.status, a.launch_tag | kErrWaitVEmpty);
                    if (rank == 0) mbar_expect_tx(&bar_v_full[st], 2 * L::kVStage);
                    // of the 128 value columns this CTA stages 64
                    tma_load_2d_pair(smem + L::kV + st * L::kVStage, &tm_v, static_cast<int>(rank) * 64, row, lead_v_full0 + st * 8);
                    ++viter;
                    w.next(segs);
                }
            }
            // after an expired wait copies may still be on their way into this CTA's shared memory: give them a
            // bounded time before the CTA ends (their completion is signalled in CTA 0, so CTA 1 just sits it out)
            if (*reinterpret_cast<volatile uint32_t*>(a.status) != 0u) {
                const unsigned long long t0 = globaltimer_ns();
                while (globaltimer_ns() - t0 < 200000ull) {}
            }
        }
      } else if ((warp == 9 || warp == 10) && rank == 0) {
        // ------------------------------------------------------------------ MMA issuers (CTA 0 only): warp 9 serves
        // query tile 0 of both CTAs, warp 10 query tile 1 of both
        const int t = warp - 9;
        const uint32_t leader = elect_one_sync();
        constexpr uint32_t idesc_s = make_idesc_bf16(256, kHalf, false);
        constexpr uint32_t idesc_o = make_idesc_bf16(256, D, true);
        constexpr uint32_t kHi = desc_hi_sw128(1024);
        const uint32_t q_lo = desc_lo_sw128(smem_u32(smem + L::kQ + t * L::kTileBytes), 16);
        const uint32_t k_lo0 = desc_lo_sw128(smem_u32(smem + L::kK), 16);
        const uint32_t v_lo0 = desc_lo_sw128(smem_u32(smem + L::kV), 16);
        const uint32_t s_col[2] = {tmem + col_s(t, 0), tmem + col_s(t, kNB - 1)};
        const uint32_t o_col = tmem + col_o(t);
        uint32_t kiter = 0, viter = 0, n_piece = 0, sp = 0;

        PieceIter<kTable> pit;
        pit.init(a, cl);
        Piece p;
        for (; pit.next(a, p); ++n_piece) {
            const AttnItem& item = item_at<kTable>(a, p.item);
            const bool active = 4 * p.pr + t < item.n_qt;   // CTA 0's tile t of the unit exists (CTA 1's may not)
            mbar_wait(&bar_q_full, n_piece & 1, a.status, a.launch_tag | kErrWaitQ);
            uint32_t k_cur = k_lo0 + (kiter % kS) * (L::kKStage >> 4);
            mbar_wait(&bar_k_full[kiter % kS], (kiter / kS) & 1, a.status, a.launch_tag | kErrWaitK);
            tc_fence_after_sync();
            if (active) {
#pragma unroll
                for (int b = 0; b < kNB; ++b) {
                    issue_qk_half_pair(s_col[b], q_lo, k_cur + ((b * L::kKBox) >> 4), kHi, idesc_s, leader);
                    mma2_commit_p(&bar_s_full[t][b], leader);
                }
            }
            mma2_commit_p(&bar_k_empty[kiter % kS], leader);
            ++kiter;
            if (p.j1 - p.j0 == 1) mma2_commit_p(&bar_q_empty, leader);
            mbar_wait(&bar_v_full[viter % kS], (viter / kS) & 1, a.status, a.launch_tag | kErrWaitV);
            if (p.j1 - p.j0 > 1) mbar_wait(&bar_k_full[kiter % kS], (kiter / kS) & 1, a.status, a.launch_tag | kErrWaitK);
            for (int j = p.j0; j < p.j1; ++j) {
                const bool last = (j == p.j1 - 1);
                const uint32_t vst = viter % kS, kst = kiter % kS;
                const uint32_t v_cur = v_lo0 + vst * (L::kVStage >> 4);
                k_cur = k_lo0 + kst * (L::kKStage >> 4);
                if (active) {
#pragma unroll
                    for (int b = 0; b < kNB; ++b) {
                        // the probabilities come from both CTAs' softmax groups
                        mbar_wait_cluster(&bar_p_full[t][b], sp & 1, a.status, a.launch_tag | kErrWaitP);
                        tc_fence_after_sync();
                        issue_pv_half_pair(o_col, s_col[b], v_cur + ((b * (kHalf / 16) * 2048) >> 4), kHi, idesc_o,
                                           (j > p.j0 || b > 0) ? 1u : 0u, leader);
                        mma2_commit_p(&bar_pv_done[t], leader);
                        if (!last) {
                            issue_qk_half_pair(s_col[b], q_lo, k_cur + ((b * L::kKBox) >> 4), kHi, idesc_s, leader);
                            mma2_commit_p(&bar_s_full[t][b], leader);
                        } else if (b == kNB - 1) {
                            mma2_commit_p(&bar_o_full[t], leader);
                        }
                    }
                    ++sp;
                }
                mma2_commit_p(&bar_v_empty[vst], leader);
                ++viter;
                if (!last) {
                    mma2_commit_p(&bar_k_empty[kst], leader);
                    ++kiter;
                    if (j + 2 == p.j1) mma2_commit_p(&bar_q_empty, leader);
                    mbar_wait(&bar_v_full[viter % kS], (viter / kS) & 1, a.status, a.launch_tag | kErrWaitV);
                    if (j + 2 < p.j1) mbar_wait(&bar_k_full[kiter % kS], (kiter / kS) & 1, a.status, a.launch_tag | kErrWaitK);
                }
            }
        }
      }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(RegsCtaPair::softmax));
        // ------------------------------------------------------------------ softmax + epilogue (one row per thread),
        // in both CTAs, each on its own 128 rows of the pair's products
        const int t = warp >> 2;
        const int r = threadIdx.x & 127;
        const uint32_t lane_addr = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const float c = a.scale * kLog2e;
        const uint32_t lead_p_full[2] = {mapa_u32(smem_u32(&bar_p_full[t][0]), 0), mapa_u32(smem_u32(&bar_p_full[t][kNB - 1]), 0)};
        uint32_t sp = 0, op = 0, halves = 0;
        TileWalker w;
        PieceIter<kTable> pit;
        pit.init(a, cl);
        Piece p;
        while (pit.next(a, p)) {
            const AttnItem& item = item_at<kTable>(a, p.item);
            // the stream runs when CTA 0's tile exists; CTA 1 then takes part even if its own tile does not (its rows
            // of the products are never stored)
            if (4 * p.pr + t >= item.n_qt) continue;
            const int tile = (2 * p.pr + static_cast<int>(rank)) * 2 + t;
            float m_used = -INFINITY;
            float l = 0.f;
            w.seek(item.segs, p.j0);
            for (int j = p.j0; j < p.j1; ++j, ++sp) {
                const int n_valid = w.n_valid(item.segs);
                w.next(item.segs);
#pragma unroll
                for (int b = 0; b < kNB; ++b, ++halves) {
                    const int n_here = n_valid - b * kHalf;
                    mbar_wait(&bar_s_full[t][b], sp & 1, a.status, a.launch_tag | kErrWaitS);
                    tc_fence_after_sync();
                    uint32_t sr[kHalf / 32][32];
#pragma unroll
                    for (int q2 = 0; q2 < kHalf / 32; ++q2) tmem_ld_32x32b_x32(tmem + lane_addr + col_s(t, b) + q2 * 32, sr[q2]);
                    tmem_ld_wait();
                    softmax_half_step<D>(sr, n_here, c, j == p.j0 && b == 0, tmem + lane_addr + col_s(t, b),
                                         tmem + lane_addr + col_o(t), &bar_pv_done[t], (halves - 1) & 1, a.status,
                                         a.launch_tag | kErrWaitO, m_used, l);
                    tmem_st_wait();
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(lead_p_full[b]);  // one arrival per warp, on CTA 0's barrier
                }
            }
            // epilogue of the piece
            mbar_wait(&bar_o_full[t], op & 1, a.status, a.launch_tag | kErrWaitO);
            ++op;
            tc_fence_after_sync();
            const int row = tile * kTile + r;
            if (p.slot < 0) {
                const float inv = 1.f / l;
                __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(item.out) + (static_cast<size_t>(row) * a.n_heads + p.h) * D;
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
                // scratch slot of this CTA's piece: two per CTA, as in the single-CTA kernel
                const int slot = 2 * (2 * cl + static_cast<int>(rank)) + (p.slot & 1);
                const size_t prow = (static_cast<size_t>(slot) * 2 + t) * kTile + r;
                float* po = a.part_o + prow * D;
#pragma unroll
                for (int q4 = 0; q4 < D / 32; ++q4) {
                    uint32_t o[32];
                    tmem_ld_32x32b_x32(tmem + lane_addr + col_o(t) + q4 * 32, o);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        *reinterpret_cast<uint4*>(po + q4 * 32 + i * 4) = make_uint4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
                }
                a.part_ml[prow] = make_float2(m_used * c, l);
            }
            tc_fence_before_sync();
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();   // neither CTA releases shared or tensor memory the other's products may still touch
    if (warp == 9) tmem_dealloc_pair<kTmemCols>(tmem);
}

cudaError_t attn_pair_prepare(int* max_pairs) {
    cudaError_t e = cudaFuncSetAttribute(attn_pair_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, PairSmem::kDynamic);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(attn_pair_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, PairSmem::kDynamic);
    if (e != cudaSuccess) return e;
    // how many CTA pairs can be resident at once (the schedule assumes all of a launch's pairs are)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * kMaxCtas);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = PairSmem::kDynamic;
    int n = 0;
    e = cudaOccupancyMaxActiveClusters(&n, attn_pair_kernel<false>, &cfg);
    if (e != cudaSuccess) return e;
    *max_pairs = n;
    return cudaSuccess;
}

cudaError_t launch_attn_pair(const AttnArgs& a, const CUtensorMap& tm_q, const CUtensorMap& tm_k32, const CUtensorMap& tm_v,
                             cudaStream_t s) {
    if (a.head_dim != 128 || a.unit_pairs != 2) return cudaErrorInvalidValue;
    if (a.n_items > kMaxInline && !a.items_tab) return cudaErrorInvalidValue;
    const dim3 grid(2 * a.n_ctas), block(kThreads);
    return a.items_tab ? launch_overlapped(attn_pair_kernel<true>, grid, block, PairSmem::kDynamic, s, tm_q, tm_k32, tm_v, a)
                       : launch_overlapped(attn_pair_kernel<false>, grid, block, PairSmem::kDynamic, s, tm_q, tm_k32, tm_v, a);
}

}  // namespace ffk
