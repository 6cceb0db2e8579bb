// Work distribution of the tensor-core attention kernel, shared by the kernel roles, the merge kernel and the
// host-side planner (and enumerable on the host, so that tests can check the cover without a GPU).
//
// A launch serves n_items layer-calls.  The unit of work is a pair of 128-row query tiles of one head of one
// item (or, for the kernel that runs on CTA pairs, two consecutive pairs of a head: one pair per CTA, both CTAs
// walking the same key tiles); units are numbered item-major, then head, then unit.  "Pair" below reads "unit"
// and "CTA" reads "CTA pair" in that case.  Every CTA first takes n_full whole pairs
// (pair r * n_ctas + cta: the CTAs walk the key tiles of neighbouring pairs in step, so a K/V tile that several
// of them need is fetched from HBM once and then hit in L2), then an equal share of the (pair, key tile)
// iterations of the remaining pairs, flattened in pair order; a share may cut pairs, and the pieces of a cut
// pair are merged afterwards.
//
// The item descriptors are either the array inside the launch arguments (kTable = false, up to kMaxInline
// items) or a table in memory (kTable = true: device memory for the kernels, host memory while planning).
#pragma once
#include "ff_internal.h"

namespace ffk {

struct Piece {
    int item, h, pr, j0, j1, slot;  // item, head, pair in the head, key-tile range, scratch slot (-1 = final output)
    bool two;                       // the pair has a second query tile
};

template <bool kTable>
__host__ __device__ __forceinline__ const AttnItem& item_at(const AttnArgs& a, int i) {
    if constexpr (kTable) return a.items_tab[i];
    else return a.items[i];
}

// Item that holds launch-wide pair g.  pair0 is non-decreasing over the items: binary search.
template <bool kTable>
__host__ __device__ inline int item_of_pair(const AttnArgs& a, int g) {
    int lo = 0, hi = a.n_items - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (g >= item_at<kTable>(a, mid).pair0) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// Start of remainder pair g (launch-wide pair index, g >= n_full * n_ctas) in the flattened iteration list.
template <bool kTable>
__host__ __device__ inline long long rem_iter_start(const AttnArgs& a, int g, int* item_out) {
    const int i = item_of_pair<kTable>(a, g);
    const AttnItem& I = item_at<kTable>(a, i);
    if (item_out) *item_out = i;
    return I.rem_iter0 + static_cast<long long>(g - I.pair0 - I.rem_pair0) * I.n_kv_tiles;
}

// The pieces of one CTA in the order it walks them.  A CTA's pairs and iterations only move forward through the
// items, so the item of the next piece is found by stepping a cursor, not by searching.
template <bool kTable>
struct PieceIter {
    int cta, round, cur;
    long long it, end;
    bool first_rem;
    __host__ __device__ inline void init(const AttnArgs& a, int cta_) {
        cta = cta_;
        round = 0;
        cur = 0;
        it = static_cast<long long>(cta) * a.iters_per_cta;
        end = it + a.iters_per_cta < a.total_iters ? it + a.iters_per_cta : a.total_iters;
        first_rem = true;
    }
    __host__ __device__ inline bool next(const AttnArgs& a, Piece& p) {
        int local;
        if (round < a.n_full) {
            const int g = round * a.n_ctas + cta;
            ++round;
            while (cur + 1 < a.n_items && g >= item_at<kTable>(a, cur + 1).pair0) ++cur;
            const AttnItem& I = item_at<kTable>(a, cur);
            p.item = cur;
            local = g - I.pair0;
            p.j0 = 0;
            p.j1 = I.n_kv_tiles;
            p.slot = -1;
        } else {
            if (it >= end) return false;
            // (the cursor left by the whole pairs is at or before the item of the first remainder iteration)
            while (cur + 1 < a.n_items && it >= item_at<kTable>(a, cur + 1).rem_iter0) ++cur;
            const AttnItem& I = item_at<kTable>(a, cur);
            const int T = I.n_kv_tiles;
            const long long rel = it - I.rem_iter0;
            const int k = static_cast<int>(rel / T);
            p.item = cur;
            local = I.rem_pair0 + k;
            p.j0 = static_cast<int>(rel - static_cast<long long>(k) * T);
            const long long left = end - it;
            p.j1 = static_cast<int>(left < T - p.j0 ? p.j0 + left : T);
            p.slot = (p.j0 == 0 && p.j1 == T) ? -1 : 2 * cta + (first_rem ? 0 : 1);
            first_rem = false;
            it += p.j1 - p.j0;
        }
        const AttnItem& I = item_at<kTable>(a, p.item);
        p.h = local / I.n_up;
        p.pr = local - p.h * I.n_up;           // unit index inside the head (= pair index when a unit is one pair)
        p.two = 2 * p.pr + 1 < I.n_qt;         // meaningful for one-pair units only
        return true;
    }
};

}  // namespace ffk
