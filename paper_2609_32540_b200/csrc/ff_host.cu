// Host side of the chunk-attention library: arena carving, per-stage ring bookkeeping (Eq. 2: Append and
// Tail_H), the anchor-slot table (bank A, window chosen by the caller), argument validation, tensor-map
// creation and kernel launches.  No device memory is allocated here: everything lives in the caller's arena.
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/ff.h"
#include "ff_internal.h"
#include "attn_schedule.h"

// What FF_ATTN_AUTO does with head_dim 128: 1 = choose per launch between the kernel on CTA pairs (cta_group::2)
// and the one-CTA-per-SM kernel, 0 = always the latter.
#ifndef FF_CTA_PAIR_DEFAULT
#define FF_CTA_PAIR_DEFAULT 1
#endif

using namespace ffk;

namespace {

thread_local int32_t g_last_cuda_error = 0;

inline bool cuda_ok(cudaError_t e) {
    if (e == cudaSuccess) return true;
    g_last_cuda_error = static_cast<int32_t>(e);
    return false;
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline int32_t round_up_tile(int32_t x) { return (x + kTile - 1) / kTile * kTile; }

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct Derived {
    int32_t tf, cap, cap_pad, tf_pad, elem, d, pairs[3], q_slots;
    int32_t R;  // slots per bank: H + 1 unless the caller asked for more (several chunks of one stage per launch)
    int64_t ring_rows, anchor_rows, total_rows;
    size_t off_tab_f, off_tab_y, off_tab_x, off_status, off_items, off_gain, off_k, off_v, off_q, off_part_o, off_part_ml, off_stage, stage_bytes, total;
    int impl, pair_mode;
};

ff_status derive(const ff_cache_config* cfg, Derived* D) {
    if (!cfg) return FF_ERR_INVALID_ARG;
    if (cfg->n_layers < 1 || cfg->n_heads < 1 || cfg->head_dim < 2 || (cfg->head_dim & 1) || cfg->grid_h < 1 ||
        cfg->grid_w < 1 || cfg->chunk_frames < 1 || cfg->n_stages < 1 || cfg->history_chunks < 0 ||
        cfg->n_anchor_slots < 0 || cfg->max_visible_anchors < 0 || cfg->max_frame_pos < 1 || cfg->device < FF_DEVICE_NONE ||
        !(cfg->rope_theta > 0.f))
        return FF_ERR_INVALID_ARG;
    if (cfg->dtype != FF_BF16 && cfg->dtype != FF_F32) return FF_ERR_INVALID_ARG;
    if (cfg->frame_pos_stride < 0) return FF_ERR_INVALID_ARG;
    if (cfg->qk_norm && !(cfg->qk_norm_eps >= 0.f)) return FF_ERR_INVALID_ARG;
    if (cfg->max_visible_anchors + cfg->history_chunks + 1 > kMaxSegs) return FF_ERR_UNSUPPORTED;
    if (cfg->ring_slots != 0 && (cfg->ring_slots < cfg->history_chunks + 1 || cfg->ring_slots > 4096)) return FF_ERR_INVALID_ARG;
    if (cfg->max_batch < 0 || cfg->max_batch > kMaxBatch) return FF_ERR_INVALID_ARG;
    D->R = cfg->ring_slots ? cfg->ring_slots : cfg->history_chunks + 1;
    if (cfg->max_visible_anchors > cfg->n_anchor_slots) return FF_ERR_INVALID_ARG;
    static_assert(FF_MAX_BATCH == kMaxBatch, "ff.h and ff_internal.h disagree on the batch limit");
    if (cfg->head_dim != 64 && cfg->head_dim != 128) return FF_ERR_UNSUPPORTED;
    int impl = cfg->attn_impl;
    // pair_mode: 0 = one-CTA-per-SM kernel, 1 = CTA-pair kernel, 2 = chosen per launch
    D->pair_mode = 0;
    if (impl == FF_ATTN_AUTO) {
        impl = cfg->dtype == FF_BF16 ? FF_ATTN_TCGEN05 : FF_ATTN_SIMT;
        if (impl == FF_ATTN_TCGEN05 && cfg->head_dim == 128 && FF_CTA_PAIR_DEFAULT) D->pair_mode = 2;
    } else if (impl == FF_ATTN_TCGEN05_PAIR) {
        if (cfg->head_dim != 128) return FF_ERR_UNSUPPORTED;
        impl = FF_ATTN_TCGEN05;
        D->pair_mode = 1;
    }
    if (impl != FF_ATTN_TCGEN05 && impl != FF_ATTN_SIMT) return FF_ERR_INVALID_ARG;
    if (impl == FF_ATTN_TCGEN05 && cfg->dtype != FF_BF16) return FF_ERR_UNSUPPORTED;
    D->impl = impl;
    D->d = cfg->head_dim;
    D->elem = cfg->dtype == FF_BF16 ? 2 : 4;
    if (cfg->rope_pairs[0] | cfg->rope_pairs[1] | cfg->rope_pairs[2]) {
        for (int i = 0; i < 3; ++i) {
            if (cfg->rope_pairs[i] < 0) return FF_ERR_INVALID_ARG;
            D->pairs[i] = cfg->rope_pairs[i];
        }
    } else {
        const int side = cfg->head_dim / 6;
        D->pairs[0] = cfg->head_dim / 2 - 2 * side;
        D->pairs[1] = side;
        D->pairs[2] = side;
    }
    if (D->pairs[0] + D->pairs[1] + D->pairs[2] != cfg->head_dim / 2) return FF_ERR_INVALID_ARG;
    const int64_t tf = (int64_t)cfg->grid_h * cfg->grid_w;
    const int64_t cap = tf * cfg->chunk_frames;
    if (cap > (1 << 24)) return FF_ERR_UNSUPPORTED;
    D->tf = (int32_t)tf;
    D->cap = (int32_t)cap;
    D->cap_pad = round_up_tile(D->cap);
    D->tf_pad = round_up_tile(D->tf);
    D->ring_rows = (int64_t)cfg->n_stages * cfg->n_layers * cfg->n_heads * D->R * D->cap_pad;
    D->anchor_rows = (int64_t)cfg->n_anchor_slots * cfg->n_layers * cfg->n_heads * D->tf_pad;
    D->total_rows = D->ring_rows + D->anchor_rows;
    if (D->total_rows >= (int64_t)1 << 31) return FF_ERR_UNSUPPORTED;  // tile coordinates are 32-bit
    size_t off = 0;
    D->off_tab_f = off; off = align_up(off + (size_t)cfg->max_frame_pos * D->pairs[0] * sizeof(float2), 256);
    D->off_tab_y = off; off = align_up(off + (size_t)cfg->grid_h * D->pairs[1] * sizeof(float2), 256);
    D->off_tab_x = off; off = align_up(off + (size_t)cfg->grid_w * D->pairs[2] * sizeof(float2), 256);
    D->off_status = off; off = align_up(off + 256, 1024);
    // descriptors of a launch over more than kMaxInline layer-calls (the whole clip of a stage at once)
    D->off_items = off; off = align_up(off + (size_t)kMaxBatch * sizeof(AttnItem), 1024);
    // channel gains of the q/k normalisation: [layer][q|k][d] floats; absent when the normalisation is off
    D->off_gain = off; off = align_up(off + (cfg->qk_norm ? (size_t)cfg->n_layers * 2 * D->d * sizeof(float) : 0), 1024);
    const size_t mat_bytes = (size_t)D->total_rows * D->d * D->elem;
    D->off_k = off; off = align_up(off + mat_bytes, 1024);
    D->off_v = off; off = align_up(off + mat_bytes, 1024);
    // rotated queries: one region per layer-call of a batched launch (at most one call per stage)
    D->q_slots = cfg->max_batch ? cfg->max_batch : (cfg->n_stages < kMaxInline ? cfg->n_stages : kMaxInline);
    D->off_q = off; off = align_up(off + (size_t)D->q_slots * cfg->n_heads * D->cap_pad * D->d * D->elem, 1024);
    D->off_part_o = off; off = align_up(off + (size_t)2 * kMaxCtas * 2 * kTile * D->d * sizeof(float), 1024);
    D->off_part_ml = off; off = align_up(off + (size_t)2 * kMaxCtas * 2 * kTile * sizeof(float2), 1024);
    D->stage_bytes = align_up((size_t)D->cap * cfg->n_heads * D->d * D->elem, 1024);
    D->off_stage = off; off += 8 * D->stage_bytes;  // two sets of (q, k, v, out) for the host-buffer entry points
    D->total = off;
    return FF_OK;
}

struct SlotMeta {
    int32_t chunk = -1;
    int32_t n_tokens = 0;
};

}  // namespace

struct ff_cache {
    ff_cache_config cfg;
    Derived D;
    uint8_t* arena = nullptr;
    int sm_count = 148;
    bool dry = false;  // bookkeeping only: nothing is enqueued
    std::vector<int32_t> head, count, next_chunk;  // per stage
    std::vector<SlotMeta> slots;                   // [stage][layer][slot]
    std::vector<int32_t> anchor_pos;               // per anchor slot
    std::vector<uint8_t> anchor_valid;             // [slot][layer]
    CUtensorMap tm_q, tm_k, tm_v;
    CUtensorMap tm_k32;               // K in boxes of 32 rows (the kernel on CTA pairs stages a quarter tile per copy)
    int pair_slots = 0;               // CTA pairs that can be resident at once; 0 = the pair kernel is not used
    int64_t n_layer_calls = 0, n_advances = 0, n_anchor_publishes = 0, n_launches = 0;
    std::vector<cudaEvent_t> prof_events;  // 3 per recorded layer-call
    size_t prof_used = 0;
    bool profiling = false;
    // copy streams and events of the pipelined host-buffer scheduler (created on first use)
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t ev_entry = nullptr, ev_in[2] = {nullptr, nullptr}, ev_done[2] = {nullptr, nullptr},
                ev_out[2] = {nullptr, nullptr};
    unsigned long long* trace = nullptr;  // device buffer for the attention kernel's event trace (caller-owned)
    int32_t trace_cap = 0;
    // page-locked host copies of the descriptor table of launches over more than kMaxInline layer-calls; two, used
    // in turn, each guarded by an event that says its upload has finished (created on first use)
    AttnItem* host_tab[2] = {nullptr, nullptr};
    cudaEvent_t tab_ev[2] = {nullptr, nullptr};
    int tab_turn = 0;
    uint32_t launch_seq = 0;        // numbers the attention launches; tags the error codes a launch records
    int32_t fail_launch_in = 0;     // test hook: the n-th launch site from now reports a failure without launching
    int64_t prof_publish_launches = 0, prof_attn_launches = 0;
    int64_t n_attn_single = 0, n_attn_pair = 0;   // attention launches by tensor-core kernel

    SlotMeta& slot(int stage, int layer, int s) {
        return slots[((size_t)stage * cfg.n_layers + layer) * D.R + s];
    }
    const SlotMeta& slot(int stage, int layer, int s) const {
        return slots[((size_t)stage * cfg.n_layers + layer) * D.R + s];
    }
    // first row (head 0, token 0) of a bank slot / an anchor slot, and the row stride between heads
    int64_t ring_row0(int stage, int layer, int s) const {
        return (((int64_t)stage * cfg.n_layers + layer) * cfg.n_heads * D.R + s) * D.cap_pad;
    }
    int32_t ring_head_stride() const { return D.R * D.cap_pad; }
    int64_t anchor_row0(int s, int layer) const {
        return D.ring_rows + ((int64_t)s * cfg.n_layers + layer) * cfg.n_heads * D.tf_pad;
    }
    int32_t anchor_head_stride() const { return D.tf_pad; }
    RopeTables tables() const {
        RopeTables t;
        t.frame = reinterpret_cast<const float2*>(arena + D.off_tab_f);
        t.row = reinterpret_cast<const float2*>(arena + D.off_tab_y);
        t.col = reinterpret_cast<const float2*>(arena + D.off_tab_x);
        t.pairs_f = D.pairs[0]; t.pairs_h = D.pairs[1]; t.pairs_w = D.pairs[2];
        return t;
    }
    const float* gain(int layer, int which) const {
        return reinterpret_cast<const float*>(arena + D.off_gain) + ((size_t)layer * 2 + which) * D.d;
    }
    uint32_t* status() const { return reinterpret_cast<uint32_t*>(arena + D.off_status); }
    // A launch site: true if the launch may proceed; false when the test hook turns it into a reported failure.
    bool launch_allowed() {
        if (fail_launch_in > 0 && --fail_launch_in == 0) {
            g_last_cuda_error = static_cast<int32_t>(cudaErrorLaunchFailure);
            return false;
        }
        return true;
    }
};

namespace {

void reset_meta(ff_cache* c) {
    std::fill(c->head.begin(), c->head.end(), 0);
    std::fill(c->count.begin(), c->count.end(), 0);
    std::fill(c->next_chunk.begin(), c->next_chunk.end(), 0);
    std::fill(c->slots.begin(), c->slots.end(), SlotMeta());
    std::fill(c->anchor_pos.begin(), c->anchor_pos.end(), -1);
    std::fill(c->anchor_valid.begin(), c->anchor_valid.end(), 0);
    c->n_layer_calls = c->n_advances = c->n_anchor_publishes = c->n_launches = 0;
    c->n_attn_single = c->n_attn_pair = 0;
}

// Rotary tables: angle = pos * theta^(-j/n) in double, cos and sin in double, each rounded once to float.
void fill_table(std::vector<float2>& tab, int n_pos, int n_pairs, double theta) {
    tab.resize((size_t)n_pos * n_pairs);
    for (int p = 0; p < n_pos; ++p)
        for (int j = 0; j < n_pairs; ++j) {
            const double freq = std::pow(theta, -(double)j / (double)n_pairs);
            const double ang = (double)p * freq;
            tab[(size_t)p * n_pairs + j] = make_float2((float)std::cos(ang), (float)std::sin(ang));
        }
}

bool make_map(EncodeTiledFn enc, CUtensorMap* m, void* base, int64_t rows, int d, int box_rows = kTile) {
    cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)d * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    cuuint32_t es[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" {

int32_t ff_plan_anchor_count(int32_t L, int32_t delta) {
    if (L < 1 || delta < 1) return 0;
    const int32_t regular = (L - 1) / delta + 1;          // m * delta < L
    return (L - 1) % delta == 0 ? regular : regular + 1;  // plus L-1 when it is not a multiple of delta
}

int32_t ff_plan_anchor_position(int32_t L, int32_t delta, int32_t m) {
    const int32_t M = ff_plan_anchor_count(L, delta);
    if (m < 0 || m >= M) return -1;
    const int32_t pos = m * delta;
    return pos < L ? pos : L - 1;
}

int32_t ff_plan_window(int32_t i, int32_t L, int32_t B_R, int32_t delta, int32_t out[3]) {
    if (i < 0 || L < 1 || B_R < 1 || delta < 1 || !out) return 0;
    const int32_t M = ff_plan_anchor_count(L, delta);
    const int32_t u = (int32_t)(((int64_t)B_R * i) / (2 * (int64_t)delta));
    int32_t n = 0;
    for (int32_t k = 0; k < 3; ++k) {
        int32_t m = 2 * u + k;
        if (m > M - 1) m = M - 1;  // beyond the clip: the last anchor (position L-1) stands in
        bool seen = false;
        for (int32_t q = 0; q < n; ++q) seen = seen || out[q] == m;
        if (!seen) out[n++] = m;
    }
    return n;
}

const char* ff_version(void) { return "ff-chunk-attn 0.1 (sm_100a)"; }
int32_t ff_last_cuda_error(void) { return g_last_cuda_error; }

ff_status ff_cache_query_bytes(const ff_cache_config* cfg, size_t* arena_bytes) {
    if (!arena_bytes) return FF_ERR_INVALID_ARG;
    Derived D;
    ff_status st = derive(cfg, &D);
    if (st != FF_OK) return st;
    *arena_bytes = D.total;
    return FF_OK;
}

ff_status ff_cache_create(const ff_cache_config* cfg, void* arena, size_t arena_bytes, ff_cache** out) {
    if (!out) return FF_ERR_INVALID_ARG;
    *out = nullptr;
    Derived D;
    ff_status st = derive(cfg, &D);
    if (st != FF_OK) return st;
    const bool dry = cfg->device == FF_DEVICE_NONE;
    int major = 0, sms = 148;
    if (!dry) {
        if (!arena || (reinterpret_cast<uintptr_t>(arena) & 255u)) return FF_ERR_INVALID_ARG;
        if (arena_bytes < D.total) return FF_ERR_OOM;
        if (!cuda_ok(cudaSetDevice(cfg->device))) return FF_ERR_CUDA;
        if (!cuda_ok(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, cfg->device))) return FF_ERR_CUDA;
        if (!cuda_ok(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, cfg->device))) return FF_ERR_CUDA;
        if (major != 10) return FF_ERR_UNSUPPORTED;  // the kernels are built for sm_100a only
    }

    ff_cache* c = new (std::nothrow) ff_cache();
    if (!c) return FF_ERR_OOM;
    c->cfg = *cfg;
    c->D = D;
    c->arena = static_cast<uint8_t*>(arena);
    c->sm_count = sms;
    c->dry = dry;
    c->head.assign(cfg->n_stages, 0);
    c->count.assign(cfg->n_stages, 0);
    c->next_chunk.assign(cfg->n_stages, 0);
    c->slots.assign((size_t)cfg->n_stages * cfg->n_layers * D.R, SlotMeta());
    c->anchor_pos.assign(cfg->n_anchor_slots, -1);
    c->anchor_valid.assign((size_t)cfg->n_anchor_slots * cfg->n_layers, 0);
    if (dry) {
        *out = c;
        return FF_OK;
    }

    std::vector<float2> tab;
    const size_t offs[3] = {D.off_tab_f, D.off_tab_y, D.off_tab_x};
    const int n_pos[3] = {cfg->max_frame_pos, cfg->grid_h, cfg->grid_w};
    for (int ax = 0; ax < 3; ++ax) {
        if (D.pairs[ax] == 0) continue;
        fill_table(tab, n_pos[ax], D.pairs[ax], (double)cfg->rope_theta);
        if (!cuda_ok(cudaMemcpy(c->arena + offs[ax], tab.data(), tab.size() * sizeof(float2), cudaMemcpyHostToDevice))) {
            delete c;
            return FF_ERR_CUDA;
        }
    }
    if (!cuda_ok(cudaMemset(c->arena + D.off_status, 0, 256))) { delete c; return FF_ERR_CUDA; }
    if (cfg->qk_norm) {
        const std::vector<float> ones((size_t)cfg->n_layers * 2 * D.d, 1.0f);
        if (!cuda_ok(cudaMemcpy(c->arena + D.off_gain, ones.data(), ones.size() * sizeof(float), cudaMemcpyHostToDevice))) {
            delete c;
            return FF_ERR_CUDA;
        }
    }

    if (D.impl == FF_ATTN_TCGEN05) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (!cuda_ok(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres)) || !fn) {
            delete c;
            return FF_ERR_CUDA;
        }
        EncodeTiledFn enc = reinterpret_cast<EncodeTiledFn>(fn);
        if (!make_map(enc, &c->tm_k, c->arena + D.off_k, D.total_rows, D.d) ||
            !make_map(enc, &c->tm_v, c->arena + D.off_v, D.total_rows, D.d) ||
            !make_map(enc, &c->tm_q, c->arena + D.off_q, (int64_t)D.q_slots * cfg->n_heads * D.cap_pad, D.d)) {
            delete c;
            return FF_ERR_CUDA;
        }
        if (!cuda_ok(attn_tcgen05_prepare(D.d))) { delete c; return FF_ERR_CUDA; }
        if (D.pair_mode != 0) {
            int pairs = 0;
            if (!make_map(enc, &c->tm_k32, c->arena + D.off_k, D.total_rows, D.d, 32) || !cuda_ok(attn_pair_prepare(&pairs))) {
                delete c;
                return FF_ERR_CUDA;
            }
            c->pair_slots = pairs < kMaxCtas / 2 ? pairs : kMaxCtas / 2;
            if (c->pair_slots < 1) {
                if (D.pair_mode == 1) { delete c; return FF_ERR_UNSUPPORTED; }
                c->D.pair_mode = 0;
            }
        }
    }
    *out = c;
    return FF_OK;
}

ff_status ff_cache_destroy(ff_cache* c) {
    if (c) {
        for (cudaEvent_t e : c->prof_events) cudaEventDestroy(e);
        if (c->s_in) cudaStreamDestroy(c->s_in);
        if (c->s_out) cudaStreamDestroy(c->s_out);
        if (c->ev_entry) cudaEventDestroy(c->ev_entry);
        for (int i = 0; i < 2; ++i) {
            if (c->host_tab[i]) cudaFreeHost(c->host_tab[i]);
            if (c->tab_ev[i]) cudaEventDestroy(c->tab_ev[i]);
            if (c->ev_in[i]) cudaEventDestroy(c->ev_in[i]);
            if (c->ev_done[i]) cudaEventDestroy(c->ev_done[i]);
            if (c->ev_out[i]) cudaEventDestroy(c->ev_out[i]);
        }
        delete c;
    }
    return FF_OK;
}

ff_status ff_cache_profile_begin(ff_cache* c, int32_t max_calls) {
    if (!c || max_calls < 1 || max_calls > (1 << 20)) return FF_ERR_INVALID_ARG;
    if (c->dry) return FF_ERR_UNSUPPORTED;
    if (c->profiling) return FF_ERR_STATE;
    c->prof_events.resize((size_t)max_calls * 3);
    for (size_t i = 0; i < c->prof_events.size(); ++i) {
        if (!cuda_ok(cudaEventCreate(&c->prof_events[i]))) {
            for (size_t j = 0; j < i; ++j) cudaEventDestroy(c->prof_events[j]);
            c->prof_events.clear();
            return FF_ERR_CUDA;
        }
    }
    c->prof_used = 0;
    c->prof_publish_launches = c->prof_attn_launches = 0;
    c->profiling = true;
    return FF_OK;
}

ff_status ff_cache_profile_end(ff_cache* c, void* stream, double* publish_ms, int64_t* publish_launches,
                               double* attn_ms, int64_t* attn_launches) {
    if (!c) return FF_ERR_INVALID_ARG;
    if (!c->profiling) return FF_ERR_STATE;
    c->profiling = false;
    ff_status r = FF_OK;
    if (!cuda_ok(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)))) r = FF_ERR_CUDA;
    double pm = 0.0, am = 0.0;
    for (size_t i = 0; r == FF_OK && i + 3 <= c->prof_used; i += 3) {
        float a = 0.f, b = 0.f;
        if (!cuda_ok(cudaEventElapsedTime(&a, c->prof_events[i], c->prof_events[i + 1])) ||
            !cuda_ok(cudaEventElapsedTime(&b, c->prof_events[i + 1], c->prof_events[i + 2]))) {
            r = FF_ERR_CUDA;
            break;
        }
        pm += a;
        am += b;
    }
    for (cudaEvent_t e : c->prof_events) cudaEventDestroy(e);
    c->prof_events.clear();
    c->prof_used = 0;
    if (publish_ms) *publish_ms = pm;
    if (attn_ms) *attn_ms = am;
    if (publish_launches) *publish_launches = c->prof_publish_launches;
    if (attn_launches) *attn_launches = c->prof_attn_launches;
    return r;
}

ff_status ff_cache_set_qk_gain(ff_cache* c, int32_t layer, const float* gain_q, const float* gain_k, void* stream) {
    if (!c || layer < 0 || layer >= c->cfg.n_layers || (!gain_q && !gain_k)) return FF_ERR_INVALID_ARG;
    if (!c->cfg.qk_norm) return FF_ERR_STATE;
    if (c->dry) return FF_OK;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t bytes = (size_t)c->D.d * sizeof(float);
    if (gain_q && !cuda_ok(cudaMemcpyAsync(const_cast<float*>(c->gain(layer, 0)), gain_q, bytes, cudaMemcpyHostToDevice, s)))
        return FF_ERR_CUDA;
    if (gain_k && !cuda_ok(cudaMemcpyAsync(const_cast<float*>(c->gain(layer, 1)), gain_k, bytes, cudaMemcpyHostToDevice, s)))
        return FF_ERR_CUDA;
    return FF_OK;
}

ff_status ff_cache_reset(ff_cache* c) {
    if (!c) return FF_ERR_INVALID_ARG;
    reset_meta(c);
    return FF_OK;
}

ff_status ff_anchor_publish(ff_cache* c, int32_t slot, int32_t frame_pos, int32_t layer, const void* k,
                            const void* v, void* stream) {
    if (!c || !k || !v || slot < 0 || slot >= c->cfg.n_anchor_slots || layer < 0 || layer >= c->cfg.n_layers ||
        frame_pos < 0 || frame_pos >= c->cfg.max_frame_pos || !aligned16(k) || !aligned16(v))
        return FF_ERR_INVALID_ARG;
    PublishArgs a{};
    a.q = nullptr; a.k = k; a.v = v; a.q_rot = nullptr;
    a.kmat = c->arena + c->D.off_k; a.vmat = c->arena + c->D.off_v;
    a.dst_row0 = c->anchor_row0(slot, layer);
    a.dst_head_stride = c->anchor_head_stride();
    a.q_rows_per_head = c->D.cap_pad;
    a.n_tok = c->D.tf; a.n_tok_pad = c->D.tf_pad;
    a.n_heads = c->cfg.n_heads; a.head_dim = c->D.d;
    a.grid_h = c->cfg.grid_h; a.grid_w = c->cfg.grid_w; a.first_frame_pos = frame_pos;
    a.frame_pos_stride = 1;
    a.qk_norm = c->cfg.qk_norm; a.qk_norm_eps = c->cfg.qk_norm_eps;
    a.gain_q = c->gain(layer, 0); a.gain_k = c->gain(layer, 1);
    a.tab = c->tables();
    if (!c->launch_allowed()) return FF_ERR_CUDA;
    if (!c->dry) {
        if (!cuda_ok(launch_rope_publish(a, c->cfg.dtype, c->sm_count, static_cast<cudaStream_t>(stream))))
            return FF_ERR_CUDA;
        ++c->n_launches;
    }
    if (c->anchor_pos[slot] != frame_pos) {
        std::fill(c->anchor_valid.begin() + (size_t)slot * c->cfg.n_layers,
                  c->anchor_valid.begin() + (size_t)(slot + 1) * c->cfg.n_layers, 0);
        c->anchor_pos[slot] = frame_pos;
    }
    c->anchor_valid[(size_t)slot * c->cfg.n_layers + layer] = 1;
    ++c->n_anchor_publishes;
    return FF_OK;
}

namespace {

struct CallDesc {
    int32_t stage, chunk_index, n_frames, first_frame_pos;
    const void *q, *k, *v;
    void* out;
    const int32_t* anchor_slots;
    int32_t n_anchors;
};

// Everything ff_chunk_forward_attn refuses, checked without touching the cache's state.  `pos` = how many
// earlier calls of the same batch belong to the same stage: they must be the chunks just before this one.
ff_status validate_call(const ff_cache* c, int32_t layer, const CallDesc& d, int32_t pos) {
    if (!d.q || !d.k || !d.v || !d.out) return FF_ERR_INVALID_ARG;
    const ff_cache_config& cfg = c->cfg;
    const int fstride = cfg.frame_pos_stride > 1 ? cfg.frame_pos_stride : 1;
    if (d.stage < 0 || d.stage >= cfg.n_stages || layer < 0 || layer >= cfg.n_layers || d.chunk_index < 0 ||
        d.n_frames < 1 || d.n_frames > cfg.chunk_frames || d.first_frame_pos < 0 ||
        d.first_frame_pos + (d.n_frames - 1) * fstride >= cfg.max_frame_pos || d.n_anchors < 0 ||
        d.n_anchors > cfg.max_visible_anchors || (d.n_anchors > 0 && !d.anchor_slots))
        return FF_ERR_INVALID_ARG;
    if (!aligned16(d.q) || !aligned16(d.k) || !aligned16(d.v) || !aligned16(d.out)) return FF_ERR_INVALID_ARG;
    for (int i = 0; i < d.n_anchors; ++i) {
        const int s = d.anchor_slots[i];
        if (s < 0 || s >= cfg.n_anchor_slots) return FF_ERR_INVALID_ARG;
        if (c->anchor_pos[s] < 0 || !c->anchor_valid[(size_t)s * cfg.n_layers + layer]) return FF_ERR_STATE;
    }
    const int next = c->next_chunk[d.stage];
    if (d.chunk_index != next + pos) return FF_ERR_STATE;
    const int H = cfg.history_chunks, R = c->D.R;
    // the slot this chunk overwrites (it held chunk - R) must not be in the window of an earlier call of the batch
    if (pos > 0 && R < H + pos + 1) return FF_ERR_UNSUPPORTED;
    const int own = d.chunk_index % R;
    if (c->slot(d.stage, layer, own).chunk == d.chunk_index && !cfg.allow_republish) return FF_ERR_STATE;  // already ran
    const int first_hist = d.chunk_index - H < 0 ? 0 : d.chunk_index - H;
    for (int j = first_hist; j < d.chunk_index; ++j) {
        if (j >= next) continue;  // published by an earlier call of this batch
        if (c->slot(d.stage, layer, j % R).chunk != j) return FF_ERR_STATE;
    }
    return FF_OK;
}

// n layer-calls of one layer: every call's rotation + publish, then ONE attention launch over all of them.
// Calls of different stages are independent (each reads and writes its own stage's bank); calls of one stage
// must be consecutive chunks in order - a later chunk reads what the earlier ones publish in the same batch,
// which is complete before the attention launch starts - and the bank needs H + (their number) slots so that no
// publish overwrites a chunk an earlier call still reads.
// Nothing of the cache's state (slot table, counters, profile records) is touched before every launch of the
// batch has been accepted by the runtime: on any error status the cache is as it was.
ff_status forward_batch(ff_cache* c, int32_t layer, const CallDesc* d, int32_t n, cudaStream_t s) {
    if (!c || !d || n < 1) return FF_ERR_INVALID_ARG;
    if (n > c->D.q_slots || n > kMaxBatch) return FF_ERR_UNSUPPORTED;
    const ff_cache_config& cfg = c->cfg;
    for (int i = 0; i < n; ++i) {
        int pos = 0;
        for (int j = 0; j < i; ++j)
            if (d[j].stage == d[i].stage) ++pos;
        const ff_status r = validate_call(c, layer, d[i], pos);
        if (r != FF_OK) return r;
    }
    const int H = cfg.history_chunks, R = c->D.R;
    const bool table = n > kMaxInline;
    cudaEvent_t* ev = nullptr;
    if (!c->dry && c->profiling && c->prof_used + 3 <= c->prof_events.size()) ev = &c->prof_events[c->prof_used];

    AttnArgs a{};
    a.q_rot = c->arena + c->D.off_q; a.kmat = c->arena + c->D.off_k; a.vmat = c->arena + c->D.off_v;
    a.q_rows_per_head = c->D.cap_pad;
    a.n_heads = cfg.n_heads; a.head_dim = c->D.d;
    a.scale = 1.0f / std::sqrt((float)c->D.d);
    a.status = c->status();
    a.launch_tag = ((c->launch_seq + 1) & 0x7fffu) << 16;
    a.n_items = n;
    a.part_o = reinterpret_cast<float*>(c->arena + c->D.off_part_o);
    a.part_ml = reinterpret_cast<float2*>(c->arena + c->D.off_part_ml);
    a.trace = c->trace;
    a.trace_cap = c->trace_cap;

    // where the descriptors are written: inside the launch arguments, or (many calls) a page-locked host table that
    // is copied into the arena ahead of the attention launch
    std::vector<AttnItem> dry_items;
    AttnItem* items = a.items;
    const int turn = c->tab_turn;
    if (table) {
        if (c->dry) {
            dry_items.resize(n);
            items = dry_items.data();
        } else {
            for (int b = 0; b < 2; ++b) {
                if (!c->host_tab[b] &&
                    (!cuda_ok(cudaHostAlloc(reinterpret_cast<void**>(&c->host_tab[b]), kMaxBatch * sizeof(AttnItem), cudaHostAllocDefault)) ||
                     !cuda_ok(cudaEventCreateWithFlags(&c->tab_ev[b], cudaEventDisableTiming))))
                    return FF_ERR_CUDA;
            }
            if (!cuda_ok(cudaEventSynchronize(c->tab_ev[turn]))) return FF_ERR_CUDA;  // its previous upload is done
            items = c->host_tab[turn];
        }
    }

    // slots this batch publishes: visible to its later calls, recorded in the cache only at the end
    struct Pending { int32_t stage, slot, chunk, n_tokens; };
    Pending pend[kMaxBatch];
    auto tokens_in = [&](int upto, int stage, int sl) -> int32_t {
        for (int j = upto; j >= 0; --j)
            if (pend[j].stage == stage && pend[j].slot == sl) return pend[j].n_tokens;
        return c->slot(stage, layer, sl).n_tokens;
    };
    std::vector<PublishArgs> pubs(n);
    for (int i = 0; i < n; ++i) {
        const CallDesc& x = d[i];
        const int n_q = x.n_frames * c->D.tf;
        const int own = x.chunk_index % R;
        const int64_t q_row0 = (int64_t)i * cfg.n_heads * c->D.cap_pad;

        // steps 1-2: rotate Q and K, publish (K', V) in place into the stage's ring slot
        PublishArgs& p = pubs[i];
        p = PublishArgs{};
        p.q = x.q; p.k = x.k; p.v = x.v;
        p.q_rot = c->arena + c->D.off_q + (size_t)q_row0 * c->D.d * c->D.elem;
        p.kmat = c->arena + c->D.off_k; p.vmat = c->arena + c->D.off_v;
        p.dst_row0 = c->ring_row0(x.stage, layer, own);
        p.dst_head_stride = c->ring_head_stride();
        p.q_rows_per_head = c->D.cap_pad;
        p.n_tok = n_q; p.n_tok_pad = round_up_tile(n_q);
        p.n_heads = cfg.n_heads; p.head_dim = c->D.d;
        p.grid_h = cfg.grid_h; p.grid_w = cfg.grid_w; p.first_frame_pos = x.first_frame_pos;
        p.frame_pos_stride = cfg.frame_pos_stride > 1 ? cfg.frame_pos_stride : 1;
        p.qk_norm = cfg.qk_norm; p.qk_norm_eps = cfg.qk_norm_eps;
        p.gain_q = c->gain(layer, 0); p.gain_k = c->gain(layer, 1);
        p.tab = c->tables();
        pend[i] = Pending{x.stage, own, x.chunk_index, n_q};

        // steps 3-4: attention over [anchors | history | own], read where they lie
        AttnItem& it = items[i];
        it = AttnItem{};
        it.out = x.out;
        it.q_row0 = (int32_t)q_row0;
        it.n_q = n_q;
        int m = 0;
        for (int j = 0; j < x.n_anchors; ++j, ++m) {
            it.segs.row0[m] = (int32_t)c->anchor_row0(x.anchor_slots[j], layer);
            it.segs.head_stride[m] = c->anchor_head_stride();
            it.segs.tokens[m] = c->D.tf;
        }
        const int first_hist = x.chunk_index - H < 0 ? 0 : x.chunk_index - H;
        for (int j = first_hist; j <= x.chunk_index; ++j, ++m) {
            const int sl = j % R;
            it.segs.row0[m] = (int32_t)c->ring_row0(x.stage, layer, sl);
            it.segs.head_stride[m] = c->ring_head_stride();
            it.segs.tokens[m] = tokens_in(i, x.stage, sl);
        }
        it.segs.n = m;
    }
    const bool tc = c->D.impl == FF_ATTN_TCGEN05;
    // Which tensor-core kernel: the CTA-pair kernel moves half the K/V bytes per query row into shared memory and is
    // about 6 % faster per (unit, key tile) step, but its units are four query tiles where the other kernel's are
    // two, so a head whose tile count is 1 mod 4 leaves more of its last unit empty.  Chosen per launch from the
    // query-tile slots each kernel would spend (measured: 720p, 85 tiles per head, +5 %; 480p, 37 tiles, a tie).
    bool pair = tc && c->D.pair_mode == 1;
    if (tc && c->D.pair_mode == 2 && !c->trace) {
        long long slots_single = 0, slots_pair = 0;
        for (int i = 0; i < n; ++i) {
            const long long n_qt = (items[i].n_q + kTile - 1) / kTile;
            long long tiles = 0;
            for (int sg = 0; sg < items[i].segs.n; ++sg) tiles += (items[i].segs.tokens[sg] + kTile - 1) / kTile;
            slots_single += (n_qt + 1) / 2 * 2 * tiles;
            slots_pair += (n_qt + 3) / 4 * 4 * tiles;
        }
        pair = slots_pair * 100 <= slots_single * 104;
    }
    a.unit_pairs = pair ? 2 : 1;
    const int merge_pairs = !tc ? 0 : pair ? attn_tcgen05_plan(a, items, c->pair_slots > 0 ? c->pair_slots : 74)
                                           : attn_tcgen05_plan(a, items, c->sm_count < kMaxCtas ? c->sm_count : kMaxCtas);

    int64_t launched = 0, pub_launches = 0, attn_launches = 0;
    if (ev) cudaEventRecord(ev[0], s);
    // the publishes, kMaxInline per launch (the items write disjoint slots and query regions)
    for (int i0 = 0; i0 < n; i0 += kMaxInline) {
        PublishBatch pb{};
        pb.n = n - i0 < kMaxInline ? n - i0 : kMaxInline;
        for (int i = 0; i < pb.n; ++i) pb.items[i] = pubs[i0 + i];
        if (!c->launch_allowed()) return FF_ERR_CUDA;
        if (!c->dry && !cuda_ok(launch_rope_publish_batch(pb, cfg.dtype, c->sm_count, s))) return FF_ERR_CUDA;
        ++pub_launches;
    }
    if (ev) cudaEventRecord(ev[1], s);
    if (tc) {
        if (!c->launch_allowed()) return FF_ERR_CUDA;
        if (!c->dry) {
            if (table) {
                AttnItem* dev_tab = reinterpret_cast<AttnItem*>(c->arena + c->D.off_items);
                if (!cuda_ok(cudaMemcpyAsync(dev_tab, items, (size_t)n * sizeof(AttnItem), cudaMemcpyHostToDevice, s)) ||
                    !cuda_ok(cudaEventRecord(c->tab_ev[turn], s)))
                    return FF_ERR_CUDA;
                c->tab_turn ^= 1;
                a.items_tab = dev_tab;
            }
            int nl = 1;
            if (!cuda_ok(launch_attn_tcgen05(a, merge_pairs, c->tm_q, pair ? c->tm_k32 : c->tm_k, c->tm_v, s, &nl))) return FF_ERR_CUDA;
            attn_launches += nl;
        } else {
            attn_launches += merge_pairs ? 2 : 1;
        }
    } else {
        for (int i = 0; i < n; ++i) {
            if (!c->launch_allowed()) return FF_ERR_CUDA;
            if (!c->dry && !cuda_ok(launch_attn_simt(a, items[i], cfg.dtype, s))) return FF_ERR_CUDA;
            ++attn_launches;
        }
    }
    if (ev) cudaEventRecord(ev[2], s);
    launched = pub_launches + attn_launches;

    // every launch was accepted: now the cache records what they do
    for (int i = 0; i < n; ++i) {
        SlotMeta& m = c->slot(pend[i].stage, layer, pend[i].slot);
        m.chunk = pend[i].chunk;
        m.n_tokens = pend[i].n_tokens;
    }
    ++c->launch_seq;
    if (tc) ++(pair ? c->n_attn_pair : c->n_attn_single);
    if (ev) {
        c->prof_used += 3;
        c->prof_publish_launches += pub_launches;
        c->prof_attn_launches += attn_launches;
    }
    if (!c->dry) c->n_launches += launched;
    c->n_layer_calls += n;
    return FF_OK;
}

}  // namespace

ff_status ff_chunk_forward_attn(ff_cache* c, int32_t stage, int32_t layer, int32_t chunk_index, int32_t n_frames,
                                int32_t first_frame_pos, const void* q, const void* k, const void* v,
                                const int32_t* anchor_slots, int32_t n_anchors, void* out, void* stream) {
    if (!c) return FF_ERR_INVALID_ARG;
    const CallDesc d{stage, chunk_index, n_frames, first_frame_pos, q, k, v, out, anchor_slots, n_anchors};
    return forward_batch(c, layer, &d, 1, static_cast<cudaStream_t>(stream));
}

ff_status ff_batch_forward_attn(ff_cache* c, int32_t layer, const ff_batch_item* items, int32_t n_items, void* stream) {
    if (!c || !items || n_items < 1 || n_items > kMaxBatch) return FF_ERR_INVALID_ARG;
    CallDesc d[kMaxBatch];
    for (int i = 0; i < n_items; ++i)
        d[i] = CallDesc{items[i].stage, items[i].chunk_index, items[i].n_frames, items[i].first_frame_pos, items[i].q,
                        items[i].k, items[i].v, items[i].out, items[i].anchor_slots, items[i].n_anchors};
    return forward_batch(c, layer, d, n_items, static_cast<cudaStream_t>(stream));
}

ff_status ff_sched_run_round(ff_cache* c, const ff_round_node* nodes, int32_t n_nodes, void* stream) {
    if (!c || !nodes || n_nodes < 1 || n_nodes > kMaxBatch) return FF_ERR_INVALID_ARG;
    for (int i = 0; i < n_nodes; ++i)
        if (!nodes[i].io) return FF_ERR_INVALID_ARG;
    CallDesc d[kMaxBatch];
    for (int l = 0; l < c->cfg.n_layers; ++l) {
        for (int i = 0; i < n_nodes; ++i) {
            const ff_round_node& x = nodes[i];
            d[i] = CallDesc{x.stage, x.chunk_index, x.n_frames, x.first_frame_pos, x.io[l].q, x.io[l].k, x.io[l].v,
                            x.io[l].out, x.anchor_slots, x.n_anchors};
        }
        const ff_status r = forward_batch(c, l, d, n_nodes, static_cast<cudaStream_t>(stream));
        if (r != FF_OK) return r;
    }
    for (int i = 0; i < n_nodes; ++i) {
        const ff_status r = ff_cache_advance(c, nodes[i].stage);
        if (r != FF_OK) return r;
    }
    return FF_OK;
}

ff_status ff_cache_advance(ff_cache* c, int32_t stage) {
    if (!c || stage < 0 || stage >= c->cfg.n_stages) return FF_ERR_INVALID_ARG;
    const int H = c->cfg.history_chunks, R = c->D.R;
    const int i = c->next_chunk[stage];
    for (int l = 0; l < c->cfg.n_layers; ++l)
        if (c->slot(stage, l, i % R).chunk != i) return FF_ERR_STATE;
    c->head[stage] = (c->head[stage] + 1) % R;
    c->count[stage] = c->count[stage] + 1 > H ? H : c->count[stage] + 1;
    c->next_chunk[stage] = i + 1;
    ++c->n_advances;
    return FF_OK;
}

ff_status ff_chunk_forward_attn_host(ff_cache* c, int32_t stage, int32_t layer, int32_t chunk_index,
                                     int32_t n_frames, int32_t first_frame_pos, const void* q, const void* k,
                                     const void* v, const int32_t* anchor_slots, int32_t n_anchors, void* out,
                                     void* stream) {
    if (!c || !q || !k || !v || !out) return FF_ERR_INVALID_ARG;
    if (n_frames < 1 || n_frames > c->cfg.chunk_frames) return FF_ERR_INVALID_ARG;
    if (c->dry) return FF_ERR_UNSUPPORTED;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t bytes = (size_t)n_frames * c->D.tf * c->cfg.n_heads * c->D.d * c->D.elem;
    uint8_t* st = c->arena + c->D.off_stage;
    void *dq = st, *dk = st + c->D.stage_bytes, *dv = st + 2 * c->D.stage_bytes, *dout = st + 3 * c->D.stage_bytes;
    if (!cuda_ok(cudaMemcpyAsync(dq, q, bytes, cudaMemcpyHostToDevice, s))) return FF_ERR_CUDA;
    if (!cuda_ok(cudaMemcpyAsync(dk, k, bytes, cudaMemcpyHostToDevice, s))) return FF_ERR_CUDA;
    if (!cuda_ok(cudaMemcpyAsync(dv, v, bytes, cudaMemcpyHostToDevice, s))) return FF_ERR_CUDA;
    ff_status r = ff_chunk_forward_attn(c, stage, layer, chunk_index, n_frames, first_frame_pos, dq, dk, dv,
                                        anchor_slots, n_anchors, dout, stream);
    if (r != FF_OK) {
        cudaStreamSynchronize(s);
        return r;
    }
    if (!cuda_ok(cudaMemcpyAsync(out, dout, bytes, cudaMemcpyDeviceToHost, s))) return FF_ERR_CUDA;
    if (!cuda_ok(cudaStreamSynchronize(s))) return FF_ERR_CUDA;
    return FF_OK;
}

ff_status ff_sched_run_node(ff_cache* c, int32_t stage, int32_t chunk_index, int32_t n_frames,
                            int32_t first_frame_pos, const int32_t* anchor_slots, int32_t n_anchors,
                            const ff_layer_io* io, void* stream) {
    if (!c || !io) return FF_ERR_INVALID_ARG;
    for (int l = 0; l < c->cfg.n_layers; ++l) {
        ff_status r = ff_chunk_forward_attn(c, stage, l, chunk_index, n_frames, first_frame_pos, io[l].q, io[l].k,
                                            io[l].v, anchor_slots, n_anchors, io[l].out, stream);
        if (r != FF_OK) return r;
    }
    return ff_cache_advance(c, stage);
}

ff_status ff_sched_run_chunk(ff_cache* c, int32_t chunk_index, int32_t n_frames, int32_t first_frame_pos,
                             const int32_t* anchor_slots, int32_t n_anchors, const ff_layer_io* io, int32_t n_io,
                             void* stream) {
    if (!c || !io || n_io < 1) return FF_ERR_INVALID_ARG;
    // stages in denoising order k = S .. 1, i.e. bank index S-1 .. 0
    for (int stage = c->cfg.n_stages - 1; stage >= 0; --stage) {
        for (int l = 0; l < c->cfg.n_layers; ++l) {
            const ff_layer_io& x = io[((size_t)stage * c->cfg.n_layers + l) % n_io];
            ff_status r = ff_chunk_forward_attn(c, stage, l, chunk_index, n_frames, first_frame_pos, x.q, x.k, x.v,
                                                anchor_slots, n_anchors, x.out, stream);
            if (r != FF_OK) return r;
        }
        ff_status r = ff_cache_advance(c, stage);
        if (r != FF_OK) return r;
    }
    return FF_OK;
}

ff_status ff_sched_run_chunk_host(ff_cache* c, int32_t chunk_index, int32_t n_frames, int32_t first_frame_pos,
                                  const int32_t* anchor_slots, int32_t n_anchors, const ff_layer_io* io,
                                  int32_t n_io, void* stream) {
    if (!c || !io || n_io < 1 || n_frames < 1 || n_frames > c->cfg.chunk_frames) return FF_ERR_INVALID_ARG;
    if (c->dry) return FF_ERR_UNSUPPORTED;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // Three-stage pipeline over the layer-calls: copy-in of call n+1 and copy-out of call n-1 run on their own
    // streams while call n computes; two staging sets alternate.
    if (!c->s_in) {
        bool ok = cuda_ok(cudaStreamCreateWithFlags(&c->s_in, cudaStreamNonBlocking)) &&
                  cuda_ok(cudaStreamCreateWithFlags(&c->s_out, cudaStreamNonBlocking)) &&
                  cuda_ok(cudaEventCreateWithFlags(&c->ev_entry, cudaEventDisableTiming));
        for (int i = 0; ok && i < 2; ++i)
            ok = cuda_ok(cudaEventCreateWithFlags(&c->ev_in[i], cudaEventDisableTiming)) &&
                 cuda_ok(cudaEventCreateWithFlags(&c->ev_done[i], cudaEventDisableTiming)) &&
                 cuda_ok(cudaEventCreateWithFlags(&c->ev_out[i], cudaEventDisableTiming));
        if (!ok) return FF_ERR_CUDA;
    }
    const size_t bytes = (size_t)n_frames * c->D.tf * c->cfg.n_heads * c->D.d * c->D.elem;
    uint8_t* st = c->arena + c->D.off_stage;
    // work already on `stream` may still use the staging sets: the copy streams start after it
    if (!cuda_ok(cudaEventRecord(c->ev_entry, s)) || !cuda_ok(cudaStreamWaitEvent(c->s_in, c->ev_entry, 0)) ||
        !cuda_ok(cudaStreamWaitEvent(c->s_out, c->ev_entry, 0)))
        return FF_ERR_CUDA;
    ff_status result = FF_OK;
    int n = 0;
    for (int stage = c->cfg.n_stages - 1; stage >= 0 && result == FF_OK; --stage) {
        for (int l = 0; l < c->cfg.n_layers && result == FF_OK; ++l, ++n) {
            const ff_layer_io& x = io[((size_t)stage * c->cfg.n_layers + l) % n_io];
            const int b = n & 1;
            uint8_t* set = st + (size_t)4 * b * c->D.stage_bytes;
            void *dq = set, *dk = set + c->D.stage_bytes, *dv = set + 2 * c->D.stage_bytes,
                 *dout = set + 3 * c->D.stage_bytes;
            bool ok = true;
            if (n >= 2) ok = cuda_ok(cudaStreamWaitEvent(c->s_in, c->ev_done[b], 0));  // inputs of set b consumed
            ok = ok && cuda_ok(cudaMemcpyAsync(dq, x.q, bytes, cudaMemcpyHostToDevice, c->s_in)) &&
                 cuda_ok(cudaMemcpyAsync(dk, x.k, bytes, cudaMemcpyHostToDevice, c->s_in)) &&
                 cuda_ok(cudaMemcpyAsync(dv, x.v, bytes, cudaMemcpyHostToDevice, c->s_in)) &&
                 cuda_ok(cudaEventRecord(c->ev_in[b], c->s_in)) && cuda_ok(cudaStreamWaitEvent(s, c->ev_in[b], 0));
            if (ok && n >= 2) ok = cuda_ok(cudaStreamWaitEvent(s, c->ev_out[b], 0));  // output of set b copied out
            if (!ok) { result = FF_ERR_CUDA; break; }
            result = ff_chunk_forward_attn(c, stage, l, chunk_index, n_frames, first_frame_pos, dq, dk, dv,
                                           anchor_slots, n_anchors, dout, stream);
            if (result != FF_OK) break;
            ok = cuda_ok(cudaEventRecord(c->ev_done[b], s)) && cuda_ok(cudaStreamWaitEvent(c->s_out, c->ev_done[b], 0)) &&
                 cuda_ok(cudaMemcpyAsync(x.out, dout, bytes, cudaMemcpyDeviceToHost, c->s_out)) &&
                 cuda_ok(cudaEventRecord(c->ev_out[b], c->s_out));
            if (!ok) result = FF_ERR_CUDA;
        }
        if (result == FF_OK) result = ff_cache_advance(c, stage);
    }
    // drain: the caller's stream waits for the last copies, then the host waits for the stream
    cudaStreamSynchronize(c->s_in);
    cudaStreamSynchronize(c->s_out);
    if (!cuda_ok(cudaStreamSynchronize(s)) && result == FF_OK) result = FF_ERR_CUDA;
    return result;
}

ff_status ff_cache_ring_state(const ff_cache* c, int32_t stage, int32_t layer, int32_t* head, int32_t* count,
                              int32_t* next_chunk, int32_t* slot_chunk, int32_t* slot_tokens) {
    if (!c || stage < 0 || stage >= c->cfg.n_stages || layer < 0 || layer >= c->cfg.n_layers) return FF_ERR_INVALID_ARG;
    if (head) *head = c->head[stage];
    if (count) *count = c->count[stage];
    if (next_chunk) *next_chunk = c->next_chunk[stage];
    for (int s = 0; s < c->D.R; ++s) {
        const SlotMeta& m = c->slot(stage, layer, s);
        if (slot_chunk) slot_chunk[s] = m.chunk;
        if (slot_tokens) slot_tokens[s] = m.chunk < 0 ? 0 : m.n_tokens;
    }
    return FF_OK;
}

ff_status ff_cache_anchor_state(const ff_cache* c, int32_t slot, int32_t* frame_pos, uint8_t* layer_valid) {
    if (!c || slot < 0 || slot >= c->cfg.n_anchor_slots) return FF_ERR_INVALID_ARG;
    if (frame_pos) *frame_pos = c->anchor_pos[slot];
    if (layer_valid) std::memcpy(layer_valid, &c->anchor_valid[(size_t)slot * c->cfg.n_layers], c->cfg.n_layers);
    return FF_OK;
}

ff_status ff_cache_slot_ptr(const ff_cache* c, int32_t kind, int32_t stage, int32_t layer, int32_t slot, void** k,
                            void** v, int64_t strides[3], int32_t* capacity_tokens) {
    if (!c || !k || !v || !strides || layer < 0 || layer >= c->cfg.n_layers) return FF_ERR_INVALID_ARG;
    int64_t row0;
    if (kind == 0) {
        if (stage < 0 || stage >= c->cfg.n_stages || slot < 0 || slot >= c->D.R) return FF_ERR_INVALID_ARG;
        row0 = c->ring_row0(stage, layer, slot);
        strides[1] = (int64_t)c->ring_head_stride() * c->D.d;
        if (capacity_tokens) *capacity_tokens = c->D.cap_pad;
    } else if (kind == 1) {
        if (slot < 0 || slot >= c->cfg.n_anchor_slots) return FF_ERR_INVALID_ARG;
        row0 = c->anchor_row0(slot, layer);
        strides[1] = (int64_t)c->anchor_head_stride() * c->D.d;
        if (capacity_tokens) *capacity_tokens = c->D.tf_pad;
    } else {
        return FF_ERR_INVALID_ARG;
    }
    strides[0] = c->D.d;
    strides[2] = 1;
    if (c->dry) return FF_ERR_UNSUPPORTED;
    *k = c->arena + c->D.off_k + (size_t)row0 * c->D.d * c->D.elem;
    *v = c->arena + c->D.off_v + (size_t)row0 * c->D.d * c->D.elem;
    return FF_OK;
}

ff_status ff_cache_status(ff_cache* c, void* stream, uint32_t* word) {
    if (!c) return FF_ERR_INVALID_ARG;
    if (c->dry) {
        if (word) *word = 0;
        return FF_OK;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint32_t w = 0;
    if (!cuda_ok(cudaStreamSynchronize(s))) return FF_ERR_CUDA;
    if (!cuda_ok(cudaMemcpy(&w, c->status(), sizeof(w), cudaMemcpyDeviceToHost))) return FF_ERR_CUDA;
    if (w != 0 && !cuda_ok(cudaMemset(c->status(), 0, sizeof(w)))) return FF_ERR_CUDA;
    if (word) *word = w & 0xffffu;  // the upper half says which launch recorded it
    return w == 0 ? FF_OK : FF_ERR_TIMEOUT;
}

ff_status ff_cache_counters(const ff_cache* c, int64_t* layer_calls, int64_t* advances, int64_t* anchor_publishes,
                            int64_t* kernel_launches) {
    if (!c) return FF_ERR_INVALID_ARG;
    if (layer_calls) *layer_calls = c->n_layer_calls;
    if (advances) *advances = c->n_advances;
    if (anchor_publishes) *anchor_publishes = c->n_anchor_publishes;
    if (kernel_launches) *kernel_launches = c->n_launches;
    return FF_OK;
}

ff_status ff_cache_kernel_choice(const ff_cache* c, int64_t* one_cta_launches, int64_t* cta_pair_launches) {
    if (!c) return FF_ERR_INVALID_ARG;
    if (one_cta_launches) *one_cta_launches = c->n_attn_single;
    if (cta_pair_launches) *cta_pair_launches = c->n_attn_pair;
    return FF_OK;
}

/* Test hook, host only: the work distribution the tensor-core kernel would use for a launch of n_items
 * layer-calls with n_q[i] query rows and n_kv[i] visible keys (taken as one segment each).  Writes up to cap
 * records of 8 int32 (cta, item, head, pair, first key tile, end key tile, scratch slot or -1, second tile
 * present) in the order each CTA walks them and returns the total number of records (which may exceed cap);
 * header[0..3] = CTAs, whole pairs per CTA, remainder pairs to merge (0 = none), iterations per CTA. */
int32_t ff_debug_schedule(int32_t n_heads, int32_t n_items, const int32_t* n_q, const int32_t* n_kv, int32_t n_ctas_max,
                          int32_t unit_pairs, int32_t* records, int32_t cap, int32_t header[4]) {
    if (unit_pairs != 1 && unit_pairs != 2) return -1;
    if (n_heads < 1 || n_items < 1 || n_items > kMaxBatch || !n_q || !n_kv || n_ctas_max < 1 || n_ctas_max > kMaxCtas ||
        cap < 0 || (cap > 0 && !records))
        return -1;
    AttnArgs a{};
    a.n_heads = n_heads;
    a.n_items = n_items;
    a.unit_pairs = unit_pairs;
    std::vector<AttnItem> tab(n_items > kMaxInline ? n_items : 0);
    AttnItem* items = n_items > kMaxInline ? tab.data() : a.items;
    for (int i = 0; i < n_items; ++i) {
        if (n_q[i] < 1 || n_kv[i] < 1) return -1;
        items[i] = AttnItem{};
        items[i].n_q = n_q[i];
        items[i].segs.n = 1;
        items[i].segs.tokens[0] = n_kv[i];
    }
    const int merge_pairs = attn_tcgen05_plan(a, items, n_ctas_max);
    if (header) { header[0] = a.n_ctas; header[1] = a.n_full; header[2] = merge_pairs; header[3] = a.iters_per_cta; }
    int32_t n = 0;
    auto walk = [&](auto pit) {
        for (int cta = 0; cta < a.n_ctas; ++cta) {
            pit.init(a, cta);
            Piece p;
            while (pit.next(a, p)) {
                if (n < cap) {
                    int32_t* r = records + (size_t)n * 8;
                    r[0] = cta; r[1] = p.item; r[2] = p.h; r[3] = p.pr; r[4] = p.j0; r[5] = p.j1; r[6] = p.slot; r[7] = p.two;
                }
                ++n;
            }
        }
    };
    if (n_items > kMaxInline) walk(PieceIter<true>()); else walk(PieceIter<false>());
    return n;
}

/* Profiling hook: the tensor-core attention kernel appends (event id << 48 | SM clock) records of CTA 0 to
 * buf, a caller-owned DEVICE buffer of 3 * cap 64-bit words (two softmax groups and the MMA issuer, cap records
 * each); buf = NULL switches tracing off. */
ff_status ff_debug_set_trace(ff_cache* c, void* buf, int32_t cap) {
    if (!c || cap < 0) return FF_ERR_INVALID_ARG;
    c->trace = static_cast<unsigned long long*>(buf);
    c->trace_cap = buf ? cap : 0;
    return FF_OK;
}

/* Test hook for the error path of a launch: the nth launch site from now (1 = the next one; publish, attention and
 * merge launches each count as one site, also on a bookkeeping-only cache) reports a failure on the host without
 * launching anything, and the call it belongs to returns FF_ERR_CUDA.  nth = 0 disarms the hook. */
ff_status ff_debug_fail_launch(ff_cache* c, int32_t nth) {
    if (!c || nth < 0) return FF_ERR_INVALID_ARG;
    c->fail_launch_in = nth;
    return FF_OK;
}

/* Test hook for the bounded-wait path: a one-thread kernel waits limit_ns on a barrier nothing arrives on and
 * then records an error in the status word, which ff_cache_status reports as FF_ERR_TIMEOUT. */
ff_status ff_debug_wait_probe(ff_cache* c, uint64_t limit_ns, void* stream) {
    if (!c || limit_ns == 0 || limit_ns > 1000000000ull) return FF_ERR_INVALID_ARG;
    if (c->dry) return FF_ERR_UNSUPPORTED;
    if (!cuda_ok(launch_wait_probe(c->status(), limit_ns, static_cast<cudaStream_t>(stream)))) return FF_ERR_CUDA;
    return FF_OK;
}

}  // extern "C"
