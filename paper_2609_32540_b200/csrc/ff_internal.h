// Internal declarations shared by the host code and the kernels of the chunk-attention library.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdint>

namespace ffk {

constexpr int kMaxSegs = 16;   // anchors + history chunks + own chunk visible to one call
constexpr int kTile = 128;     // query rows per CTA and keys per KV tile; slot capacities are multiples of it

// Device status codes (first error wins).
constexpr uint32_t kErrWaitQ = 0x101, kErrWaitK = 0x102, kErrWaitV = 0x103, kErrWaitS = 0x104,
                   kErrWaitP = 0x105, kErrWaitO = 0x106, kErrWaitKEmpty = 0x107, kErrWaitVEmpty = 0x108,
                   kErrProbe = 0x1FF;

// The cache keeps K and V as two row-major matrices [rows, head_dim]; a slot (bank slot or anchor slot) owns,
// for every head, a run of consecutive rows.  Row of (head h, token t) of a segment = row0 + h*head_stride + t.
struct KvSegs {
    int32_t n;
    int32_t row0[kMaxSegs];
    int32_t head_stride[kMaxSegs];
    int32_t tokens[kMaxSegs];
};

struct RopeTables {
    const float2* frame;  // [max_frame_pos][pairs_f]  (cos, sin)
    const float2* row;    // [grid_h][pairs_h]
    const float2* col;    // [grid_w][pairs_w]
    int32_t pairs_f, pairs_h, pairs_w;
};

struct PublishArgs {
    const void* q;       // [n_tok, Hd, d] or null (anchor publish)
    const void* k;
    const void* v;
    void* q_rot;         // [Hd][q_rows_per_head][d]
    void* kmat;          // cache K matrix base
    void* vmat;          // cache V matrix base
    int64_t dst_row0;    // first row of the slot (head 0, token 0)
    int32_t dst_head_stride;
    int32_t q_rows_per_head;
    int32_t n_tok;       // tokens to publish
    int32_t n_tok_pad;   // rows written per head: n_tok rounded up to the tile (zero-filled beyond n_tok)
    int32_t n_heads, head_dim;
    int32_t grid_h, grid_w, first_frame_pos;
    int32_t frame_pos_stride;  // frame f sits at first_frame_pos + f * frame_pos_stride
    int32_t qk_norm;           // nonzero: RMS-normalise every (token, head) row of q and k before the rotation
    float qk_norm_eps;
    const float* gain_q;       // [head_dim] channel gains applied after the normalisation (qk_norm only)
    const float* gain_k;
    RopeTables tab;
};

constexpr int kMaxInline = 8;   // layer-calls whose descriptors travel as kernel parameters
constexpr int kMaxBatch = 128;  // layer-calls one attention launch can serve; beyond kMaxInline the descriptors
                                // are read from a table in device memory (the whole clip of a stage in one launch)

// One layer-call inside an attention launch: its queries, its visible key segments, its output.
struct AttnItem {
    KvSegs segs;
    void* out;            // [n_q, Hd, d]
    int32_t q_row0;       // row of (head 0, token 0) of the item's rotated queries in the query matrix
    int32_t n_q;
    // schedule of the tensor-core kernel (filled by attn_tcgen05_plan)
    int32_t n_qt, n_qp;   // query tiles and query-tile pairs per head
    int32_t n_up;         // work units per head: a unit is one pair (single-CTA kernel) or two consecutive pairs (CTA-pair kernel)
    int32_t n_kv_tiles;   // key tiles over all visible segments
    int32_t pair0;        // index of the item's first pair in the launch-wide order (item, head, pair)
    int32_t rem_pair0;    // first pair of the item (item-local index) that lies in the cut remainder
    long long rem_iter0;  // where the item's remainder pairs start in the flattened (pair, key tile) list
};

// The publishes of one batched layer-call (one kernel launch; blockIdx.y selects the item).
struct PublishBatch {
    int32_t n;
    PublishArgs items[kMaxInline];
};

struct AttnArgs {
    const void* q_rot;   // query matrix: per item [Hd][q_rows_per_head][d]
    const void* kmat;
    const void* vmat;
    int32_t q_rows_per_head;
    int32_t n_heads, head_dim;
    float scale;         // 1/sqrt(d)
    uint32_t* status;
    uint32_t launch_tag;      // launch sequence number << 16: or-ed into every error code this launch records
    int32_t n_items;
    const AttnItem* items_tab;  // n_items > kMaxInline: the descriptors (device memory; host memory while planning)
    AttnItem items[kMaxInline]; // n_items <= kMaxInline: the descriptors themselves
    // schedule of the tensor-core kernel (filled by attn_tcgen05_plan)
    int32_t unit_pairs;       // pairs per work unit: 1 (single-CTA kernel) or 2 (CTA-pair kernel: one pair per CTA)
    int32_t n_pairs;          // work units over all items and heads (pairs, when unit_pairs == 1)
    int32_t n_full;           // whole pairs every CTA handles first (pair r * n_ctas + cta)
    int32_t iters_per_cta;    // share of the remaining pairs' (pair, key tile) iterations per CTA
    int32_t n_ctas;           // schedule slots: CTAs (single-CTA kernel) or CTA pairs
    long long total_iters;    // (pair, key tile) iterations of the remaining pairs
    float* part_o;            // [slot][2][128][d] unnormalised accumulators of split pairs
    float2* part_ml;          // [slot][2][128]    (reference maximum in log2 units, row sum)
    // optional event trace of CTA 0 (null = off): [role][trace_cap] entries of (event id << 48 | SM clock)
    unsigned long long* trace;
    int32_t trace_cap;
};

constexpr int kMaxCtas = 160;  // scratch for split pairs is sized for this many resident CTAs

// Launch that may overlap the tail of the kernel before it in the stream (programmatic dependent launch): the
// grid's blocks can be scheduled, and run their set-up, while that kernel is still draining.  A kernel launched
// this way must call grid_dependency_wait() before its first access to global memory; the call returns once the
// preceding kernel has completed and its writes are visible (at once if the launch was an ordinary one).
#ifdef __CUDACC__
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_overlapped(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                     Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// Launchers (defined in the .cu files).  Each returns the cudaError_t of the launch.
cudaError_t launch_rope_publish(const PublishArgs& a, int dtype, int sm_count, cudaStream_t s);
cudaError_t launch_rope_publish_batch(const PublishBatch& b, int dtype, int sm_count, cudaStream_t s);
cudaError_t launch_attn_simt(const AttnArgs& shared, const AttnItem& item, int dtype, cudaStream_t s);
// Fills the schedule fields of `a` and of the n_items descriptors in `items` (HOST memory: a.items itself, or the
// host copy of the table for more than kMaxInline items); returns the number of remainder pairs whose pieces need
// merging afterwards (0 = no merge launch).
int attn_tcgen05_plan(AttnArgs& a, AttnItem* items, int n_ctas_max);
// Launches a planned `a`; a.items_tab must be null (inline descriptors) or the DEVICE copy of the planned table.
cudaError_t launch_attn_tcgen05(const AttnArgs& a, int merge_pairs, const CUtensorMap& tm_q, const CUtensorMap& tm_k,
                                const CUtensorMap& tm_v, cudaStream_t s, int* n_launches);
cudaError_t attn_tcgen05_prepare(int head_dim);  // sets the dynamic shared-memory attribute once
// The kernel on CTA pairs (head_dim 128): prepare reports how many pairs can be resident at once; launch takes a
// planned `a` with unit_pairs == 2, n_ctas = CTA pairs, and the K map whose boxes hold 32 rows.
cudaError_t attn_pair_prepare(int* max_pairs);
cudaError_t launch_attn_pair(const AttnArgs& a, const CUtensorMap& tm_q, const CUtensorMap& tm_k32, const CUtensorMap& tm_v,
                             cudaStream_t s);
cudaError_t launch_wait_probe(uint32_t* status, unsigned long long limit_ns, cudaStream_t s);

}  // namespace ffk
