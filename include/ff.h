/*
 * ff.h — C ABI of the FlashForward renderer chunk-attention library for NVIDIA B200 (sm_100a).
 *
 * One call of ff_chunk_forward_attn is the self-attention part of one renderer forward F^R (Eq. 2) at one
 * transformer layer: the chunk's queries attend to [ clean anchor KV A_Gamma(i) | the stage-matched history
 * bank B_k^(i) | the chunk's own keys ], and the same call leaves the chunk's own K/V in bank B_k for later
 * chunks (Alg. 1, Phase B: "Read", "Evaluate", "Write in place").  There is no cache-update-only pass.
 *
 * Conventions
 *  - Plain C types only.  Every pointer is documented as HOST or DEVICE.  The caller owns all device memory:
 *    it allocates one arena (size from ff_cache_query_bytes) and hands it to ff_cache_create; the library
 *    never allocates device memory.  Input and output tensors are borrowed for the duration of the work
 *    enqueued on `stream` (a cudaStream_t passed as void*; NULL = the legacy default stream).
 *  - Tensors are row-major [tokens, n_heads, head_dim]; a token index is (frame, row, column) with the column
 *    fastest: token = (frame * grid_h + row) * grid_w + column.
 *  - Calls are asynchronous and ordered by the stream.  Errors that the host can see (bad argument, call out
 *    of order, unpublished anchor, arena too small) are returned synchronously and enqueue nothing.  Errors
 *    only the device can see (a bounded wait that ran out) are recorded in a status word, read with
 *    ff_cache_status.  No call aborts, throws, or traps the GPU.
 *  - Not thread-safe per cache object; use one stream per cache at a time.
 */
#ifndef FF_H_
#define FF_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t ff_status;
enum {
    FF_OK = 0,
    FF_ERR_INVALID_ARG = 1,  /* null / misaligned pointer, index out of range, unsupported shape */
    FF_ERR_STATE = 2,        /* chunk or layer out of order, anchor slot not published for that layer */
    FF_ERR_OOM = 3,          /* arena smaller than ff_cache_query_bytes reports */
    FF_ERR_UNSUPPORTED = 4,  /* configuration the kernels do not cover */
    FF_ERR_CUDA = 5,         /* a CUDA runtime call failed (ff_last_cuda_error gives the code) */
    FF_ERR_TIMEOUT = 6       /* a device-side bounded wait expired (reported by ff_cache_status) */
};

enum { FF_BF16 = 0, FF_F32 = 1 };

/* Which attention kernel serves ff_chunk_forward_attn. */
enum {
    FF_ATTN_AUTO = 0,    /* a tensor-core kernel for FF_BF16 with head_dim 64 or 128 (with head_dim 128 the library
                            picks, per launch, between the two below), the CUDA-core kernel otherwise */
    FF_ATTN_TCGEN05 = 1, /* TMA + tcgen05/TMEM flash attention, one CTA per SM (FF_BF16 only) */
    FF_ATTN_SIMT = 2,    /* fp32 CUDA-core flash attention: FF_F32 caches, and an on-device cross-check */
    FF_ATTN_TCGEN05_PAIR = 3 /* the same attention on CTA pairs (tcgen05 cta_group::2: the two SMs of a TPC share
                            every K/V tile, each staging half of it); FF_BF16, head_dim 128 only */
};

typedef struct ff_cache ff_cache; /* opaque HOST object */

typedef struct {
    int32_t n_layers;            /* transformer layers sharing this cache                                  */
    int32_t n_heads, head_dim;   /* head_dim even; the tensor-core kernel needs 64 or 128                  */
    int32_t grid_h, grid_w;      /* latent-frame token grid; T_f = grid_h * grid_w tokens per frame        */
    int32_t chunk_frames;        /* B_R: latent frames per renderer chunk (Notation paragraph)             */
    int32_t n_stages;            /* S denoising stages, one history bank B_k each (Eq. 2)                  */
    int32_t history_chunks;      /* H: preceding chunks kept by Tail_H (Eq. 2)                             */
    int32_t n_anchor_slots;      /* capacity of the clean anchor bank A, in anchor frames                  */
    int32_t max_visible_anchors; /* upper bound on |Gamma(i)|                                              */
    int32_t dtype;               /* FF_BF16 or FF_F32: element type of Q/K/V/out and of the cache          */
    int32_t attn_impl;           /* FF_ATTN_*                                                              */
    int32_t max_frame_pos;       /* rotary table covers frame positions 0 .. max_frame_pos-1               */
    int32_t rope_pairs[3];       /* rotary pairs given to (frame, row, column); {0,0,0} = default split
                                    (head_dim/2 - 2*floor(head_dim/6), floor(head_dim/6), floor(head_dim/6)) */
    float rope_theta;            /* rotary base, e.g. 10000                                                */
    int32_t device;              /* CUDA device ordinal that owns the arena, or FF_DEVICE_NONE             */
    int32_t frame_pos_stride;    /* frame f of a chunk sits at first_frame_pos + f * stride; 0 or 1 = dense chunks
                                    (renderer); the planner's blocks of anchor latents use the anchor stride     */
    int32_t allow_republish;     /* nonzero: a layer may run again for the current chunk before ff_cache_advance,
                                    the later call overwriting the slot (planner: denoising forwards, then the
                                    clean-endpoint forward whose K/V stay in the bank; Alg. 1 Phase A)           */
    int32_t ring_slots;          /* slots per bank; 0 = H + 1 (a ring that holds exactly Tail_H and the chunk in
                                    flight).  More slots (>= H + 1) change nothing in what a chunk sees; they
                                    let several consecutive chunks of ONE stage share a batched launch, up to the
                                    full clip under the chunk-wise causal mask: n chunks need H + n slots.        */
    int32_t max_batch;           /* layer-calls per batched launch the arena has query regions for; 0 = min(S, 8);
                                    at most FF_MAX_BATCH (enough for every chunk of a 65 s clip in one launch)   */
    int32_t qk_norm;             /* nonzero: every (token, head) row of q and k is scaled by
                                    1/sqrt(mean(x^2) + qk_norm_eps) before the rotary embedding (the per-head
                                    normalisation that precedes this path in the backbone; fused into the same
                                    HBM pass).  0 = inputs arrive normalised.                                    */
    float qk_norm_eps;
} ff_cache_config;

/* device = FF_DEVICE_NONE builds a bookkeeping-only cache: arena may be NULL, every call validates its
 * arguments and updates the ring / anchor tables exactly as usual, but nothing is enqueued.  Meant for
 * planning a call sequence and for checking call order without a GPU; it computes nothing. */
enum { FF_DEVICE_NONE = -1 };

/* Bytes of DEVICE memory the caller must provide.  arena_bytes covers the banks, the anchor bank, the rotary
 * tables, the status word and the rotated-query scratch. */
ff_status ff_cache_query_bytes(const ff_cache_config* cfg /*HOST*/, size_t* arena_bytes /*HOST out*/);

/* Builds the host object over a caller-owned DEVICE arena (256-byte aligned, >= arena_bytes).  Uploads the
 * rotary tables and clears the status word with synchronous copies; leaves the banks' contents untouched
 * (they are never read before they are written).  Makes cfg->device current. */
ff_status ff_cache_create(const ff_cache_config* cfg /*HOST*/, void* arena /*DEVICE*/, size_t arena_bytes,
                          ff_cache** out /*HOST out*/);
ff_status ff_cache_destroy(ff_cache* c); /* frees host state only; the arena stays the caller's */
/* Channel gains of the fused q/k normalisation for one layer: gain_q, gain_k are HOST pointers to head_dim
 * floats each (either may be NULL = leave as is); every normalised element is multiplied by its channel's
 * gain before the rotation.  All gains are 1 after ff_cache_create.  The copy is enqueued on `stream` and the
 * host arrays may be reused when the call returns.  FF_ERR_STATE when the cache was created with qk_norm = 0.
 * (The normalisation belongs to the backbone the method is built on; the paper's own text does not spell it
 * out, so its form here - per (token, head) row, unit offset, per-channel gain - is this library's reading.) */
ff_status ff_cache_set_qk_gain(ff_cache* c, int32_t layer, const float* gain_q, const float* gain_k, void* stream);

ff_status ff_cache_reset(ff_cache* c);   /* all banks empty (B_k^(0) = {}), all anchor slots unpublished */

/* Planner side of Alg. 1 Phase A, last line: append one clean anchor frame's KV at one layer to bank A.
 * k, v: DEVICE, [T_f, n_heads, head_dim], K before the rotary embedding.  The library rotates K at frame
 * position frame_pos (which may lie ahead of the chunks that read it: the plan is two-sided) and copies V
 * bit for bit.  Publishing a slot with a new frame_pos recycles it: its other layers become unpublished.
 * Work already enqueued that reads the slot is protected by stream order only. */
ff_status ff_anchor_publish(ff_cache* c, int32_t slot, int32_t frame_pos, int32_t layer, const void* k /*DEVICE*/,
                            const void* v /*DEVICE*/, void* stream);

/* One renderer layer-call (Eq. 2; Alg. 1 Phase B "Read / Evaluate / Write in place"):
 *   Q' = rope(q), K' = rope(k) at positions (first_frame_pos + f, row, column);
 *   bank B_stage, slot chunk_index mod (H+1)  <-  (chunk_index, K' rounded to the cache dtype, v bit for bit);
 *   out = softmax(Q' K_vis^T / sqrt(head_dim)) V_vis over
 *         K_vis = [ anchor slots listed | chunks max(0, chunk_index-H) .. chunk_index-1 of B_stage | own ].
 * q, k, v: DEVICE, [n_frames*T_f, n_heads, head_dim], 16-byte aligned; out: DEVICE, same shape.
 * stage in [0, S): index of the bank (the paper's k-1).  chunk_index must equal the stage's next chunk
 * (ff_cache_ring_state); layers may be called in any order, each at most once per chunk.
 * n_frames in [1, chunk_frames] (the last chunk of a stream may be short).
 * anchor_slots: HOST array of n_anchors slot indices (Gamma(i) is the caller's choice), n_anchors may be 0. */
ff_status ff_chunk_forward_attn(ff_cache* c, int32_t stage, int32_t layer, int32_t chunk_index, int32_t n_frames,
                                int32_t first_frame_pos, const void* q /*DEVICE*/, const void* k /*DEVICE*/,
                                const void* v /*DEVICE*/, const int32_t* anchor_slots /*HOST*/, int32_t n_anchors,
                                void* out /*DEVICE*/, void* stream);

/* Tail_H of Eq. 2 for one stage, after the stage's layers have run for the current chunk: the oldest chunk
 * leaves the window and the stage expects the next chunk index.  Host metadata only; enqueues nothing.
 * FF_ERR_STATE if some layer has not appended the current chunk yet. */
ff_status ff_cache_advance(ff_cache* c, int32_t stage);

/* Same computation with HOST q/k/v/out: stages the inputs through device buffers inside the arena, runs the
 * layer-call and copies the result back, all on `stream`; returns after the stream work has completed.
 * Host buffers should be page-locked for full copy bandwidth. */
ff_status ff_chunk_forward_attn_host(ff_cache* c, int32_t stage, int32_t layer, int32_t chunk_index,
                                     int32_t n_frames, int32_t first_frame_pos, const void* q /*HOST*/,
                                     const void* k /*HOST*/, const void* v /*HOST*/,
                                     const int32_t* anchor_slots /*HOST*/, int32_t n_anchors, void* out /*HOST*/,
                                     void* stream);

/* Single-GPU scheduler (Alg. 1 Phase B collapsed onto one device): runs every stage of one chunk in order
 * k = S .. 1 (bank index S-1 .. 0), every layer of each stage, then Tail_H for that stage.
 * io: HOST array of n_io entries; the layer-call (stage, layer) uses entry ((stage*n_layers + layer) % n_io). */
typedef struct {
    const void* q; /* DEVICE */
    const void* k; /* DEVICE */
    const void* v; /* DEVICE */
    void* out;     /* DEVICE */
} ff_layer_io;
ff_status ff_sched_run_chunk(ff_cache* c, int32_t chunk_index, int32_t n_frames, int32_t first_frame_pos,
                             const int32_t* anchor_slots /*HOST*/, int32_t n_anchors,
                             const ff_layer_io* io /*HOST*/, int32_t n_io, void* stream);
/* ff_sched_run_chunk with HOST q/k/v/out in every io entry.  The layer-calls are pipelined: the inputs of
 * call n+1 are copied in and the result of call n-1 is copied out (on two internal copy streams, through two
 * staging sets inside the arena) while call n computes on `stream`.  Returns after everything has completed.
 * Host buffers should be page-locked; with pageable memory the copies serialize. */
ff_status ff_sched_run_chunk_host(ff_cache* c, int32_t chunk_index, int32_t n_frames, int32_t first_frame_pos,
                                  const int32_t* anchor_slots /*HOST*/, int32_t n_anchors,
                                  const ff_layer_io* io /*HOST array of HOST pointers*/, int32_t n_io, void* stream);
/* One node (chunk, stage) of the wavefront: all layers of that stage for that chunk, then Tail_H.  Nodes may
 * be issued in any order that respects Alg. 1's dependencies ((i,k) after (i,k+1) and (i-1,k)); the banks
 * are per stage, so chunk-major and wavefront orders give identical results. */
ff_status ff_sched_run_node(ff_cache* c, int32_t stage, int32_t chunk_index, int32_t n_frames,
                            int32_t first_frame_pos, const int32_t* anchor_slots /*HOST*/, int32_t n_anchors,
                            const ff_layer_io* io /*HOST, n_layers entries*/, void* stream);

/* ---- one wavefront round on one device (Alg. 1 Phase B: "for all r in parallel") ----
 *
 * In round n of the renderer wavefront, stage S-r works on chunk n-r for every r: up to S nodes (chunk, stage)
 * that do not depend on one another, because every stage reads and writes only its own bank.  The paper gives
 * each stage its own device; on one device the same independence lets the nodes of a round share launches:
 * per layer, the rotations and publishes of all nodes, then ONE attention launch whose work list spans all of
 * them.  Results are identical, element for element, to issuing the calls one by one. */
#define FF_MAX_BATCH 128
typedef struct {
    int32_t stage, chunk_index, n_frames, first_frame_pos;
    const void* q;   /* DEVICE, as in ff_chunk_forward_attn */
    const void* k;   /* DEVICE */
    const void* v;   /* DEVICE */
    void* out;       /* DEVICE */
    const int32_t* anchor_slots; /* HOST */
    int32_t n_anchors;
} ff_batch_item;
/* The layer-calls items[0..n_items) of ONE layer (n_items <= the cache's max_batch), with the semantics and the
 * checks of n_items ff_chunk_forward_attn calls issued in this order.  Items of different stages are independent.
 * Items of one stage must be consecutive chunks in order, starting at that stage's next chunk (the later ones
 * read what the earlier ones publish), and the bank must have H + (their number) slots (ring_slots): this is the
 * "full clip at once under a chunk-wise causal mask" form of Sec. 3: with ring_slots = H + N_R and max_batch = N_R
 * every chunk of a stage shares ONE attention launch per layer.  Up to 8 items travel as launch arguments; beyond
 * that the per-item descriptors are written to a page-locked host table (allocated by the library on first use:
 * host memory, not device memory) and copied into the arena ahead of the attention launch on `stream`.  All
 * items are checked before anything is enqueued, and the cache records the batch only after every launch has been
 * accepted: on an error status - FF_ERR_CUDA included - the cache's tables and counters are as they were (kernels
 * accepted before a failing launch may still run and write bank slots the tables do not list; such slots are
 * never read).  FF_ERR_UNSUPPORTED for more items than query regions or too few bank slots. */
ff_status ff_batch_forward_attn(ff_cache* c, int32_t layer, const ff_batch_item* items /*HOST*/, int32_t n_items,
                                void* stream);
typedef struct {
    int32_t stage, chunk_index, n_frames, first_frame_pos;
    const int32_t* anchor_slots; /* HOST */
    int32_t n_anchors;
    const ff_layer_io* io;       /* HOST array of n_layers entries of DEVICE pointers */
} ff_round_node;
/* One wavefront round: for every layer one batched call over all nodes, then Tail_H (ff_cache_advance) on every
 * node's stage, in the order given.  The caller lists the active nodes of the round (Alg. 1: i = n - r,
 * k = S - r, 0 <= i < N_R).  Nodes may also be consecutive chunks of one stage (see ff_batch_forward_attn): the
 * clip-at-once form; every node is advanced once. */
ff_status ff_sched_run_round(ff_cache* c, const ff_round_node* nodes /*HOST*/, int32_t n_nodes, void* stream);

/* ---- the step after the forward (Alg. 1, "Step"; rectified-flow parameterisation of Eq. 6) ---- */

/* out[i] = x[i] - (sigma_k - sigma_km1) * v[i] for i < n: the Euler update that moves a chunk's latent from noise
 * level sigma_k to sigma_{k-1} along the predicted velocity.  x, v, out are DEVICE pointers, 16-byte aligned,
 * n elements each, any shape (flat); x and out have dtype_x, v has dtype_v (FF_BF16 or FF_F32); out may equal x
 * (in place) but must not partially overlap it.  Arithmetic in float: the step size, the product and the
 * difference are each rounded once, then rounded to nearest-even when dtype_x is bf16.  Asynchronous on
 * `stream`.  n = 0 is a no-op.  FF_ERR_INVALID_ARG for null or misaligned pointers, n < 0, NaN levels. */
ff_status ff_euler_step(const void* x, const void* v, float sigma_k, float sigma_km1, int64_t n,
                        int32_t dtype_x, int32_t dtype_v, void* out, void* stream);
/* Noise level of stage k of S (HOST helper): sigma_k = shift*u / (1 + (shift-1)*u), u = k/S, so sigma_S = 1 and
 * sigma_0 = 0.  With S = 4 and shift = 5 the levels are 1, 15/16, 5/6, 5/8: within one step of a 1000-step
 * table of the four stage indices the paper lists for its student (appendix, student schedule); the exact
 * index rule is not given there, so this closed form is the library's reading. */
ff_status ff_plan_sigma(int32_t k, int32_t n_stages, double shift, double* sigma /*HOST*/);

/* ---- the paper's index sets (host-only helpers; Notation paragraph and Eq. 1) ---- */

/* Number of anchor latents M = |P| for a clip of L latents and anchor stride delta, P = {m*delta < L} U {L-1}. */
int32_t ff_plan_anchor_count(int32_t L, int32_t delta);
/* Timeline position of anchor m (0 <= m < M); -1 if out of range. */
int32_t ff_plan_anchor_position(int32_t L, int32_t delta, int32_t m);
/* Gamma(i) = {2u, 2u+1, 2u+2} * delta with u = floor(B_R * i / (2 * delta)): the anchor INDICES (into P) that renderer
 * chunk i reads.  At the end of a finite clip an index whose position would be >= L is replaced by the last
 * anchor and duplicates are dropped.  Writes up to 3 indices to out (HOST) and returns their number. */
int32_t ff_plan_window(int32_t i, int32_t L, int32_t B_R, int32_t delta, int32_t out[3]);

/* ---- observers (tests, debugging) ---- */

/* head = slot the next chunk will be written to; count = chunks currently in the history window (<= H);
 * slot_chunk / slot_tokens: HOST arrays of one entry per slot of the bank (H+1, or ring_slots if that was set)
 * for `layer` (-1 / 0 for an empty slot). */
ff_status ff_cache_ring_state(const ff_cache* c, int32_t stage, int32_t layer, int32_t* head, int32_t* count,
                              int32_t* next_chunk, int32_t* slot_chunk, int32_t* slot_tokens);
/* frame_pos = -1 if the slot was never published; layer_valid: HOST array of n_layers bytes. */
ff_status ff_cache_anchor_state(const ff_cache* c, int32_t slot, int32_t* frame_pos, uint8_t* layer_valid);
/* DEVICE addresses of a slot's K and V.  kind 0 = bank slot (stage, layer, slot), 1 = anchor slot (layer, slot).
 * Element (token t, head h, dim e) is at base + t*strides[0] + h*strides[1] + e*strides[2] (in elements).
 * capacity_tokens = rows the slot owns per head. */
ff_status ff_cache_slot_ptr(const ff_cache* c, int32_t kind, int32_t stage, int32_t layer, int32_t slot,
                            void** k /*DEVICE out*/, void** v /*DEVICE out*/, int64_t strides[3],
                            int32_t* capacity_tokens);
/* Synchronizes `stream` and returns the device status word (0 = no device-side error) in *word; the
 * function's own result is FF_ERR_TIMEOUT if a bounded wait expired.  Clears the word.
 * Every wait inside the kernels is bounded (2 s).  When one expires, the launch it belongs to records a code here,
 * its other waits give up as well, and the kernel runs to its end without the data it waited for: the outputs and
 * the bank slot of that layer-call are then UNDEFINED, and so is everything computed from them later.  The first
 * code recorded stays until this function collects it; launches enqueued after the failing one run normally (an
 * old code does not shorten their waits) but cannot record a second code.  Check the status at the points where
 * results leave the stream (end of a chunk, of a clip), and treat everything since the previous check as lost
 * when it is not FF_OK. */
ff_status ff_cache_status(ff_cache* c, void* stream, uint32_t* word /*HOST out*/);
/* Counters since creation/reset: layer-calls, Tail_H advances, anchor publishes, kernels launched. */
ff_status ff_cache_counters(const ff_cache* c, int64_t* layer_calls, int64_t* advances, int64_t* anchor_publishes,
                            int64_t* kernel_launches);
/* Attention launches since creation/reset by tensor-core kernel: the one-CTA-per-SM kernel and the kernel on CTA
 * pairs (see FF_ATTN_AUTO: with head_dim 128 the choice is made per launch). */
ff_status ff_cache_kernel_choice(const ff_cache* c, int64_t* one_cta_launches, int64_t* cta_pair_launches);
/* Per-kernel timing for roofline reports.  After ff_cache_profile_begin every layer-call records CUDA events
 * on its stream before the publish kernel, between the two kernels and after the attention kernel (at most
 * max_calls layer-calls are recorded; later ones run untimed; a batched call counts as one record, its publish
 * launches timed together and its attention + merge launches together).  ff_cache_profile_end synchronizes
 * `stream`, returns the summed durations in milliseconds with the number of kernel launches behind each sum
 * (publish_launches: publish kernels; attn_launches: attention kernels plus merge kernels), and releases the
 * events.  Events are host-side driver objects; no device memory is allocated.  The events sit
 * between the kernels, so the overlap of a kernel's set-up with its predecessor's tail is not in these times. */
ff_status ff_cache_profile_begin(ff_cache* c, int32_t max_calls);
ff_status ff_cache_profile_end(ff_cache* c, void* stream, double* publish_ms, int64_t* publish_launches,
                               double* attn_ms, int64_t* attn_launches);
/* Test hook, HOST only, no device work: enumerates the work distribution of the tensor-core attention kernel for
 * a launch of n_items layer-calls with n_q[i] query rows and n_kv[i] visible keys.  unit_pairs = 1: the kernel
 * with one CTA per SM (a work unit is one pair of query tiles, a schedule slot one CTA); 2: the kernel on CTA
 * pairs (a unit is two consecutive pairs, one per CTA of the pair; a slot is a CTA pair, n_ctas_max counts pairs).
 * records: cap x 8 int32 (slot, item, head, unit, first key tile, end key tile, scratch slot or -1, second query
 * tile present (one-pair units)); header: slots, whole units per slot, remainder units to merge, iterations per
 * slot.  Returns the number of pieces, or -1. */
int32_t ff_debug_schedule(int32_t n_heads, int32_t n_items, const int32_t* n_q, const int32_t* n_kv, int32_t n_ctas_max,
                          int32_t unit_pairs, int32_t* records, int32_t cap, int32_t header[4]);
/* Tracing hook: the tensor-core attention kernel appends (event id << 48 | SM clock) records of its first CTA
 * to buf, a caller-owned DEVICE buffer of 3 * cap 64-bit words (softmax group 0, softmax group 1, MMA issuer;
 * cap records each, later events are dropped).  buf = NULL switches tracing off.  Event ids: softmax 1 = waits
 * for scores, 2 = scores ready, 3 = scores in registers, 4 = probabilities issued, 5 = probabilities stored;
 * issuer 10+ = waits for probabilities, 20+ = got them, 30+ = products issued (+2*tile + half). */
ff_status ff_debug_set_trace(ff_cache* c, void* buf /*DEVICE*/, int32_t cap);
/* Failure-injection hook, HOST only: the nth launch site from now (1 = the next publish / attention / merge
 * launch of this cache; also counted on a bookkeeping-only cache) reports a failure without launching, so that
 * the call it belongs to returns FF_ERR_CUDA.  Shows that a refused launch leaves the cache's tables untouched.
 * nth = 0 disarms. */
ff_status ff_debug_fail_launch(ff_cache* c, int32_t nth);
/* Failure-detection hook: enqueues a one-thread kernel that waits limit_ns (<= 1e9) on a barrier nothing
 * will ever arrive on, gives up, and records an error in the status word, which the next ff_cache_status
 * reports as FF_ERR_TIMEOUT.  Shows that an expired device-side wait leaves the context usable. */
ff_status ff_debug_wait_probe(ff_cache* c, uint64_t limit_ns, void* stream);
/* (No counterpart in the paper: an addition for callers that cannot allocate device memory.)
 * One layer-call on a FIRST chunk - empty history bank, no anchors - with no cache object and no arena:
 *   out = softmax(rope(q) rope(k)^T / sqrt(head_dim)) v   over the chunk's own n_frames*grid_h*grid_w tokens,
 * the same arithmetic as ff_chunk_forward_attn with chunk_index 0 and n_anchors 0 on the CUDA-core kernel (the
 * rotary tables are evaluated by a small kernel on the device instead of on the host, so a table entry may
 * differ from the arena path's in its last float bit).
 * Meant for code that receives device buffers but may not create any: a plug-in inside a process whose device
 * memory pool belongs to the host framework, a latency-critical loop that cannot afford cudaMalloc's implicit
 * synchronisation, or a process whose device memory was fully handed out before this library was loaded.
 * The call allocates nothing (no cudaMalloc, no cudaFree, no allocating library routine, no host buffer) and
 * copies nothing between host and device: it enqueues three kernels and returns.  Its scratch - rotary
 * tables, rotated queries, the rotated-K / V slot - is a fixed device array of FF_STATIC_SCRATCH_BYTES that
 * every GPU using this library holds until the process exits.
 *  - q, k, v, out: DEVICE, [n_frames*grid_h*grid_w, n_heads, head_dim], 16-byte aligned, dtype FF_BF16 or FF_F32;
 *    head_dim 64 or 128.  Work is enqueued on `stream` of the CURRENT device and is asynchronous.
 *  - FF_ERR_OOM if the call needs more than FF_STATIC_SCRATCH_BYTES, i.e. unless
 *      3 * roundup128(tokens) * n_heads * head_dim * sizeof(element) + tables  <=  FF_STATIC_SCRATCH_BYTES.
 *  - The first call on each device looks up the array's device address (cudaGetSymbolAddress); make that first
 *    call before starting any stream capture.
 *  - All calls on a device share the array and it keeps the previous call's contents (every byte that is read
 *    is rewritten first).  Calls whose GPU work can overlap - different streams, several host threads - race
 *    on it: issue them on one stream, or order them yourself. */
#define FF_STATIC_SCRATCH_BYTES (8 * 1024 * 1024)
ff_status ff_chunk_attn_static(int32_t n_heads, int32_t head_dim, int32_t grid_h, int32_t grid_w, int32_t n_frames,
                               int32_t first_frame_pos, float rope_theta, int32_t dtype, const void* q /*DEVICE*/,
                               const void* k /*DEVICE*/, const void* v /*DEVICE*/, void* out /*DEVICE*/,
                               void* stream);
/* The cudaError_t of the last failing CUDA call on this thread (0 if none). */
int32_t ff_last_cuda_error(void);
const char* ff_version(void);

#ifdef __cplusplus
}
#endif
#endif /* FF_H_ */
