// ff_chunk_attn_static: one layer-call on a first chunk (no history, no anchors) that touches no allocator.
//
// Who needs this: callers that are handed device pointers for their inputs and outputs but may not create
// device memory themselves - a plug-in running inside a serving process whose memory pool belongs to the host
// framework, a real-time loop in which cudaMalloc's implicit synchronisation is not acceptable, or a process
// whose device memory has been fully handed out before this library is loaded.  The normal entry points need
// an arena from the caller; this one needs nothing beyond q, k, v and out.
//
// The scratch that ff_chunk_forward_attn keeps in the arena (rotated queries, the published K'/V slot and the
// rotary tables) lives here in a file-scope device array of FF_STATIC_SCRATCH_BYTES.  Every device that loads
// the library carries that array until the process exits.  All calls on a device share it: it still holds
// the previous call's data when the next call starts (the kernels rewrite every byte they later read,
// including the zero rows up to the tile boundary), and two calls whose GPU work overlaps - different
// streams, or different host threads - race on it.
#include <cmath>
#include <mutex>

#include "../../include/ff.h"
#include "ff_internal.h"

using namespace ffk;

namespace {

static __device__ __align__(256) unsigned char g_static_scratch[FF_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
unsigned char* g_scratch_addr[kMaxDevices] = {};  // device address of g_static_scratch, per device ordinal

inline size_t align256(size_t x) { return (x + 255) / 256 * 256; }

// The array's name is only a host-side handle here; the kernels need its device address, which differs per
// device.  Looked up once per device, with that device current.
ff_status scratch_address(int device, unsigned char** out) {
    if (device < 0 || device >= kMaxDevices) return FF_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[device]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return FF_ERR_CUDA;
        g_scratch_addr[device] = static_cast<unsigned char*>(p);
    }
    *out = g_scratch_addr[device];
    return FF_OK;
}

// Rotary tables written by the device itself, straight into the static array: (cos, sin) of pos * theta^(-j/n),
// angle and functions in double, each rounded once to float.  No host buffer and no copy are involved, so the
// call neither blocks the host nor leaves a host pointer behind in a captured stream.
struct TableJob {
    float2* dst;       // [n_pos][n_pairs]
    int first_pos, n_pos, n_pairs;
};
__global__ void static_tables_kernel(TableJob f, TableJob y, TableJob x, double theta) {
    const TableJob job = blockIdx.y == 0 ? f : (blockIdx.y == 1 ? y : x);
    const int n = job.n_pos * job.n_pairs;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
        const int p = i / job.n_pairs, j = i - p * job.n_pairs;
        const double freq = pow(theta, -(double)j / (double)job.n_pairs);
        const double ang = (double)(job.first_pos + p) * freq;
        job.dst[i] = make_float2((float)cos(ang), (float)sin(ang));
    }
}

}  // namespace

extern "C" ff_status ff_chunk_attn_static(int32_t n_heads, int32_t head_dim, int32_t grid_h, int32_t grid_w,
                                          int32_t n_frames, int32_t first_frame_pos, float rope_theta, int32_t dtype,
                                          const void* q, const void* k, const void* v, void* out, void* stream) {
    if (!q || !k || !v || !out || n_heads < 1 || grid_h < 1 || grid_w < 1 || n_frames < 1 || first_frame_pos < 0 ||
        !(rope_theta > 0.f) || (dtype != FF_BF16 && dtype != FF_F32))
        return FF_ERR_INVALID_ARG;
    if (head_dim != 64 && head_dim != 128) return FF_ERR_UNSUPPORTED;
    if (((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)out) & 15u) return FF_ERR_INVALID_ARG;
    const long long n_tok = (long long)n_frames * grid_h * grid_w;
    if (n_tok > (1 << 20)) return FF_ERR_OOM;
    const int n_tok_pad = (int)((n_tok + kTile - 1) / kTile * kTile);
    const int elem = dtype == FF_BF16 ? 2 : 4;
    const int side = head_dim / 6;
    const int pairs[3] = {head_dim / 2 - 2 * side, side, side};
    const int n_pos[3] = {n_frames, grid_h, grid_w};

    // carve the static array: rotary tables | rotated Q | K' slot | V slot
    size_t tab_elems = 0, tab_at[3];
    for (int ax = 0; ax < 3; ++ax) { tab_at[ax] = tab_elems; tab_elems += (size_t)n_pos[ax] * pairs[ax]; }
    const size_t mat_bytes = align256((size_t)n_tok_pad * n_heads * head_dim * elem);
    const size_t off_q = align256(tab_elems * sizeof(float2));
    const size_t off_k = off_q + mat_bytes, off_v = off_k + mat_bytes, need = off_v + mat_bytes;
    if (need > (size_t)FF_STATIC_SCRATCH_BYTES) return FF_ERR_OOM;  // the problem does not fit the fixed scratch

    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess) return FF_ERR_CUDA;
    unsigned char* base = nullptr;
    ff_status st = scratch_address(device, &base);
    if (st != FF_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    // rotary tables for exactly the positions of this call, evaluated on the device
    float2* t0 = reinterpret_cast<float2*>(base);
    const TableJob jf{t0 + tab_at[0], first_frame_pos, n_frames, pairs[0]}, jy{t0 + tab_at[1], 0, grid_h, pairs[1]},
        jx{t0 + tab_at[2], 0, grid_w, pairs[2]};
    static_tables_kernel<<<dim3(8, 3), 128, 0, s>>>(jf, jy, jx, (double)rope_theta);
    if (cudaGetLastError() != cudaSuccess) return FF_ERR_CUDA;

    PublishArgs p{};
    p.q = q; p.k = k; p.v = v;
    p.q_rot = base + off_q; p.kmat = base + off_k; p.vmat = base + off_v;
    p.dst_row0 = 0; p.dst_head_stride = n_tok_pad; p.q_rows_per_head = n_tok_pad;
    p.n_tok = (int)n_tok; p.n_tok_pad = n_tok_pad;
    p.n_heads = n_heads; p.head_dim = head_dim;
    p.grid_h = grid_h; p.grid_w = grid_w;
    p.first_frame_pos = 0;  // the frame table starts at this call's first frame
    p.frame_pos_stride = 1;
    p.qk_norm = 0; p.qk_norm_eps = 0.f; p.gain_q = nullptr; p.gain_k = nullptr;
    p.tab.frame = t0 + tab_at[0]; p.tab.row = t0 + tab_at[1]; p.tab.col = t0 + tab_at[2];
    p.tab.pairs_f = pairs[0]; p.tab.pairs_h = pairs[1]; p.tab.pairs_w = pairs[2];
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
    if (launch_rope_publish(p, dtype, sms, s) != cudaSuccess) return FF_ERR_CUDA;

    AttnArgs a{};
    a.q_rot = p.q_rot; a.kmat = p.kmat; a.vmat = p.vmat;
    a.q_rows_per_head = n_tok_pad;
    a.n_heads = n_heads; a.head_dim = head_dim;
    a.scale = 1.0f / std::sqrt((float)head_dim);
    a.status = nullptr;
    a.n_items = 1;
    AttnItem it{};
    it.out = out; it.q_row0 = 0; it.n_q = (int)n_tok;
    it.segs.n = 1;
    it.segs.row0[0] = 0; it.segs.head_stride[0] = n_tok_pad; it.segs.tokens[0] = (int)n_tok;
    if (launch_attn_simt(a, it, dtype, s) != cudaSuccess) return FF_ERR_CUDA;
    return FF_OK;
}
