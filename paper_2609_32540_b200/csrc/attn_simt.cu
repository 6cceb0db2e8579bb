// fp32 CUDA-core flash attention over the visible cache segments.  Serves FF_F32 caches and acts as an
// on-device cross-check of the tensor-core kernel; it is not the fast path.
//
// A block owns 64 query rows of one head; 4 threads share a row, thread `sub` holding dims {4e + sub}.
// Keys and values are staged 32 at a time in shared memory as floats.  Online softmax, everything in fp32.
#include <cuda_bf16.h>
#include "ff_internal.h"

namespace ffk {

template <typename T>
__device__ __forceinline__ float to_f32(T x);
template <>
__device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T>
__device__ __forceinline__ T from_f32(float x);
template <>
__device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

template <typename T, int D>
__global__ void __launch_bounds__(256) attn_simt_kernel(const __grid_constant__ AttnArgs a) {
    const AttnItem& item = a.items[0];
    constexpr int kRows = 64, kKeys = 32, kDpt = D / 4;
    __shared__ float sK[kKeys][D];
    __shared__ float sV[kKeys][D];
    const int h = blockIdx.y;
    const int row = blockIdx.x * kRows + threadIdx.x / 4;
    const int sub = threadIdx.x % 4;
    const bool row_ok = row < item.n_q;
    const T* q_rot = reinterpret_cast<const T*>(a.q_rot);
    const T* kmat = reinterpret_cast<const T*>(a.kmat);
    const T* vmat = reinterpret_cast<const T*>(a.vmat);

    float q[kDpt], acc[kDpt];
#pragma unroll
    for (int e = 0; e < kDpt; ++e) {
        q[e] = row_ok ? to_f32<T>(q_rot[((size_t)item.q_row0 + (size_t)h * a.q_rows_per_head + row) * D + 4 * e + sub]) : 0.f;
        acc[e] = 0.f;
    }
    float m = -INFINITY, l = 0.f;

    for (int sgi = 0; sgi < item.segs.n; ++sgi) {
        const long long base = (long long)item.segs.row0[sgi] + (long long)h * item.segs.head_stride[sgi];
        const int n_tok = item.segs.tokens[sgi];
        for (int t0 = 0; t0 < n_tok; t0 += kKeys) {
            const int n_here = min(kKeys, n_tok - t0);
            __syncthreads();
            for (int i = threadIdx.x; i < n_here * D; i += blockDim.x) {
                const int j = i / D, e = i - j * D;
                sK[j][e] = to_f32<T>(kmat[(base + t0 + j) * D + e]);
                sV[j][e] = to_f32<T>(vmat[(base + t0 + j) * D + e]);
            }
            __syncthreads();
            for (int j = 0; j < n_here; ++j) {
                float part = 0.f;
#pragma unroll
                for (int e = 0; e < kDpt; ++e) part = fmaf(q[e], sK[j][4 * e + sub], part);
                part += __shfl_xor_sync(0xffffffffu, part, 1);
                part += __shfl_xor_sync(0xffffffffu, part, 2);
                const float s = part * a.scale;
                const float m_new = fmaxf(m, s);
                const float corr = expf(m - m_new);  // m = -inf on the first key: exp(-inf) = 0
                const float p = expf(s - m_new);
                l = l * corr + p;
#pragma unroll
                for (int e = 0; e < kDpt; ++e) acc[e] = fmaf(p, sV[j][4 * e + sub], acc[e] * corr);
                m = m_new;
            }
        }
    }
    if (row_ok) {
        T* out = reinterpret_cast<T*>(item.out) + ((size_t)row * a.n_heads + h) * D;
        const float inv = 1.f / l;
#pragma unroll
        for (int e = 0; e < kDpt; ++e) out[4 * e + sub] = from_f32<T>(acc[e] * inv);
    }
}

// One launch per layer-call: `item` travels as the launch's only inline descriptor.
cudaError_t launch_attn_simt(const AttnArgs& shared, const AttnItem& item, int dtype, cudaStream_t s) {
    AttnArgs a = shared;
    a.n_items = 1;
    a.items_tab = nullptr;
    a.items[0] = item;
    dim3 grid((item.n_q + 63) / 64, a.n_heads);
    if (a.head_dim == 64) {
        if (dtype == 0) attn_simt_kernel<__nv_bfloat16, 64><<<grid, 256, 0, s>>>(a);
        else attn_simt_kernel<float, 64><<<grid, 256, 0, s>>>(a);
    } else if (a.head_dim == 128) {
        if (dtype == 0) attn_simt_kernel<__nv_bfloat16, 128><<<grid, 256, 0, s>>>(a);
        else attn_simt_kernel<float, 128><<<grid, 256, 0, s>>>(a);
    } else {
        return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

}  // namespace ffk
