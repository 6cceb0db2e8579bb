// The rectified-flow Euler update that follows a forward (Alg. 1, "Step"):
//     x_{k-1} = x_k - (sigma_k - sigma_{k-1}) * v_hat
// and the shifted noise levels sigma_k the stages sit at.
//
// Elementwise and HBM-bound: x and v are read once, the result is written once, 16 bytes per access.  Each
// thread handles pieces of 4 elements (fp32) or 8 elements (bf16) in a grid-stride loop; the grid is a whole
// number of waves.  Arithmetic is in float with the step size, the product and the difference each rounded
// once (no fused multiply-add), then round-to-nearest-even to bf16 if the latent is stored in bf16, so that
// the result can be checked bit for bit.
#include <cuda_bf16.h>

#include <atomic>

#include "../../include/ff.h"
#include "ff_internal.h"

namespace {

template <bool kBf16>
struct Elem;
template <>
struct Elem<true> {
    using T = __nv_bfloat16;
    static __device__ __forceinline__ float load(const T* p) { return __bfloat162float(*p); }
    static __device__ __forceinline__ void store(T* p, float x) { *p = __float2bfloat16_rn(x); }
};
template <>
struct Elem<false> {
    using T = float;
    static __device__ __forceinline__ float load(const T* p) { return *p; }
    static __device__ __forceinline__ void store(T* p, float x) { *p = x; }
};

__device__ __forceinline__ float euler(float x, float v, float dsigma) { return __fsub_rn(x, __fmul_rn(dsigma, v)); }

// kVec elements per thread per iteration: 8 keeps every access at 16 bytes (bf16) or 2 x 16 bytes (fp32).
template <bool kXBf16, bool kVBf16>
__global__ void __launch_bounds__(256) euler_step_kernel(const void* x_, const void* __restrict__ v_, void* out_,
                                                         long long n, float dsigma) {
    using XT = typename Elem<kXBf16>::T;
    using VT = typename Elem<kVBf16>::T;
    constexpr int kVec = 8;
    const XT* x = static_cast<const XT*>(x_);
    const VT* v = static_cast<const VT*>(v_);
    XT* out = static_cast<XT*>(out_);
    const long long n_vec = n / kVec;
    const long long stride = (long long)gridDim.x * blockDim.x;
    ffk::grid_dependency_wait();  // launched as a programmatic dependent: x and v may come from the kernel before
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec; i += stride) {
        alignas(16) XT xs[kVec];
        alignas(16) VT vs[kVec];
        constexpr int kXLoads = sizeof(XT) * kVec / 16, kVLoads = sizeof(VT) * kVec / 16;
#pragma unroll
        for (int j = 0; j < kXLoads; ++j)
            reinterpret_cast<uint4*>(xs)[j] = reinterpret_cast<const uint4*>(x + i * kVec)[j];  // out may be x: plain load
#pragma unroll
        for (int j = 0; j < kVLoads; ++j)
            reinterpret_cast<uint4*>(vs)[j] = __ldg(reinterpret_cast<const uint4*>(v + i * kVec) + j);
#pragma unroll
        for (int e = 0; e < kVec; ++e)
            Elem<kXBf16>::store(&xs[e], euler(Elem<kXBf16>::load(&xs[e]), Elem<kVBf16>::load(&vs[e]), dsigma));
#pragma unroll
        for (int j = 0; j < kXLoads; ++j)
            reinterpret_cast<uint4*>(out + i * kVec)[j] = reinterpret_cast<const uint4*>(xs)[j];
    }
    // ragged tail (fewer than kVec elements): one element per thread of the first block
    const long long tail0 = n_vec * kVec;
    if (blockIdx.x == 0 && tail0 + threadIdx.x < n) {
        const long long i = tail0 + threadIdx.x;
        Elem<kXBf16>::store(out + i, euler(Elem<kXBf16>::load(x + i), Elem<kVBf16>::load(v + i), dsigma));
    }
}

}  // namespace

extern "C" ff_status ff_euler_step(const void* x, const void* v, float sigma_k, float sigma_km1, int64_t n,
                                   int32_t dtype_x, int32_t dtype_v, void* out, void* stream) {
    if (!x || !v || !out || n < 0 || (dtype_x != FF_BF16 && dtype_x != FF_F32) ||
        (dtype_v != FF_BF16 && dtype_v != FF_F32) || !(sigma_k == sigma_k) || !(sigma_km1 == sigma_km1))
        return FF_ERR_INVALID_ARG;
    if (((uintptr_t)x | (uintptr_t)v | (uintptr_t)out) & 15u) return FF_ERR_INVALID_ARG;
    if (n == 0) return FF_OK;
    // the SM count of each device is asked once (the call is a large part of the host time of a launch this small)
    static std::atomic<int> sms_of[64];
    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess) return FF_ERR_CUDA;
    int sms = (device >= 0 && device < 64) ? sms_of[device].load(std::memory_order_relaxed) : 0;
    if (sms == 0) {
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms < 1) sms = 148;
        if (device >= 0 && device < 64) sms_of[device].store(sms, std::memory_order_relaxed);
    }
    const long long n_vec = n / 8;
    long long blocks = (n_vec + 255) / 256;
    const long long cap = (long long)sms * 8;  // a whole number of waves of 8 resident blocks per SM
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    const float dsigma = sigma_k - sigma_km1;  // rounded once, on the host, in float
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const bool xb = dtype_x == FF_BF16, vb = dtype_v == FF_BF16;
    // One chunk's latent is a few hundred thousand elements: the launch itself is most of the cost, so the grid is
    // set up under the tail of the kernel before it in the stream, like the library's other kernels.
    const dim3 grid((unsigned)blocks), block(256);
    const long long nn = n;
    cudaError_t e;
    if (xb && vb) e = ffk::launch_overlapped(euler_step_kernel<true, true>, grid, block, 0, s, x, v, out, nn, dsigma);
    else if (xb) e = ffk::launch_overlapped(euler_step_kernel<true, false>, grid, block, 0, s, x, v, out, nn, dsigma);
    else if (vb) e = ffk::launch_overlapped(euler_step_kernel<false, true>, grid, block, 0, s, x, v, out, nn, dsigma);
    else e = ffk::launch_overlapped(euler_step_kernel<false, false>, grid, block, 0, s, x, v, out, nn, dsigma);
    return e == cudaSuccess ? FF_OK : FF_ERR_CUDA;
}

// sigma_k = shift * u / (1 + (shift - 1) * u) with u = k / S: the uniform levels 1, (S-1)/S, ..., 1/S, 0 pushed
// through the flow-shift map; sigma_S = 1 (pure noise), sigma_0 = 0 (clean).
extern "C" ff_status ff_plan_sigma(int32_t k, int32_t n_stages, double shift, double* sigma) {
    if (!sigma || n_stages < 1 || k < 0 || k > n_stages || !(shift > 0.0)) return FF_ERR_INVALID_ARG;
    const double u = (double)k / (double)n_stages;
    *sigma = shift * u / (1.0 + (shift - 1.0) * u);
    return FF_OK;
}
