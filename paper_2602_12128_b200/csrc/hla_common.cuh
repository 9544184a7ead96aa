// Shared definitions of the HLA CUDA library (device helpers and the problem
// description the kernels receive).  Notation follows the paper: q, k^f are the
// d_phi-wide feature vectors, T_q / T_k their F-fold outer products with
// P = d_phi^F entries (first factor's index slowest), C the P x d context
// tensor, z the key-side sum used by the normaliser eta.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace hla {

constexpr int kMaxF = 4;
constexpr int kMaxP = 256;
constexpr int kMaxD = 128;

struct Dims {
    int B, H, N, d;
    int F, dphi, P;
    int ld;      // row stride (floats) of the fp32 state [P][ld]; column d holds z
    int S;       // token splits of a state build
    float eps;
};

// Words of the device status slot at the start of the workspace.
enum StatusWord { kStatusTimeout = 0, kStatusWhere = 1 };

template <typename T> __device__ __forceinline__ float ldf(const T* p);
template <> __device__ __forceinline__ float ldf<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }

template <typename T> __device__ __forceinline__ void stf(T* p, float v);
template <> __device__ __forceinline__ void stf<float>(float* p, float v) { *p = v; }
template <> __device__ __forceinline__ void stf<__nv_bfloat16>(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// Exact GELU, x * Phi(x), and its derivative Phi(x) + x * pdf(x).
__device__ __forceinline__ float gelu_erf(float x) { return 0.5f * x * (1.0f + erff(x * 0.70710678118654752f)); }
__device__ __forceinline__ float gelu_erf_grad(float x) {
    const float cdf = 0.5f * (1.0f + erff(x * 0.70710678118654752f));
    const float pdf = 0.3989422804014327f * __expf(-0.5f * x * x);
    return cdf + x * pdf;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

}  // namespace hla
