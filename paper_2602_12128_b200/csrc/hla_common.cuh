// Shared definitions of the HLA CUDA library (device helpers and the problem
// description the kernels receive).  Notation follows the paper: q, k^f are the
// d_phi-wide feature vectors, T_q / T_k their F-fold outer products with
// P = d_phi^F entries (first factor's index slowest), C the P x d context
// tensor, z the key-side sum used by the normaliser eta.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <vector>

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

// Host side: counts the kernels a call launches and, when enabled, marks each launch with CUDA events on the
// launching stream so a caller can read per-kernel device time.  Kernels of one call run back to back on the stream,
// so one event between two launches serves as the end of the first and the start of the second: n launches of a call
// cost n + 1 event records.
struct LaunchRec {
    struct Rec { const char* name; int a, b; };            // indices into `events`
    struct Acc { const char* name; double ms; long long n; };
    cudaStream_t st = nullptr;
    int launches = 0;
    bool timing = false;
    std::vector<cudaEvent_t> events;      // pool, reused after every collect()
    size_t used = 0;
    std::vector<Rec> recs;
    int last_end = -1;                    // event that ended the previous launch of this call
    std::vector<Acc> acc;

    void start_call(cudaStream_t s) { st = s; launches = 0; last_end = -1; }
    int mark() {
        if (used == events.size()) {
            cudaEvent_t e = nullptr;
            if (cudaEventCreate(&e) != cudaSuccess) { timing = false; return -1; }
            events.push_back(e);
        }
        cudaEventRecord(events[used], st);
        return (int)used++;
    }
    void begin(const char* name) {
        ++launches;
        if (!timing) return;
        const int a = last_end >= 0 ? last_end : mark();
        if (a >= 0) recs.push_back(Rec{name, a, -1});
    }
    bool end() {
        if (timing && !recs.empty() && recs.back().b < 0) {
            recs.back().b = mark();
            last_end = recs.back().b;
        }
        return cudaPeekAtLastError() == cudaSuccess;
    }
    // Caller has synchronised the stream.  Folds the recorded launches into per-name totals (replacing earlier totals).
    int collect() {
        acc.clear();
        for (const Rec& r : recs) {
            float ms = 0.f;
            if (r.a < 0 || r.b < 0 || cudaEventElapsedTime(&ms, events[r.a], events[r.b]) != cudaSuccess) continue;
            size_t j = 0;
            for (; j < acc.size(); ++j) if (strcmp(acc[j].name, r.name) == 0) break;
            if (j == acc.size()) acc.push_back(Acc{r.name, 0.0, 0});
            acc[j].ms += ms;
            acc[j].n += 1;
        }
        recs.clear();
        used = 0;
        last_end = -1;
        return (int)acc.size();
    }
    ~LaunchRec() { for (auto e : events) cudaEventDestroy(e); }
};

}  // namespace hla
