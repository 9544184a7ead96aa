// Tensor-core kernels of the feature networks phi (appendix "Defining phi";
// Algorithm 1 step 4) for bf16:  feat = ReLU(W2^T GELU(W1^T x + b1) + b2).
//
// Per 128-token tile of X (Q or K, TMA-loaded once) and per map m:
//   D1 = X * W1[m]            tcgen05, fp32 in TMEM        [128 tok x d hidden]
//   G  = bf16(GELU(D1 + b1))  8 warps, thread = (token, half of the hidden units); written as the next MMA's A operand
//   D2 = G * W2[m]            tcgen05, N padded to 16
//   feat = ReLU(D2 + b2)      fp32 features to global memory
// The key side runs its F maps on the same X tile, so K is read once.
// GELU is the exact erf form evaluated with an odd polynomial for erf (fit_gelu_poly.py: |error| < 7e-5,
// far below the bf16 rounding of G) - no special-function unit on the hot loop.
#pragma once
#include "hla_tc.cuh"

namespace hla {
namespace tc {

__device__ __forceinline__ float gelu_poly(float x) {
    const float u = fminf(fmaxf(x * 0.70710678f, -3.0f), 3.0f);
    const float t = u * u;
    float p = 4.074210630e-08f;
    p = fmaf(p, t, -1.944822741e-06f);
    p = fmaf(p, t, 4.106052437e-05f);
    p = fmaf(p, t, -5.110368664e-04f);
    p = fmaf(p, t, 4.235427410e-03f);
    p = fmaf(p, t, -2.510286119e-02f);
    p = fmaf(p, t, 1.110793351e-01f);
    p = fmaf(p, t, -3.753148748e-01f);
    p = fmaf(p, t, 1.128268423e+00f);
    const float hx = 0.5f * x;
    return fmaf(hx, u * p, hx);
}

struct PhiPtrs {
    const __nv_bfloat16* b1[3];
    const __nv_bfloat16* W2[3];
    const __nv_bfloat16* b2[3];
};
struct PhiMaps {
    CUtensorMap w1[3];
};

constexpr int kPfThreads = 320;   // warp 0: TMA, warp 1: MMA, warps 2..9: epilogue (thread = token row x half of the hidden units)

template <int DV, int NMAPS> struct PfCfg {
    static constexpr int kXBytes = kTileTokens * DV * 2;
    static constexpr int kW1Bytes = DV * DV * 2;
    static constexpr int kW2Bytes = (DV / 64) * 2048;            // [16 rows][DV] bf16, K-major, per map
    static constexpr int kOffX = 0;                              // 2 stages
    static constexpr int kOffG = 2 * kXBytes;                    // GELU output tile
    static constexpr int kOffW1 = kOffG + kXBytes;
    static constexpr int kOffW2 = kOffW1 + NMAPS * kW1Bytes;
    static constexpr int kOffBias = kOffW2 + NMAPS * kW2Bytes;   // per map: b1[DV], b2[8] floats
    static constexpr int kOffBars = kOffBias + NMAPS * (DV + 8) * 4;
    static constexpr int kSmemUsed = 1024 + kOffBars + 256;
    static constexpr int kSmem = kSmemUsed > 120 * 1024 ? kSmemUsed : 120 * 1024;   // one CTA per SM (512 TMEM columns)
};

// X [rows][DV] bf16 (rows = B*H*N tokens).  KSIDE: features to kf[bh][f][n][6], else qf[row][6].
template <int DV, int NMAPS, bool KSIDE>
__global__ void __launch_bounds__(kPfThreads, 1) tc_phi_forward_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ PhiMaps maps,
                                                                       PhiPtrs P, float* __restrict__ feat, long long rows, int N, int* status) {
    using Cfg = PfCfg<DV, NMAPS>;
    constexpr int HC = DV / 2;          // hidden units per epilogue thread
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    float* bias = reinterpret_cast<float*>(smem + Cfg::kOffBias);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::kOffBars);
    uint64_t* x_full = bars;           // [2]
    uint64_t* x_empty = bars + 2;      // [2] MMA commit
    uint64_t* d1_full = bars + 4;      // [2] MMA commit
    uint64_t* d1_empty = bars + 6;     // [2] 256 arrivals
    uint64_t* g_full = bars + 8;       // 256 arrivals
    uint64_t* g_free = bars + 9;       // MMA commit
    uint64_t* d2_full = bars + 10;     // [2] MMA commit
    uint64_t* d2_empty = bars + 12;    // [2] 128 arrivals
    uint64_t* w_full = bars + 14;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 15);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const long long tiles = (rows + kTileTokens - 1) / kTileTokens;
    const long long t0 = tiles * blockIdx.x / gridDim.x, t1 = tiles * (blockIdx.x + 1) / gridDim.x;
    const int ntiles = (int)(t1 - t0);
    const int nunits = ntiles * NMAPS;

    // second-layer weights as a K-major MMA operand [16 rows (outputs, 6 used)][DV], and the biases
    for (int i = tid; i < NMAPS * Cfg::kW2Bytes / 16; i += kPfThreads) reinterpret_cast<uint4*>(smem + Cfg::kOffW2)[i] = make_uint4(0, 0, 0, 0);
    __syncthreads();
    for (int i = tid; i < NMAPS * DV * 6; i += kPfThreads) {
        const int m = i / (DV * 6), j = (i / 6) % DV, o = i % 6;
        uint8_t* base = smem + Cfg::kOffW2 + m * Cfg::kW2Bytes + (j >> 6) * 2048;
        *reinterpret_cast<__nv_bfloat16*>(base + sw128_off(o, (j & 63) >> 3) + (j & 7) * 2) = P.W2[m][j * 6 + o];
    }
    for (int i = tid; i < NMAPS * (DV + 8); i += kPfThreads) {
        const int m = i / (DV + 8), j = i % (DV + 8);
        bias[i] = j < DV ? __bfloat162float(P.b1[m][j]) : (j - DV < 6 ? __bfloat162float(P.b2[m][j - DV]) : 0.f);
    }
    fence_proxy_async();
    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(&x_full[i], 1);
            mbar_init(&x_empty[i], 1);
            mbar_init(&d1_full[i], 1);
            mbar_init(&d1_empty[i], 256);
            mbar_init(&d2_full[i], 1);
            mbar_init(&d2_empty[i], 128);
        }
        mbar_init(g_full, 256);
        mbar_init(g_free, 1);
        mbar_init(w_full, 1);
        fence_mbar_init();
        prefetch_tmap(&mapX);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;     // D1[b] at columns 128*b, D2[b] at columns 256 + 32*b
    bool ok = true;

    if (warp == 0) {
        if (lane == 0 && ntiles > 0) {
            mbar_arrive_expect_tx(w_full, NMAPS * Cfg::kW1Bytes);
            for (int m = 0; m < NMAPS; ++m)
                for (int b = 0; b < DV / 64; ++b)
                    tma_load_2d(smem + Cfg::kOffW1 + m * Cfg::kW1Bytes + b * (DV * 128), &maps.w1[m], w_full, b * 64, 0);
            for (int it = 0; it < ntiles; ++it) {
                const int st = it & 1, u = it >> 1;
                if (!mbar_wait(&x_empty[st], (u & 1) ^ 1)) { report_timeout(status, 501); break; }
                mbar_arrive_expect_tx(&x_full[st], Cfg::kXBytes);
                for (int b = 0; b < DV / 64; ++b)
                    tma_load_2d(smem + Cfg::kOffX + st * Cfg::kXBytes + b * kBlk, &mapX, &x_full[st], b * 64, (int)((t0 + it) * kTileTokens));
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && ntiles > 0) {
            const uint32_t idesc1 = idesc_bf16(128, DV, false, true);   // X K-major, W1 [in][hidden] MN-major
            const uint32_t idesc2 = idesc_bf16(128, 16, false, false);  // G K-major, W2 operand K-major
            const uint32_t ga = smem_u32(smem + Cfg::kOffG);
            bool good = mbar_wait(w_full, 0);
            if (!good) report_timeout(status, 502);
            auto issue_mma1 = [&](int unit) -> bool {
                const int it = unit / NMAPS, m = unit % NMAPS, st = it & 1, b = unit & 1;
                if (m == 0 && !mbar_wait(&x_full[st], (it >> 1) & 1)) return false;
                if (!mbar_wait(&d1_empty[b], ((unit >> 1) & 1) ^ 1)) return false;
                tc_fence_after();
                const uint32_t xa = smem_u32(smem + Cfg::kOffX + st * Cfg::kXBytes);
                const uint32_t wa = smem_u32(smem + Cfg::kOffW1 + m * Cfg::kW1Bytes);
#pragma unroll
                for (int ks = 0; ks < DV / 16; ++ks)
                    umma_bf16(tmem + 128 * b, smem_desc_sw128(xa + (ks >> 2) * kBlk + (ks & 3) * 32, 16, 1024),
                              smem_desc_sw128(wa + ks * 2048, DV * 128, 1024), idesc1, ks > 0 ? 1u : 0u);
                umma_commit(&d1_full[b]);
                if (m == NMAPS - 1) umma_commit(&x_empty[st]);
                return true;
            };
            if (good && nunits > 0) good = issue_mma1(0);
            if (good && nunits > 1) good = issue_mma1(1);
            for (int unit = 0; unit < nunits && good; ++unit) {
                const int m = unit % NMAPS, b = unit & 1;
                if (!(mbar_wait(g_full, unit & 1) && mbar_wait(&d2_empty[b], ((unit >> 1) & 1) ^ 1))) { good = false; break; }
                tc_fence_after();
                const uint32_t w2a = smem_u32(smem + Cfg::kOffW2 + m * Cfg::kW2Bytes);
#pragma unroll
                for (int ks = 0; ks < DV / 16; ++ks)
                    umma_bf16(tmem + 256 + 32 * b, smem_desc_sw128(ga + (ks >> 2) * kBlk + (ks & 3) * 32, 16, 1024),
                              smem_desc_sw128(w2a + (ks >> 2) * 2048 + (ks & 3) * 32, 16, 1024), idesc2, ks > 0 ? 1u : 0u);
                umma_commit(g_free);
                umma_commit(&d2_full[b]);
                if (unit + 2 < nunits) good = issue_mma1(unit + 2);
            }
            if (!good) report_timeout(status, 503);
        }
    } else {
        const int quarter = warp & 3, half = (warp - 2) >> 2;
        const int row = quarter * 32 + lane;
        for (int unit = 0; unit < nunits; ++unit) {
            const int it = unit / NMAPS, m = unit % NMAPS, b = unit & 1;
            const float* b1s = bias + m * (DV + 8);
            if (ok && !mbar_wait(&d1_full[b], (unit >> 1) & 1)) { ok = false; report_timeout(status, 504); }
            if (ok && unit > 0 && !mbar_wait(g_free, (unit - 1) & 1)) { ok = false; report_timeout(status, 505); }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t ta = tmem + 128 * b + ((uint32_t)(quarter * 32) << 16) + half * HC;
            const uint32_t gblk = smem_u32(smem + Cfg::kOffG);
#pragma unroll
            for (int c = 0; c < HC / 16; ++c) {
                uint32_t r[16];
                tmem_ld16(ta + 16 * c, r);
                tmem_ld_wait();
                const int col = half * HC + 16 * c;
                uint32_t w[8];
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    w[e] = pack_bf16(gelu_poly(__uint_as_float(r[2 * e]) + b1s[col + 2 * e]), gelu_poly(__uint_as_float(r[2 * e + 1]) + b1s[col + 2 * e + 1]));
                const uint32_t blk = gblk + (col >> 6) * kBlk;
                st_shared_v4(blk + sw128_off(row, (col & 63) >> 3), w[0], w[1], w[2], w[3]);
                st_shared_v4(blk + sw128_off(row, ((col & 63) >> 3) + 1), w[4], w[5], w[6], w[7]);
            }
            tc_fence_before();
            mbar_arrive(&d1_empty[b]);
            fence_proxy_async();
            mbar_arrive(g_full);
            if (half == 0) {
                if (!mbar_wait(&d2_full[b], (unit >> 1) & 1)) { ok = false; report_timeout(status, 506); }
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                uint32_t r[8];
                tmem_ld8(tmem + 256 + 32 * b + ((uint32_t)(quarter * 32) << 16), r);
                tmem_ld_wait();
                tc_fence_before();
                mbar_arrive(&d2_empty[b]);
                const long long grow = (t0 + it) * kTileTokens + row;
                if (grow < rows) {
                    float f[6];
#pragma unroll
                    for (int o = 0; o < 6; ++o) f[o] = fmaxf(__uint_as_float(r[o]) + b1s[DV + o], 0.f);
                    if (KSIDE) {
                        const long long bh = grow / N, n = grow - bh * N;
                        store6(feat + ((bh * NMAPS + m) * N + n) * 6, f);
                    } else {
                        store6(feat + grow * 6, f);
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, 512);
}

template <int DV>
inline hla_status launch_phi_forward(const Dims& D, int BH, const hla_mlp* phi_q, const hla_mlp* phi_k, const void* Q, const void* K, char* ws,
                                     const hla_ws_layout& L, int sm_count, LaunchRec& rec) {
    const long long rows = (long long)BH * D.N;
    CUtensorMap mapQ, mapK;
    PhiMaps mq, mk;
    PhiPtrs pq{}, pk{};
    if (!make_map_2d(&mapQ, Q, (size_t)rows, DV, kTileTokens) || !make_map_2d(&mapK, K, (size_t)rows, DV, kTileTokens)) return HLA_ERR_CUDA;
    if (!make_map_2d(&mq.w1[0], phi_q->W1, DV, DV, DV)) return HLA_ERR_CUDA;
    mq.w1[1] = mq.w1[0];
    mq.w1[2] = mq.w1[0];
    pq.b1[0] = static_cast<const __nv_bfloat16*>(phi_q->b1);
    pq.W2[0] = static_cast<const __nv_bfloat16*>(phi_q->W2);
    pq.b2[0] = static_cast<const __nv_bfloat16*>(phi_q->b2);
    for (int f = 0; f < 3; ++f) {
        if (!make_map_2d(&mk.w1[f], phi_k[f].W1, DV, DV, DV)) return HLA_ERR_CUDA;
        pk.b1[f] = static_cast<const __nv_bfloat16*>(phi_k[f].b1);
        pk.W2[f] = static_cast<const __nv_bfloat16*>(phi_k[f].W2);
        pk.b2[f] = static_cast<const __nv_bfloat16*>(phi_k[f].b2);
    }
    int* status = reinterpret_cast<int*>(ws + L.status);
    if (!set_smem(tc_phi_forward_kernel<DV, 1, false>, PfCfg<DV, 1>::kSmem) || !set_smem(tc_phi_forward_kernel<DV, 3, true>, PfCfg<DV, 3>::kSmem))
        return HLA_ERR_CUDA;
    const long long tiles = (rows + kTileTokens - 1) / kTileTokens;
    const int grid = (int)(tiles < sm_count ? tiles : sm_count);
    cudaStream_t st = rec.st;
    rec.begin("tc_phi_forward");
    tc_phi_forward_kernel<DV, 1, false><<<grid, kPfThreads, PfCfg<DV, 1>::kSmem, st>>>(mapQ, mq, pq, reinterpret_cast<float*>(ws + L.qf), rows, D.N, status);
    if (!rec.end()) return HLA_ERR_CUDA;
    rec.begin("tc_phi_forward");
    tc_phi_forward_kernel<DV, 3, true><<<grid, kPfThreads, PfCfg<DV, 3>::kSmem, st>>>(mapK, mk, pk, reinterpret_cast<float*>(ws + L.kf), rows, D.N, status);
    return rec.end() ? HLA_OK : HLA_ERR_CUDA;
}

inline hla_status phi_forward(const Dims& D, int BH, const hla_mlp* phi_q, const hla_mlp* phi_k, const void* Q, const void* K, char* ws,
                              const hla_ws_layout& L, int sm_count, LaunchRec& rec) {
    if (D.d == 128) return launch_phi_forward<128>(D, BH, phi_q, phi_k, Q, K, ws, L, sm_count, rec);
    return launch_phi_forward<64>(D, BH, phi_q, phi_k, Q, K, ws, L, sm_count, rec);
}

// =======================================================================================
// Backward of the feature networks with respect to their input (weights fixed):
//   dp  = dfeat (.) 1[feat > 0]                 ReLU mask from the features the forward kept
//   dg  = dp * W2^T                             6 FMAs per hidden unit on the ALUs
//   dh  = dg (.) GELU'(h),  h = X W1 + b1       h recomputed on the tensor cores
//   dX  = sum over the maps of dh * W1^T        tensor cores, accumulated over the maps in TMEM
// Per 128-token tile: X is TMA-loaded once, every map's h goes through TMEM, the dh tile is
// written as the second MMA's A operand, and the W1 image in shared memory serves both MMAs
// (MN-major B for X W1, K-major B for dh W1^T).
// =======================================================================================
// GELU'(x) = Phi(x) + x pdf(x) = 1/2 + u (P(u^2)/2 + exp(-u^2)/sqrt(pi)),  u = x / sqrt 2, erf(u) = u P(u^2).
__device__ __forceinline__ float gelu_grad_poly(float x) {
    const float uu = x * 0.70710678f;
    const float u = fminf(fmaxf(uu, -3.0f), 3.0f);
    const float t = u * u;
    float p = 4.074210630e-08f;
    p = fmaf(p, t, -1.944822741e-06f);
    p = fmaf(p, t, 4.106052437e-05f);
    p = fmaf(p, t, -5.110368664e-04f);
    p = fmaf(p, t, 4.235427410e-03f);
    p = fmaf(p, t, -2.510286119e-02f);
    p = fmaf(p, t, 1.110793351e-01f);
    p = fmaf(p, t, -3.753148748e-01f);
    p = fmaf(p, t, 1.128268423e+00f);
    const float e = exp2f(uu * uu * -1.44269504f);
    return fmaf(uu, 0.564189584f * e, fmaf(0.5f * u, p, 0.5f));
}

struct PhiBwdPtrs {
    const __nv_bfloat16* b1[3];
    const __nv_bfloat16* W2[3];
};

constexpr int kPbThreads = 320;   // warp 0: TMA loads, warp 1: MMA, warps 2..9: epilogue (thread = token row x half of the columns)

template <int DV, int NMAPS> struct PbCfg {
    static constexpr int kXStages = (DV == 128 && NMAPS == 3) ? 1 : 2;
    static constexpr int kXBytes = kTileTokens * DV * 2;
    static constexpr int kW1Bytes = DV * DV * 2;
    static constexpr int kOffX = 0;
    static constexpr int kOffDh = kXStages * kXBytes;            // dh tile (A operand of the second MMA)
    static constexpr int kOffOut = kOffDh + kXBytes;             // dX staging tile for the TMA store
    static constexpr int kOffW1 = kOffOut + kXBytes;
    static constexpr int kOffW2 = kOffW1 + NMAPS * kW1Bytes;     // fp32 [NMAPS][DV][8]  (6 used)
    static constexpr int kOffB1 = kOffW2 + NMAPS * DV * 8 * 4;   // fp32 [NMAPS][DV]
    static constexpr int kOffBars = kOffB1 + NMAPS * DV * 4;
    static constexpr int kSmemUsed = 1024 + kOffBars + 256;
    static constexpr int kSmem = kSmemUsed > 120 * 1024 ? kSmemUsed : 120 * 1024;   // one CTA per SM (512 TMEM columns)
};

// X, dX [rows][DV] bf16.  KSIDE: feat / dfeat are [bh][NMAPS][N][6], else [rows][6].
template <int DV, int NMAPS, bool KSIDE>
__global__ void __launch_bounds__(kPbThreads, 1) tc_phi_backward_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapdX,
                                                                        const __grid_constant__ PhiMaps maps, PhiBwdPtrs P,
                                                                        const float* __restrict__ feat, const float* __restrict__ dfeat,
                                                                        long long rows, int N, int* status) {
    using Cfg = PbCfg<DV, NMAPS>;
    constexpr int HC = DV / 2;
    constexpr int XST = Cfg::kXStages;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    float* w2s = reinterpret_cast<float*>(smem + Cfg::kOffW2);
    float* b1s = reinterpret_cast<float*>(smem + Cfg::kOffB1);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::kOffBars);
    uint64_t* x_full = bars;           // [2]
    uint64_t* x_empty = bars + 2;      // [2] MMA commit
    uint64_t* h_full = bars + 4;       // [2] MMA commit
    uint64_t* h_empty = bars + 6;      // [2] 256 arrivals
    uint64_t* dh_full = bars + 8;      // 256 arrivals
    uint64_t* dh_free = bars + 9;      // MMA commit
    uint64_t* dx_full = bars + 10;     // [2] MMA commit
    uint64_t* dx_empty = bars + 12;    // [2] 256 arrivals
    uint64_t* w_full = bars + 14;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 15);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const long long tiles = (rows + kTileTokens - 1) / kTileTokens;
    const long long t0 = tiles * blockIdx.x / gridDim.x, t1 = tiles * (blockIdx.x + 1) / gridDim.x;
    const int ntiles = (int)(t1 - t0);
    const int nunits = ntiles * NMAPS;

    for (int i = tid; i < NMAPS * DV * 8; i += kPbThreads) {
        const int m = i / (DV * 8), j = (i >> 3) % DV, o = i & 7;
        w2s[i] = o < 6 ? __bfloat162float(P.W2[m][j * 6 + o]) : 0.f;
    }
    for (int i = tid; i < NMAPS * DV; i += kPbThreads) b1s[i] = __bfloat162float(P.b1[i / DV][i % DV]);
    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(&x_full[i], 1);
            mbar_init(&x_empty[i], 1);
            mbar_init(&h_full[i], 1);
            mbar_init(&h_empty[i], 256);
            mbar_init(&dx_full[i], 1);
            mbar_init(&dx_empty[i], 256);
        }
        mbar_init(dh_full, 256);
        mbar_init(dh_free, 1);
        mbar_init(w_full, 1);
        fence_mbar_init();
        prefetch_tmap(&mapX);
        prefetch_tmap(&mapdX);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;     // h[b] at columns 128*b, dX[b] at columns 256 + 128*b
    bool ok = true;

    if (warp == 0) {
        if (lane == 0 && ntiles > 0) {
            mbar_arrive_expect_tx(w_full, NMAPS * Cfg::kW1Bytes);
            for (int m = 0; m < NMAPS; ++m)
                for (int b = 0; b < DV / 64; ++b)
                    tma_load_2d(smem + Cfg::kOffW1 + m * Cfg::kW1Bytes + b * (DV * 128), &maps.w1[m], w_full, b * 64, 0);
            for (int it = 0; it < ntiles; ++it) {
                const int st = it % XST, u = it / XST;
                if (!mbar_wait(&x_empty[st], (u & 1) ^ 1)) { report_timeout(status, 601); break; }
                mbar_arrive_expect_tx(&x_full[st], Cfg::kXBytes);
                for (int b = 0; b < DV / 64; ++b)
                    tma_load_2d(smem + Cfg::kOffX + st * Cfg::kXBytes + b * kBlk, &mapX, &x_full[st], b * 64, (int)((t0 + it) * kTileTokens));
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && ntiles > 0) {
            const uint32_t idesc1 = idesc_bf16(128, DV, false, true);    // h  = X (K-major) * W1 [in][hidden] (MN-major)
            const uint32_t idesc2 = idesc_bf16(128, DV, false, false);   // dX = dh (K-major over hidden) * W1 as [in][hidden] (K-major)
            const uint32_t dha = smem_u32(smem + Cfg::kOffDh);
            bool good = mbar_wait(w_full, 0);
            if (!good) report_timeout(status, 602);
            auto issue_mma1 = [&](int unit) -> bool {
                const int it = unit / NMAPS, m = unit % NMAPS, st = it % XST, b = unit & 1;
                if (m == 0 && !mbar_wait(&x_full[st], (it / XST) & 1)) return false;
                if (!mbar_wait(&h_empty[b], ((unit >> 1) & 1) ^ 1)) return false;
                tc_fence_after();
                const uint32_t xa = smem_u32(smem + Cfg::kOffX + st * Cfg::kXBytes);
                const uint32_t wa = smem_u32(smem + Cfg::kOffW1 + m * Cfg::kW1Bytes);
#pragma unroll
                for (int ks = 0; ks < DV / 16; ++ks)
                    umma_bf16(tmem + 128 * b, smem_desc_sw128(xa + (ks >> 2) * kBlk + (ks & 3) * 32, 16, 1024),
                              smem_desc_sw128(wa + ks * 2048, DV * 128, 1024), idesc1, ks > 0 ? 1u : 0u);
                umma_commit(&h_full[b]);
                if (m == NMAPS - 1) umma_commit(&x_empty[st]);
                return true;
            };
            if (good && nunits > 0) good = issue_mma1(0);
            if (good && nunits > 1) good = issue_mma1(1);
            for (int unit = 0; unit < nunits && good; ++unit) {
                const int it = unit / NMAPS, m = unit % NMAPS, tb = it & 1;
                if (!mbar_wait(dh_full, unit & 1)) { good = false; break; }
                if (m == 0 && !mbar_wait(&dx_empty[tb], ((it >> 1) & 1) ^ 1)) { good = false; break; }
                tc_fence_after();
                const uint32_t wa = smem_u32(smem + Cfg::kOffW1 + m * Cfg::kW1Bytes);
#pragma unroll
                for (int ks = 0; ks < DV / 16; ++ks)
                    umma_bf16(tmem + 256 + 128 * tb, smem_desc_sw128(dha + (ks >> 2) * kBlk + (ks & 3) * 32, 16, 1024),
                              smem_desc_sw128(wa + (ks >> 2) * (DV * 128) + (ks & 3) * 32, 16, 1024), idesc2, (m > 0 || ks > 0) ? 1u : 0u);
                umma_commit(dh_free);
                if (m == NMAPS - 1) umma_commit(&dx_full[tb]);
                if (unit + 2 < nunits) good = issue_mma1(unit + 2);
            }
            if (!good) report_timeout(status, 603);
        }
    } else {
        const int quarter = warp & 3, half = (warp - 2) >> 2;
        const int row = quarter * 32 + lane;
        const bool leader = tid == 64;
        // After a wait has run out (ok == false) the loop keeps going without waiting or touching TMEM / shared
        // memory, so that every thread still reaches the named barriers.
        for (int unit = 0; unit < nunits; ++unit) {
            const int it = unit / NMAPS, m = unit % NMAPS, b = unit & 1, tb = it & 1;
            const long long grow = (t0 + it) * kTileTokens + row;
            float dp[6];
            if (ok && grow < rows) {
                size_t off;
                if (KSIDE) {
                    const long long bh = grow / N, n = grow - bh * N;
                    off = (size_t)((bh * NMAPS + m) * N + n) * 6;
                } else {
                    off = (size_t)grow * 6;
                }
                float f[6];
                load6(f, feat + off);
                load6(dp, dfeat + off);
#pragma unroll
                for (int o = 0; o < 6; ++o) dp[o] = f[o] > 0.f ? dp[o] : 0.f;
            } else {
#pragma unroll
                for (int o = 0; o < 6; ++o) dp[o] = 0.f;
            }
            if (ok && !mbar_wait(&h_full[b], (unit >> 1) & 1)) { ok = false; report_timeout(status, 604); }
            ok = __all_sync(0xffffffffu, ok);
            if (ok) {
                tc_fence_after();
                const uint32_t ta = tmem + 128 * b + ((uint32_t)(quarter * 32) << 16) + half * HC;
                const uint32_t dblk = smem_u32(smem + Cfg::kOffDh);
                const float* bm = b1s + m * DV;
                const float4* wm = reinterpret_cast<const float4*>(w2s + m * DV * 8);
#pragma unroll
                for (int c = 0; c < HC / 16; ++c) {
                    uint32_t r[16];
                    tmem_ld16(ta + 16 * c, r);
                    tmem_ld_wait();
                    const int col = half * HC + 16 * c;
                    float dh[16];
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        const float4 wa = wm[2 * (col + e)], wb = wm[2 * (col + e) + 1];
                        float dg = dp[0] * wa.x;
                        dg = fmaf(dp[1], wa.y, dg);
                        dg = fmaf(dp[2], wa.z, dg);
                        dg = fmaf(dp[3], wa.w, dg);
                        dg = fmaf(dp[4], wb.x, dg);
                        dg = fmaf(dp[5], wb.y, dg);
                        dh[e] = dg * gelu_grad_poly(__uint_as_float(r[e]) + bm[col + e]);
                    }
                    if (c == 0 && unit > 0) {   // the dh tile is free once the previous unit's second MMA has read it
                        if (!mbar_wait(dh_free, (unit - 1) & 1)) { ok = false; report_timeout(status, 605); }
                        ok = __all_sync(0xffffffffu, ok);
                    }
                    if (ok) {
                        uint32_t w[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) w[e] = pack_bf16(dh[2 * e], dh[2 * e + 1]);
                        const uint32_t blk = dblk + (col >> 6) * kBlk;
                        st_shared_v4(blk + sw128_off(row, (col & 63) >> 3), w[0], w[1], w[2], w[3]);
                        st_shared_v4(blk + sw128_off(row, ((col & 63) >> 3) + 1), w[4], w[5], w[6], w[7]);
                    }
                }
            }
            if (ok) {
                tc_fence_before();
                mbar_arrive(&h_empty[b]);
                fence_proxy_async();
                mbar_arrive(dh_full);
            }
            if (m == NMAPS - 1) {   // the tile's dX is complete after this unit's second MMA
                if (ok && !mbar_wait(&dx_full[tb], (it >> 1) & 1)) { ok = false; report_timeout(status, 606); }
                ok = __all_sync(0xffffffffu, ok);
                if (leader) tma_store_wait_read0();     // the staging tile has been read by the previous store
                named_barrier(1, 256);
                if (ok) {
                    tc_fence_after();
                    const uint32_t tx = tmem + 256 + 128 * tb + ((uint32_t)(quarter * 32) << 16) + half * HC;
                    const uint32_t os = smem_u32(smem + Cfg::kOffOut);
#pragma unroll
                    for (int c = 0; c < HC / 16; ++c) {
                        uint32_t r[16];
                        tmem_ld16(tx + 16 * c, r);
                        tmem_ld_wait();
                        const int col = half * HC + 16 * c;
                        uint32_t w[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) w[e] = pack_bf16(__uint_as_float(r[2 * e]), __uint_as_float(r[2 * e + 1]));
                        const uint32_t blk = os + (col >> 6) * kBlk;
                        st_shared_v4(blk + sw128_off(row, (col & 63) >> 3), w[0], w[1], w[2], w[3]);
                        st_shared_v4(blk + sw128_off(row, ((col & 63) >> 3) + 1), w[4], w[5], w[6], w[7]);
                    }
                    tc_fence_before();
                    mbar_arrive(&dx_empty[tb]);
                    fence_proxy_async();
                }
                named_barrier(1, 256);
                if (ok && leader) {
                    for (int bb = 0; bb < DV / 64; ++bb)
                        tma_store_2d(&mapdX, smem + Cfg::kOffOut + bb * kBlk, bb * 64, (int)((t0 + it) * kTileTokens));
                    tma_store_commit();
                }
            }
        }
        if (leader) tma_store_wait_all0();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, 512);
}

template <int DV>
inline hla_status launch_phi_backward(const Dims& D, int BH, const hla_mlp* phi_q, const hla_mlp* phi_k, const void* Q, const void* K, void* dQ,
                                      void* dK, char* ws, const hla_ws_layout& L, int sm_count, LaunchRec& rec) {
    const long long rows = (long long)BH * D.N;
    CUtensorMap mapQ, mapK, mapdQ, mapdK;
    PhiMaps mq, mk;
    PhiBwdPtrs pq{}, pk{};
    if (!make_map_2d(&mapQ, Q, (size_t)rows, DV, kTileTokens) || !make_map_2d(&mapK, K, (size_t)rows, DV, kTileTokens) ||
        !make_map_2d(&mapdQ, dQ, (size_t)rows, DV, kTileTokens) || !make_map_2d(&mapdK, dK, (size_t)rows, DV, kTileTokens))
        return HLA_ERR_CUDA;
    if (!make_map_2d(&mq.w1[0], phi_q->W1, DV, DV, DV)) return HLA_ERR_CUDA;
    mq.w1[1] = mq.w1[0];
    mq.w1[2] = mq.w1[0];
    pq.b1[0] = static_cast<const __nv_bfloat16*>(phi_q->b1);
    pq.W2[0] = static_cast<const __nv_bfloat16*>(phi_q->W2);
    for (int f = 0; f < 3; ++f) {
        if (!make_map_2d(&mk.w1[f], phi_k[f].W1, DV, DV, DV)) return HLA_ERR_CUDA;
        pk.b1[f] = static_cast<const __nv_bfloat16*>(phi_k[f].b1);
        pk.W2[f] = static_cast<const __nv_bfloat16*>(phi_k[f].W2);
    }
    int* status = reinterpret_cast<int*>(ws + L.status);
    if (!set_smem(tc_phi_backward_kernel<DV, 1, false>, PbCfg<DV, 1>::kSmem) || !set_smem(tc_phi_backward_kernel<DV, 3, true>, PbCfg<DV, 3>::kSmem))
        return HLA_ERR_CUDA;
    const long long tiles = (rows + kTileTokens - 1) / kTileTokens;
    const int grid = (int)(tiles < sm_count ? tiles : sm_count);
    cudaStream_t st = rec.st;
    rec.begin("tc_phi_backward");
    tc_phi_backward_kernel<DV, 1, false><<<grid, kPbThreads, PbCfg<DV, 1>::kSmem, st>>>(
        mapQ, mapdQ, mq, pq, reinterpret_cast<const float*>(ws + L.qf), reinterpret_cast<const float*>(ws + L.dqf), rows, D.N, status);
    if (!rec.end()) return HLA_ERR_CUDA;
    rec.begin("tc_phi_backward");
    tc_phi_backward_kernel<DV, 3, true><<<grid, kPbThreads, PbCfg<DV, 3>::kSmem, st>>>(
        mapK, mapdK, mk, pk, reinterpret_cast<const float*>(ws + L.kf), reinterpret_cast<const float*>(ws + L.dkf), rows, D.N, status);
    return rec.end() ? HLA_OK : HLA_ERR_CUDA;
}

inline hla_status phi_backward(const Dims& D, int BH, const hla_mlp* phi_q, const hla_mlp* phi_k, const void* Q, const void* K, void* dQ, void* dK,
                               char* ws, const hla_ws_layout& L, int sm_count, LaunchRec& rec) {
    if (D.d == 128) return launch_phi_backward<128>(D, BH, phi_q, phi_k, Q, K, dQ, dK, ws, L, sm_count, rec);
    return launch_phi_backward<64>(D, BH, phi_q, phi_k, Q, K, dQ, dK, ws, L, sm_count, rec);
}

}  // namespace tc
}  // namespace hla
