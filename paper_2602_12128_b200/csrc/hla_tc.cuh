// Tensor-core (tcgen05 / TMEM / TMA) kernels of the HLA path for bf16,
// F = 3 factors with d_phi = 6 (P = 216 features), d in {64, 128}.
//
//   state build  : C^T[d x P] += V_tile^T[d x 128 tok] * T_k tile[128 tok x P]   (Theorem 4.2, C = T_k (x)_1 V)
//                  T_k rows are formed in registers from the 3 x 6 key features of each token, rounded once to
//                  bf16 and written straight into the swizzled shared-memory operand tile; z = sum_j T_k[j] is
//                  accumulated in fp32 registers on the way.
//   reduce/emit  : sums the split partials in a fixed order, keeps the fp32 state, and emits the readout operand.
//   readout      : T_q[i] = q_i (x) q_i (x) q_i is symmetric, so only its 56 distinct monomials q_a q_b q_c
//                  (a <= b <= c) are formed, against the state folded over index permutations
//                  (Csym[m] = sum over distinct permutations of C[abc]).  One MMA per tile gives
//                  num (d columns) and eta (the extra column holding zsym); o = num / (eta + eps).
#pragma once
#include "../../include/hla.h"
#include "hla_common.cuh"
#include "hla_tc_prim.cuh"

namespace hla {
namespace tc {

constexpr int kTileTokens = 128;
constexpr int kP = 216;          // d_phi^F
constexpr int kNP = 224;         // P rounded up to the MMA's N granularity
constexpr int kMono = 56;        // distinct monomials of degree 3 in 6 variables
constexpr int kMonoPad = 64;
constexpr int kBlk = 16384;      // one 128-row x 128-byte swizzled block

struct Plan {
    size_t b3;     // bf16 [BH][d+16][64]  readout operand: rows g < d: Csym[.][g]; row d: zsym; rest 0
    size_t end;
};

inline bool supported(bool bf16, int d, int F, int dphi) { return bf16 && (d == 64 || d == 128) && F == 3 && dphi == 6; }

inline size_t plan(Plan& p, const Dims& D, int BH, size_t off) {
    auto up = [](size_t x) { return (x + 255) / 256 * 256; };
    p.b3 = off;
    off = up(off + (size_t)BH * (D.d + 16) * kMonoPad * 2);
    p.end = off;
    return off;
}

// ---- host: tensor maps ---------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// bf16 tensor [BH][N][d] (d innermost), box = 64 columns x box_rows tokens of one head, 128-byte swizzle.
inline bool make_map_bhnd(CUtensorMap* m, const void* ptr, int BH, int N, int d, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)N, (cuuint64_t)BH};
    cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)N * d * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
    cuuint32_t es[3] = {1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// bf16 matrix [rows][64], box = 64 x box_rows, 128-byte swizzle.
inline bool make_map_rows64(CUtensorMap* m, const void* ptr, size_t rows, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {64, (cuuint64_t)rows};
    cuuint64_t strides[1] = {128};
    cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    cuuint32_t es[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

__device__ __forceinline__ void report_timeout(int* status, int where) {
    atomicExch(status + kStatusTimeout, 1);
    atomicExch(status + kStatusWhere, where);
}

__device__ __forceinline__ void named_barrier(int id, int nthreads) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory"); }

__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// =======================================================================================
// State build
// =======================================================================================
constexpr int kSbThreads = 320;            // warp 0: TMA, warp 1: MMA, warps 2..9: T_k generators
constexpr int kSbStages = 2;
constexpr int kSbStageBytes = 2 * kBlk + 4 * kBlk;   // V (two 64-column blocks) + T_k (four 64-feature blocks)
constexpr int kSbZHalf0 = 14 * 8;          // features 0..111 belong to the first generator half, 112..215 to the second
constexpr int kSbSmem = 1024 + kSbStages * kSbStageBytes + 8 * kSbZHalf0 * 4 + 256;

// One generator thread: half of the 216 products of one token -> bf16 operand row + fp32 z accumulators.
template <int HALF>
__device__ __forceinline__ void sb_generate(const float (&k)[18], float (&zacc)[kSbZHalf0], uint32_t t_tile, uint32_t row) {
    constexpr int C0 = HALF ? 14 : 0, C1 = HALF ? 27 : 14;
    float k12[36];
#pragma unroll
    for (int ab = 0; ab < 36; ++ab) k12[ab] = k[ab / 6] * k[6 + ab % 6];
#pragma unroll
    for (int c = C0; c < C1; ++c) {
        float t[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int p = 8 * c + e;
            t[e] = k12[p / 6] * k[12 + p % 6];
            zacc[p - 8 * C0] += t[e];
        }
        st_shared_v4(t_tile + (c >> 3) * kBlk + sw128_off(row, c & 7), pack_bf16(t[0], t[1]), pack_bf16(t[2], t[3]),
                     pack_bf16(t[4], t[5]), pack_bf16(t[6], t[7]));
    }
}

__device__ __forceinline__ void sb_load_features(float (&k)[18], const float* __restrict__ kf, int bh, int N, int tok) {
    if (tok < N) {
#pragma unroll
        for (int f = 0; f < 3; ++f) {
            const float2* src = reinterpret_cast<const float2*>(kf + (((size_t)bh * 3 + f) * N + tok) * 6);
            const float2 a = __ldg(src), b = __ldg(src + 1), c = __ldg(src + 2);
            k[6 * f + 0] = a.x; k[6 * f + 1] = a.y; k[6 * f + 2] = b.x; k[6 * f + 3] = b.y; k[6 * f + 4] = c.x; k[6 * f + 5] = c.y;
        }
    } else {
#pragma unroll
        for (int i = 0; i < 18; ++i) k[i] = 0.f;
    }
}

template <int DV>
__global__ void __launch_bounds__(kSbThreads, 1) tc_state_build_kernel(const __grid_constant__ CUtensorMap mapV, const float* __restrict__ kf,
                                                                       float* __restrict__ part, int N, int S, int ld, int* status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    float* zred = reinterpret_cast<float*>(smem + kSbStages * kSbStageBytes);          // [8 warps][112]
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kSbStages * kSbStageBytes + 8 * kSbZHalf0 * 4);
    uint64_t* full_v = bars;            // [2]
    uint64_t* full_t = bars + 2;        // [2]
    uint64_t* empty = bars + 4;         // [2]
    uint64_t* acc_done = bars + 6;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 7);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int s = blockIdx.x, bh = blockIdx.y;
    const int tiles = (N + kTileTokens - 1) / kTileTokens;
    const int tiles_per = (tiles + S - 1) / S;
    const int tile0 = s * tiles_per;
    const int ntiles = max(0, min(tiles, tile0 + tiles_per) - tile0);
    float* out = part + ((size_t)bh * S + s) * kP * ld;

    if (ntiles == 0) {   // an empty split contributes zeros
        for (int i = tid; i < kP * ld; i += kSbThreads) out[i] = 0.f;
        return;
    }

    // zero what the generators never write: feature columns 216..223 of each T_k tile, and for d = 64 the
    // second V block (rows 64..127 of the MMA's M dimension read it)
    for (int st = 0; st < kSbStages; ++st) {
        uint8_t* tt = smem + st * kSbStageBytes + 2 * kBlk;
        for (int r = tid; r < kTileTokens; r += kSbThreads) *reinterpret_cast<uint4*>(tt + 3 * kBlk + sw128_off(r, 3)) = make_uint4(0, 0, 0, 0);
        if (DV == 64) {
            uint4* vz = reinterpret_cast<uint4*>(smem + st * kSbStageBytes + kBlk);
            for (int i = tid; i < kBlk / 16; i += kSbThreads) vz[i] = make_uint4(0, 0, 0, 0);
        }
    }
    fence_proxy_async();
    if (tid == 0) {
        for (int i = 0; i < kSbStages; ++i) {
            mbar_init(&full_v[i], 1);
            mbar_init(&full_t[i], 256);
            mbar_init(&empty[i], 1);
        }
        mbar_init(acc_done, 1);
        fence_mbar_init();
        prefetch_tmap(&mapV);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, 256);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    bool ok = true;

    if (warp == 0) {
        if (lane == 0) {
            for (int it = 0; it < ntiles && ok; ++it) {
                const int st = it & 1, u = it >> 1;
                ok = mbar_wait(&empty[st], (u & 1) ^ 1);
                if (!ok) { report_timeout(status, 101); break; }
                uint8_t* vs = smem + st * kSbStageBytes;
                mbar_arrive_expect_tx(&full_v[st], DV * kTileTokens * 2);
                for (int b = 0; b < DV / 64; ++b) tma_load_3d(vs + b * kBlk, &mapV, &full_v[st], b * 64, (tile0 + it) * kTileTokens, bh);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = idesc_bf16(128, kNP, true, true);
            for (int it = 0; it < ntiles && ok; ++it) {
                const int st = it & 1, u = it >> 1;
                ok = mbar_wait(&full_v[st], u & 1) && mbar_wait(&full_t[st], u & 1);
                if (!ok) { report_timeout(status, 102); break; }
                tc_fence_after();
                const uint32_t va = smem_u32(smem + st * kSbStageBytes), ta = va + 2 * kBlk;
#pragma unroll
                for (int ks = 0; ks < kTileTokens / 16; ++ks)
                    umma_bf16(tmem, smem_desc_sw128(va + ks * 2048, kBlk, 1024), smem_desc_sw128(ta + ks * 2048, kBlk, 1024), idesc,
                              (it > 0 || ks > 0) ? 1u : 0u);
                umma_commit(&empty[st]);
            }
            umma_commit(acc_done);
        }
    } else {
        const int gi = tid - 64;
        const int row = gi & 127, half = gi >> 7;
        float zacc[kSbZHalf0];
#pragma unroll
        for (int i = 0; i < kSbZHalf0; ++i) zacc[i] = 0.f;
        float kcur[18], knext[18];
        sb_load_features(knext, kf, bh, N, tile0 * kTileTokens + row);
        for (int it = 0; it < ntiles; ++it) {
            const int st = it & 1, u = it >> 1;
#pragma unroll
            for (int i = 0; i < 18; ++i) kcur[i] = knext[i];
            if (it + 1 < ntiles) sb_load_features(knext, kf, bh, N, (tile0 + it + 1) * kTileTokens + row);
            if (ok) {
                ok = mbar_wait(&empty[st], (u & 1) ^ 1);
                if (!ok) report_timeout(status, 103);
            }
            if (ok) {
                const uint32_t ta = smem_u32(smem + st * kSbStageBytes + 2 * kBlk);
                if (half == 0) sb_generate<0>(kcur, zacc, ta, row);
                else sb_generate<1>(kcur, zacc, ta, row);
                fence_proxy_async();
                mbar_arrive(&full_t[st]);
            }
        }
        // z: sum the per-token-slot accumulators over the 128 slots of this half
#pragma unroll
        for (int i = 0; i < kSbZHalf0; ++i) {
            const float v = warp_sum(zacc[i]);
            if (lane == 0) zred[(warp - 2) * kSbZHalf0 + i] = v;
        }
        named_barrier(1, 256);
        if (gi < kP) {
            const int h = gi >= kSbZHalf0 ? 1 : 0, i = gi - h * kSbZHalf0;
            float z = 0.f;
#pragma unroll
            for (int w = 0; w < 4; ++w) z += zred[(h * 4 + w) * kSbZHalf0 + i];
            out[(size_t)gi * ld + DV] = z;
            for (int c = DV + 1; c < ld; ++c) out[(size_t)gi * ld + c] = 0.f;
        }
        if (warp < 6) {   // warps 2..5 cover the four TMEM lane quarters
            const int quarter = warp & 3;
            if (ok) {
                ok = mbar_wait(acc_done, 0);
                if (!ok && lane == 0) report_timeout(status, 104);
            }
            ok = __all_sync(0xffffffffu, ok);
            tc_fence_after();
            const int g = quarter * 32 + lane;
            if (ok && quarter * 32 < DV) {
#pragma unroll 1
                for (int c = 0; c < kP / 8; ++c) {
                    uint32_t r[8];
                    tmem_ld8(tmem + ((uint32_t)(quarter * 32) << 16) + 8 * c, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 8; ++e) out[(size_t)(8 * c + e) * ld + g] = __uint_as_float(r[e]);
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, 256);
}

// =======================================================================================
// Reduce the split partials, keep the fp32 state, emit the readout operand
// =======================================================================================
template <int DV>
__global__ void __launch_bounds__(256) tc_reduce_emit_kernel(const float* __restrict__ part, float* __restrict__ state,
                                                             __nv_bfloat16* __restrict__ b3, int S, int ld) {
    __shared__ uint8_t perm[kMono][6];
    __shared__ uint8_t nperm[kMono];
    const int bh = blockIdx.x, tid = threadIdx.x;
    const size_t n_per = (size_t)kP * ld;
    float* st = state + (size_t)bh * n_per;
    for (size_t i = tid; i < n_per; i += 256) {
        float a = 0.f;
        for (int s = 0; s < S; ++s) a += part[((size_t)bh * S + s) * n_per + i];
        st[i] = a;
    }
    if (tid < kMono) {
        int m = 0, A = 0, Bq = 0, C = 0;
        for (int a = 0; a < 6; ++a)
            for (int b = a; b < 6; ++b)
                for (int c = b; c < 6; ++c) {
                    if (m == tid) { A = a; Bq = b; C = c; }
                    ++m;
                }
        const int idx[3] = {A, Bq, C};
        const int order[6][3] = {{0, 1, 2}, {0, 2, 1}, {1, 0, 2}, {1, 2, 0}, {2, 0, 1}, {2, 1, 0}};
        int n = 0;
        for (int o = 0; o < 6; ++o) {
            const int p = (idx[order[o][0]] * 6 + idx[order[o][1]]) * 6 + idx[order[o][2]];
            bool seen = false;
            for (int j = 0; j < n; ++j) seen |= (perm[tid][j] == p);
            if (!seen) perm[tid][n++] = (uint8_t)p;
        }
        nperm[tid] = (uint8_t)n;
    }
    __syncthreads();
    __nv_bfloat16* o = b3 + (size_t)bh * (DV + 16) * kMonoPad;
    for (int i = tid; i < (DV + 16) * kMonoPad; i += 256) {
        const int row = i / kMonoPad, m = i % kMonoPad;
        float v = 0.f;
        if (m < kMono && row <= DV) {
            for (int j = 0; j < nperm[m]; ++j) v += st[(size_t)perm[m][j] * ld + row];   // row == DV reads the z column
        }
        o[i] = __float2bfloat16_rn(v);
    }
}

// =======================================================================================
// Readout + normaliser
// =======================================================================================
constexpr int kRoThreads = 288;   // warps 0..3: epilogue, warps 4..7: monomial generators, warp 8: TMA + MMA
template <int DV> struct RoCfg {
    static constexpr int kNmma = DV + 16;
    static constexpr int kB3Bytes = kNmma * 128;
    static constexpr int kOBytes = kTileTokens * DV * 2;
    static constexpr int kOffA = 0;                       // 2 x 16 KB monomial tiles
    static constexpr int kOffB3 = 2 * kBlk;
    static constexpr int kOffO = kOffB3 + ((kB3Bytes + 1023) / 1024) * 1024;   // 2 staging tiles
    static constexpr int kOffBars = kOffO + 2 * kOBytes;
    static constexpr int kSmemUsed = 1024 + kOffBars + 256;
    static constexpr int kSmem = kSmemUsed > 120 * 1024 ? kSmemUsed : 120 * 1024;   // one CTA per SM (it owns all of TMEM)
};

template <int DV>
__global__ void __launch_bounds__(kRoThreads, 1) tc_readout_kernel(const __grid_constant__ CUtensorMap mapB3, const __grid_constant__ CUtensorMap mapO,
                                                                   const float* __restrict__ qf, float* __restrict__ eta_out, int N, int BH,
                                                                   float eps, int* status) {
    using Cfg = RoCfg<DV>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::kOffBars);
    uint64_t* a_full = bars;          // [2] 128 generator arrivals
    uint64_t* a_empty = bars + 2;     // [2] MMA commit
    uint64_t* acc_full = bars + 4;    // [2] MMA commit
    uint64_t* acc_empty = bars + 6;   // [2] 128 epilogue arrivals
    uint64_t* b3_full = bars + 8;
    uint64_t* b3_free = bars + 9;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 10);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 11);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tiles_per_head = (N + kTileTokens - 1) / kTileTokens;
    const long long total = (long long)BH * tiles_per_head;
    const int w0 = (int)(total * blockIdx.x / gridDim.x), w1 = (int)(total * (blockIdx.x + 1) / gridDim.x);
    const int nwork = w1 - w0;

    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(&a_full[i], 128);
            mbar_init(&a_empty[i], 1);
            mbar_init(&acc_full[i], 1);
            mbar_init(&acc_empty[i], 128);
        }
        mbar_init(b3_full, 1);
        mbar_init(b3_free, 1);
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tmap(&mapB3);
        prefetch_tmap(&mapO);
    }
    if (warp == 8) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    bool ok = true;

    if (warp == 8) {
        if (lane == 0) {
            const uint32_t idesc = idesc_bf16(128, Cfg::kNmma, false, false);
            const uint32_t b3a = smem_u32(smem + Cfg::kOffB3);
            int cur_bh = -1, nload = 0;
            for (int it = 0; it < nwork && ok; ++it) {
                const int work = w0 + it, bh = work / tiles_per_head;
                const int ab = it & 1, u = it >> 1;
                if (bh != cur_bh) {
                    if (cur_bh >= 0) {   // every MMA that reads the old state operand must have finished
                        umma_commit(b3_free);
                        ok = mbar_wait(b3_free, (nload - 1) & 1);
                        if (!ok) { report_timeout(status, 201); break; }
                    }
                    mbar_arrive_expect_tx(b3_full, Cfg::kB3Bytes);
                    tma_load_2d(smem + Cfg::kOffB3, &mapB3, b3_full, 0, bh * Cfg::kNmma);
                    ok = mbar_wait(b3_full, nload & 1);
                    if (!ok) { report_timeout(status, 202); break; }
                    ++nload;
                    cur_bh = bh;
                }
                ok = mbar_wait(&a_full[ab], u & 1) && mbar_wait(&acc_empty[ab], (u & 1) ^ 1);
                if (!ok) { report_timeout(status, 203); break; }
                tc_fence_after();
                const uint32_t aa = smem_u32(smem + Cfg::kOffA + ab * kBlk);
#pragma unroll
                for (int ks = 0; ks < kMonoPad / 16; ++ks)
                    umma_bf16(tmem + ab * 256, smem_desc_sw128(aa + ks * 32, 16, 1024), smem_desc_sw128(b3a + ks * 32, 16, 1024), idesc,
                              ks > 0 ? 1u : 0u);
                umma_commit(&a_empty[ab]);
                umma_commit(&acc_full[ab]);
            }
        }
    } else if (warp >= 4) {
        const int row = tid - 128;
        float q[6], qn[6];
        auto load_q = [&](float (&dst)[6], int work) {
            const int bh = work / tiles_per_head, tok = (work % tiles_per_head) * kTileTokens + row;
            if (tok < N) {
                const float2* src = reinterpret_cast<const float2*>(qf + ((size_t)bh * N + tok) * 6);
                const float2 a = __ldg(src), b = __ldg(src + 1), c = __ldg(src + 2);
                dst[0] = a.x; dst[1] = a.y; dst[2] = b.x; dst[3] = b.y; dst[4] = c.x; dst[5] = c.y;
            } else {
#pragma unroll
                for (int i = 0; i < 6; ++i) dst[i] = 0.f;
            }
        };
        if (nwork > 0) load_q(qn, w0);
        for (int it = 0; it < nwork; ++it) {
            const int ab = it & 1, u = it >> 1;
#pragma unroll
            for (int i = 0; i < 6; ++i) q[i] = qn[i];
            if (it + 1 < nwork) load_q(qn, w0 + it + 1);
            if (ok) {
                ok = mbar_wait(&a_empty[ab], (u & 1) ^ 1);
                if (!ok) report_timeout(status, 204);
            }
            if (!ok) continue;
            // the 56 monomials q_a q_b q_c, a <= b <= c, in lexicographic order of (a, b, c)
            float mono[kMonoPad];
            {
                int m = 0;
#pragma unroll
                for (int a = 0; a < 6; ++a)
#pragma unroll
                    for (int b = a; b < 6; ++b) {
                        const float qab = q[a] * q[b];
#pragma unroll
                        for (int c = b; c < 6; ++c) mono[m++] = qab * q[c];
                    }
#pragma unroll
                for (; m < kMonoPad; ++m) mono[m] = 0.f;
            }
            const uint32_t aa = smem_u32(smem + Cfg::kOffA + ab * kBlk);
#pragma unroll
            for (int c = 0; c < 8; ++c)
                st_shared_v4(aa + sw128_off(row, c), pack_bf16(mono[8 * c], mono[8 * c + 1]), pack_bf16(mono[8 * c + 2], mono[8 * c + 3]),
                             pack_bf16(mono[8 * c + 4], mono[8 * c + 5]), pack_bf16(mono[8 * c + 6], mono[8 * c + 7]));
            fence_proxy_async();
            mbar_arrive(&a_full[ab]);
        }
    } else {
        const int row = tid;   // TMEM lane = token row of the tile
        for (int it = 0; it < nwork; ++it) {
            const int work = w0 + it, bh = work / tiles_per_head, tile = work % tiles_per_head;
            const int ab = it & 1, u = it >> 1;
            if (!mbar_wait(&acc_full[ab], u & 1)) {
                report_timeout(status, 205);
                *abort_flag = 1;
            }
            named_barrier(3, 128);                     // every epilogue thread arrives, timed out or not
            if (*abort_flag) break;                    // uniform across the four warps
            tc_fence_after();
            const uint32_t ta = tmem + ab * 256 + ((uint32_t)(warp * 32) << 16);
            uint32_t r[16];
            tmem_ld16(ta + DV, r);
            tmem_ld_wait();
            const float eta = __uint_as_float(r[0]);
            const float rinv = 1.f / (eta + eps);
            // the staging tile of two tiles ago must have been read by its TMA store
            if (tid == 0) tma_store_wait_read1();
            named_barrier(2, 128);
            const uint32_t os = smem_u32(smem + Cfg::kOffO + ab * Cfg::kOBytes);
#pragma unroll
            for (int c = 0; c < DV / 16; ++c) {
                tmem_ld16(ta + 16 * c, r);
                tmem_ld_wait();
                uint32_t w[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) w[e] = pack_bf16(__uint_as_float(r[2 * e]) * rinv, __uint_as_float(r[2 * e + 1]) * rinv);
                const uint32_t blk = os + (c >> 2) * kBlk;
                st_shared_v4(blk + sw128_off(row, (2 * c) & 7), w[0], w[1], w[2], w[3]);
                st_shared_v4(blk + sw128_off(row, (2 * c + 1) & 7), w[4], w[5], w[6], w[7]);
            }
            tc_fence_before();
            mbar_arrive(&acc_empty[ab]);
            fence_proxy_async();
            named_barrier(2, 128);
            if (tid == 0) {
                for (int b = 0; b < DV / 64; ++b) tma_store_3d(&mapO, smem + Cfg::kOffO + ab * Cfg::kOBytes + b * kBlk, b * 64, tile * kTileTokens, bh);
                tma_store_commit();
            }
            const int tok = tile * kTileTokens + row;
            if (tok < N) eta_out[(size_t)bh * N + tok] = eta;
        }
        if (tid == 0) tma_store_wait_all0();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 8) tmem_dealloc(tmem, 512);
}

// ---- host launch helpers ---------------------------------------------------------------
template <int DV>
inline hla_status launch_core_forward(const Plan& P, const Dims& D, int BH, const float* qf, const float* kf, const void* V, void* O, char* ws,
                                      const hla_ws_layout& L, size_t off_part, int sm_count, LaunchRec& rec) {
    CUtensorMap mapV, mapO, mapB3;
    __nv_bfloat16* b3 = reinterpret_cast<__nv_bfloat16*>(ws + P.b3);
    if (!make_map_bhnd(&mapV, V, BH, D.N, DV, kTileTokens) || !make_map_bhnd(&mapO, O, BH, D.N, DV, kTileTokens) ||
        !make_map_rows64(&mapB3, b3, (size_t)BH * (DV + 16), DV + 16))
        return HLA_ERR_CUDA;
    int* status = reinterpret_cast<int*>(ws + L.status);
    float* part = reinterpret_cast<float*>(ws + off_part);
    float* state = reinterpret_cast<float*>(ws + L.state);
    float* eta = reinterpret_cast<float*>(ws + L.eta);

    static bool attr_done = false;
    if (!attr_done) {
        if (cudaFuncSetAttribute(tc_state_build_kernel<DV>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSbSmem) != cudaSuccess) return HLA_ERR_CUDA;
        if (cudaFuncSetAttribute(tc_readout_kernel<DV>, cudaFuncAttributeMaxDynamicSharedMemorySize, RoCfg<DV>::kSmem) != cudaSuccess) return HLA_ERR_CUDA;
        attr_done = true;
    }
    cudaStream_t st = rec.st;
    rec.begin("tc_state_build");
    tc_state_build_kernel<DV><<<dim3(D.S, BH), kSbThreads, kSbSmem, st>>>(mapV, kf, part, D.N, D.S, D.ld, status);
    if (!rec.end()) return HLA_ERR_CUDA;
    rec.begin("tc_reduce_emit");
    tc_reduce_emit_kernel<DV><<<BH, 256, 0, st>>>(part, state, b3, D.S, D.ld);
    if (!rec.end()) return HLA_ERR_CUDA;
    const int tiles = (D.N + kTileTokens - 1) / kTileTokens;
    const long long total = (long long)BH * tiles;
    const int grid = (int)(total < sm_count ? total : sm_count);
    rec.begin("tc_readout");
    tc_readout_kernel<DV><<<grid, kRoThreads, RoCfg<DV>::kSmem, st>>>(mapB3, mapO, qf, eta, D.N, BH, D.eps, status);
    return rec.end() ? HLA_OK : HLA_ERR_CUDA;
}

inline hla_status core_forward(const Plan& P, const Dims& D, int BH, const float* qf, const float* kf, const void* V, void* O, char* ws,
                               const hla_ws_layout& L, size_t off_part, int sm_count, LaunchRec& rec) {
    if (D.d == 128) return launch_core_forward<128>(P, D, BH, qf, kf, V, O, ws, L, off_part, sm_count, rec);
    return launch_core_forward<64>(P, D, BH, qf, kf, V, O, ws, L, off_part, sm_count, rec);
}

}  // namespace tc
}  // namespace hla
