// Tensor-core building blocks of the feature networks phi (appendix "Defining phi";
// Algorithm 1 step 4) for bf16:  feat = ReLU(W2^T GELU(W1^T x + b1) + b2), and their backward.
//
// Forward, per 128-token tile of X (Q or K, TMA-loaded once) and per map m - the pipeline the fused key-side and
// query-side kernels of the forward (hla_tc_fused_k.cuh, hla_tc_fused.cuh) run:
//   D1 = X * W1[m] + b1       tcgen05, fp32 in TMEM        [128 tok x d hidden]; the bias is a ninth K step
//   G  = bf16(GELU(D1))       16 warps, thread = (token, quarter of the hidden units); written as the next MMA's A operand
//   D2 = G * W2[m]            tcgen05, N padded to 16
//   feat = ReLU(D2 + b2)      fp32 features
// The key side runs its F maps on the same X tile, so K is read once.  This file holds the GELU / GELU' arithmetic and
// the backward kernel.
// GELU is the exact erf form, x Phi(x), with Phi evaluated as 1/2 + tanh(x (a + b x^2)) / 2 (a, b fitted to erf; one
// tanh.approx per hidden unit) - total error of Phi below 4e-4, several times below the bf16 rounding of G.
#pragma once
#include "hla_tc.cuh"

namespace hla {
namespace tc {

// Arithmetic on pairs uses the packed fp32 instructions (fma.rn.f32x2 and friends), which halve the issue slots.
__device__ __forceinline__ float2 splat2(float v) { return make_float2(v, v); }
__device__ __forceinline__ float tanh_approx(float x) {
    float y;
    asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// GELU(x) = x Phi(x) through the special-function unit: Phi(x) = 1/2 + tanh(x (a + b x^2)) / 2 with a, b fitted to the erf
// form (|Phi error| < 1.5e-4 before the 2^-11 relative error of tanh.approx).  A polynomial Phi kept the FMA pipe busier
// and was slower; the special-function pipe is otherwise idle.  The kernels form 2 GELU(x) = x + x tanh(..) and stage the
// second-layer weights halved (exact in bf16), which saves the multiplication by 1/2.
__device__ __forceinline__ float2 gelu2_twice(float2 x) {
    const float2 t = __fmul2_rn(x, x);
    const float2 u = __fmul2_rn(x, __ffma2_rn(t, splat2(0.0352821f), splat2(0.79880136f)));
    return __ffma2_rn(x, make_float2(tanh_approx(u.x), tanh_approx(u.y)), x);
}
__device__ __forceinline__ __nv_bfloat16 half_bf16(__nv_bfloat16 w) { return __float2bfloat16_rn(0.5f * __bfloat162float(w)); }
// GELU'(x) = Phi(x) + x pdf(x) through one tanh.approx per element:
//   th = tanh(x (a + b x^2)),   2 GELU'(x) ~ (1 + th) (1 + V (1 - th)) = 1 + V + th (1 - V th),   V = x (C0 + C1 x^2) / 2
// (the derivative of a tanh-form GELU whose inner derivative is a free polynomial); a, b, C0, C1 are fitted against the
// exact derivative (fit_gelu_tanh.py: |error| < 1.5e-4 before the 2^-11 relative error of tanh.approx, < 1.3e-3 with
// it).  The kernel evaluates it with -V (negated constants) so that every step is one packed multiply or fma, and the
// factor 1/2 sits in the staged W2^T of the dg product (exact in bf16): 9 packed + 2 special-function instructions
// per pair of elements; the polynomial Phi plus exp form needed sixteen.
__device__ __forceinline__ float2 gelu_grad2_twice(float2 x) {
    const float2 t = __fmul2_rn(x, x);
    const float2 u = __fmul2_rn(x, __ffma2_rn(t, splat2(0.02936904f), splat2(0.69631102f)));
    const float2 th = make_float2(tanh_approx(u.x), tanh_approx(u.y));
    const float2 vn = __fmul2_rn(x, __ffma2_rn(t, splat2(0.010848315f), splat2(-0.89902785f)));   // -V
    const float2 a1 = __ffma2_rn(vn, th, splat2(1.f));          // 1 - V th
    const float2 b1 = __ffma2_rn(th, a1, splat2(1.f));          // 1 + th (1 - V th)
    return __ffma2_rn(vn, splat2(-1.f), b1);                    // + V
}

// 2 GELU(x) and 2 GELU'(x) of the same elements through ONE tanh.approx each (the weight gradients need both): the tanh
// of the forward's form, th = tanh(x (a + b x^2)), and the derivative form above with only C0, C1 fitted to it
// (fit_gelu_tanh.py: |GELU' error| < 5.2e-4 instead of 1.5e-4 - still an order below the bf16 rounding of dh).  V grows to
// 27 at |x| = 6 with these constants, so the form relies on tanh.approx being accurate near saturation: measured on B200 its
// absolute error stays below 8e-6 on [-6, 6] (its documented bound, 2^-11 relative, would allow 1.4e-2 in GELU' there).
__device__ __forceinline__ void gelu_both2_twice(float2 x, float2& g2, float2& grad2) {
    const float2 t = __fmul2_rn(x, x);
    const float2 u = __fmul2_rn(x, __ffma2_rn(t, splat2(0.0352821f), splat2(0.79880136f)));
    const float2 th = make_float2(tanh_approx(u.x), tanh_approx(u.y));
    g2 = __ffma2_rn(x, th, x);
    const float2 vn = __fmul2_rn(x, __ffma2_rn(t, splat2(-0.104597145f), splat2(-0.800572795f)));   // -V, V = x (C0 + C1 x^2) / 2
    const float2 a1 = __ffma2_rn(vn, th, splat2(1.f));          // 1 - V th
    const float2 b1 = __ffma2_rn(th, a1, splat2(1.f));          // 1 + th (1 - V th)
    grad2 = __ffma2_rn(vn, splat2(-1.f), b1);                   // + V
}

struct PhiPtrs {
    const __nv_bfloat16* b1[3];
    const __nv_bfloat16* W2[3];
    const __nv_bfloat16* b2[3];
};
struct PhiMaps {
    CUtensorMap w1[3];
};

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
struct PhiBwdPtrs {
    const __nv_bfloat16* b1[3];
    const __nv_bfloat16* W2[3];
};

// warp 0: TMA loads, warp 1: dg and dX MMAs, warp 2: h MMAs, warps 3..18: epilogue (thread = token row x quarter of the columns),
// warps 19..22: dp tiles (thread = token row).  The dp tiles were written by the epilogue threads at first; per unit that
// cost each of the sixteen epilogue warps, whose instruction stream is what bounds the kernel, 600 of its 2850 cycles
// (two loads, the split into two bf16 halves, two 4-byte stores, and above all one proxy fence per thread).
// Warps 23..26: drain of the dX accumulator (thread = token row): TMEM -> bf16 -> swizzled staging tile -> TMA store.  It
// ran on the epilogue warps at first (557 of their cycles per unit on the key side, a third of a unit on the query side).
constexpr int kPbThreads = 864;
constexpr int kPbEpiWarp0 = 3, kPbDpWarp0 = 19, kPbDrainWarp0 = 23;

// DP = d_phi: 6 (F = 3) or 12 (F = 2).  The dp tile of a unit is [dp_hi | dp_lo] = 2 DP K columns: one K = 16 step for DP = 6 (two
// tiles share one swizzled block at K columns 0..15 and 16..31), two steps for DP = 12 (one block per tile, K columns 0..23).
template <int DV, int NMAPS, int DP> struct PbCfg {
    static constexpr int kXStages = 2;
    static constexpr int kXBytes = kTileTokens * DV * 2;
    static constexpr int kW1Bytes = DV * DV * 2;
    static constexpr int kDgSteps = DP == 6 ? 1 : 2;             // K = 16 steps of the dg product
    static constexpr int kW2tBlock = kDgSteps * 2048;            // [16 kDgSteps K rows][64 hidden] bf16
    static constexpr int kW2tBytes = (DV / 64) * kW2tBlock;      // per map: MN-major B operand of the dg product
    static constexpr int kDpBlocks = DP == 6 ? 1 : 2;
    static constexpr int kOffX = 0;
    static constexpr int kOffW1 = kXStages * kXBytes;            // (the dh tiles live in TMEM)
    static constexpr int kOffDp = kOffW1 + NMAPS * kW1Bytes;     // dp tiles (see above)
    static constexpr int kOffW2t = kOffDp + kDpBlocks * kBlk;
    // b1 is added on the tensor cores by a ninth K step of the h product: A = K columns 32..47 of the first dp block (column
    // 44 is a constant 1, never written again; the dp tiles use lower columns), B = the last K step of the map's W2^T
    // tile, whose row 12 holds b1 (the rows from 2 DP on meet zero columns of the dp tiles in the dg product, so they are free there)
    static constexpr int kB1Row = 12;
    // dX staging tile (128 x DV) for the TMA store of the drain
    static constexpr int kStageBlocks = DV / 64;
    static constexpr int kOffStage = kOffW2t + NMAPS * kW2tBytes;
    static constexpr int kOffBars = kOffStage + kStageBlocks * kBlk;
    static constexpr int kSmemUsed = 1024 + kOffBars + 256;
    static_assert(kSmemUsed <= 227 * 1024, "shared memory");
    static constexpr int kSmem = kSmemUsed > 120 * 1024 ? kSmemUsed : 120 * 1024;   // one CTA per SM (512 TMEM columns)
};

// X, dX [rows][DV] bf16.  KSIDE: feat / dfeat are [bh][NMAPS][N][6], else [rows][6].
// Per unit (one map of one 128-token tile) three products run on the tensor cores:
//   h  = X * W1                         [128 x DV], K = DV
//   dg = [dp_hi | dp_lo] * [W2^T; W2^T]  [128 x DV], K = 16: dp = dfeat (.) 1[feat > 0] split into two bf16 halves, so dg is exact to ~2^-17
//   dX += dh * W1^T                     [128 x DV], K = DV,  dh = dg (.) GELU'(h + b1) formed by the 16 epilogue warps
// h and the dh tile are double-buffered; dg is taken into registers at the start of a unit so that the next unit's dg
// product overlaps this unit's arithmetic; the dX accumulator of a tile is drained one unit late, straight from
// registers to global memory.  The epilogue threads also write the dp tiles (one feature pair each, one unit ahead).
template <int DV, int NMAPS, bool KSIDE, int DP>
__global__ void __launch_bounds__(kPbThreads, 1) tc_phi_backward_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ PhiMaps maps,
                                                                        const __grid_constant__ CUtensorMap mapdX, PhiBwdPtrs P,
                                                                        const float* __restrict__ feat, const float* __restrict__ dfeat,
                                                                        __nv_bfloat16* __restrict__ dX, long long rows, int N, int* status) {
    using Cfg = PbCfg<DV, NMAPS, DP>;
    constexpr int HC = DV / 4;
    constexpr int XST = Cfg::kXStages;
    extern __shared__ uint8_t smem_raw[];
    grid_launch_dependents();
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::kOffBars);
    uint64_t* x_full = bars;           // [2]
    uint64_t* x_empty = bars + 2;      // [2] MMA commit
    uint64_t* h_full = bars + 4;       // [2] MMA commit
    uint64_t* dh_full = bars + 8;      // [2] 512 arrivals
    uint64_t* dh_free = bars + 10;     // [2] MMA commit
    uint64_t* dp_full = bars + 12;     // [2] 128 arrivals
    uint64_t* dp_free = bars + 28;     // [2] MMA commit: the dg product that read the slot has completed
    uint64_t* dg_full = bars + 20;     // MMA commit
    uint64_t* dg_empty = bars + 21;    // 512 arrivals
    uint64_t* dx_full = bars + 22;     // MMA commit
    uint64_t* dx_empty = bars + 23;    // 128 arrivals
    uint64_t* w_full = bars + 24;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 25);
    uint64_t* stage_free = bars + 26;  // 1 arrival: the previous TMA store has read the dX staging tile
    uint64_t* stage_full = bars + 27;  // 128 arrivals: the staging tile of this drain is written

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const long long tiles = (rows + kTileTokens - 1) / kTileTokens;
    const long long t0 = tiles * blockIdx.x / gridDim.x, t1 = tiles * (blockIdx.x + 1) / gridDim.x;
    const int ntiles = (int)(t1 - t0);
    const int nunits = ntiles * NMAPS;

    // W2^T stacked twice (rows 0..DP-1 meet dp_hi, rows DP..2DP-1 meet dp_lo, the rest is zero but for b1), as an MN-major operand
    constexpr int kRows = 16 * Cfg::kDgSteps, kB1Abs = kRows - 16 + Cfg::kB1Row;
    for (int i = tid; i < NMAPS * kRows * DV; i += kPbThreads) {
        const int m = i / (kRows * DV), k = (i / DV) % kRows, j = i % DV;
        uint8_t* base = smem + Cfg::kOffW2t + m * Cfg::kW2tBytes + (j >> 6) * Cfg::kW2tBlock;
        *reinterpret_cast<__nv_bfloat16*>(base + sw128_off(k, (j & 63) >> 3) + (j & 7) * 2) =
            k < 2 * DP ? half_bf16(P.W2[m][j * DP + (k % DP)]) : (k == kB1Abs ? P.b1[m][j] : __float2bfloat16_rn(0.f));
    }
    for (int i = tid; i < Cfg::kDpBlocks * kBlk / 16; i += kPbThreads) reinterpret_cast<uint4*>(smem + Cfg::kOffDp)[i] = make_uint4(0, 0, 0, 0);
    __syncthreads();
    for (int i = tid; i < kTileTokens; i += kPbThreads)      // K column 32 + kB1Row of the dp block
        *reinterpret_cast<__nv_bfloat16*>(smem + Cfg::kOffDp + sw128_off(i, 4 + Cfg::kB1Row / 8) + (Cfg::kB1Row & 7) * 2) = __float2bfloat16_rn(1.f);
    fence_proxy_async();
    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(&x_full[i], 1);
            mbar_init(&x_empty[i], 1);
            mbar_init(&h_full[i], 1);
            mbar_init(&dh_full[i], 512);
            mbar_init(&dh_free[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&dp_full[i], 128);
            mbar_init(&dp_free[i], 1);
        }
        mbar_init(dg_full, 1);
        mbar_init(dg_empty, 512);
        mbar_init(dx_full, 1);
        mbar_init(dx_empty, 128);
        mbar_init(w_full, 1);
        mbar_init(stage_free, 1);
        mbar_init(stage_full, 128);
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
    const uint32_t tmem = *tmem_slot;     // h[b] at columns 128*b, dg at 256, dX at 384
    grid_dependency_wait();
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
    } else if (warp == 2) {
        if (lane == 0 && ntiles > 0) {      // h[b] = X * W1[m]
            const uint32_t idesc1 = idesc_bf16(128, DV, false, true);    // X K-major, W1 [in][hidden] MN-major
            const uint64_t xd0 = smem_desc_sw128(smem_u32(smem + Cfg::kOffX), 16, 1024);
            const uint64_t wd0 = smem_desc_sw128(smem_u32(smem + Cfg::kOffW1), DV * 128, 1024);
            const uint64_t od = smem_desc_sw128(smem_u32(smem + Cfg::kOffDp) + 64, 16, 1024);
            const uint64_t bd0 = smem_desc_sw128(smem_u32(smem + Cfg::kOffW2t) + (Cfg::kDgSteps - 1) * 2048, Cfg::kW2tBlock, 1024);      // the K step with the b1 row
            bool good = mbar_wait(w_full, 0);
            for (int unit = 0; unit < nunits && good; ++unit) {
                const int it = unit / NMAPS, m = unit % NMAPS, st = it % XST, b = unit & 1;
                if (m == 0 && !mbar_wait(&x_full[st], (it / XST) & 1)) { good = false; break; }
                // h[b] also holds the dh operand of unit - 2 (written over the h columns that were read): it is free when
                // that unit's dX product has completed
                if (!mbar_wait(&dh_free[b], ((unit >> 1) & 1) ^ 1)) { good = false; break; }
                // One map per tile: dg of this unit must be complete too, so that h_full tells the epilogue warps both (one
                // wait per unit on their instruction stream instead of two).  Several maps per tile: the chain dX(unit - 2)
                // -> h(unit) -> GELU'(unit) sets the pace, and a wait for dg here would put the issue of dg(unit), which
                // follows the issue of dX(unit - 2) on the other thread, into that chain as well; the epilogue warps wait
                // for dg themselves (measured: key side 7 % faster, query side 7 % slower without this wait).
                if (NMAPS == 1 && !mbar_wait(dg_full, unit & 1)) { good = false; break; }
                tc_fence_after();
                const uint64_t xd = desc_advance(xd0, st * Cfg::kXBytes), wd = desc_advance(wd0, m * Cfg::kW1Bytes);
#pragma unroll
                for (int ks = 0; ks < DV / 16; ++ks)
                    umma_bf16(tmem + 128 * b, desc_advance(xd, (ks >> 2) * kBlk + (ks & 3) * 32), desc_advance(wd, ks * 2048), idesc1, ks > 0 ? 1u : 0u);
                umma_bf16(tmem + 128 * b, od, desc_advance(bd0, m * Cfg::kW2tBytes), idesc1, 1u);      // + 1 * b1
                umma_commit(&h_full[b]);
                if (m == NMAPS - 1) umma_commit(&x_empty[st]);
            }
            if (!good) report_timeout(status, 602);
        }
    } else if (warp == 1) {
        if (lane == 0 && ntiles > 0) {
            const uint32_t idesc_dg = idesc_bf16(128, DV, false, true);  // dg = dp (K-major) * W2^T (MN-major)
            const uint32_t idesc2 = idesc_bf16(128, DV, false, false);   // dX = dh (TMEM) * W1 as [in][hidden] (K-major)
            const uint64_t pd0 = smem_desc_sw128(smem_u32(smem + Cfg::kOffDp), 16, 1024);
            const uint64_t vd0 = smem_desc_sw128(smem_u32(smem + Cfg::kOffW2t), Cfg::kW2tBlock, 1024);
            const uint64_t wd0 = smem_desc_sw128(smem_u32(smem + Cfg::kOffW1), 16, 1024);
            bool good = mbar_wait(w_full, 0);
            // dg of `unit`; the epilogue of unit - 1 must have taken its dg into registers
            auto issue_dg = [&](int unit) -> bool {
                const int m = unit % NMAPS, slot = unit & 1;
                if (unit > 0 && !mbar_wait(dg_empty, (unit - 1) & 1)) return false;
                if (!mbar_wait(&dp_full[slot], (unit >> 1) & 1)) return false;
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < Cfg::kDgSteps; ++ks)      // the slot's K columns: 16 slot.. (DP = 6, one block), or block `slot` (DP = 12)
                    umma_bf16(tmem + 256, desc_advance(pd0, (DP == 6 ? slot * 32 : slot * kBlk) + ks * 32), desc_advance(vd0, m * Cfg::kW2tBytes + ks * 2048), idesc_dg,
                              ks > 0 ? 1u : 0u);
                umma_commit(dg_full);
                umma_commit(&dp_free[slot]);
                return true;
            };
            if (good && nunits > 0) good = issue_dg(0);
            for (int unit = 0; unit < nunits && good; ++unit) {
                const int it = unit / NMAPS, m = unit % NMAPS, b = unit & 1;
                if (unit + 1 < nunits && !issue_dg(unit + 1)) { good = false; break; }
                if (!mbar_wait(&dh_full[b], (unit >> 1) & 1)) { good = false; break; }
                if (m == 0 && !mbar_wait(dx_empty, (it & 1) ^ 1)) { good = false; break; }
                tc_fence_after();
                const uint64_t wd = desc_advance(wd0, m * Cfg::kW1Bytes);
                // hidden units 16 ks .. 16 ks + 15 were written by the threads of part (16 ks) / HC as 8 packed columns
                // at the start of their own column range plus ((16 ks) % HC) / 2
#pragma unroll
                for (int ks = 0; ks < DV / 16; ++ks)
                    umma_bf16_ta(tmem + 384, tmem + 128 * b + ((16 * ks) / HC) * HC + ((16 * ks) % HC) / 2,
                                 desc_advance(wd, (ks >> 2) * (DV * 128) + (ks & 3) * 32), idesc2, (m > 0 || ks > 0) ? 1u : 0u);
                umma_commit(&dh_free[b]);
                if (m == NMAPS - 1) umma_commit(dx_full);
            }
            if (!good) report_timeout(status, 603);
        }
    } else if (warp >= kPbDrainWarp0) {
        // dX of a tile: TMEM -> bf16 -> swizzled staging tile -> TMA store (rows past the end are clipped by the store).
        // The two hand-overs around the staging tile go through mbarriers with bounded waits, so a warp that has given up
        // elsewhere cannot leave the others waiting for ever.
        const int quarter = warp & 3, row = quarter * 32 + lane;
        const uint32_t tx = tmem + 384 + ((uint32_t)(quarter * 32) << 16);
        const uint32_t sbase = smem_u32(smem + Cfg::kOffStage);
        const bool leader = tid == kPbDrainWarp0 * 32;
        for (int it = 0; it < ntiles; ++it) {
            if (ok && !mbar_wait(dx_full, it & 1)) { ok = false; report_timeout(status, 606); }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            if (leader) {
                tma_store_wait_read0();      // the previous tile's store has read the staging tile
                mbar_arrive(stage_free);
            }
#pragma unroll 1
            for (int h = 0; h < DV / 32; ++h) {
                uint32_t r[32];
                tmem_ld16(tx + 32 * h, *reinterpret_cast<uint32_t(*)[16]>(r));
                tmem_ld16(tx + 32 * h + 16, *reinterpret_cast<uint32_t(*)[16]>(r + 16));
                tmem_ld_wait();
                if (h == DV / 32 - 1) {
                    tc_fence_before();
                    mbar_arrive(dx_empty);          // the accumulator has been read
                }
                if (h == 0) {
                    if (!mbar_wait(stage_free, it & 1)) { ok = false; report_timeout(status, 609); }
                    ok = __all_sync(0xffffffffu, ok);
                }
                if (ok) {
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        st_shared_v4(sbase + (h >> 1) * kBlk + sw128_off(row, 4 * (h & 1) + c), pack_bf16(__uint_as_float(r[8 * c]), __uint_as_float(r[8 * c + 1])),
                                     pack_bf16(__uint_as_float(r[8 * c + 2]), __uint_as_float(r[8 * c + 3])),
                                     pack_bf16(__uint_as_float(r[8 * c + 4]), __uint_as_float(r[8 * c + 5])),
                                     pack_bf16(__uint_as_float(r[8 * c + 6]), __uint_as_float(r[8 * c + 7])));
                }
            }
            if (!ok) break;
            fence_proxy_async();
            mbar_arrive(stage_full);
            if (leader) {
                if (mbar_wait(stage_full, it & 1)) {
                    for (int blk = 0; blk < Cfg::kStageBlocks; ++blk)
                        tma_store_2d(&mapdX, smem + Cfg::kOffStage + blk * kBlk, blk * 64, (int)((t0 + it) * kTileTokens));
                    tma_store_commit();
                } else {
                    report_timeout(status, 610);
                }
            }
        }
        if (leader) tma_store_wait_all0();
    } else if (warp >= kPbDpWarp0) {
        // dp = dfeat (.) 1[feat > 0] of one token row as the A operand [dp_hi | dp_lo] of the dg product: the two bf16 halves
        // of every value, so that dg is exact to ~2^-17.  DP = 6: the two slots share one block (K columns 16 slot ..);
        // DP = 12: one block per slot.  The producer runs up to two units ahead of the dg products.
        const int row = tid - kPbDpWarp0 * 32;
        const uint32_t dpblk = smem_u32(smem + Cfg::kOffDp);
        for (int unit = 0; unit < nunits; ++unit) {
            const int it = unit / NMAPS, m = unit % NMAPS, slot = unit & 1;
            long long grow = (t0 + it) * kTileTokens + row;
            const bool live = grow < rows;
            grow = live ? grow : rows - 1;
            size_t off;
            if (KSIDE) {
                const uint32_t bh = (uint32_t)grow / (uint32_t)N, n = (uint32_t)grow - bh * (uint32_t)N;   // rows < 2^31 (checked on the host)
                off = (((size_t)bh * NMAPS + m) * N + n) * DP;
            } else {
                off = (size_t)grow * DP;
            }
            float d[DP];
#pragma unroll
            for (int i = 0; i < DP / 2; ++i) {
                const float2 f = __ldg(reinterpret_cast<const float2*>(feat + off) + i);
                const float2 g = __ldg(reinterpret_cast<const float2*>(dfeat + off) + i);
                d[2 * i] = (live && f.x > 0.f) ? g.x : 0.f;
                d[2 * i + 1] = (live && f.y > 0.f) ? g.y : 0.f;
            }
            uint32_t w[DP];      // [hi pairs | lo pairs]
#pragma unroll
            for (int i = 0; i < DP / 2; ++i) {
                const float l0 = d[2 * i] - __bfloat162float(__float2bfloat16_rn(d[2 * i])), l1 = d[2 * i + 1] - __bfloat162float(__float2bfloat16_rn(d[2 * i + 1]));
                w[i] = pack_bf16(d[2 * i], d[2 * i + 1]);
                w[DP / 2 + i] = pack_bf16(l0, l1);
            }
            if (ok && !mbar_wait(&dp_free[slot], ((unit >> 1) & 1) ^ 1)) { ok = false; report_timeout(status, 611); }
            if (!ok) break;
            if constexpr (DP == 6) {
                st_shared_v4(dpblk + sw128_off(row, 2 * slot), w[0], w[1], w[2], w[3]);
                st_shared_v4(dpblk + sw128_off(row, 2 * slot + 1), w[4], w[5], 0u, 0u);
            } else {
                const uint32_t blk = dpblk + slot * kBlk;
#pragma unroll
                for (int c = 0; c < 3; ++c) st_shared_v4(blk + sw128_off(row, c), w[4 * c], w[4 * c + 1], w[4 * c + 2], w[4 * c + 3]);
            }
            fence_proxy_async();
            mbar_arrive(&dp_full[slot]);
        }
    } else {
        const int quarter = warp & 3, part = (warp - kPbEpiWarp0) >> 2;
        const int row = quarter * 32 + lane;
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        for (int unit = 0; unit < nunits && ok; ++unit) {
            const int it = unit / NMAPS, m = unit % NMAPS, b = unit & 1, par = (unit >> 1) & 1;
            // dg(unit) was issued before dX(unit - 1), h(unit) after dX(unit - 2) had completed: dg is there first as a rule
            if (!mbar_wait(&h_full[b], par)) { ok = false; report_timeout(status, 604); }
            if (NMAPS > 1 && ok && !mbar_wait(dg_full, unit & 1)) { ok = false; report_timeout(status, 612); }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            uint32_t dgr[HC];
#pragma unroll
            for (int c = 0; c < HC / 16; ++c) tmem_ld16(tmem + 256 + lane_base + part * HC + 16 * c, *reinterpret_cast<uint32_t(*)[16]>(dgr + 16 * c));
            // (the h products of this unit were issued after the dX product of unit - 2 had completed, so the dh tile of this
            // parity is free)
            const uint32_t ta = tmem + 128 * b + lane_base + part * HC;
#pragma unroll
            for (int c = 0; c < HC / 16; ++c) {
                uint32_t r[16];
                tmem_ld16(ta + 16 * c, r);
                tmem_ld_wait();           // first round: dg and the first h columns in one batch of loads
                if (c == 0) {
                    tc_fence_before();
                    mbar_arrive(dg_empty);
                }
                uint32_t w[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float2 h = make_float2(__uint_as_float(r[2 * e]), __uint_as_float(r[2 * e + 1]));
                    const float2 dg = make_float2(__uint_as_float(dgr[16 * c + 2 * e]), __uint_as_float(dgr[16 * c + 2 * e + 1]));
                    const float2 dh = __fmul2_rn(dg, gelu_grad2_twice(h));      // dg holds dg / 2 (halved W2^T)
                    w[e] = pack_bf16(dh.x, dh.y);
                }
                // dh as the A operand of the dX product, packed into the h columns this thread has already read
                tmem_st8(ta + 8 * c, w[0], w[1], w[2], w[3], w[4], w[5], w[6], w[7]);
            }
            tmem_st_wait();
            tc_fence_before();
            mbar_arrive(&dh_full[b]);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, 512);
}

template <int DV, int F>
inline hla_status launch_phi_backward(const Dims& D, int BH, const hla_mlp* phi_q, const hla_mlp* phi_k, const void* Q, const void* K, void* dQ,
                                      void* dK, char* ws, const hla_ws_layout& L, int sm_count, LaunchRec& rec) {
    constexpr int NM = MT<F>::kMaps, DP = MT<F>::kDphi;
    const long long rows = (long long)BH * D.N;
    CUtensorMap mapQ, mapK, mapdQ, mapdK;
    PhiMaps mq, mk;
    PhiBwdPtrs pq{}, pk{};
    if (!make_map_2d(&mapQ, Q, (size_t)rows, DV, kTileTokens) || !make_map_2d(&mapK, K, (size_t)rows, DV, kTileTokens)) return HLA_ERR_CUDA;
    if (!make_map_2d(&mapdQ, dQ, (size_t)rows, DV, kTileTokens) || !make_map_2d(&mapdK, dK, (size_t)rows, DV, kTileTokens)) return HLA_ERR_CUDA;
    if (!make_map_2d(&mq.w1[0], phi_q->W1, DV, DV, DV)) return HLA_ERR_CUDA;
    mq.w1[1] = mq.w1[0];
    mq.w1[2] = mq.w1[0];
    pq.b1[0] = static_cast<const __nv_bfloat16*>(phi_q->b1);
    pq.W2[0] = static_cast<const __nv_bfloat16*>(phi_q->W2);
    for (int f = 0; f < NM; ++f) {
        if (!make_map_2d(&mk.w1[f], phi_k[f].W1, DV, DV, DV)) return HLA_ERR_CUDA;
        pk.b1[f] = static_cast<const __nv_bfloat16*>(phi_k[f].b1);
        pk.W2[f] = static_cast<const __nv_bfloat16*>(phi_k[f].W2);
    }
    for (int f = NM; f < 3; ++f) mk.w1[f] = mk.w1[0];
    int* status = reinterpret_cast<int*>(ws + L.status);
    if (!set_smem(tc_phi_backward_kernel<DV, 1, false, DP>, PbCfg<DV, 1, DP>::kSmem) || !set_smem(tc_phi_backward_kernel<DV, NM, true, DP>, PbCfg<DV, NM, DP>::kSmem))
        return HLA_ERR_CUDA;
    const long long tiles = (rows + kTileTokens - 1) / kTileTokens;
    const int grid = (int)(tiles < sm_count ? tiles : sm_count);
    cudaStream_t st = rec.st;
    rec.begin("tc_phi_backward_q");
    launch_pdl(tc_phi_backward_kernel<DV, 1, false, DP>, grid, dim3(kPbThreads), PbCfg<DV, 1, DP>::kSmem, st,
        mapQ, mq, mapdQ, pq, reinterpret_cast<const float*>(ws + L.qf), reinterpret_cast<const float*>(ws + L.dqf), static_cast<__nv_bfloat16*>(dQ), rows, D.N, status);
    if (!rec.end()) return HLA_ERR_CUDA;
    rec.begin("tc_phi_backward_k");
    launch_pdl(tc_phi_backward_kernel<DV, NM, true, DP>, grid, dim3(kPbThreads), PbCfg<DV, NM, DP>::kSmem, st,
        mapK, mk, mapdK, pk, reinterpret_cast<const float*>(ws + L.kf), reinterpret_cast<const float*>(ws + L.dkf), static_cast<__nv_bfloat16*>(dK), rows, D.N, status);
    return rec.end() ? HLA_OK : HLA_ERR_CUDA;
}

inline hla_status phi_backward(const Dims& D, int BH, const hla_mlp* phi_q, const hla_mlp* phi_k, const void* Q, const void* K, void* dQ, void* dK,
                               char* ws, const hla_ws_layout& L, int sm_count, LaunchRec& rec) {
    if (D.F == 3) {
        if (D.d == 128) return launch_phi_backward<128, 3>(D, BH, phi_q, phi_k, Q, K, dQ, dK, ws, L, sm_count, rec);
        return launch_phi_backward<64, 3>(D, BH, phi_q, phi_k, Q, K, dQ, dK, ws, L, sm_count, rec);
    }
    if (D.d == 128) return launch_phi_backward<128, 2>(D, BH, phi_q, phi_k, Q, K, dQ, dK, ws, L, sm_count, rec);
    return launch_phi_backward<64, 2>(D, BH, phi_q, phi_k, Q, K, dQ, dK, ws, L, sm_count, rec);
}

}  // namespace tc
}  // namespace hla
