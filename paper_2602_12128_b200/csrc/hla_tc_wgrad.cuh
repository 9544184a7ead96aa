// Gradients of the loss with respect to the weights of the feature networks (Section 5, "Training Details": the phi
// maps are trained with the rest of the model).  For one map, with dp = dfeat (.) 1[feat > 0] (the feature gradients the
// backward left in the workspace, masked by the features the forward kept):
//   h   = X W1 + b1,  G = GELU(h),  dg = dp W2^T,  dh = dg (.) GELU'(h)        (recomputed exactly as in the phi backward)
//   dW2 = G^T dp,   db2 = sum_t dp,   dW1 = X^T dh,   db1 = sum_t dh          (sums over all tokens of all heads)
//
// Both weight gradients contract over the tokens, so neither operand can stay in TMEM (a TMEM operand has one token per
// lane): the 16 arithmetic warps write the G and dh tiles to shared memory, where X^T, G^T (A operands) and dh, dp (B
// operands) are all read token-major ("MN-major").  Persistent CTAs take one map at a time over all their tiles, keep
//   dW1     [d x d]   accumulator lane = input index, column = hidden unit
//   dW2ext  [d x 64]  accumulator lane = hidden unit, columns 0..5 = G^T dp_hi, 6..11 = G^T dp_lo
// in TMEM for the whole map and leave one partial per (CTA, map) in the workspace; a second kernel adds the partials in
// CTA order, so the result is bit-reproducible.
//
// warp 0: TMA loads, warp 1: dg, dW1 and dW2 MMAs, warp 2: h MMAs, warps 3..18: arithmetic (thread = token row x quarter
// of the hidden units), warps 19..22: column sums of the dh tile (db1), warps 23..26: dp tiles and db2 (thread = token row;
// off the arithmetic warps' instruction stream, which is what bounds the kernel).
#pragma once
#include "hla_tc_phi.cuh"

namespace hla {
namespace tc {

constexpr int kWgThreads = 27 * 32;
constexpr int kWgEpiWarp0 = 3, kWgSumWarp0 = 19, kWgDpWarp0 = 23;
constexpr int kWgColDg = 128, kWgColW1 = 256, kWgColW2 = 384;      // TMEM columns (h at 0)

template <int DV, int NMAPS, int DP> struct WgCfg {
    static constexpr int kXBytes = 2 * kBlk;                     // two 64-column blocks per stage (the second stays zero for d = 64)
    static constexpr int kW1Bytes = DV * DV * 2;
    static constexpr int kDgSteps = DP == 6 ? 1 : 2;             // K = 16 steps of the dg product: [dp_hi | dp_lo] is 2 DP columns wide
    static constexpr int kW2tBlock = kDgSteps * 2048;
    static constexpr int kW2tBytes = (DV / 64) * kW2tBlock;      // per map: [16 kDgSteps K rows][DV] bf16 (W2^T twice, halved; row 12 of the last step: b1)
    static constexpr int kOffX = 0;                              // 2 stages
    static constexpr int kOffW1 = 2 * kXBytes;                   // the current map's W1
    static constexpr int kOffDp = kOffW1 + kW1Bytes;             // 3 dp blocks [128 tok][64]: K columns 0..5 dp_hi, 6..11 dp_lo; column 44 of block 0 is 1
    static constexpr int kOffW2t = kOffDp + 3 * kBlk;
    static constexpr int kOffG = ((kOffW2t + NMAPS * kW2tBytes + 1023) / 1024) * 1024;   // G tile, two 64-column blocks
    static constexpr int kOffDh = kOffG + 2 * kBlk;              // dh tile
    static constexpr int kOffBars = kOffDh + 2 * kBlk;
    static constexpr int kSmemUsed = 1024 + kOffBars + 256;
    static_assert(kSmemUsed <= 227 * 1024, "shared memory");
    static constexpr int kSmem = kSmemUsed > 120 * 1024 ? kSmemUsed : 120 * 1024;   // one CTA per SM (512 TMEM columns)
    static constexpr int kB1Row = 12;
    // one partial per (CTA, map), in floats: dW1 [DV][DV], dW2ext [DV][kW2Cols], db1 [DV], db2 [4 token quarters][16]
    static constexpr int kW2Cols = 16 * kDgSteps;
    static constexpr int kPartW2 = DV * DV, kPartB1 = kPartW2 + DV * kW2Cols, kPartB2 = kPartB1 + DV, kPartFloats = kPartB2 + 64;
};

// X [rows][DV] bf16.  KSIDE: feat / dfeat are [bh][NMAPS][N][6], else [rows][6].  wpart: [gridDim.x][NMAPS][kPartFloats].
template <int DV, int NMAPS, bool KSIDE, int DP>
__global__ void __launch_bounds__(kWgThreads, 1) tc_phi_wgrad_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ PhiMaps maps,
                                                                     PhiBwdPtrs P, const float* __restrict__ feat, const float* __restrict__ dfeat,
                                                                     float* __restrict__ wpart, long long rows, int N, int* status) {
    using Cfg = WgCfg<DV, NMAPS, DP>;
    constexpr int HC = DV / 4;
    extern __shared__ uint8_t smem_raw[];
    grid_launch_dependents();
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::kOffBars);
    uint64_t* x_full = bars;           // [2] TMA
    uint64_t* x_empty = bars + 2;      // [2] MMA commit (dW1 of the unit has read the tile)
    uint64_t* w_full = bars + 4;       // TMA: W1 of the current map
    uint64_t* w_empty = bars + 5;      // MMA commit after the map's last product
    uint64_t* h_full = bars + 6;       // MMA commit
    uint64_t* h_empty = bars + 7;      // 512 arrivals
    uint64_t* dp_full = bars + 8;      // [3] 128 arrivals
    uint64_t* dp_free = bars + 18;     // [3] MMA commit: the unit's products have read the block
    uint64_t* dg_full = bars + 11;     // MMA commit
    uint64_t* dg_empty = bars + 12;    // 512 arrivals
    uint64_t* gd_full = bars + 13;     // 512 arrivals: G and dh tiles written
    uint64_t* gd_empty = bars + 14;    // MMA commit + the column-sum warps
    uint64_t* acc_full = bars + 15;    // MMA commit, once per map
    uint64_t* acc_empty = bars + 16;   // 512 arrivals, once per map
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 17);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const long long tiles = (rows + kTileTokens - 1) / kTileTokens;
    const long long t0 = tiles * blockIdx.x / gridDim.x, t1 = tiles * (blockIdx.x + 1) / gridDim.x;
    const int ntiles = (int)(t1 - t0);
    const int nunits = ntiles * NMAPS;      // unit u = map (u / ntiles), tile (u % ntiles)
    float* out_cta = wpart + (size_t)blockIdx.x * NMAPS * Cfg::kPartFloats;

    constexpr int kRows = 16 * Cfg::kDgSteps, kB1Abs = kRows - 16 + Cfg::kB1Row;
    for (int i = tid; i < NMAPS * kRows * DV; i += kWgThreads) {
        const int m = i / (kRows * DV), k = (i / DV) % kRows, j = i % DV;
        uint8_t* base = smem + Cfg::kOffW2t + m * Cfg::kW2tBytes + (j >> 6) * Cfg::kW2tBlock;
        *reinterpret_cast<__nv_bfloat16*>(base + sw128_off(k, (j & 63) >> 3) + (j & 7) * 2) =
            k < 2 * DP ? half_bf16(P.W2[m][j * DP + (k % DP)]) : (k == kB1Abs ? P.b1[m][j] : __float2bfloat16_rn(0.f));
    }
    for (int i = tid; i < 3 * kBlk / 16; i += kWgThreads) reinterpret_cast<uint4*>(smem + Cfg::kOffDp)[i] = make_uint4(0, 0, 0, 0);
    for (int i = tid; i < 2 * Cfg::kXBytes / 16; i += kWgThreads) reinterpret_cast<uint4*>(smem + Cfg::kOffX)[i] = make_uint4(0, 0, 0, 0);
    for (int i = tid; i < 4 * kBlk / 16; i += kWgThreads) reinterpret_cast<uint4*>(smem + Cfg::kOffG)[i] = make_uint4(0, 0, 0, 0);
    __syncthreads();
    for (int i = tid; i < kTileTokens; i += kWgThreads)      // K column 32 + kB1Row of dp block 0: the ones column of the bias step
        *reinterpret_cast<__nv_bfloat16*>(smem + Cfg::kOffDp + sw128_off(i, 4 + Cfg::kB1Row / 8) + (Cfg::kB1Row & 7) * 2) = __float2bfloat16_rn(1.f);
    fence_proxy_async();
    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(&x_full[i], 1);
            mbar_init(&x_empty[i], 1);
        }
        mbar_init(w_full, 1);
        mbar_init(w_empty, 1);
        mbar_init(h_full, 1);
        mbar_init(h_empty, 512);
        for (int i = 0; i < 3; ++i) {
            mbar_init(&dp_full[i], 128);
            mbar_init(&dp_free[i], 1);
        }
        mbar_init(dg_full, 1);
        mbar_init(dg_empty, 512);
        mbar_init(gd_full, 512);
        mbar_init(gd_empty, 1 + DV / 32);
        mbar_init(acc_full, 1);
        mbar_init(acc_empty, 512);
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
    const uint32_t tmem = *tmem_slot;
    grid_dependency_wait();
    bool ok = true;

    if (warp == 0) {
        if (lane == 0 && ntiles > 0) {
            for (int unit = 0; unit < nunits; ++unit) {
                const int m = unit / ntiles, it = unit - m * ntiles, st = unit & 1;
                if (it == 0) {      // the previous map's products have finished with the W1 image
                    if (!mbar_wait(w_empty, (m & 1) ^ 1)) { report_timeout(status, 1001); break; }
                    mbar_arrive_expect_tx(w_full, Cfg::kW1Bytes);
                    for (int b = 0; b < DV / 64; ++b) tma_load_2d(smem + Cfg::kOffW1 + b * (DV * 128), &maps.w1[m], w_full, b * 64, 0);
                }
                if (!mbar_wait(&x_empty[st], ((unit >> 1) & 1) ^ 1)) { report_timeout(status, 1002); break; }
                mbar_arrive_expect_tx(&x_full[st], DV * kTileTokens * 2);
                for (int b = 0; b < DV / 64; ++b)
                    tma_load_2d(smem + Cfg::kOffX + st * Cfg::kXBytes + b * kBlk, &mapX, &x_full[st], b * 64, (int)((t0 + it) * kTileTokens));
            }
        }
    } else if (warp == 2) {
        if (lane == 0 && ntiles > 0) {      // h = X * W1[m] + 1 * b1[m]
            const uint32_t idesc1 = idesc_bf16(128, DV, false, true);    // X K-major, W1 [in][hidden] MN-major
            const uint64_t xd0 = smem_desc_sw128(smem_u32(smem + Cfg::kOffX), 16, 1024);
            const uint64_t wd = smem_desc_sw128(smem_u32(smem + Cfg::kOffW1), DV * 128, 1024);
            const uint64_t od = smem_desc_sw128(smem_u32(smem + Cfg::kOffDp) + 64, 16, 1024);
            const uint64_t bd0 = smem_desc_sw128(smem_u32(smem + Cfg::kOffW2t) + (Cfg::kDgSteps - 1) * 2048, Cfg::kW2tBlock, 1024);      // the K step with the b1 row
            bool good = true;
            for (int unit = 0; unit < nunits && good; ++unit) {
                const int m = unit / ntiles, it = unit - m * ntiles, st = unit & 1;
                if (it == 0 && !mbar_wait(w_full, m & 1)) { good = false; break; }
                if (!(mbar_wait(&x_full[st], (unit >> 1) & 1) && mbar_wait(h_empty, (unit & 1) ^ 1))) { good = false; break; }
                // the unit's dg product must be complete too, so that h_full tells the arithmetic warps both
                if (!mbar_wait(dg_full, unit & 1)) { good = false; break; }
                tc_fence_after();
                const uint64_t xd = desc_advance(xd0, st * Cfg::kXBytes);
#pragma unroll
                for (int ks = 0; ks < DV / 16; ++ks)
                    umma_bf16(tmem, desc_advance(xd, (ks >> 2) * kBlk + (ks & 3) * 32), desc_advance(wd, ks * 2048), idesc1, ks > 0 ? 1u : 0u);
                umma_bf16(tmem, od, desc_advance(bd0, m * Cfg::kW2tBytes), idesc1, 1u);      // + 1 * b1
                umma_commit(h_full);
            }
            if (!good) report_timeout(status, 1003);
        }
    } else if (warp == 1) {
        if (lane == 0 && ntiles > 0) {
            const uint32_t idesc_dg = idesc_bf16(128, DV, false, true);   // dg = dp (K-major) * W2^T (MN-major)
            const uint32_t idesc_w1 = idesc_bf16(128, DV, true, true);    // dW1 = X^T (MN-major, M = input index) * dh (MN-major, N = hidden)
            const uint32_t idesc_w2 = idesc_bf16(128, 64, true, true);    // dW2ext = G^T (MN-major, M = hidden) * dp block (MN-major, N = 64)
            const uint32_t dpa = smem_u32(smem + Cfg::kOffDp), xa = smem_u32(smem + Cfg::kOffX);
            const uint32_t ga = smem_u32(smem + Cfg::kOffG), da = smem_u32(smem + Cfg::kOffDh);
            const uint64_t vd0 = smem_desc_sw128(smem_u32(smem + Cfg::kOffW2t), Cfg::kW2tBlock, 1024);
            bool good = true;
            auto issue_dg = [&](int unit) -> bool {      // the arithmetic warps of unit - 1 must have taken their dg into registers
                const int m = unit / ntiles;
                if (unit > 0 && !mbar_wait(dg_empty, (unit - 1) & 1)) return false;
                if (!mbar_wait(&dp_full[unit % 3], (unit / 3) & 1)) return false;
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < Cfg::kDgSteps; ++ks)
                    umma_bf16(tmem + kWgColDg, smem_desc_sw128(dpa + (unit % 3) * kBlk + ks * 32, 16, 1024), desc_advance(vd0, m * Cfg::kW2tBytes + ks * 2048), idesc_dg,
                              ks > 0 ? 1u : 0u);
                umma_commit(dg_full);
                return true;
            };
            if (nunits > 0) good = issue_dg(0);
            for (int unit = 0; unit < nunits && good; ++unit) {
                const int m = unit / ntiles, it = unit - m * ntiles, st = unit & 1;
                if (unit + 1 < nunits && !issue_dg(unit + 1)) { good = false; break; }
                // the accumulators of the previous map must have been drained before this map's first product overwrites them
                if (it == 0 && m > 0 && !mbar_wait(acc_empty, (m - 1) & 1)) { good = false; break; }
                if (!mbar_wait(gd_full, unit & 1)) { good = false; break; }
                tc_fence_after();
                const uint32_t xs = xa + st * Cfg::kXBytes, dps = dpa + (unit % 3) * kBlk;
#pragma unroll
                for (int ks = 0; ks < kTileTokens / 16; ++ks)
                    umma_bf16(tmem + kWgColW1, smem_desc_sw128(xs + ks * 2048, kBlk, 1024), smem_desc_sw128(da + ks * 2048, kBlk, 1024), idesc_w1,
                              (it > 0 || ks > 0) ? 1u : 0u);
#pragma unroll
                for (int ks = 0; ks < kTileTokens / 16; ++ks)
                    umma_bf16(tmem + kWgColW2, smem_desc_sw128(ga + ks * 2048, kBlk, 1024), smem_desc_sw128(dps + ks * 2048, kBlk, 1024), idesc_w2,
                              (it > 0 || ks > 0) ? 1u : 0u);
                umma_commit(gd_empty);
                umma_commit(&dp_free[unit % 3]);
                umma_commit(&x_empty[st]);
                if (it == ntiles - 1) {
                    umma_commit(acc_full);
                    umma_commit(w_empty);
                }
            }
            if (!good) report_timeout(status, 1004);
        }
    } else if (warp >= kWgSumWarp0 && warp < kWgDpWarp0) {
        // db1: column sums of the dh tile as the dW1 product sees it (bf16 values, fp32 sums).  Warp w owns the 32 hidden
        // units 32 w ..: one 16-byte load per lane and step, lane l adds the eight columns of chunk 4 w + (l & 3) over the
        // rows l >> 2, l >> 2 + 8, ... and keeps its partial sums for the whole map; the lanes' sums meet after the map's last
        // tile, in a fixed order.  (Two warps with one 4-byte load per row took as long as a whole unit: a lone warp issues
        // an instruction every five cycles or so.)
        const int sw = warp - kWgSumWarp0;
        if (sw < DV / 32) {
            const uint32_t da = smem_u32(smem + Cfg::kOffDh) + (sw >> 1) * kBlk;
            const int chunk = 4 * (sw & 1) + (lane & 3);
            float sm[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) sm[e] = 0.f;
            for (int unit = 0; unit < nunits; ++unit) {
                const int m = unit / ntiles, it = unit - m * ntiles;
                if (ok && !mbar_wait(gd_full, unit & 1)) { ok = false; report_timeout(status, 1005); }
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
#pragma unroll 8
                for (int j = 0; j < kTileTokens / 8; ++j) {
                    uint32_t w[4];
                    asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(da + sw128_off((lane >> 2) + 8 * j, chunk)) : "memory");
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        sm[2 * e] += __uint_as_float(w[e] << 16);
                        sm[2 * e + 1] += __uint_as_float(w[e] & 0xffff0000u);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(gd_empty);
                if (it == ntiles - 1) {
                    float* o = out_cta + (size_t)m * Cfg::kPartFloats + Cfg::kPartB1 + (sw >> 1) * 64 + 8 * chunk;
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        float v = sm[e];
#pragma unroll
                        for (int x = 4; x < 32; x <<= 1) v += __shfl_xor_sync(0xffffffffu, v, x);
                        if (lane < 4) o[e] = v;
                        sm[e] = 0.f;
                    }
                }
            }
        }
    } else if (warp >= kWgDpWarp0) {
        // dp = dfeat (.) 1[feat > 0] of one token row as [dp_hi | dp_lo] (two bf16 halves, so dg is exact to ~2^-17) into
        // block unit % 3, and db2 = sum over the tokens of dp (this warp's 32 tokens by shuffles: one partial per token quarter)
        const int quarter = warp - kWgDpWarp0, row = quarter * 32 + lane;
        const uint32_t dpblk = smem_u32(smem + Cfg::kOffDp);
        float b2s[DP];
#pragma unroll
        for (int i = 0; i < DP; ++i) b2s[i] = 0.f;
        for (int unit = 0; unit < nunits; ++unit) {
            const int m = unit / ntiles, it = unit - m * ntiles;
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
            uint32_t w[DP];      // [hi pairs | lo pairs]
#pragma unroll
            for (int i = 0; i < DP / 2; ++i) {
                const float2 f = __ldg(reinterpret_cast<const float2*>(feat + off) + i);
                const float2 g = __ldg(reinterpret_cast<const float2*>(dfeat + off) + i);
                const float d0 = (live && f.x > 0.f) ? g.x : 0.f, d1 = (live && f.y > 0.f) ? g.y : 0.f;
                const float l0 = d0 - __bfloat162float(__float2bfloat16_rn(d0)), l1 = d1 - __bfloat162float(__float2bfloat16_rn(d1));
                w[i] = pack_bf16(d0, d1);
                w[DP / 2 + i] = pack_bf16(l0, l1);
                b2s[2 * i] += d0;
                b2s[2 * i + 1] += d1;
            }
            if (ok && !mbar_wait(&dp_free[unit % 3], ((unit / 3) & 1) ^ 1)) { ok = false; report_timeout(status, 1010); }
            if (!ok) break;
            const uint32_t blk = dpblk + (unit % 3) * kBlk;
            if constexpr (DP == 6) {
                st_shared_v4(blk + sw128_off(row, 0), w[0], w[1], w[2], w[3]);
                asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(blk + sw128_off(row, 1)), "r"(w[4]), "r"(w[5]) : "memory");
            } else {
#pragma unroll
                for (int c = 0; c < 3; ++c) st_shared_v4(blk + sw128_off(row, c), w[4 * c], w[4 * c + 1], w[4 * c + 2], w[4 * c + 3]);
            }
            fence_proxy_async();
            mbar_arrive(&dp_full[unit % 3]);
            if (it == ntiles - 1) {      // the map is complete: its db2 partial of this token quarter
                float* o = out_cta + (size_t)m * Cfg::kPartFloats + Cfg::kPartB2 + quarter * 16;
#pragma unroll
                for (int i = 0; i < DP; ++i) {
                    const float a = warp_sum(b2s[i]);
                    if (lane == 0) o[i] = a;
                    b2s[i] = 0.f;
                }
                if (lane < 16 - DP) o[DP + lane] = 0.f;
            }
        }
    } else {
        const int quarter = warp & 3, part = (warp - kWgEpiWarp0) >> 2;
        const int row = quarter * 32 + lane;
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        for (int unit = 0; unit < nunits && ok; ++unit) {
            const int m = unit / ntiles, it = unit - m * ntiles;
            // h_full(unit) also says that dg(unit) is complete (the thread that issues the h products waits for it first)
            if (!mbar_wait(h_full, unit & 1)) { ok = false; report_timeout(status, 1007); }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            uint32_t dgr[HC];
#pragma unroll
            for (int c = 0; c < HC / 16; ++c) tmem_ld16(tmem + kWgColDg + lane_base + part * HC + 16 * c, *reinterpret_cast<uint32_t(*)[16]>(dgr + 16 * c));
            uint32_t hr[HC];
#pragma unroll
            for (int c = 0; c < HC / 16; ++c) tmem_ld16(tmem + lane_base + part * HC + 16 * c, *reinterpret_cast<uint32_t(*)[16]>(hr + 16 * c));
            tmem_ld_wait();
            tc_fence_before();
            mbar_arrive(dg_empty);
            mbar_arrive(h_empty);
            uint32_t gw[HC / 2], dw[HC / 2];
#pragma unroll
            for (int e = 0; e < HC / 2; ++e) {
                const float2 h = make_float2(__uint_as_float(hr[2 * e]), __uint_as_float(hr[2 * e + 1]));
                const float2 dg = make_float2(__uint_as_float(dgr[2 * e]), __uint_as_float(dgr[2 * e + 1]));
                float2 g, gr;
                gelu_both2_twice(h, g, gr);                                      // 2 GELU(h) (the factor 1/2 is applied when the partial is reduced) and 2 GELU'(h)
                const float2 dh = __fmul2_rn(dg, gr);                            // dg holds dg / 2 (halved W2^T)
                gw[e] = pack_bf16(g.x, g.y);
                dw[e] = pack_bf16(dh.x, dh.y);
            }
            // the products of unit - 1 (and the column sums) have finished reading the two tiles
            if (!mbar_wait(gd_empty, (unit & 1) ^ 1)) { ok = false; report_timeout(status, 1008); }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const int col0 = part * HC;
            const uint32_t gblk = smem_u32(smem + Cfg::kOffG) + (col0 / 64) * kBlk, dblk = smem_u32(smem + Cfg::kOffDh) + (col0 / 64) * kBlk;
#pragma unroll
            for (int j = 0; j < HC / 8; ++j) {
                st_shared_v4(gblk + sw128_off(row, (col0 & 63) / 8 + j), gw[4 * j], gw[4 * j + 1], gw[4 * j + 2], gw[4 * j + 3]);
                st_shared_v4(dblk + sw128_off(row, (col0 & 63) / 8 + j), dw[4 * j], dw[4 * j + 1], dw[4 * j + 2], dw[4 * j + 3]);
            }
            fence_proxy_async();
            mbar_arrive(gd_full);
            if (it == ntiles - 1) {
                // the map is complete: drain dW1 (lane = input index) and dW2ext (lane = hidden unit)
                if (!mbar_wait(acc_full, m & 1)) { ok = false; report_timeout(status, 1009); }
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                float* o = out_cta + (size_t)m * Cfg::kPartFloats;
                if (row < DV) {
#pragma unroll
                    for (int c = 0; c < HC / 16; ++c) {
                        uint32_t r[16];
                        tmem_ld16(tmem + kWgColW1 + lane_base + col0 + 16 * c, r);
                        tmem_ld_wait();
                        float4* dst = reinterpret_cast<float4*>(o + (size_t)row * DV + col0 + 16 * c);
#pragma unroll
                        for (int q = 0; q < 4; ++q)
                            dst[q] = make_float4(__uint_as_float(r[4 * q]), __uint_as_float(r[4 * q + 1]), __uint_as_float(r[4 * q + 2]), __uint_as_float(r[4 * q + 3]));
                    }
                    if (part == 0) {
#pragma unroll
                        for (int c = 0; c < Cfg::kW2Cols / 16; ++c) {
                            uint32_t r[16];
                            tmem_ld16(tmem + kWgColW2 + lane_base + 16 * c, r);
                            tmem_ld_wait();
                            float4* dst = reinterpret_cast<float4*>(o + Cfg::kPartW2 + (size_t)row * Cfg::kW2Cols + 16 * c);
#pragma unroll
                            for (int q = 0; q < 4; ++q)
                                dst[q] = make_float4(__uint_as_float(r[4 * q]), __uint_as_float(r[4 * q + 1]), __uint_as_float(r[4 * q + 2]), __uint_as_float(r[4 * q + 3]));
                        }
                    }
                }
                tc_fence_before();
                mbar_arrive(acc_empty);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, 512);
}

// Adds the partials of `nctas` CTAs in CTA order and writes one map's gradients (fp32, the shapes of the weights).
// grid = (blocks, maps); partial layout as WgCfg::kPart*.  A CTA that had no tiles left its partial untouched: it is skipped.
struct WgradOut {
    float* dW1[4];
    float* db1[4];
    float* dW2[4];
    float* db2[4];
};
// Sum of the per-CTA partials in a fixed order (bit-reproducible): a block owns 32 consecutive outputs, warp w adds the
// partials of the CTAs w, w + 8, ... (coalesced 128-byte reads, a dozen and a half independent loads per thread), and
// the eight warp sums are added in warp order.
template <int DV, int DP>
__global__ void __launch_bounds__(256) tc_wgrad_reduce_kernel(const float* __restrict__ wpart, WgradOut out, int nmaps_in_part, int map0, int nctas) {
    using C1 = WgCfg<DV, 1, DP>;
    constexpr int PF = C1::kPartFloats, oW2 = C1::kPartW2, oB1 = C1::kPartB1, oB2 = C1::kPartB2, W2C = C1::kW2Cols;
    __shared__ float red[8][32];
    grid_launch_dependents();
    grid_dependency_wait();
    const int m = blockIdx.y;                        // map of this launch
    const int total = DV * DV + DV * DP + DV + DP;   // outputs of one map
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float* src = wpart + (size_t)m * PF;
    const size_t stride = (size_t)nmaps_in_part * PF;
    for (int base = blockIdx.x * 32; base < total; base += gridDim.x * 32) {
        const int i = base + lane;
        // an output is the sum over the CTAs of `nterm` partial entries `step` floats apart, starting at `off`
        int off = 0, nterm = 0, step = 0;
        float scale = 1.f;
        if (i < DV * DV) {
            off = i; nterm = 1;
        } else if (i < DV * DV + DV * DP) {
            const int j = (i - DV * DV) / DP, o = (i - DV * DV) % DP;
            off = oW2 + j * W2C + o; nterm = 2; step = DP; scale = 0.5f;      // the G tile held 2 GELU(h)
        } else if (i < DV * DV + DV * DP + DV) {
            off = oB1 + (i - DV * DV - DV * DP); nterm = 1;
        } else if (i < total) {
            off = oB2 + (i - DV * DV - DV * DP - DV); nterm = 4; step = 16;
        }
        float a = 0.f;
        if (nterm == 1) {
#pragma unroll 4
            for (int c = warp; c < nctas; c += 8) a += src[c * stride + off];
        } else {
            for (int c = warp; c < nctas; c += 8)
                for (int q = 0; q < nterm; ++q) a += src[c * stride + off + q * step];
        }
        red[warp][lane] = a;
        __syncthreads();
        if (warp == 0 && i < total) {
            float t = red[0][lane];
#pragma unroll
            for (int w = 1; w < 8; ++w) t += red[w][lane];
            t *= scale;
            if (i < DV * DV) out.dW1[map0 + m][i] = t;
            else if (i < DV * DV + DV * DP) out.dW2[map0 + m][i - DV * DV] = t;
            else if (i < DV * DV + DV * DP + DV) out.db1[map0 + m][i - DV * DV - DV * DP] = t;
            else out.db2[map0 + m][i - DV * DV - DV * DP - DV] = t;
        }
        __syncthreads();
    }
}

inline size_t wgrad_part_bytes(int d, long long rows, int sm_count) {
    const long long tiles = (rows + kTileTokens - 1) / kTileTokens;
    const int grid = (int)(tiles < sm_count ? tiles : sm_count);
    const size_t pf = d == 128 ? WgCfg<128, 1, 12>::kPartFloats : WgCfg<64, 1, 12>::kPartFloats;      // the larger of the two geometries
    return (size_t)grid * 3 * pf * 4;      // the key side's maps share one launch; the query side reuses the region
}

// dphi_q / dphi_k: fp32 device outputs with the shapes of the weights (dphi_k points to one entry per key map); either may be null.
template <int DV, int F>
inline hla_status launch_phi_wgrad(const Dims& D, int BH, const hla_mlp* phi_q, const hla_mlp* phi_k, const void* Q, const void* K,
                                   const hla_mlp_grad* dphi_q, const hla_mlp_grad* dphi_k, char* ws, const hla_ws_layout& L, size_t off_wpart,
                                   int sm_count, LaunchRec& rec) {
    constexpr int NM = MT<F>::kMaps, DP = MT<F>::kDphi;
    const long long rows = (long long)BH * D.N;
    const long long tiles = (rows + kTileTokens - 1) / kTileTokens;
    const int grid = (int)(tiles < sm_count ? tiles : sm_count);
    int* status = reinterpret_cast<int*>(ws + L.status);
    float* wpart = reinterpret_cast<float*>(ws + off_wpart);
    cudaStream_t st = rec.st;
    if (dphi_q) {
        CUtensorMap mapQ;
        PhiMaps mq;
        PhiBwdPtrs pq{};
        if (!make_map_2d(&mapQ, Q, (size_t)rows, DV, kTileTokens) || !make_map_2d(&mq.w1[0], phi_q->W1, DV, DV, DV)) return HLA_ERR_CUDA;
        mq.w1[1] = mq.w1[0];
        mq.w1[2] = mq.w1[0];
        pq.b1[0] = static_cast<const __nv_bfloat16*>(phi_q->b1);
        pq.W2[0] = static_cast<const __nv_bfloat16*>(phi_q->W2);
        if (!set_smem(tc_phi_wgrad_kernel<DV, 1, false, DP>, WgCfg<DV, 1, DP>::kSmem)) return HLA_ERR_CUDA;
        rec.begin("tc_phi_wgrad_q");
        launch_serial(tc_phi_wgrad_kernel<DV, 1, false, DP>, grid, dim3(kWgThreads), WgCfg<DV, 1, DP>::kSmem, st, mapQ, mq, pq,
                      reinterpret_cast<const float*>(ws + L.qf), reinterpret_cast<const float*>(ws + L.dqf), wpart, rows, D.N, status);
        if (!rec.end()) return HLA_ERR_CUDA;
        WgradOut o{};
        o.dW1[0] = static_cast<float*>(dphi_q->dW1); o.db1[0] = static_cast<float*>(dphi_q->db1);
        o.dW2[0] = static_cast<float*>(dphi_q->dW2); o.db2[0] = static_cast<float*>(dphi_q->db2);
        rec.begin("tc_wgrad_reduce");
        launch_pdl(tc_wgrad_reduce_kernel<DV, DP>, dim3((DV * DV + DV * DP + DV + DP + 31) / 32, 1), dim3(256), 0, st, (const float*)wpart, o, 1, 0, grid);
        if (!rec.end()) return HLA_ERR_CUDA;
    }
    if (dphi_k) {
        CUtensorMap mapK;
        PhiMaps mk;
        PhiBwdPtrs pk{};
        if (!make_map_2d(&mapK, K, (size_t)rows, DV, kTileTokens)) return HLA_ERR_CUDA;
        WgradOut o{};
        for (int f = 0; f < NM; ++f) {
            if (!make_map_2d(&mk.w1[f], phi_k[f].W1, DV, DV, DV)) return HLA_ERR_CUDA;
            pk.b1[f] = static_cast<const __nv_bfloat16*>(phi_k[f].b1);
            pk.W2[f] = static_cast<const __nv_bfloat16*>(phi_k[f].W2);
            o.dW1[f] = static_cast<float*>(dphi_k[f].dW1); o.db1[f] = static_cast<float*>(dphi_k[f].db1);
            o.dW2[f] = static_cast<float*>(dphi_k[f].dW2); o.db2[f] = static_cast<float*>(dphi_k[f].db2);
        }
        for (int f = NM; f < 3; ++f) mk.w1[f] = mk.w1[0];
        if (!set_smem(tc_phi_wgrad_kernel<DV, NM, true, DP>, WgCfg<DV, NM, DP>::kSmem)) return HLA_ERR_CUDA;
        rec.begin("tc_phi_wgrad_k");
        // it stages caller-provided weights before its dependency wait, and the reduction before it still reads the
        // partial region: no overlap with what precedes it
        launch_serial(tc_phi_wgrad_kernel<DV, NM, true, DP>, grid, dim3(kWgThreads), WgCfg<DV, NM, DP>::kSmem, st, mapK, mk, pk,
                      reinterpret_cast<const float*>(ws + L.kf), reinterpret_cast<const float*>(ws + L.dkf), wpart, rows, D.N, status);
        if (!rec.end()) return HLA_ERR_CUDA;
        rec.begin("tc_wgrad_reduce");
        launch_pdl(tc_wgrad_reduce_kernel<DV, DP>, dim3((DV * DV + DV * DP + DV + DP + 31) / 32, NM), dim3(256), 0, st, (const float*)wpart, o, NM, 0, grid);
        if (!rec.end()) return HLA_ERR_CUDA;
    }
    return HLA_OK;
}

inline hla_status phi_wgrad(const Dims& D, int BH, const hla_mlp* phi_q, const hla_mlp* phi_k, const void* Q, const void* K,
                            const hla_mlp_grad* dphi_q, const hla_mlp_grad* dphi_k, char* ws, const hla_ws_layout& L, size_t off_wpart, int sm_count,
                            LaunchRec& rec) {
    if (D.F == 3) {
        if (D.d == 128) return launch_phi_wgrad<128, 3>(D, BH, phi_q, phi_k, Q, K, dphi_q, dphi_k, ws, L, off_wpart, sm_count, rec);
        return launch_phi_wgrad<64, 3>(D, BH, phi_q, phi_k, Q, K, dphi_q, dphi_k, ws, L, off_wpart, sm_count, rec);
    }
    if (D.d == 128) return launch_phi_wgrad<128, 2>(D, BH, phi_q, phi_k, Q, K, dphi_q, dphi_k, ws, L, off_wpart, sm_count, rec);
    return launch_phi_wgrad<64, 2>(D, BH, phi_q, phi_k, Q, K, dphi_q, dphi_k, ws, L, off_wpart, sm_count, rec);
}

}  // namespace tc
}  // namespace hla
