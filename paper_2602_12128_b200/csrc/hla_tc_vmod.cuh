// Value modulation (Section 4.5 "Value Modulation"; appendix "Defining phi"):   Out = T + phi_v1(T) (.) phi_v2(V),
// phi_v(x) = W2^T GELU(W1^T LN(x) + b1) + b2 with a LayerNorm (scale g, shift s, eps 1e-5) on the d channels of each token,
// two Linear layers of width d, no final activation.  T is the attention result (the output of hla_forward), per head.
//
// The LayerNorm never materialises: with xhat = (x - mu) rstd,
//     W1^T LN(x) + b1 = rstd (x W1' - mu c) + b1',   W1'[i][j] = g_i W1[i][j],  c_j = sum_i W1'[i][j],  b1'_j = b1_j + sum_i s_i W1[i][j]
// so the first-layer product runs on the raw tile as TMA delivers it, a ninth K step adds (-mu) c + (1 / rstd) b1' on the
// tensor cores (A = per-row [-mu, 1 / rstd] written to TMEM by the statistics warps, B = [c; b1'], both split into two bf16
// halves so the step is exact to ~2^-17), and the GELU warps only multiply by rstd.  A small kernel folds the weights.
//
// One map per launch (the two weight matrices of a map take 64 KB of shared memory at d = 128, so both maps do not fit):
//   forward : Y2 = phi_v2(V)  ->  Out = T + phi_v1(T) (.) Y2
//   backward: Y2 = phi_v2(V),  Y1 = phi_v1(T)  ->  dT = dOut + J1^T (dOut (.) Y2),  dV (+)= J2^T (dOut (.) Y1)
// with J^T the transposed Jacobian of a map: dg = dy W2^T, dh = dg (.) GELU'(h), dxhat = dh W1'^T, then the LayerNorm:
//     dx = rstd (dxhat - mean(dxhat) - xhat mean(dxhat (.) xhat)).
#pragma once
#include "hla_tc_phi.cuh"

namespace hla {
namespace tc {

constexpr float kLnEps = 1e-5f;

// ---- folding of the LayerNorm into the first layer -----------------------------------------------------------------
// aux [16][d] bf16 (K rows of the extra K steps): rows 0..2 = c_hi, c_lo, c_hi; rows 3..5 = b1'_hi, b1'_lo, b1'_hi; row 8 = b2.
struct VmlpPtrs {
    const __nv_bfloat16 *ln_g, *ln_b, *W1, *b1, *W2, *b2;
};
// grid = (2 maps, d / 32 column groups), block = 32 columns x 8 row groups
__global__ void __launch_bounds__(256) vmod_fold_kernel(VmlpPtrs a, VmlpPtrs b, __nv_bfloat16* __restrict__ w1f, __nv_bfloat16* __restrict__ aux, int d) {
    __shared__ float sc[8][32], ss[8][32];
    const VmlpPtrs p = blockIdx.x == 0 ? a : b;
    __nv_bfloat16* wf = w1f + (size_t)blockIdx.x * d * d;
    __nv_bfloat16* ax = aux + (size_t)blockIdx.x * 16 * d;
    const int jx = threadIdx.x & 31, iy = threadIdx.x >> 5, j = blockIdx.y * 32 + jx;
    float c = 0.f, s = 0.f;
    for (int i = iy; i < d; i += 8) {      // fixed order per thread, then a fixed-order sum over the 8 row groups
        const float w = __bfloat162float(p.W1[(size_t)i * d + j]);
        const __nv_bfloat16 f = __float2bfloat16_rn(__bfloat162float(p.ln_g[i]) * w);
        wf[(size_t)i * d + j] = f;
        c += __bfloat162float(f);
        s = fmaf(__bfloat162float(p.ln_b[i]), w, s);
    }
    sc[iy][jx] = c;
    ss[iy][jx] = s;
    __syncthreads();
    if (iy == 0) {
        c = 0.f;
        s = 0.f;
        for (int k = 0; k < 8; ++k) {
            c += sc[k][jx];
            s += ss[k][jx];
        }
        const float b1f = __bfloat162float(p.b1[j]) + s;
        const __nv_bfloat16 chi = __float2bfloat16_rn(c), clo = __float2bfloat16_rn(c - __bfloat162float(chi));
        const __nv_bfloat16 bhi = __float2bfloat16_rn(b1f), blo = __float2bfloat16_rn(b1f - __bfloat162float(bhi));
        const __nv_bfloat16 zero = __float2bfloat16_rn(0.f);
        for (int r = 0; r < 16; ++r) ax[(size_t)r * d + j] = zero;
        ax[0 * d + j] = chi; ax[1 * d + j] = clo; ax[2 * d + j] = chi;
        ax[3 * d + j] = bhi; ax[4 * d + j] = blo; ax[5 * d + j] = bhi;
        ax[8 * d + j] = p.b2[j];
    }
}

// Row statistics of a 128-token bf16 tile in shared memory (two 64-column swizzled blocks): mean and 1 / sqrt(var + eps).
// One pass over the row: sums of (x - shift) and (x - shift)^2 with shift = the mean of the row's first eight elements, which
// is within a few standard deviations of the row mean, so the difference of the two moments loses no more than a few bits.
template <int DV>
__device__ __forceinline__ void tile_row_stats(uint32_t tile, int row, float& mu, float& rstd) {
    float2 shift = make_float2(0.f, 0.f), s = shift, q = shift;      // shift holds minus the shift
#pragma unroll 4
    for (int c = 0; c < DV / 8; ++c) {
        uint32_t w[4];
        asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(tile + (c >> 3) * kBlk + sw128_off(row, c & 7)) : "memory");
        if (c == 0) {
            float t = 0.f;
#pragma unroll
            for (int e = 0; e < 4; ++e) t += __uint_as_float(w[e] << 16) + __uint_as_float(w[e] & 0xffff0000u);
            shift = splat2(-0.125f * t);
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 dlt = __fadd2_rn(make_float2(__uint_as_float(w[e] << 16), __uint_as_float(w[e] & 0xffff0000u)), shift);
            s = __fadd2_rn(s, dlt);
            q = __ffma2_rn(dlt, dlt, q);
        }
    }
    const float m = (s.x + s.y) * (1.f / DV);
    mu = m - shift.x;
    rstd = rsqrtf(fmaxf((q.x + q.y) * (1.f / DV) - m * m, 0.f) + kLnEps);
}
// The A operand of the extra K step, 8 TMEM columns of one row: K0, K1 = -mu_hi; K2 = -mu_lo; K3, K4 = sigma_hi; K5 = sigma_lo.
__device__ __forceinline__ void store_aug_row(uint32_t taddr, float mu, float rstd) {
    const float sigma = 1.f / rstd;
    const float mh = __bfloat162float(__float2bfloat16_rn(-mu)), ml = -mu - mh;
    const float sh = __bfloat162float(__float2bfloat16_rn(sigma)), sl = sigma - sh;
    tmem_st8(taddr, pack_bf16(mh, mh), pack_bf16(ml, sh), pack_bf16(sh, sl), 0u, 0u, 0u, 0u, 0u);
}

// 16 bf16 of one tile row (two 16-byte chunks 2 c, 2 c + 1 of a two-block swizzled tile) <-> 8 packed words
__device__ __forceinline__ void lds_row16(uint32_t tile, int row, int c, uint32_t (&w)[8]) {
    const uint32_t a = tile + (c >> 2) * kBlk + sw128_off(row, (2 * c) & 7), b = tile + (c >> 2) * kBlk + sw128_off(row, (2 * c + 1) & 7);
    asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(a) : "memory");
    asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7]) : "r"(b) : "memory");
}
__device__ __forceinline__ void sts_row16(uint32_t tile, int row, int c, const uint32_t (&w)[8]) {
    st_shared_v4(tile + (c >> 2) * kBlk + sw128_off(row, (2 * c) & 7), w[0], w[1], w[2], w[3]);
    st_shared_v4(tile + (c >> 2) * kBlk + sw128_off(row, (2 * c + 1) & 7), w[4], w[5], w[6], w[7]);
}
// Products of two pairs of bf16, each rounded once to bf16 (the same value as an fp32 product rounded to bf16: the
// product of two 8-bit significands is exact in fp32).
__device__ __forceinline__ uint32_t mul_bf16x2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// ---- forward of one map --------------------------------------------------------------------------------------------
// warp 0: TMA, warp 1: second-layer MMAs, warp 2: first-layer MMAs, warps 3..18: GELU (thread = token row x quarter of the
// hidden units), warps 19..22: row statistics, warps 23..26: output (thread = token row).  Every byte of global memory
// moves through TMA: the output warps read the residual and the other map's output from a tile in shared memory, write
// the result over it and store the tile.
constexpr int kVfThreads = 27 * 32;
constexpr int kVfGeluWarp0 = 3, kVfStatWarp0 = 19, kVfOutWarp0 = 23;
constexpr int kVfColD2 = 256, kVfColOnes = 384, kVfColAug = 392;      // TMEM columns (D1[b] at 128 b, aug[b] at 392 + 8 b)

template <int DV, bool COMBINE> struct VfCfg {
    static constexpr int kXStages = COMBINE ? 2 : 3;
    static constexpr int kXBytes = 2 * kBlk;                     // a tile is always two 64-column blocks apart (d = 64 uses the first)
    static constexpr int kWBytes = DV * DV * 2;
    static constexpr int kAuxBytes = (DV / 64) * 2048;           // [16 K rows][DV] bf16
    static constexpr int kOffX = 0;
    static constexpr int kOffE = kXStages * kXBytes;             // COMBINE: two Y2 tiles (-> Out tiles), by tile parity; else the Out tile
    static constexpr int kEBytes = (COMBINE ? 2 : 1) * kXBytes;
    static constexpr int kOffW1 = kOffE + kEBytes;
    static constexpr int kOffW2 = kOffW1 + kWBytes;
    static constexpr int kOffAux = kOffW2 + kWBytes;
    static constexpr int kOffStat = kOffAux + kAuxBytes;         // rstd [2][128] floats
    static constexpr int kOffBars = kOffStat + 2 * kTileTokens * 4;
    static constexpr int kSmemUsed = 1024 + kOffBars + 256;
    static_assert(kSmemUsed <= 227 * 1024, "shared memory");
    static constexpr int kSmem = kSmemUsed > 120 * 1024 ? kSmemUsed : 120 * 1024;   // one CTA per SM (512 TMEM columns)
};

// X [rows][DV] bf16 (mapX).  COMBINE: Out = X + y (.) Y2 (X is T; mapY2 covers Y2), else Out = y.  mapOut covers Out.
template <int DV, bool COMBINE>
__global__ void __launch_bounds__(kVfThreads, 1) tc_vmlp_forward_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapW1,
                                                                        const __grid_constant__ CUtensorMap mapW2, const __grid_constant__ CUtensorMap mapAux,
                                                                        const __grid_constant__ CUtensorMap mapY2, const __grid_constant__ CUtensorMap mapOut,
                                                                        long long rows, int* status) {
    using Cfg = VfCfg<DV, COMBINE>;
    constexpr int HC = DV / 4;
    constexpr int XST = Cfg::kXStages;
    extern __shared__ uint8_t smem_raw[];
    grid_launch_dependents();
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    float* stat = reinterpret_cast<float*>(smem + Cfg::kOffStat);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::kOffBars);
    uint64_t* x_full = bars;           // [3] TMA
    uint64_t* x_empty = bars + 3;      // [3] MMA commit
    uint64_t* st_full = bars + 6;      // [2] 128 arrivals: statistics of the tile written
    uint64_t* d1_full = bars + 8;      // [2] MMA commit
    uint64_t* g_full = bars + 10;      // [2] 512 arrivals
    uint64_t* g_free = bars + 12;      // [2] MMA commit
    uint64_t* d2_full = bars + 14;     // MMA commit
    uint64_t* d2_empty = bars + 15;    // 128 arrivals
    uint64_t* w_full = bars + 16;      // TMA
    uint64_t* e_ready = bars + 19;     // [2] COMBINE: the Y2 tile of that parity has landed (TMA); else [0]: one arrival, the output tile may be used
    uint64_t* o_full = bars + 18;      // 128 arrivals: the output tile is written
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 21);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const long long tiles = (rows + kTileTokens - 1) / kTileTokens;
    const long long t0 = tiles * blockIdx.x / gridDim.x, t1 = tiles * (blockIdx.x + 1) / gridDim.x;
    const int ntiles = (int)(t1 - t0);

    if (tid == 0) {
        for (int i = 0; i < 3; ++i) {
            mbar_init(&x_full[i], 1);
            mbar_init(&x_empty[i], COMBINE ? 128 : 1);      // COMBINE: the output warps read T from the X tile
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&e_ready[i], 1);
            mbar_init(&st_full[i], 128);
            mbar_init(&d1_full[i], 1);
            mbar_init(&g_full[i], 512);
            mbar_init(&g_free[i], 1);
        }
        mbar_init(d2_full, 1);
        mbar_init(d2_empty, 128);
        mbar_init(w_full, 1);
        mbar_init(o_full, 128);
        fence_mbar_init();
        prefetch_tmap(&mapX);
        prefetch_tmap(&mapW1);
        prefetch_tmap(&mapW2);
        prefetch_tmap(&mapAux);
        prefetch_tmap(&mapOut);
        if (COMBINE) prefetch_tmap(&mapY2);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    if (warp >= kVfOutWarp0) {      // constant A operand of the second layer's bias step: a one at K = 8
        tmem_st8(tmem + kVfColOnes + ((uint32_t)((warp & 3) * 32) << 16), 0u, 0u, 0u, 0u, 0x3F80u, 0u, 0u, 0u);
        tmem_st_wait();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    grid_dependency_wait();
    bool ok = true;

    if (warp == 0) {
        if (lane == 0 && ntiles > 0) {
            mbar_arrive_expect_tx(w_full, 2 * Cfg::kWBytes + Cfg::kAuxBytes);
            for (int b = 0; b < DV / 64; ++b) {
                tma_load_2d(smem + Cfg::kOffW1 + b * (DV * 128), &mapW1, w_full, b * 64, 0);
                tma_load_2d(smem + Cfg::kOffW2 + b * (DV * 128), &mapW2, w_full, b * 64, 0);
                tma_load_2d(smem + Cfg::kOffAux + b * 2048, &mapAux, w_full, b * 64, 0);
            }
            for (int it = 0; it < ntiles; ++it) {
                const int st = it % XST, u = it / XST;
                if (!mbar_wait(&x_empty[st], (u & 1) ^ 1)) { report_timeout(status, 1101); break; }
                mbar_arrive_expect_tx(&x_full[st], DV * kTileTokens * 2);
                for (int b = 0; b < DV / 64; ++b)
                    tma_load_2d(smem + Cfg::kOffX + st * Cfg::kXBytes + b * kBlk, &mapX, &x_full[st], b * 64, (int)((t0 + it) * kTileTokens));
            }
        }
    } else if (warp == 2) {
        if (lane == 0 && ntiles > 0) {      // D1[b] = X W1' + [-mu, sigma] [c; b1']
            const uint32_t idesc1 = idesc_bf16(128, DV, false, true);   // X K-major, W1' [in][hidden] MN-major
            const uint64_t xd0 = smem_desc_sw128(smem_u32(smem + Cfg::kOffX), 16, 1024);
            const uint64_t wd = smem_desc_sw128(smem_u32(smem + Cfg::kOffW1), DV * 128, 1024);
            const uint64_t ad = smem_desc_sw128(smem_u32(smem + Cfg::kOffAux), 2048, 1024);
            bool good = mbar_wait(w_full, 0);
            for (int it = 0; it < ntiles && good; ++it) {
                const int st = it % XST, b = it & 1, par = (it >> 1) & 1;
                if (!(mbar_wait(&x_full[st], (it / XST) & 1) && mbar_wait(&st_full[b], par) && mbar_wait(&g_free[b], par ^ 1))) { good = false; break; }
                tc_fence_after();
                const uint64_t xd = desc_advance(xd0, st * Cfg::kXBytes);
#pragma unroll
                for (int ks = 0; ks < DV / 16; ++ks)
                    umma_bf16(tmem + 128 * b, desc_advance(xd, (ks >> 2) * kBlk + (ks & 3) * 32), desc_advance(wd, ks * 2048), idesc1, ks > 0 ? 1u : 0u);
                umma_bf16_ta(tmem + 128 * b, tmem + kVfColAug + 8 * b, ad, idesc1, 1u);
                umma_commit(&d1_full[b]);
                if (!COMBINE) umma_commit(&x_empty[st]);
            }
            if (!good) report_timeout(status, 1102);
        }
    } else if (warp == 1) {
        if (lane == 0 && ntiles > 0) {      // D2 = G W2 + 1 b2
            const uint32_t idesc2 = idesc_bf16(128, DV, false, true);   // G from TMEM, W2 [hidden][out] MN-major
            const uint64_t wd = smem_desc_sw128(smem_u32(smem + Cfg::kOffW2), DV * 128, 1024);
            const uint64_t ad = smem_desc_sw128(smem_u32(smem + Cfg::kOffAux), 2048, 1024);
            bool good = mbar_wait(w_full, 0);
            for (int it = 0; it < ntiles && good; ++it) {
                const int b = it & 1, par = (it >> 1) & 1;
                if (!(mbar_wait(&g_full[b], par) && mbar_wait(d2_empty, (it & 1) ^ 1))) { good = false; break; }
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < DV / 16; ++ks)
                    umma_bf16_ta(tmem + kVfColD2, tmem + 128 * b + ((16 * ks) / HC) * HC + ((16 * ks) % HC) / 2, desc_advance(wd, ks * 2048), idesc2,
                                 ks > 0 ? 1u : 0u);
                umma_bf16_ta(tmem + kVfColD2, tmem + kVfColOnes, ad, idesc2, 1u);
                umma_commit(&g_free[b]);
                umma_commit(d2_full);
            }
            if (!good) report_timeout(status, 1103);
        }
    } else if (warp >= kVfOutWarp0) {
        // Out = y (or T + y (.) Y2): thread = token row; the result tile is formed in shared memory and stored by TMA.
        // COMBINE: T is read from the X tile the map was computed from (the tile stays until this pass is done with it), Y2
        // comes by TMA into one of two tiles (by tile parity) a whole tile ahead, and the result is written over it.
        const int quarter = warp & 3, row = quarter * 32 + lane;
        const bool leader = warp == kVfOutWarp0 && lane == 0;
        const uint32_t ta = tmem + kVfColD2 + ((uint32_t)(quarter * 32) << 16);
        auto open_tile = [&](int it) {      // leader only: the tile of that parity is free; COMBINE fetches Y2 into it
            if (COMBINE) {
                mbar_arrive_expect_tx(&e_ready[it & 1], DV * kTileTokens * 2);
                for (int b = 0; b < DV / 64; ++b)
                    tma_load_2d(smem + Cfg::kOffE + (it & 1) * Cfg::kXBytes + b * kBlk, &mapY2, &e_ready[it & 1], b * 64, (int)((t0 + it) * kTileTokens));
            } else {
                mbar_arrive(&e_ready[0]);
            }
        };
        if (leader && ntiles > 0) open_tile(0);
        for (int it = 0; it < ntiles; ++it) {
            const int eb = COMBINE ? (it & 1) : 0, epar = COMBINE ? ((it >> 1) & 1) : (it & 1);
            if (COMBINE && leader && it + 1 < ntiles) {
                tma_store_wait_read0();      // the store of tile it - 1 has read the tile of the other parity
                open_tile(it + 1);
            }
            if (ok && !mbar_wait(d2_full, it & 1)) { ok = false; report_timeout(status, 1104); }
            if (ok && !mbar_wait(&e_ready[eb], epar)) { ok = false; report_timeout(status, 1108); }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t xt = smem_u32(smem + Cfg::kOffX + (it % XST) * Cfg::kXBytes);      // COMBINE: T tile
            const uint32_t ot = smem_u32(smem + Cfg::kOffE + eb * Cfg::kXBytes);              // Y2 tile, overwritten by the result
#pragma unroll 2
            for (int c = 0; c < DV / 16; ++c) {
                uint32_t r[16], xw[8], yw[8], w[8];
                tmem_ld16(ta + 16 * c, r);
                if (COMBINE) {
                    lds_row16(xt, row, c, xw);
                    lds_row16(ot, row, c, yw);
                }
                tmem_ld_wait();
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    float a = __uint_as_float(r[2 * e]), b = __uint_as_float(r[2 * e + 1]);
                    if (COMBINE) {
                        a = fmaf(a, bf_lo(yw[e]), bf_lo(xw[e]));
                        b = fmaf(b, bf_hi(yw[e]), bf_hi(xw[e]));
                    }
                    w[e] = pack_bf16(a, b);
                }
                sts_row16(ot, row, c, w);
            }
            tc_fence_before();
            mbar_arrive(d2_empty);
            if (COMBINE) mbar_arrive(&x_empty[it % XST]);
            fence_proxy_async();
            mbar_arrive(o_full);
            if (leader) {
                if (mbar_wait(o_full, it & 1)) {
                    for (int b = 0; b < DV / 64; ++b) tma_store_2d(&mapOut, smem + Cfg::kOffE + eb * Cfg::kXBytes + b * kBlk, b * 64, (int)((t0 + it) * kTileTokens));
                    tma_store_commit();
                    if (!COMBINE) {
                        tma_store_wait_read0();
                        if (it + 1 < ntiles) open_tile(it + 1);
                    }
                } else {
                    report_timeout(status, 1109);
                }
            }
        }
        if (leader) tma_store_wait_all0();
    } else if (warp >= kVfStatWarp0) {
        // row statistics of the tile -> rstd for the GELU warps, [-mu, sigma] for the extra K step
        const int quarter = warp & 3, row = quarter * 32 + lane;
        for (int it = 0; it < ntiles; ++it) {
            const int st = it % XST, b = it & 1;
            if (ok && !mbar_wait(&x_full[st], (it / XST) & 1)) { ok = false; report_timeout(status, 1105); }
            // buffer b was last used by tile it - 2: its first-layer product and its GELU pass are over once its G tile is complete
            if (ok && it >= 2 && !mbar_wait(&g_full[b], ((it - 2) >> 1) & 1)) { ok = false; report_timeout(status, 1106); }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            float mu, rstd;
            tile_row_stats<DV>(smem_u32(smem + Cfg::kOffX + st * Cfg::kXBytes), row, mu, rstd);
            store_aug_row(tmem + kVfColAug + 8 * b + ((uint32_t)(quarter * 32) << 16), mu, rstd);
            stat[b * kTileTokens + row] = rstd;
            tmem_st_wait();
            tc_fence_before();
            mbar_arrive(&st_full[b]);
        }
    } else {
        // GELU: thread = token row x quarter of the hidden units
        const int quarter = warp & 3, part = (warp - kVfGeluWarp0) >> 2, row = quarter * 32 + lane;
        for (int it = 0; it < ntiles; ++it) {
            const int b = it & 1, par = (it >> 1) & 1;
            if (!mbar_wait(&d1_full[b], par)) { ok = false; report_timeout(status, 1107); }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const float rstd = stat[b * kTileTokens + row];
            const uint32_t ta = tmem + 128 * b + ((uint32_t)(quarter * 32) << 16) + part * HC;
            uint32_t r[HC];
#pragma unroll
            for (int c = 0; c < HC / 16; ++c) tmem_ld16(ta + 16 * c, *reinterpret_cast<uint32_t(*)[16]>(r + 16 * c));
            tmem_ld_wait();
            uint32_t w[HC / 2];
#pragma unroll
            for (int e = 0; e < HC / 2; ++e) {
                const float2 h = __fmul2_rn(make_float2(__uint_as_float(r[2 * e]), __uint_as_float(r[2 * e + 1])), splat2(rstd));
                const float2 g = __fmul2_rn(gelu2_twice(h), splat2(0.5f));
                w[e] = pack_bf16(g.x, g.y);
            }
#pragma unroll
            for (int c = 0; c < HC / 16; ++c)
                tmem_st8(ta + 8 * c, w[8 * c], w[8 * c + 1], w[8 * c + 2], w[8 * c + 3], w[8 * c + 4], w[8 * c + 5], w[8 * c + 6], w[8 * c + 7]);
            tmem_st_wait();
            tc_fence_before();
            mbar_arrive(&g_full[b]);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, 512);
}

// ---- backward of one map (input gradient) ---------------------------------------------------------------------------
// warp 0: TMA (lane 0: weights and X tiles, lane 1: dOut and Yother tiles), warp 1: dg and dxhat MMAs, warp 2: h MMAs, warps
// 3..18: GELU' (thread = token row x quarter of the hidden units), warps 19..22: dy = dOut (.) Yother, row statistics and the residual, warps 23..26: LayerNorm backward,
// warp 27: TMA stores.
// Shared-memory tiles: X (two stages, kept until the tile's output is formed: the LayerNorm backward needs xhat; the result
// is written over the X tile row by row and stored - or added to dX - by TMA from there), dOut and Yother (one stage each,
// free again as soon as dy is formed and the dg product has read it, so the next tile's pair is in flight while this
// tile runs through GELU', the dxhat product and the LayerNorm backward).  Yother is multiplied in place into dy, the A
// operand of the dg product.
// RESIDUAL: the dy warps copy the rows of dOut into tensor memory, where the output warps find them at the end of the tile.
// The two row means of the LayerNorm backward come from the hidden layer, where the GELU' warps already hold the numbers:
//     sum_i dxhat_i = sum_j dh_j c_j,     sum_i dxhat_i xhat_i = sum_j dh_j (h_j - b1'_j)       (dxhat = dh W1'^T, h = xhat W1' + b1')
constexpr int kVbThreads = 28 * 32;
constexpr int kVbGeluWarp0 = 3, kVbProdWarp0 = 19, kVbOutWarp0 = 23, kVbStoreWarp = 27;
constexpr int kVbColDg = 128, kVbColDx = 256, kVbColAug = 384, kVbColRes = 400;   // TMEM columns (h at 0, aug[b] at 384 + 8 b, dOut rows: 64)

template <int DV> struct VbCfg {
    static constexpr int kXBytes = 2 * kBlk;
    static constexpr int kWBytes = DV * DV * 2;
    static constexpr int kAuxBytes = (DV / 64) * 2048;
    static constexpr int kOffX = 0;                              // 2 stages
    static constexpr int kOffDo = 2 * kXBytes;                   // dOut tile
    static constexpr int kOffDy = kOffDo + kXBytes;              // Yother tile -> dy tile
    static constexpr int kOffW1 = kOffDy + kXBytes;
    static constexpr int kOffW2 = kOffW1 + kWBytes;
    static constexpr int kOffAux = kOffW2 + kWBytes;
    static constexpr int kOffStat = kOffAux + kAuxBytes;         // [2][128] x (mu, rstd)
    static constexpr int kOffLnp = kOffStat + 2 * kTileTokens * 8;   // [2][4 parts][128] x (partial of sum dxhat, partial of sum dxhat xhat)
    static constexpr int kOffCb = kOffLnp + 2 * 4 * kTileTokens * 8; // c [DV], b1' [DV] floats
    static constexpr int kOffBars = kOffCb + 2 * DV * 4;
    static constexpr int kSmemUsed = 1024 + kOffBars + 256;
    static_assert(kSmemUsed <= 227 * 1024, "shared memory");
    static constexpr int kSmem = kSmemUsed > 120 * 1024 ? kSmemUsed : 120 * 1024;
};

// X, dOut, Yother, dX [rows][DV] bf16 behind their tensor maps.  dX = J^T (dOut (.) Yother), plus dOut if RESIDUAL (the T
// side: Out = T + ...); with `accumulate` the tile is added to what dX holds instead of overwriting it.
template <int DV, bool RESIDUAL>
__global__ void __launch_bounds__(kVbThreads, 1) tc_vmlp_backward_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapW1,
                                                                         const __grid_constant__ CUtensorMap mapW2, const __grid_constant__ CUtensorMap mapAux,
                                                                         const __grid_constant__ CUtensorMap mapdO, const __grid_constant__ CUtensorMap mapY,
                                                                         const __grid_constant__ CUtensorMap mapdX, const __nv_bfloat16* __restrict__ aux,
                                                                         int accumulate, long long rows, int* status) {
    using Cfg = VbCfg<DV>;
    constexpr int HC = DV / 4;
    extern __shared__ uint8_t smem_raw[];
    grid_launch_dependents();
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    float2* stat = reinterpret_cast<float2*>(smem + Cfg::kOffStat);
    float2* lnp = reinterpret_cast<float2*>(smem + Cfg::kOffLnp);
    float* cb = reinterpret_cast<float*>(smem + Cfg::kOffCb);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::kOffBars);
    uint64_t* x_full = bars;           // [2] TMA
    uint64_t* x_empty = bars + 2;      // [2] 1 arrival: the result tile written over the X tile has been read by its store
    uint64_t* st_full = bars + 4;      // [2] 128 arrivals
    uint64_t* in_full = bars + 6;      // TMA: the dOut and Yother tiles have landed
    uint64_t* dy_full = bars + 7;      // 128 arrivals
    uint64_t* dy_empty = bars + 8;     // MMA commit
    uint64_t* do_free = bars + 9;      // 128 arrivals: the dy warps are done with the dOut tile
    uint64_t* h_full = bars + 10;      // MMA commit
    uint64_t* dh_full = bars + 11;     // 512 arrivals
    uint64_t* dh_free = bars + 12;     // MMA commit (the dxhat product has read dh: the h columns are free)
    uint64_t* dg_full = bars + 13;     // MMA commit
    uint64_t* dg_empty = bars + 14;    // 512 arrivals
    uint64_t* dx_full = bars + 15;     // MMA commit
    uint64_t* dx_empty = bars + 16;    // [2] 128 arrivals, by tile parity
    uint64_t* w_full = bars + 18;      // TMA
    uint64_t* o_full = bars + 19;      // [2] 128 arrivals, by tile parity: the result tile is written
    uint64_t* res_full = bars + 21;    // 128 arrivals (RESIDUAL): the tile's dOut rows are in tensor memory
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 22);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const long long tiles = (rows + kTileTokens - 1) / kTileTokens;
    const long long t0 = tiles * blockIdx.x / gridDim.x, t1 = tiles * (blockIdx.x + 1) / gridDim.x;
    const int ntiles = (int)(t1 - t0);

    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(&x_full[i], 1);
            mbar_init(&x_empty[i], 1);
            mbar_init(&st_full[i], 128);
            mbar_init(&dx_empty[i], 128);
            mbar_init(&o_full[i], 128);
        }
        mbar_init(in_full, 1);
        mbar_init(dy_full, 128);
        mbar_init(dy_empty, 1);
        mbar_init(do_free, 128);
        mbar_init(res_full, 128);
        mbar_init(h_full, 1);
        mbar_init(dh_full, 512);
        mbar_init(dh_free, 1);
        mbar_init(dg_full, 1);
        mbar_init(dg_empty, 512);
        mbar_init(dx_full, 1);
        mbar_init(w_full, 1);
        fence_mbar_init();
        prefetch_tmap(&mapX);
        prefetch_tmap(&mapW1);
        prefetch_tmap(&mapW2);
        prefetch_tmap(&mapAux);
        prefetch_tmap(&mapdO);
        prefetch_tmap(&mapY);
        prefetch_tmap(&mapdX);
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
    // c and b1' (fp32, from the two bf16 halves the folding kernel wrote) for the row means of the LayerNorm backward
    for (int j = tid; j < DV; j += kVbThreads) {
        cb[j] = __bfloat162float(aux[j]) + __bfloat162float(aux[DV + j]);
        cb[DV + j] = __bfloat162float(aux[3 * DV + j]) + __bfloat162float(aux[4 * DV + j]);
    }
    __syncthreads();
    bool ok = true;

    if (warp == 0) {
        if (lane == 0 && ntiles > 0) {
            mbar_arrive_expect_tx(w_full, 2 * Cfg::kWBytes + Cfg::kAuxBytes);
            for (int b = 0; b < DV / 64; ++b) {
                tma_load_2d(smem + Cfg::kOffW1 + b * (DV * 128), &mapW1, w_full, b * 64, 0);
                tma_load_2d(smem + Cfg::kOffW2 + b * (DV * 128), &mapW2, w_full, b * 64, 0);
                tma_load_2d(smem + Cfg::kOffAux + b * 2048, &mapAux, w_full, b * 64, 0);
            }
            for (int it = 0; it < ntiles; ++it) {
                const int st = it & 1, u = it >> 1;
                if (!mbar_wait(&x_empty[st], (u & 1) ^ 1)) { report_timeout(status, 1201); break; }
                mbar_arrive_expect_tx(&x_full[st], DV * kTileTokens * 2);
                for (int b = 0; b < DV / 64; ++b)
                    tma_load_2d(smem + Cfg::kOffX + st * Cfg::kXBytes + b * kBlk, &mapX, &x_full[st], b * 64, (int)((t0 + it) * kTileTokens));
            }
        } else if (lane == 1) {
            // dOut and Yother tiles: free once the dg product of the previous tile has read dy and the dy warps are done with dOut
            for (int it = 0; it < ntiles; ++it) {
                if (it > 0 && !(mbar_wait(dy_empty, (it - 1) & 1) && mbar_wait(do_free, (it - 1) & 1))) { report_timeout(status, 1205); break; }
                mbar_arrive_expect_tx(in_full, 2 * DV * kTileTokens * 2);
                for (int b = 0; b < DV / 64; ++b) {
                    tma_load_2d(smem + Cfg::kOffDo + b * kBlk, &mapdO, in_full, b * 64, (int)((t0 + it) * kTileTokens));
                    tma_load_2d(smem + Cfg::kOffDy + b * kBlk, &mapY, in_full, b * 64, (int)((t0 + it) * kTileTokens));
                }
            }
        }
    } else if (warp == 2) {
        if (lane == 0 && ntiles > 0) {      // h = X W1' + [-mu, sigma] [c; b1']
            const uint32_t idesc1 = idesc_bf16(128, DV, false, true);
            const uint64_t xd0 = smem_desc_sw128(smem_u32(smem + Cfg::kOffX), 16, 1024);
            const uint64_t wd = smem_desc_sw128(smem_u32(smem + Cfg::kOffW1), DV * 128, 1024);
            const uint64_t ad = smem_desc_sw128(smem_u32(smem + Cfg::kOffAux), 2048, 1024);
            bool good = mbar_wait(w_full, 0);
            for (int it = 0; it < ntiles && good; ++it) {
                const int st = it & 1, par = (it >> 1) & 1;
                // the h columns also hold the dh operand of the previous tile: free when its dxhat product has completed
                if (!(mbar_wait(&x_full[st], par) && mbar_wait(&st_full[st], par) && mbar_wait(dh_free, (it & 1) ^ 1))) { good = false; break; }
                tc_fence_after();
                const uint64_t xd = desc_advance(xd0, st * Cfg::kXBytes);
#pragma unroll
                for (int ks = 0; ks < DV / 16; ++ks)
                    umma_bf16(tmem, desc_advance(xd, (ks >> 2) * kBlk + (ks & 3) * 32), desc_advance(wd, ks * 2048), idesc1, ks > 0 ? 1u : 0u);
                umma_bf16_ta(tmem, tmem + kVbColAug + 8 * st, ad, idesc1, 1u);
                umma_commit(h_full);
            }
            if (!good) report_timeout(status, 1202);
        }
    } else if (warp == 1) {
        if (lane == 0 && ntiles > 0) {
            const uint32_t idesc_k = idesc_bf16(128, DV, false, false);
            const uint64_t yd = smem_desc_sw128(smem_u32(smem + Cfg::kOffDy), 16, 1024);       // dy tile, K-major over the output channels
            const uint64_t w2d = smem_desc_sw128(smem_u32(smem + Cfg::kOffW2), 16, 1024);      // W2 [hidden][out] read K-major: N = hidden, K = out
            const uint64_t w1d = smem_desc_sw128(smem_u32(smem + Cfg::kOffW1), 16, 1024);      // W1' [in][hidden] read K-major: N = in, K = hidden
            bool good = mbar_wait(w_full, 0);
            auto issue_dg = [&](int it) -> bool {      // dg = dy W2^T; the GELU' warps of tile it - 1 must have taken their dg
                if (it > 0 && !mbar_wait(dg_empty, (it - 1) & 1)) return false;
                if (!mbar_wait(dy_full, it & 1)) return false;
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < DV / 16; ++ks)
                    umma_bf16(tmem + kVbColDg, desc_advance(yd, (ks >> 2) * kBlk + (ks & 3) * 32), desc_advance(w2d, (ks >> 2) * (DV * 128) + (ks & 3) * 32),
                              idesc_k, ks > 0 ? 1u : 0u);
                umma_commit(dg_full);
                umma_commit(dy_empty);
                return true;
            };
            for (int it = 0; it < ntiles && good; ++it) {
                if (!issue_dg(it)) { good = false; break; }
                // dxhat = dh W1'^T; the output warps must have read the previous tile's dxhat
                if (!mbar_wait(dh_full, it & 1)) { good = false; break; }
                if (it > 0 && !mbar_wait(&dx_empty[(it - 1) & 1], ((it - 1) >> 1) & 1)) { good = false; break; }
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < DV / 16; ++ks)
                    umma_bf16_ta(tmem + kVbColDx, tmem + ((16 * ks) / HC) * HC + ((16 * ks) % HC) / 2,
                                 desc_advance(w1d, (ks >> 2) * (DV * 128) + (ks & 3) * 32), idesc_k, ks > 0 ? 1u : 0u);
                umma_commit(dh_free);
                umma_commit(dx_full);
            }
            if (!good) report_timeout(status, 1203);
        }
    } else if (warp == kVbStoreWarp) {
        // the result tile leaves through TMA; its X stage is free for the next load once the store has read it
        if (lane == 0) {
            for (int it = 0; it < ntiles; ++it) {
                const int st = it & 1;
                if (!mbar_wait(&o_full[st], (it >> 1) & 1)) { report_timeout(status, 1210); break; }
                const uint8_t* src = smem + Cfg::kOffX + st * Cfg::kXBytes;
                for (int b = 0; b < DV / 64; ++b) {
                    if (accumulate) tma_reduce_add_2d(&mapdX, src + b * kBlk, b * 64, (int)((t0 + it) * kTileTokens));
                    else tma_store_2d(&mapdX, src + b * kBlk, b * 64, (int)((t0 + it) * kTileTokens));
                }
                tma_store_commit();
                tma_store_wait_read0();
                mbar_arrive(&x_empty[st]);
            }
            tma_store_wait_all0();
        }
    } else if (warp >= kVbOutWarp0) {
        // LayerNorm backward: dx = rstd (dxhat - mean(dxhat) - xhat mean(dxhat xhat)) (+ dOut); thread = token row.  The result
        // replaces the row of the X tile it was computed from.
        const int quarter = warp & 3, row = quarter * 32 + lane;
        const uint32_t ta = tmem + kVbColDx + ((uint32_t)(quarter * 32) << 16);
        for (int it = 0; it < ntiles; ++it) {
            const int st = it & 1;
            if (ok && !mbar_wait(dx_full, it & 1)) { ok = false; report_timeout(status, 1204); }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const float2 ms = stat[st * kTileTokens + row];
            const float mu = ms.x, rstd = ms.y;
            float s1 = 0.f, s2 = 0.f;
#pragma unroll
            for (int p = 0; p < 4; ++p) {
                const float2 v = lnp[(st * 4 + p) * kTileTokens + row];
                s1 += v.x;
                s2 += v.y;
            }
            const float m1 = s1 * (1.f / DV), m2 = s2 * (1.f / DV);
            // dx = rs acc - rs m1' - rs rstd m2' (x - mu) = rs acc + (k3 x + k4), with rs = rstd / 2: the GELU' warps leave out the
            // factor 1/2 of GELU', so acc, m1' and m2' are twice dxhat and its two means
            const float rs = 0.5f * rstd, k3 = -rs * rstd * m2, k4 = -rs * m1 - k3 * mu;
            const uint32_t xt = smem_u32(smem + Cfg::kOffX + st * Cfg::kXBytes);
            if (RESIDUAL) {
                if (ok && !mbar_wait(res_full, it & 1)) { ok = false; report_timeout(status, 1213); }
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
            }
#pragma unroll 2
            for (int c = 0; c < DV / 16; ++c) {
                uint32_t r[16], xw[8], dw[8], w[8];
                tmem_ld16(ta + 16 * c, r);
                if (RESIDUAL) tmem_ld8(tmem + kVbColRes + ((uint32_t)(quarter * 32) << 16) + 8 * c, dw);
                lds_row16(xt, row, c, xw);
                tmem_ld_wait();
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float2 lin = __ffma2_rn(make_float2(bf_lo(xw[e]), bf_hi(xw[e])), splat2(k3), splat2(k4));
                    float2 v = __ffma2_rn(make_float2(__uint_as_float(r[2 * e]), __uint_as_float(r[2 * e + 1])), splat2(rs), lin);
                    if (RESIDUAL) v = __fadd2_rn(v, make_float2(bf_lo(dw[e]), bf_hi(dw[e])));
                    w[e] = pack_bf16(v.x, v.y);
                }
                sts_row16(xt, row, c, w);
            }
            tc_fence_before();
            mbar_arrive(&dx_empty[st]);
            fence_proxy_async();
            mbar_arrive(&o_full[st]);
        }
    } else if (warp >= kVbProdWarp0) {
        // dy = dOut (.) Yother in place over the Yother tile -> A operand of the dg product (the pair of tiles is ahead of the X
        // tile), then the row statistics of the X tile
        const int t = tid - kVbProdWarp0 * 32;      // 0..127
        const int quarter = warp & 3, row = quarter * 32 + lane;
        constexpr int CPR = DV / 8;                 // 16-byte chunks per row
        const uint32_t dot = smem_u32(smem + Cfg::kOffDo), dyt = smem_u32(smem + Cfg::kOffDy);
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        for (int it = 0; it < ntiles; ++it) {
            const int st = it & 1, par = (it >> 1) & 1;
            if (ok && !mbar_wait(in_full, it & 1)) { ok = false; report_timeout(status, 1211); }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
#pragma unroll 4
            for (int k = 0; k < CPR; ++k) {
                const int idx = k * 128 + t, r = idx / CPR, ch = idx % CPR;
                const uint32_t off = (ch >> 3) * kBlk + sw128_off(r, ch & 7);
                uint32_t a[4], b[4];
                asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3]) : "r"(dot + off) : "memory");
                asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(b[0]), "=r"(b[1]), "=r"(b[2]), "=r"(b[3]) : "r"(dyt + off) : "memory");
                st_shared_v4(dyt + off, mul_bf16x2(a[0], b[0]), mul_bf16x2(a[1], b[1]), mul_bf16x2(a[2], b[2]), mul_bf16x2(a[3], b[3]));
            }
            fence_proxy_async();
            mbar_arrive(dy_full);
            if (!RESIDUAL) mbar_arrive(do_free);
            // statistics: buffer st was last read by the output warps of tile it - 2
            if (ok && !mbar_wait(&x_full[st], par)) { ok = false; report_timeout(status, 1206); }
            if (ok && it >= 2 && !mbar_wait(&dx_empty[st], par ^ 1)) { ok = false; report_timeout(status, 1207); }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            float mu, rstd;
            tile_row_stats<DV>(smem_u32(smem + Cfg::kOffX + st * Cfg::kXBytes), row, mu, rstd);
            store_aug_row(tmem + kVbColAug + 8 * st + lane_base, mu, rstd);
            stat[st * kTileTokens + row] = make_float2(mu, rstd);
            tmem_st_wait();
            tc_fence_before();
            mbar_arrive(&st_full[st]);
            if (RESIDUAL) {
                // the rows of dOut, as they are, into tensor memory for the output warps (one buffer: free once they have
                // finished the previous tile), so that the dOut tile does not have to stay until the end of this one
                if (ok && it > 0 && !mbar_wait(&dx_empty[(it - 1) & 1], ((it - 1) >> 1) & 1)) { ok = false; report_timeout(status, 1212); }
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
#pragma unroll 2
                for (int c = 0; c < DV / 16; ++c) {
                    uint32_t dw[8];
                    lds_row16(dot, row, c, dw);
                    tmem_st8(tmem + kVbColRes + lane_base + 8 * c, dw[0], dw[1], dw[2], dw[3], dw[4], dw[5], dw[6], dw[7]);
                }
                tmem_st_wait();
                tc_fence_before();
                mbar_arrive(res_full);
                mbar_arrive(do_free);
            }
        }
    } else {
        // dh = dg (.) GELU'(h), h = rstd acc: thread = token row x quarter of the hidden units; dh goes back into the h columns
        const int quarter = warp & 3, part = (warp - kVbGeluWarp0) >> 2, row = quarter * 32 + lane;
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        for (int it = 0; it < ntiles; ++it) {
            const int st = it & 1;
            if (!mbar_wait(dg_full, it & 1)) { ok = false; report_timeout(status, 1208); }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            uint32_t dgr[HC];
#pragma unroll
            for (int c = 0; c < HC / 16; ++c) tmem_ld16(tmem + kVbColDg + lane_base + part * HC + 16 * c, *reinterpret_cast<uint32_t(*)[16]>(dgr + 16 * c));
            tmem_ld_wait();
            tc_fence_before();
            mbar_arrive(dg_empty);
            if (!mbar_wait(h_full, it & 1)) { ok = false; report_timeout(status, 1209); }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const float rstd = stat[st * kTileTokens + row].y;
            const uint32_t ta = tmem + lane_base + part * HC;
            float2 p1 = make_float2(0.f, 0.f), p2 = make_float2(0.f, 0.f);
#pragma unroll
            for (int c = 0; c < HC / 16; ++c) {
                uint32_t r[16];
                tmem_ld16(ta + 16 * c, r);
                tmem_ld_wait();
                uint32_t w[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const int j = part * HC + 16 * c + 2 * e;
                    const float2 h = __fmul2_rn(make_float2(__uint_as_float(r[2 * e]), __uint_as_float(r[2 * e + 1])), splat2(rstd));
                    const float2 dg = make_float2(__uint_as_float(dgr[16 * c + 2 * e]), __uint_as_float(dgr[16 * c + 2 * e + 1]));
                    const float2 dh = __fmul2_rn(dg, gelu_grad2_twice(h));      // twice dh: the output warps halve
                    w[e] = pack_bf16(dh.x, dh.y);
                    const float2 dr = make_float2(bf_lo(w[e]), bf_hi(w[e]));      // dh as the dxhat product sees it
                    const float2 cj = *reinterpret_cast<const float2*>(cb + j), bj = *reinterpret_cast<const float2*>(cb + DV + j);
                    p1 = __ffma2_rn(dr, cj, p1);
                    p2 = __ffma2_rn(dr, make_float2(h.x - bj.x, h.y - bj.y), p2);
                }
                tmem_st8(ta + 8 * c, w[0], w[1], w[2], w[3], w[4], w[5], w[6], w[7]);
            }
            lnp[(st * 4 + part) * kTileTokens + row] = make_float2(p1.x + p1.y, p2.x + p2.y);
            tmem_st_wait();
            tc_fence_before();
            mbar_arrive(dh_full);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, 512);
}

// ---- host side ---------------------------------------------------------------------------------------------------------
// Scratch of the value modulation inside the workspace: folded first-layer weights and extra-K-step rows of both maps, and
// the two map outputs Y1 = phi_v1(T), Y2 = phi_v2(V).
struct VmodPlan {
    size_t w1f, aux, y1, y2, end;
};
inline size_t vmod_plan(VmodPlan& p, int d, long long rows, size_t off) {
    auto up = [](size_t x) { return (x + 255) / 256 * 256; };
    p.w1f = off; off = up(off + (size_t)2 * d * d * 2);
    p.aux = off; off = up(off + (size_t)2 * 16 * d * 2);
    p.y1 = off; off = up(off + (size_t)rows * d * 2);
    p.y2 = off; off = up(off + (size_t)rows * d * 2);
    p.end = off;
    return off;
}

template <int DV>
inline hla_status launch_vmod(const VmodPlan& P, long long rows, const hla_vmlp* v, const void* T, const void* V, const void* dOut, void* Out, void* dT,
                              void* dV, int accumulate_dV, bool backward, char* ws, int* status, int sm_count, LaunchRec& rec) {
    using bf = __nv_bfloat16;
    bf* w1f = reinterpret_cast<bf*>(ws + P.w1f);
    bf* aux = reinterpret_cast<bf*>(ws + P.aux);
    bf* y1 = reinterpret_cast<bf*>(ws + P.y1);
    bf* y2 = reinterpret_cast<bf*>(ws + P.y2);
    cudaStream_t st = rec.st;
    VmlpPtrs a[2];
    for (int i = 0; i < 2; ++i)
        a[i] = VmlpPtrs{static_cast<const bf*>(v[i].ln_g), static_cast<const bf*>(v[i].ln_b), static_cast<const bf*>(v[i].W1), static_cast<const bf*>(v[i].b1),
                        static_cast<const bf*>(v[i].W2), static_cast<const bf*>(v[i].b2)};
    rec.begin("vmod_fold");
    vmod_fold_kernel<<<dim3(2, DV / 32), 256, 0, st>>>(a[0], a[1], w1f, aux, DV);
    if (!rec.end()) return HLA_ERR_CUDA;
    CUtensorMap mapT, mapV, mapY1, mapY2, mapW1[2], mapW2[2], mapAux[2];
    if (!make_map_2d(&mapT, T, (size_t)rows, DV, kTileTokens) || !make_map_2d(&mapV, V, (size_t)rows, DV, kTileTokens) ||
        !make_map_2d(&mapY1, y1, (size_t)rows, DV, kTileTokens) || !make_map_2d(&mapY2, y2, (size_t)rows, DV, kTileTokens))
        return HLA_ERR_CUDA;
    for (int i = 0; i < 2; ++i)
        if (!make_map_2d(&mapW1[i], w1f + (size_t)i * DV * DV, DV, DV, DV) || !make_map_2d(&mapW2[i], v[i].W2, DV, DV, DV) ||
            !make_map_2d(&mapAux[i], aux + (size_t)i * 16 * DV, 16, DV, 16))
            return HLA_ERR_CUDA;
    if (!set_smem(tc_vmlp_forward_kernel<DV, false>, VfCfg<DV, false>::kSmem) || !set_smem(tc_vmlp_forward_kernel<DV, true>, VfCfg<DV, true>::kSmem) ||
        !set_smem(tc_vmlp_backward_kernel<DV, false>, VbCfg<DV>::kSmem) || !set_smem(tc_vmlp_backward_kernel<DV, true>, VbCfg<DV>::kSmem))
        return HLA_ERR_CUDA;
    const long long tiles = (rows + kTileTokens - 1) / kTileTokens;
    const int grid = (int)(tiles < sm_count ? tiles : sm_count);
    // Y2 = phi_v2(V)
    rec.begin("tc_vmlp_forward");
    launch_pdl(tc_vmlp_forward_kernel<DV, false>, grid, dim3(kVfThreads), VfCfg<DV, false>::kSmem, st, mapV, mapW1[1], mapW2[1], mapAux[1], mapY2, mapY2, rows, status);
    if (!rec.end()) return HLA_ERR_CUDA;
    if (!backward) {      // Out = T + phi_v1(T) (.) Y2
        CUtensorMap mapOut;
        if (!make_map_2d(&mapOut, Out, (size_t)rows, DV, kTileTokens)) return HLA_ERR_CUDA;
        rec.begin("tc_vmlp_forward_combine");
        launch_pdl(tc_vmlp_forward_kernel<DV, true>, grid, dim3(kVfThreads), VfCfg<DV, true>::kSmem, st, mapT, mapW1[0], mapW2[0], mapAux[0], mapY2, mapOut, rows, status);
        return rec.end() ? HLA_OK : HLA_ERR_CUDA;
    }
    rec.begin("tc_vmlp_forward");      // Y1 = phi_v1(T)
    launch_pdl(tc_vmlp_forward_kernel<DV, false>, grid, dim3(kVfThreads), VfCfg<DV, false>::kSmem, st, mapT, mapW1[0], mapW2[0], mapAux[0], mapY1, mapY1, rows, status);
    if (!rec.end()) return HLA_ERR_CUDA;
    CUtensorMap mapdO, mapdT, mapdV;
    if (!make_map_2d(&mapdO, dOut, (size_t)rows, DV, kTileTokens) || !make_map_2d(&mapdT, dT, (size_t)rows, DV, kTileTokens) ||
        !make_map_2d(&mapdV, dV, (size_t)rows, DV, kTileTokens))
        return HLA_ERR_CUDA;
    rec.begin("tc_vmlp_backward_t");   // dT = dOut + J1^T (dOut (.) Y2)
    launch_pdl(tc_vmlp_backward_kernel<DV, true>, grid, dim3(kVbThreads), VbCfg<DV>::kSmem, st, mapT, mapW1[0], mapW2[0], mapAux[0], mapdO, mapY2, mapdT,
               (const bf*)aux, 0, rows, status);
    if (!rec.end()) return HLA_ERR_CUDA;
    rec.begin("tc_vmlp_backward_v");   // dV (+)= J2^T (dOut (.) Y1)
    launch_pdl(tc_vmlp_backward_kernel<DV, false>, grid, dim3(kVbThreads), VbCfg<DV>::kSmem, st, mapV, mapW1[1], mapW2[1], mapAux[1], mapdO, mapY1, mapdV,
               (const bf*)(aux + (size_t)16 * DV), accumulate_dV, rows, status);
    return rec.end() ? HLA_OK : HLA_ERR_CUDA;
}

}  // namespace tc
}  // namespace hla
