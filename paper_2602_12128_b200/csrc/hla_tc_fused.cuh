// Fused query side of the forward (Algorithm 1 step 4 for phi_q, then the readout of Eq. "hla.la.form" with the
// normaliser):  Q tile -> h = Q W1 -> GELU -> q = ReLU(G W2 + b2) -> monomials q_a q_b q_c -> [num | eta] = mono [Csym | zsym]
// -> o = num / (eta + eps).  The feature map is bound by plain arithmetic and the readout by the write of O, so one
// kernel that does both hides the write stream under the arithmetic; the query features never make a round trip through
// global memory before they are used (they are still stored, for the backward).
//
// Persistent over (head, 128-token tile).  Warp roles:
//   warp 0       TMA: W1 once, one Q tile per work item
//   warp 1       MMAs: second layer D2 = G W2
//   warp 27      MMAs: readout acc = mono * state operand; TMA of the state operand when the head changes
//   warp 2       MMAs: first layer  D1 = Q W1
//   warps 3..18  GELU: thread = token row x quarter of the hidden units
//   warps 19..22 features: ReLU, store q, monomial row -> A operand of the readout product
//   warps 23..26 readout epilogue: acc -> 1 / (eta + eps) -> bf16 -> staging tile -> TMA store of O
#pragma once
#include "hla_tc_phi.cuh"

namespace hla {
namespace tc {

constexpr int kFqThreads = 28 * 32;
constexpr int kFqGeluWarp0 = 3, kFqFeatWarp0 = 19, kFqOutWarp0 = 23, kFqReadoutMmaWarp = 27;

template <int DV, int F> struct FqCfg {
    static constexpr int kXBytes = kTileTokens * DV * 2;
    static constexpr int kW1Bytes = DV * DV * 2;
    static constexpr int kW2Bytes = (DV / 64) * 2048;            // [16 rows][DV] bf16, K-major
    static constexpr int kNmma = DV + 16;                        // readout product: d value channels, then the normaliser column
    static constexpr int kB3Block = ((kNmma * 128 + 1023) / 1024) * 1024;   // one 64-monomial block of the state operand
    static constexpr int kB3Bytes = MT<F>::kBlocks * kNmma * 128;           // bytes its TMA loads deliver
    static constexpr int kOffX = 0;                              // 2 Q tiles (the load of a tile takes longer than a tile's arithmetic)
    static constexpr int kOffW1 = 2 * kXBytes;                   // (the GELU tile lives in TMEM)
    static constexpr int kOffW2 = kOffW1 + kW1Bytes;
    static constexpr int kOffB3 = kOffW2 + ((kW2Bytes + 1023) / 1024) * 1024;      // state operand of the current head
    static constexpr int kOffA = kOffB3 + MT<F>::kBlocks * kB3Block;               // monomial tile
    static constexpr int kOffO = kOffA + MT<F>::kBlocks * kBlk;  // O staging tile
    // b1 is added on the tensor cores by a ninth K step of the first-layer product: A = a constant tile whose K column
    // 0 is 1, B = a tile whose K row 0 is b1 (both zero elsewhere)
    static constexpr int kOffOnes = kOffO + kXBytes;             // [128 rows][64 K] bf16, K-major (16 K columns used)
    static constexpr int kB1Bytes = (DV / 64) * 2048;            // [16 K rows][DV] bf16, MN-major
    static constexpr int kOffB1 = kOffOnes + kBlk;
    static constexpr int kOffBias = kOffB1 + kB1Bytes;           // b1[DV] (unused by the kernel), b2[16] floats
    static constexpr int kOffBars = kOffBias + (DV + 16) * 4;
    static constexpr int kSmemUsed = 1024 + kOffBars + 256;
    static_assert(kSmemUsed <= 227 * 1024, "shared memory");
    static constexpr int kSmem = kSmemUsed > 120 * 1024 ? kSmemUsed : 120 * 1024;   // one CTA per SM (512 TMEM columns)
};

// Q [BH][N][DV] bf16 (3-D map, rows past N read as zero), O the same (stores are clipped at N).  READOUT = false: the feature
// map only (the causal operator reads its states tile by tile in a sweep of its own and needs just the query features):
// the readout product, its epilogue and the monomial tile are left out, O and eta are not written.
template <int DV, int F, bool READOUT = true>
__global__ void __launch_bounds__(kFqThreads, 1) tc_phiq_readout_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapW1,
                                                                        const __grid_constant__ CUtensorMap mapB3, const __grid_constant__ CUtensorMap mapO,
                                                                        const __nv_bfloat16* __restrict__ b1g, const __nv_bfloat16* __restrict__ W2g,
                                                                        const __nv_bfloat16* __restrict__ b2g, float* __restrict__ qf_out,
                                                                        float* __restrict__ eta_out, int N, int BH, float eps, int* status) {
    using Cfg = FqCfg<DV, F>;
    using M = MT<F>;
    constexpr int DP = M::kDphi;
    constexpr int HC = DV / 4;          // hidden units per GELU thread
    extern __shared__ uint8_t smem_raw[];
    grid_launch_dependents();
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    float* bias = reinterpret_cast<float*>(smem + Cfg::kOffBias);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::kOffBars);
    uint64_t* x_full = bars;           // [2] TMA   (x_full[1], x_empty[1] live at bars + 22, + 23)
    uint64_t* x_empty = bars + 1;      // [2] MMA commit
    uint64_t* d1_full = bars + 2;      // [2] MMA commit
    uint64_t* g_full = bars + 6;       // 512 arrivals (bars + 7 unused)
    uint64_t* g_free = bars + 8;       // MMA commit (bars + 9 unused)
    uint64_t* d2_full = bars + 10;     // [2] MMA commit
    uint64_t* d2_empty = bars + 12;    // [2] 128 arrivals
    uint64_t* a_full = bars + 14;      // 128 arrivals
    uint64_t* a_empty = bars + 15;     // MMA commit
    uint64_t* acc_full = bars + 16;    // MMA commit
    uint64_t* acc_empty = bars + 17;   // 128 arrivals
    uint64_t* b3_full = bars + 18;     // TMA
    uint64_t* b3_free = bars + 19;     // MMA commit
    uint64_t* w_full = bars + 20;      // TMA
    uint64_t* x_full1 = bars + 22;
    uint64_t* x_empty1 = bars + 23;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 24);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tiles_per_head = (N + kTileTokens - 1) / kTileTokens;
    const long long total = (long long)BH * tiles_per_head;
    const int w0 = (int)(total * blockIdx.x / gridDim.x), w1 = (int)(total * (blockIdx.x + 1) / gridDim.x);
    const int nwork = w1 - w0;

    // second-layer weights as a K-major MMA operand [16 rows (outputs, 6 used)][DV], and the biases
    for (int i = tid; i < Cfg::kW2Bytes / 16; i += kFqThreads) reinterpret_cast<uint4*>(smem + Cfg::kOffW2)[i] = make_uint4(0, 0, 0, 0);
    __syncthreads();
    for (int i = tid; i < DV * DP; i += kFqThreads) {
        const int j = i / DP, o = i % DP;
        uint8_t* base = smem + Cfg::kOffW2 + (j >> 6) * 2048;
        *reinterpret_cast<__nv_bfloat16*>(base + sw128_off(o, (j & 63) >> 3) + (j & 7) * 2) = half_bf16(W2g[j * DP + o]);
    }
    for (int i = tid; i < (kBlk + Cfg::kB1Bytes) / 16; i += kFqThreads) reinterpret_cast<uint4*>(smem + Cfg::kOffOnes)[i] = make_uint4(0, 0, 0, 0);
    __syncthreads();
    for (int i = tid; i < kTileTokens; i += kFqThreads)
        *reinterpret_cast<__nv_bfloat16*>(smem + Cfg::kOffOnes + sw128_off(i, 0)) = __float2bfloat16_rn(1.f);
    for (int j = tid; j < DV; j += kFqThreads)      // K row 0 of the MN-major tile: 64-column block j / 64, no swizzle in row 0
        *reinterpret_cast<__nv_bfloat16*>(smem + Cfg::kOffB1 + (j >> 6) * 2048 + (j & 63) * 2) = b1g[j];
    for (int j = tid; j < DV + 16; j += kFqThreads) bias[j] = j < DV ? __bfloat162float(b1g[j]) : (j - DV < DP ? __bfloat162float(b2g[j - DV]) : 0.f);
    fence_proxy_async();
    if (tid == 0) {
        mbar_init(x_full, 1);
        mbar_init(x_empty, 1);
        mbar_init(x_full1, 1);
        mbar_init(x_empty1, 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(&d1_full[i], 1);
            mbar_init(&g_full[i], 512);
            mbar_init(&g_free[i], 1);
            mbar_init(&d2_full[i], 1);
            mbar_init(&d2_empty[i], 128);
        }
        mbar_init(a_full, 128);
        mbar_init(a_empty, 1);
        mbar_init(acc_full, 1);
        mbar_init(acc_empty, 128);
        mbar_init(b3_full, 1);
        mbar_init(b3_free, 1);
        mbar_init(w_full, 1);
        fence_mbar_init();
        prefetch_tmap(&mapQ);
        prefetch_tmap(&mapW1);
        prefetch_tmap(&mapB3);
        prefetch_tmap(&mapO);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;     // D1[b] at columns 128*b, D2[b] at 256 + 32*b, readout accumulator at 320
    grid_dependency_wait();
    bool ok = true;

    if (warp == 0) {
        if (lane == 0 && nwork > 0) {
            mbar_arrive_expect_tx(w_full, Cfg::kW1Bytes);
            for (int b = 0; b < DV / 64; ++b) tma_load_2d(smem + Cfg::kOffW1 + b * (DV * 128), &mapW1, w_full, b * 64, 0);
            for (int it = 0; it < nwork; ++it) {
                const int work = w0 + it, bh = work / tiles_per_head, tile = work % tiles_per_head;
                const int st = it & 1, u = it >> 1;
                uint64_t* xf = st ? x_full1 : x_full;
                if (!mbar_wait(st ? x_empty1 : x_empty, (u & 1) ^ 1)) { report_timeout(status, 701); break; }
                mbar_arrive_expect_tx(xf, Cfg::kXBytes);
                for (int b = 0; b < DV / 64; ++b) tma_load_3d(smem + Cfg::kOffX + st * Cfg::kXBytes + b * kBlk, &mapQ, xf, b * 64, tile * kTileTokens, bh);
            }
        }
    } else if (warp == 2) {
        if (lane == 0 && nwork > 0) {      // D1[b] = Q tile * W1
            const uint32_t idesc1 = idesc_bf16(128, DV, false, true);   // Q K-major, W1 [in][hidden] MN-major
            const uint64_t xd = smem_desc_sw128(smem_u32(smem + Cfg::kOffX), 16, 1024);
            const uint64_t wd = smem_desc_sw128(smem_u32(smem + Cfg::kOffW1), DV * 128, 1024);
            const uint64_t od = smem_desc_sw128(smem_u32(smem + Cfg::kOffOnes), 16, 1024);
            const uint64_t bd = smem_desc_sw128(smem_u32(smem + Cfg::kOffB1), 2048, 1024);
            bool good = mbar_wait(w_full, 0);
            for (int it = 0; it < nwork && good; ++it) {
                const int b = it & 1, par = (it >> 1) & 1;      // accumulator buffer and Q stage alternate together
                // D1[b] also holds the GELU tile of work item it - 2 (packed over the columns that were read): free when that
                // item's second-layer product has completed
                if (!(mbar_wait(b ? x_full1 : x_full, par) && mbar_wait(&g_free[b], par ^ 1))) { good = false; break; }
                tc_fence_after();
                const uint64_t xs = desc_advance(xd, b * Cfg::kXBytes);
#pragma unroll
                for (int ks = 0; ks < DV / 16; ++ks)
                    umma_bf16(tmem + 128 * b, desc_advance(xs, (ks >> 2) * kBlk + (ks & 3) * 32), desc_advance(wd, ks * 2048), idesc1, ks > 0 ? 1u : 0u);
                umma_bf16(tmem + 128 * b, od, bd, idesc1, 1u);      // + 1 * b1
                umma_commit(&d1_full[b]);
                umma_commit(b ? x_empty1 : x_empty);
            }
            if (!good) report_timeout(status, 702);
        }
    } else if (warp == 1) {
        if (lane == 0 && nwork > 0) {      // D2[b] = G[b] * W2
            const uint32_t idesc2 = idesc_bf16(128, 16, false, false);           // G from TMEM, W2 operand K-major
            const uint64_t vd = smem_desc_sw128(smem_u32(smem + Cfg::kOffW2), 16, 1024);
            bool good = true;
            for (int it = 0; it < nwork && good; ++it) {
                const int b = it & 1, par = (it >> 1) & 1;
                if (!(mbar_wait(&g_full[b], par) && mbar_wait(&d2_empty[b], par ^ 1))) { good = false; break; }
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < DV / 16; ++ks)
                    umma_bf16_ta(tmem + 256 + 32 * b, tmem + 128 * b + ((16 * ks) / HC) * HC + ((16 * ks) % HC) / 2,
                                 desc_advance(vd, (ks >> 2) * 2048 + (ks & 3) * 32), idesc2, ks > 0 ? 1u : 0u);
                umma_commit(&g_free[b]);
                umma_commit(&d2_full[b]);
            }
            if (!good) report_timeout(status, 703);
        }
    } else if (warp == kFqReadoutMmaWarp) {
        if (READOUT && lane == 0 && nwork > 0) {      // [num | eta] = monomial tile * state operand of the tile's head
            const uint32_t idesc3 = idesc_bf16(128, Cfg::kNmma, false, false);   // monomial tile K-major, state operand K-major over the monomials
            const uint64_t ad = smem_desc_sw128(smem_u32(smem + Cfg::kOffA), 16, 1024);
            const uint64_t bd = smem_desc_sw128(smem_u32(smem + Cfg::kOffB3), 16, 1024);
            static_assert(Cfg::kB3Block % 16 == 0, "descriptor advance");
            int cur_bh = -1, nload = 0;
            bool good = true;
            for (int it = 0; it < nwork && good; ++it) {
                const int bh = (w0 + it) / tiles_per_head;
                if (bh != cur_bh) {
                    if (cur_bh >= 0) {   // every product that reads the old state operand must have finished
                        umma_commit(b3_free);
                        if (!mbar_wait(b3_free, (nload - 1) & 1)) { good = false; break; }
                    }
                    mbar_arrive_expect_tx(b3_full, Cfg::kB3Bytes);
                    for (int b = 0; b < M::kBlocks; ++b) tma_load_2d(smem + Cfg::kOffB3 + b * Cfg::kB3Block, &mapB3, b3_full, b * 64, bh * Cfg::kNmma);
                    if (!mbar_wait(b3_full, nload & 1)) { good = false; break; }
                    ++nload;
                    cur_bh = bh;
                }
                if (!(mbar_wait(a_full, it & 1) && mbar_wait(acc_empty, (it & 1) ^ 1))) { good = false; break; }
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < M::kPad / 16; ++ks)
                    umma_bf16(tmem + 320, desc_advance(ad, (ks >> 2) * kBlk + (ks & 3) * 32), desc_advance(bd, (ks >> 2) * Cfg::kB3Block + (ks & 3) * 32), idesc3,
                              ks > 0 ? 1u : 0u);
                umma_commit(a_empty);
                umma_commit(acc_full);
            }
            if (!good) report_timeout(status, 709);
        }
    } else if (warp >= kFqOutWarp0) {      // warps 23..26 (warp 27 was handled above)
        // readout epilogue: o = num / (eta + eps); thread = token row (TMEM lane)
        const int quarter = warp & 3, row = quarter * 32 + lane;
        const bool leader = warp == kFqOutWarp0 && lane == 0;
        const uint32_t ta = tmem + 320 + ((uint32_t)(quarter * 32) << 16);
        const uint32_t os = smem_u32(smem + Cfg::kOffO);
        for (int it = 0; READOUT && it < nwork; ++it) {
            const int work = w0 + it, bh = work / tiles_per_head, tile = work % tiles_per_head;
            if (ok && !mbar_wait(acc_full, it & 1)) { ok = false; report_timeout(status, 704); }
            ok = __all_sync(0xffffffffu, ok);
            if (leader) tma_store_wait_read0();        // the staging tile has been read by the previous tile's store
            named_barrier(3, 128);                     // every epilogue thread arrives, timed out or not
            float eta = 0.f;
            if (ok) {
                tc_fence_after();
                uint32_t re[8];
                tmem_ld8(ta + DV, re);
                tmem_ld_wait();
                eta = __uint_as_float(re[0]);
                const float rinv = 1.f / (eta + eps);
#pragma unroll
                for (int c = 0; c < DV / 16; ++c) {
                    uint32_t r[16];
                    tmem_ld16(ta + 16 * c, r);
                    tmem_ld_wait();
                    if (c == DV / 16 - 1) {            // the accumulator is in registers: the next tile's product may overwrite it
                        tc_fence_before();
                        mbar_arrive(acc_empty);
                    }
                    uint32_t w[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) w[e] = pack_bf16(__uint_as_float(r[2 * e]) * rinv, __uint_as_float(r[2 * e + 1]) * rinv);
                    const uint32_t blk = os + (c >> 2) * kBlk;
                    st_shared_v4(blk + sw128_off(row, (2 * c) & 7), w[0], w[1], w[2], w[3]);
                    st_shared_v4(blk + sw128_off(row, (2 * c + 1) & 7), w[4], w[5], w[6], w[7]);
                }
                fence_proxy_async();
            }
            named_barrier(2, 128);
            if (ok && leader) {
                for (int b = 0; b < DV / 64; ++b) tma_store_3d(&mapO, smem + Cfg::kOffO + b * kBlk, b * 64, tile * kTileTokens, bh);
                tma_store_commit();
            }
            const int tok = tile * kTileTokens + row;
            if (ok && tok < N) eta_out[(size_t)bh * N + tok] = eta;
        }
        if (READOUT && leader) tma_store_wait_all0();
    } else if (warp >= kFqFeatWarp0) {
        // q = ReLU(D2 + b2) -> global memory (kept for the backward); monomial row -> A operand of the readout product
        const int quarter = warp & 3, row = quarter * 32 + lane;
        const float* b2s = bias + DV;
        for (int it = 0; it < nwork; ++it) {
            const int work = w0 + it, bh = work / tiles_per_head, tile = work % tiles_per_head, b = it & 1;
            if (!mbar_wait(&d2_full[b], (it >> 1) & 1)) { ok = false; report_timeout(status, 705); }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            uint32_t r[16];
            if constexpr (DP <= 8) tmem_ld8(tmem + 256 + 32 * b + ((uint32_t)(quarter * 32) << 16), *reinterpret_cast<uint32_t(*)[8]>(r));
            else tmem_ld16(tmem + 256 + 32 * b + ((uint32_t)(quarter * 32) << 16), r);
            tmem_ld_wait();
            tc_fence_before();
            mbar_arrive(&d2_empty[b]);
            const int tok = tile * kTileTokens + row;
            float q[DP];
#pragma unroll
            for (int o = 0; o < DP; ++o) q[o] = tok < N ? fmaxf(__uint_as_float(r[o]) + b2s[o], 0.f) : 0.f;
            if (tok < N) store_feat<DP>(qf_out + ((size_t)bh * N + tok) * DP, q);
            if (!READOUT) continue;
            float mono[M::kN];
            query_monomials_t<F>(q, mono);
            if (!mbar_wait(a_empty, (it & 1) ^ 1)) { ok = false; report_timeout(status, 706); }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            store_mono_row_t<F>(smem_u32(smem + Cfg::kOffA), row, mono, 1.f);
            fence_proxy_async();
            mbar_arrive(a_full);
        }
    } else {
        // GELU: thread = token row x quarter of the hidden units
        const int quarter = warp & 3, part = (warp - kFqGeluWarp0) >> 2;
        for (int it = 0; it < nwork; ++it) {
            const int b = it & 1, par = (it >> 1) & 1;
            if (!mbar_wait(&d1_full[b], par)) { ok = false; report_timeout(status, 707); }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t ta = tmem + 128 * b + ((uint32_t)(quarter * 32) << 16) + part * HC;
            uint32_t r[HC];
#pragma unroll
            for (int c = 0; c < HC / 16; ++c) tmem_ld16(ta + 16 * c, *reinterpret_cast<uint32_t(*)[16]>(r + 16 * c));
            tmem_ld_wait();
            // The GELU outputs go back into TMEM as the second layer's A operand: bf16 pairs packed over the first half of
            // the h columns this thread has just read (hidden units 16 c .. 16 c + 15 of its range -> 8 columns).
            uint32_t w[HC / 2];
#pragma unroll
            for (int c = 0; c < HC / 16; ++c) {
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float2 g = gelu2_twice(make_float2(__uint_as_float(r[16 * c + 2 * e]), __uint_as_float(r[16 * c + 2 * e + 1])));
                    w[8 * c + e] = pack_bf16(g.x, g.y);
                }
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

template <int DV, int F, bool READOUT>
inline hla_status launch_phiq_readout(const Plan& P, const Dims& D, int BH, const hla_mlp* phi_q, const void* Q, void* O, char* ws,
                                      const hla_ws_layout& L, int sm_count, LaunchRec& rec) {
    CUtensorMap mapQ, mapW1, mapB3, mapO;
    __nv_bfloat16* b3 = reinterpret_cast<__nv_bfloat16*>(ws + P.b3);
    if (!make_map_bhnd(&mapQ, Q, BH, D.N, DV, kTileTokens) || !make_map_bhnd(&mapO, O, BH, D.N, DV, kTileTokens) ||
        !make_map_2d(&mapW1, phi_q->W1, DV, DV, DV) || !make_map_2d(&mapB3, b3, (size_t)BH * (DV + 16), MT<F>::kPad, DV + 16))
        return HLA_ERR_CUDA;
    if (!set_smem(tc_phiq_readout_kernel<DV, F, READOUT>, FqCfg<DV, F>::kSmem)) return HLA_ERR_CUDA;
    const int tiles = (D.N + kTileTokens - 1) / kTileTokens;
    const long long total = (long long)BH * tiles;
    const int grid = (int)(total < sm_count ? total : sm_count);
    rec.begin(READOUT ? "tc_phiq_readout" : "tc_phiq");
    launch_pdl(tc_phiq_readout_kernel<DV, F, READOUT>, grid, dim3(kFqThreads), FqCfg<DV, F>::kSmem, rec.st,
        mapQ, mapW1, mapB3, mapO, static_cast<const __nv_bfloat16*>(phi_q->b1), static_cast<const __nv_bfloat16*>(phi_q->W2),
        static_cast<const __nv_bfloat16*>(phi_q->b2), reinterpret_cast<float*>(ws + L.qf), reinterpret_cast<float*>(ws + L.eta), D.N, BH, D.eps,
        reinterpret_cast<int*>(ws + L.status));
    return rec.end() ? HLA_OK : HLA_ERR_CUDA;
}

inline hla_status phiq_readout(const Plan& P, const Dims& D, int BH, const hla_mlp* phi_q, const void* Q, void* O, char* ws, const hla_ws_layout& L,
                               int sm_count, LaunchRec& rec, bool readout = true) {
    if (D.F == 3) {
        if (!readout) {
            if (D.d == 128) return launch_phiq_readout<128, 3, false>(P, D, BH, phi_q, Q, O, ws, L, sm_count, rec);
            return launch_phiq_readout<64, 3, false>(P, D, BH, phi_q, Q, O, ws, L, sm_count, rec);
        }
        if (D.d == 128) return launch_phiq_readout<128, 3, true>(P, D, BH, phi_q, Q, O, ws, L, sm_count, rec);
        return launch_phiq_readout<64, 3, true>(P, D, BH, phi_q, Q, O, ws, L, sm_count, rec);
    }
    if (!readout) return HLA_ERR_UNSUPPORTED;
    if (D.d == 128) return launch_phiq_readout<128, 2, true>(P, D, BH, phi_q, Q, O, ws, L, sm_count, rec);
    return launch_phiq_readout<64, 2, true>(P, D, BH, phi_q, Q, O, ws, L, sm_count, rec);
}

}  // namespace tc
}  // namespace hla
