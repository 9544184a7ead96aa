// Fused key side of the forward (Algorithm 1 step 4 for phi_k1..3, then the state build of Theorem 4.2 with the
// key-side sum of the normaliser paragraph):
//   K tile -> for each key map m: h = K W1[m] + b1[m] -> GELU -> k^m = ReLU(G W2[m] + b2[m])
//          -> folded key tile Tsym_k (56 monomials per token) -> Csym^T[d x 64] += V_tile^T * Tsym_k tile,  zsym += column sums.
// The three feature maps are bound by plain arithmetic and the state build by the read of V, so one kernel that does
// both hides the V stream under the arithmetic; the key features never make a round trip through global memory before
// they are used (they are still stored: the backward needs them).
//
// Persistent over (head, 128-token tile): CTA c owns the contiguous work items [total c / G, total (c + 1) / G).  A run of
// items of one head is a "piece" of that head: its accumulator is drained to the partial-state slot (head, piece), piece
// = c - (first CTA that touches the head), and the reduction sums a head's pieces in that fixed order.
//
// Warp roles:
//   warp 0        TMA: the three W1 once, one K tile per work item
//   warp 1        MMAs: second layer D2 = G W2[m]
//   warp 2        MMAs: first layer  D1 = K W1[m] (+ b1 as a ninth K step)
//   warps 3..18   GELU: thread = token row x quarter of the hidden units
//   warps 19..22  features: ReLU, store k^m, folded key row -> B operand of the state product; drain of a finished piece
//   warp 23       state product Csym^T += V^T Tsym_k, and the TMA loads of V
//   warps 24..27  zsym: column sums of the folded key tile (16 columns per warp)
#pragma once
#include <utility>

#include "hla_tc_phi.cuh"

namespace hla {
namespace tc {

constexpr int kFkThreads = 28 * 32;
constexpr int kFkGeluWarp0 = 3, kFkFeatWarp0 = 19, kFkStateWarp = 23, kFkZWarp0 = 24, kFkZWarps = 4;
constexpr int kFkB1Row = 12;        // K row of the staged W2 tiles that carries b1 (rows 6..15 are padding of the second layer)

// TMEM columns (D1[b] at 128 b).  F = 3: D2[b] at 256 + 32 b (16 used), the constant A operand of the bias step (8 columns, K column
// kFkB1Row is 1) at 272, G[b] (bf16 pairs) at 320 + 64 b, the Csym^T accumulator (64 columns, lane = value channel) at 448.
// F = 2 needs 80 accumulator columns: G[b] at 256 + 64 b, D2[b] at 384 + 16 b, the constant operand at 416, Csym^T at 432.
template <int F> struct FkCols {
    static constexpr int kD2 = F == 3 ? 256 : 384, kD2Stride = F == 3 ? 32 : 16;
    static constexpr int kOnes = F == 3 ? 272 : 416;
    static constexpr int kG = F == 3 ? 320 : 256;
    static constexpr int kC = F == 3 ? 448 : 432;
};

template <int DV, int F> struct FkCfg {
    static constexpr int NM = MT<F>::kMaps;
    static constexpr int kXBytes = kTileTokens * DV * 2;
    static constexpr int kW1Bytes = DV * DV * 2;
    static constexpr int kW2Bytes = (DV / 64) * 2048;            // [16 rows][DV] bf16 per map
    static constexpr int kOffX = 0;                              // 2 K tiles
    static constexpr int kOffW1 = 2 * kXBytes;
    static constexpr int kOffW2 = kOffW1 + NM * kW1Bytes;
    static constexpr int kOffV = ((kOffW2 + NM * kW2Bytes + 1023) / 1024) * 1024;   // V tile: two 64-column blocks (the second stays zero for d = 64)
    static constexpr int kOffF = kOffV + 2 * kBlk;               // folded key tile
    static constexpr int kOffB2 = kOffF + MT<F>::kBlocks * kBlk; // b2: NM x 16 floats
    static constexpr int kOffBars = kOffB2 + 256;
    static constexpr int kSmemUsed = 1024 + kOffBars + 256;
    static_assert(kSmemUsed <= 227 * 1024, "shared memory");
    static constexpr int kSmem = kSmemUsed > 120 * 1024 ? kSmemUsed : 120 * 1024;   // one CTA per SM (512 TMEM columns)
};

// (a, b, c) of monomial m in lexicographic order, packed as 36 a + 6 b + c.
__host__ __device__ constexpr int mono_abc(int m) {
    int idx = 0;
    for (int a = 0; a < 6; ++a)
        for (int b = a; b < 6; ++b)
            for (int c = b; c < 6; ++c) {
                if (idx == m) return 36 * a + 6 * b + c;
                ++idx;
            }
    return 0;
}

// Folded key feature M from the pair sums s12 (see key_folded) and k3; zero for the padding monomials.
template <int M>
__device__ __forceinline__ float folded_value(const float (&s12)[6][6], const float (&k3)[6]) {
    if constexpr (M >= kMono) {
        return 0.f;
    } else {
        constexpr int abc = mono_abc(M), a = abc / 36, b = (abc / 6) % 6, c = abc % 6;
        if constexpr (a == b && b == c) return s12[a][a] * k3[a];
        else if constexpr (a == b) return fmaf(s12[a][a], k3[c], s12[a][c] * k3[a]);
        else if constexpr (b == c) return fmaf(s12[a][c], k3[c], s12[c][c] * k3[a]);
        else return fmaf(s12[a][b], k3[c], fmaf(s12[a][c], k3[b], s12[b][c] * k3[a]));
    }
}
template <int C, int... E>
__device__ __forceinline__ void folded_chunk_store(uint32_t blk, uint32_t row, const float (&s12)[6][6], const float (&k3)[6], std::integer_sequence<int, E...>) {
    const float v[8] = {folded_value<8 * C + E>(s12, k3)...};
    st_shared_v4(blk + sw128_off(row, C), pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
}
// One row of the folded key tile (56 values, 8 zeros), 16 bytes at a time so that only a few values are live at once.
template <int... C>
__device__ __forceinline__ void folded_row_store(uint32_t blk, uint32_t row, const float (&s12)[6][6], const float (&k3)[6], std::integer_sequence<int, C...>) {
    (folded_chunk_store<C>(blk, row, s12, k3, std::make_integer_sequence<int, 8>{}), ...);
}

// The same for the 2-factor geometry: monomial M = (a <= b) of 12 features, value k1[a] k2[b] + k1[b] k2[a] (a < b), k1[a] k2[a] (a == b).
__host__ __device__ constexpr int mono_ab2(int m) {
    int idx = 0;
    for (int a = 0; a < 12; ++a)
        for (int b = a; b < 12; ++b) {
            if (idx == m) return 12 * a + b;
            ++idx;
        }
    return 0;
}
template <int M>
__device__ __forceinline__ float folded_value2(const float (&k1)[12], const float (&k2)[12]) {
    if constexpr (M >= MT<2>::kN) {
        return 0.f;
    } else {
        constexpr int ab = mono_ab2(M), a = ab / 12, b = ab % 12;
        if constexpr (a == b) return k1[a] * k2[a];
        else return fmaf(k1[a], k2[b], k1[b] * k2[a]);
    }
}
template <int C, int... E>
__device__ __forceinline__ void folded_chunk_store2(uint32_t tile, uint32_t row, const float (&k1)[12], const float (&k2)[12], std::integer_sequence<int, E...>) {
    const float v[8] = {folded_value2<8 * C + E>(k1, k2)...};
    st_shared_v4(tile + (C >> 3) * kBlk + sw128_off(row, C & 7), pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
}
template <int... C>
__device__ __forceinline__ void folded_row_store2(uint32_t tile, uint32_t row, const float (&k1)[12], const float (&k2)[12], std::integer_sequence<int, C...>) {
    (folded_chunk_store2<C>(tile, row, k1, k2, std::make_integer_sequence<int, 8>{}), ...);
}

template <int DV, int F>
__global__ void __launch_bounds__(kFkThreads, 1) tc_phik_state_kernel(const __grid_constant__ CUtensorMap mapK, const __grid_constant__ PhiMaps maps,
                                                                      const __grid_constant__ CUtensorMap mapV, PhiPtrs P, float* __restrict__ kf_out,
                                                                      float* __restrict__ part, int N, int BH, int ld, int smax, int* status) {
    using Cfg = FkCfg<DV, F>;
    using M = MT<F>;
    using Col = FkCols<F>;
    constexpr int NM = M::kMaps, DP = M::kDphi;
    constexpr int HC = DV / 4;          // hidden units per GELU thread
    extern __shared__ uint8_t smem_raw[];
    grid_launch_dependents();
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    float* b2s = reinterpret_cast<float*>(smem + Cfg::kOffB2);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::kOffBars);
    uint64_t* x_full = bars;           // [2] TMA
    uint64_t* x_empty = bars + 2;      // [2] MMA commit
    uint64_t* d1_full = bars + 4;      // [2] two MMA commits: the first-layer product of the unit, and the second-layer product of
                                       // unit - 2 (the G tile of this parity has been read: the GELU warps may write it again), so
                                       // that the GELU warps wait once per unit; the first phase gets the second arrival at set-up
    uint64_t* d1_empty = bars + 6;     // [2] 512 arrivals
    uint64_t* g_full = bars + 8;       // [2] 512 arrivals
    uint64_t* g_free = bars + 10;      // (unused: see d1_full)
    uint64_t* d2_full = bars + 12;     // [2] MMA commit
    uint64_t* d2_empty = bars + 14;    // [2] 128 arrivals
    uint64_t* w_full = bars + 16;      // TMA
    uint64_t* v_full = bars + 17;      // TMA
    uint64_t* v_empty = bars + 18;     // MMA commit
    uint64_t* f_full = bars + 19;      // 128 arrivals: the folded key tile is written
    uint64_t* f_empty = bars + 20;     // 2 arrivals: MMA commit + the zsym warp
    uint64_t* acc_done = bars + 21;    // MMA commit: the accumulator of a piece is complete
    uint64_t* acc_free = bars + 22;    // 128 arrivals: it has been drained
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 23);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int T = (N + kTileTokens - 1) / kTileTokens;      // tiles per head
    const long long total = (long long)BH * T;
    const int G = gridDim.x;
    const int w0 = (int)(total * blockIdx.x / G), w1 = (int)(total * (blockIdx.x + 1) / G);
    const int nwork = w1 - w0;
    auto head_of = [&](int it) { return (w0 + it) / T; };
    auto piece_ends = [&](int it) { return it == nwork - 1 || head_of(it + 1) != head_of(it); };

    // second-layer weights as a K-major MMA operand [16 rows (outputs, 6 used)][DV] per map, halved (the GELU warps
    // form 2 GELU); row kFkB1Row of the same tile holds b1: read as an MN-major operand [16 K rows][DV] it is the B
    // operand of the bias step of the first layer
    for (int i = tid; i < NM * Cfg::kW2Bytes / 16; i += kFkThreads) reinterpret_cast<uint4*>(smem + Cfg::kOffW2)[i] = make_uint4(0, 0, 0, 0);
    if (DV == 64)
        for (int i = tid; i < kBlk / 16; i += kFkThreads) reinterpret_cast<uint4*>(smem + Cfg::kOffV + kBlk)[i] = make_uint4(0, 0, 0, 0);
    __syncthreads();
    for (int i = tid; i < NM * DV * (DP + 1); i += kFkThreads) {
        const int m = i / (DV * (DP + 1)), j = (i / (DP + 1)) % DV, o = i % (DP + 1);
        uint8_t* base = smem + Cfg::kOffW2 + m * Cfg::kW2Bytes + (j >> 6) * 2048;
        const int r = o < DP ? o : kFkB1Row;
        *reinterpret_cast<__nv_bfloat16*>(base + sw128_off(r, (j & 63) >> 3) + (j & 7) * 2) = o < DP ? half_bf16(P.W2[m][j * DP + o]) : P.b1[m][j];
    }
    for (int i = tid; i < NM * 16; i += kFkThreads) b2s[i] = (i & 15) < DP ? __bfloat162float(P.b2[i >> 4][i & 15]) : 0.f;
    fence_proxy_async();
    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(&x_full[i], 1);
            mbar_init(&x_empty[i], 1);
            mbar_init(&d1_full[i], 2);
            mbar_init(&d1_empty[i], 512);
            mbar_init(&g_full[i], 512);
            mbar_init(&g_free[i], 1);
            mbar_init(&d2_full[i], 1);
            mbar_init(&d2_empty[i], 128);
        }
        mbar_init(w_full, 1);
        mbar_init(v_full, 1);
        mbar_init(v_empty, 1);
        mbar_init(f_full, 128);
        mbar_init(f_empty, 1 + kFkZWarps);
        mbar_init(acc_done, 1);
        mbar_init(acc_free, 128);
        fence_mbar_init();
        mbar_arrive(&d1_full[0]);      // no second-layer product precedes the first two units
        mbar_arrive(&d1_full[1]);
        prefetch_tmap(&mapK);
        prefetch_tmap(&mapV);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;     // D1[b] at columns 128 b; the rest as the kFkCol constants say
    if (warp >= kFkFeatWarp0 && warp < kFkFeatWarp0 + 4) {
        // constant A operand of the bias step: every row is 16 K values (two per column) with a one at K = kFkB1Row
        const uint32_t one = 0x3F80u << (16 * (kFkB1Row & 1));
        uint32_t c[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) c[i] = i == kFkB1Row / 2 ? one : 0u;
        tmem_st8(tmem + Col::kOnes + ((uint32_t)((warp & 3) * 32) << 16), c[0], c[1], c[2], c[3], c[4], c[5], c[6], c[7]);
        tmem_st_wait();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    grid_dependency_wait();
    bool ok = true;

    if (warp == 0) {
        if (lane == 0) {
            mbar_arrive_expect_tx(w_full, NM * Cfg::kW1Bytes);
            for (int m = 0; m < NM; ++m)
                for (int b = 0; b < DV / 64; ++b)
                    tma_load_2d(smem + Cfg::kOffW1 + m * Cfg::kW1Bytes + b * (DV * 128), &maps.w1[m], w_full, b * 64, 0);
            for (int it = 0; it < nwork; ++it) {
                const int work = w0 + it, bh = work / T, tile = work - bh * T;
                const int st = it & 1, u = it >> 1;
                if (!mbar_wait(&x_empty[st], (u & 1) ^ 1)) { report_timeout(status, 801); break; }
                mbar_arrive_expect_tx(&x_full[st], Cfg::kXBytes);
                for (int b = 0; b < DV / 64; ++b)
                    tma_load_3d(smem + Cfg::kOffX + st * Cfg::kXBytes + b * kBlk, &mapK, &x_full[st], b * 64, tile * kTileTokens, bh);
            }
        }
    } else if (warp == 2) {
        if (lane == 0) {      // D1[b] = K tile * W1[m] + 1 * b1[m]
            const uint32_t idesc1 = idesc_bf16(128, DV, false, true);   // K tile K-major, W1 [in][hidden] MN-major
            const uint64_t xd0 = smem_desc_sw128(smem_u32(smem + Cfg::kOffX), 16, 1024);
            const uint64_t wd0 = smem_desc_sw128(smem_u32(smem + Cfg::kOffW1), DV * 128, 1024);
            const uint64_t bd0 = smem_desc_sw128(smem_u32(smem + Cfg::kOffW2), 2048, 1024);
            bool good = mbar_wait(w_full, 0);
            for (int unit = 0; unit < NM * nwork && good; ++unit) {
                const int it = unit / NM, m = unit - NM * it, st = it & 1, b = unit & 1;
                if (m == 0 && !mbar_wait(&x_full[st], (it >> 1) & 1)) { good = false; break; }
                if (!mbar_wait(&d1_empty[b], ((unit >> 1) & 1) ^ 1)) { good = false; break; }
                tc_fence_after();
                const uint64_t xd = desc_advance(xd0, st * Cfg::kXBytes), wd = desc_advance(wd0, m * Cfg::kW1Bytes);
#pragma unroll
                for (int ks = 0; ks < DV / 16; ++ks)
                    umma_bf16(tmem + 128 * b, desc_advance(xd, (ks >> 2) * kBlk + (ks & 3) * 32), desc_advance(wd, ks * 2048), idesc1, ks > 0 ? 1u : 0u);
                umma_bf16_ta(tmem + 128 * b, tmem + Col::kOnes, desc_advance(bd0, m * Cfg::kW2Bytes), idesc1, 1u);
                umma_commit(&d1_full[b]);
                if (m == NM - 1) umma_commit(&x_empty[st]);
            }
            if (!good) report_timeout(status, 802);
        }
    } else if (warp == 1) {
        if (lane == 0) {      // D2[b] = G[b] * W2[m]
            const uint32_t idesc2 = idesc_bf16(128, 16, false, false);  // G from TMEM, W2 operand K-major
            const uint64_t vd0 = smem_desc_sw128(smem_u32(smem + Cfg::kOffW2), 16, 1024);
            bool good = true;
            for (int unit = 0; unit < NM * nwork && good; ++unit) {
                const int m = unit % NM, b = unit & 1, par = (unit >> 1) & 1;
                if (!(mbar_wait(&g_full[b], par) && mbar_wait(&d2_empty[b], par ^ 1))) { good = false; break; }
                tc_fence_after();
                const uint64_t vd = desc_advance(vd0, m * Cfg::kW2Bytes);
#pragma unroll
                for (int ks = 0; ks < DV / 16; ++ks)
                    umma_bf16_ta(tmem + Col::kD2 + Col::kD2Stride * b, tmem + Col::kG + 64 * b + 8 * ks, desc_advance(vd, (ks >> 2) * 2048 + (ks & 3) * 32), idesc2,
                                 ks > 0 ? 1u : 0u);
                umma_commit(&d1_full[b]);      // G[b] is free again: second arrival of the phase of unit + 2
                umma_commit(&d2_full[b]);
            }
            if (!good) report_timeout(status, 803);
        }
    } else if (warp == kFkStateWarp) {
        if (lane == 0) {      // Csym^T += V tile^T (MN-major, M = value channels) * folded key tile (MN-major, N = 64), K = 128 tokens
            const uint32_t idesc = idesc_bf16(128, M::kPad, true, true);
            const uint32_t va = smem_u32(smem + Cfg::kOffV), fa = smem_u32(smem + Cfg::kOffF);
            auto load_v = [&](int it) {
                const int work = w0 + it, bh = work / T, tile = work - bh * T;
                mbar_arrive_expect_tx(v_full, DV * kTileTokens * 2);
                for (int b = 0; b < DV / 64; ++b) tma_load_3d(smem + Cfg::kOffV + b * kBlk, &mapV, v_full, b * 64, tile * kTileTokens, bh);
            };
            load_v(0);
            int pieces = 0;
            bool first = true, good = true;
            for (int it = 0; it < nwork && good; ++it) {
                const bool last = piece_ends(it);
                // the previous piece must have been drained before the first product of this one overwrites it
                if (first && pieces > 0 && !mbar_wait(acc_free, (pieces - 1) & 1)) { good = false; break; }
                if (!(mbar_wait(v_full, it & 1) && mbar_wait(f_full, it & 1))) { good = false; break; }
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < kTileTokens / 16; ++ks)
                    umma_bf16(tmem + Col::kC, smem_desc_sw128(va + ks * 2048, kBlk, 1024), smem_desc_sw128(fa + ks * 2048, kBlk, 1024), idesc,
                              (!first || ks > 0) ? 1u : 0u);
                umma_commit(v_empty);
                umma_commit(f_empty);
                if (last) {
                    umma_commit(acc_done);
                    ++pieces;
                }
                first = last;
                if (it + 1 < nwork) {
                    if (!mbar_wait(v_empty, it & 1)) { good = false; break; }
                    load_v(it + 1);
                }
            }
            if (!good) report_timeout(status, 804);
        }
    } else if (warp >= kFkZWarp0) {
        // zsym: column sums of the folded key tile as the state product sees it (bf16 values, fp32 sums).  One warp summed
        // them at first and needed 4500 (three factors) to 10600 (two factors) cycles per tile, as long as the rest of the
        // tile: a lone warp issues an instruction every five cycles or so.  Now four warps take 16 columns each: one
        // 16-byte load per lane and step, lane l adds the eight monomials of chunk 2 w + (l & 1) over the rows l >> 1,
        // l >> 1 + 16, ...; with a second block of 16 columns its two chunks go to warps 0 and 1 (rows l, l + 32, ...).
        // The lanes keep their partial sums for the whole piece and add them up at its end, in a fixed order.
        const int zw = warp - kFkZWarp0;
        const uint32_t fa = smem_u32(smem + Cfg::kOffF);
        float z0[8], z1[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) z0[e] = z1[e] = 0.f;
        auto add_chunk = [](float (&z)[8], uint32_t addr) {
            uint32_t w[4];
            asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(addr) : "memory");
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                z[2 * e] += __uint_as_float(w[e] << 16);
                z[2 * e + 1] += __uint_as_float(w[e] & 0xffff0000u);
            }
        };
        const bool second = M::kBlocks == 2 && zw < 2;
        for (int it = 0; it < nwork; ++it) {
            if (ok && !mbar_wait(f_full, it & 1)) { ok = false; report_timeout(status, 805); }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
#pragma unroll
            for (int j = 0; j < kTileTokens / 16; ++j) add_chunk(z0, fa + sw128_off((lane >> 1) + 16 * j, 2 * zw + (lane & 1)));
            if (second) {
#pragma unroll
                for (int j = 0; j < kTileTokens / 32; ++j) add_chunk(z1, fa + kBlk + sw128_off(lane + 32 * j, zw));
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(f_empty);
            if (piece_ends(it)) {
                const int bh = head_of(it);
                const int piece = blockIdx.x - owner_of_work((long long)bh * T, total, G);
                float* out = part + ((size_t)bh * smax + piece) * M::kN * ld;
                auto put = [&](int m, float v) {
                    if (m < M::kN) {
                        out[(size_t)m * ld + DV] = v;
                        for (int c = DV + 1; c < ld; ++c) out[(size_t)m * ld + c] = 0.f;
                    }
                };
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    float v = z0[e];
#pragma unroll
                    for (int o = 2; o < 32; o <<= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                    if (lane < 2) put(8 * (2 * zw + lane) + e, v);
                    z0[e] = 0.f;
                }
                if (M::kBlocks == 2) {      // (every warp runs the shuffles; warps 2 and 3 hold zeros)
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        float v = z1[e];
#pragma unroll
                        for (int o = 1; o < 32; o <<= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                        if (second && lane == 0) put(64 + 8 * zw + e, v);
                        z1[e] = 0.f;
                    }
                }
            }
        }
    } else if (warp >= kFkFeatWarp0) {
        // k^m = ReLU(D2 + b2) -> global memory (kept for the backward); after the third map the folded key row of the token
        // goes into the B operand of the state product; the piece's accumulator is drained when its last tile is in
        const int quarter = warp & 3, row = quarter * 32 + lane;
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        const uint32_t fblk = smem_u32(smem + Cfg::kOffF);
        int pieces = 0;
        for (int it = 0; it < nwork && ok; ++it) {
            const int work = w0 + it, bh = work / T, tile = work - bh * T;
            const int tok = tile * kTileTokens + row;
            float k1[DP], s12[6][6];
#pragma unroll
            for (int m = 0; m < NM; ++m) {
                const int unit = NM * it + m, b = unit & 1;
                if (!mbar_wait(&d2_full[b], (unit >> 1) & 1)) { ok = false; report_timeout(status, 806); }
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                uint32_t r[16];
                if constexpr (DP <= 8) tmem_ld8(tmem + Col::kD2 + Col::kD2Stride * b + lane_base, *reinterpret_cast<uint32_t(*)[8]>(r));
                else tmem_ld16(tmem + Col::kD2 + Col::kD2Stride * b + lane_base, r);
                tmem_ld_wait();
                tc_fence_before();
                mbar_arrive(&d2_empty[b]);
                float f[DP];
#pragma unroll
                for (int o = 0; o < DP; ++o) f[o] = tok < N ? fmaxf(__uint_as_float(r[o]) + b2s[16 * m + o], 0.f) : 0.f;
                if (tok < N) store_feat<DP>(kf_out + ((size_t)(bh * NM + m) * N + tok) * DP, f);
                if (m == 0) {
#pragma unroll
                    for (int o = 0; o < DP; ++o) k1[o] = f[o];
                } else if (F == 3 && m == 1) {
                    if constexpr (F == 3) {
#pragma unroll
                        for (int x = 0; x < 6; ++x)
#pragma unroll
                            for (int y = x; y < 6; ++y) s12[x][y] = (x == y) ? k1[x] * f[x] : fmaf(k1[x], f[y], k1[y] * f[x]);
                    }
                } else {
                    if (!mbar_wait(f_empty, (it & 1) ^ 1)) { ok = false; report_timeout(status, 807); }
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    if constexpr (F == 3) folded_row_store(fblk, row, s12, f, std::make_integer_sequence<int, 8>{});
                    else folded_row_store2(fblk, row, k1, f, std::make_integer_sequence<int, 10>{});
                    fence_proxy_async();
                    mbar_arrive(f_full);
                }
            }
            if (ok && piece_ends(it)) {
                if (!mbar_wait(acc_done, pieces & 1)) { ok = false; report_timeout(status, 808); }
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                const int piece = blockIdx.x - owner_of_work((long long)bh * T, total, G);
                float* out = part + ((size_t)bh * smax + piece) * M::kN * ld;
                const int g = quarter * 32 + lane;       // TMEM lane = value channel
                if (quarter * 32 < DV) {
#pragma unroll
                    for (int c = 0; c < (M::kN + 7) / 8; ++c) {
                        uint32_t rr[8];
                        tmem_ld8(tmem + Col::kC + lane_base + 8 * c, rr);
                        tmem_ld_wait();
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            if (8 * c + e < M::kN) out[(size_t)(8 * c + e) * ld + g] = __uint_as_float(rr[e]);
                    }
                }
                tc_fence_before();
                mbar_arrive(acc_free);
                ++pieces;
            }
        }
    } else {
        // GELU: thread = token row x quarter of the hidden units
        const int quarter = warp & 3, prt = (warp - kFkGeluWarp0) >> 2;
        for (int unit = 0; unit < NM * nwork; ++unit) {
            const int b = unit & 1, par = (unit >> 1) & 1;
            if (!mbar_wait(&d1_full[b], par)) { ok = false; report_timeout(status, 809); }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t ta = tmem + 128 * b + ((uint32_t)(quarter * 32) << 16) + prt * HC;
            const uint32_t tg = tmem + Col::kG + 64 * b + ((uint32_t)(quarter * 32) << 16) + prt * (HC / 2);
            uint32_t r[HC];
#pragma unroll
            for (int c = 0; c < HC / 16; ++c) tmem_ld16(ta + 16 * c, *reinterpret_cast<uint32_t(*)[16]>(r + 16 * c));
            tmem_ld_wait();
            tc_fence_before();
            mbar_arrive(&d1_empty[b]);          // h is in registers: the next first-layer product may overwrite it
#pragma unroll
            for (int c = 0; c < HC / 16; ++c) {
                uint32_t w[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float2 g = gelu2_twice(make_float2(__uint_as_float(r[16 * c + 2 * e]), __uint_as_float(r[16 * c + 2 * e + 1])));
                    w[e] = pack_bf16(g.x, g.y);
                }
                tmem_st8(tg + 8 * c, w[0], w[1], w[2], w[3], w[4], w[5], w[6], w[7]);      // the second layer's A operand lives in TMEM
            }
            tmem_st_wait();
            tc_fence_before();
            mbar_arrive(&g_full[b]);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, 512);
}

// Largest number of pieces any head has when BH * T work items are dealt to G CTAs.
inline int fused_key_max_pieces(int BH, int T, int G) {
    const long long total = (long long)BH * T;
    int smax = 1;
    for (int bh = 0; bh < BH; ++bh) {
        const int n = owner_of_work((long long)bh * T + T - 1, total, G) - owner_of_work((long long)bh * T, total, G) + 1;
        if (n > smax) smax = n;
    }
    return smax;
}
inline int fused_key_grid(int BH, int N, int sm_count) {
    const long long total = (long long)BH * ((N + kTileTokens - 1) / kTileTokens);
    return (int)(total < sm_count ? total : sm_count);
}

template <int DV, int F>
inline hla_status launch_phik_state(const Dims& D, int BH, const hla_mlp* phi_k, const void* K, const void* V, char* ws, const hla_ws_layout& L,
                                    size_t off_part, int smax, int sm_count, LaunchRec& rec) {
    CUtensorMap mapK, mapV;
    PhiMaps mk;
    PhiPtrs pk{};
    if (!make_map_bhnd(&mapK, K, BH, D.N, DV, kTileTokens) || !make_map_bhnd(&mapV, V, BH, D.N, DV, kTileTokens)) return HLA_ERR_CUDA;
    for (int f = 0; f < MT<F>::kMaps; ++f) {
        if (!make_map_2d(&mk.w1[f], phi_k[f].W1, DV, DV, DV)) return HLA_ERR_CUDA;
        pk.b1[f] = static_cast<const __nv_bfloat16*>(phi_k[f].b1);
        pk.W2[f] = static_cast<const __nv_bfloat16*>(phi_k[f].W2);
        pk.b2[f] = static_cast<const __nv_bfloat16*>(phi_k[f].b2);
    }
    for (int f = MT<F>::kMaps; f < 3; ++f) mk.w1[f] = mk.w1[0];
    if (!set_smem(tc_phik_state_kernel<DV, F>, FkCfg<DV, F>::kSmem)) return HLA_ERR_CUDA;
    const int grid = fused_key_grid(BH, D.N, sm_count);
    rec.begin("tc_phik_state");
    // first kernel of hla_forward, and it stages the weights before its dependency wait: no overlap with what precedes it
    launch_serial(tc_phik_state_kernel<DV, F>, grid, dim3(kFkThreads), FkCfg<DV, F>::kSmem, rec.st, mapK, mk, mapV, pk, reinterpret_cast<float*>(ws + L.kf),
                  reinterpret_cast<float*>(ws + off_part), D.N, BH, D.ld, smax, reinterpret_cast<int*>(ws + L.status));
    return rec.end() ? HLA_OK : HLA_ERR_CUDA;
}

inline hla_status phik_state(const Dims& D, int BH, const hla_mlp* phi_k, const void* K, const void* V, char* ws, const hla_ws_layout& L,
                             size_t off_part, int smax, int sm_count, LaunchRec& rec) {
    if (D.F == 3) {
        if (D.d == 128) return launch_phik_state<128, 3>(D, BH, phi_k, K, V, ws, L, off_part, smax, sm_count, rec);
        return launch_phik_state<64, 3>(D, BH, phi_k, K, V, ws, L, off_part, smax, sm_count, rec);
    }
    if (D.d == 128) return launch_phik_state<128, 2>(D, BH, phi_k, K, V, ws, L, off_part, smax, sm_count, rec);
    return launch_phik_state<64, 2>(D, BH, phi_k, K, V, ws, L, off_part, smax, sm_count, rec);
}

}  // namespace tc
}  // namespace hla
