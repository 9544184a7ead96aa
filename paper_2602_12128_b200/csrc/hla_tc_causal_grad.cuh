// Feature gradients of causal HLA (Section 4.4) on the tensor cores, F = 3, d_phi = 6.
//
// With r_i = 1 / (eta_i + eps), delta_i = dO_i . o_i and dA_ij = r_i (dO_i . v_j - delta_i) for j <= i (0 otherwise):
//     dmono_i = sum_{j <= i} dA_ij Tsym_j      -> dq_i   (gradient of the monomials q_a q_b q_c)
//     dTsym_j = sum_{i >= j} dA_ij mono_i      -> dk^f_j (gradient of the folded key features)
// Both are sweeps over 128-token tiles that carry a state, like the forward: the first walks the tokens forwards and
// carries [Csym | zsym] (the state of the forward), the second walks them backwards and carries [dCsym | dzsym]
// = sum_i r_i mono_i (x) [dO_i | -delta_i].  One kernel serves both (DIR 0 / 1); per tile, with X, Y the two bf16 tiles
// that TMA brings in (DIR 0: X = dO, Y = V; DIR 1: X = V, Y = dO) and W the generated operand-row tile
// (DIR 0: [1, 0 x 7, Tsym_j]; DIR 1: [-delta_i, 0 x 7, r_i mono_i]):
//
//     Sc     = X Y^T                                     (MMA, K = d)        Sc[x][y] = v . dO of the two tokens
//     acc    = X * (state image)^T                       (MMA, K = d, 64 columns: one per state row)
//     state += W^T [Y | W]                               (MMA, K = 128 tokens, 64 rows)
//     Sm     = bf16(Sc - delta of the query token) on the kept side of the diagonal, else 0      (threads, in place)
//     acc   += Sm * W                                    (MMA, K = 128 tokens)
//     DIR 0: dmono_i = r_i (acc_i - delta_i zsym_before) -> dq_i ;   DIR 1: dTsym_j = acc_j + dzsym_after -> dk_j   (threads)
//
// The state rows, their shift by 8, the bf16 image of the state (read here with the value channels as the K dimension),
// the two MMA-issuing threads and the barrier protocol are those of the forward sweep.
//
// Warp roles: 0 TMA (X and Y tiles), 2 MMA issue (Sc), 1 MMA issue (readout, Sm * W), 3 MMA issue (state), 4..7 operand
// rows W, 8..15 mask, 16..19 state image, 20..23 and 24..27 epilogue (two groups, alternate tiles).  A lone thread needs
// well over a hundred cycles per product it issues, more than the product takes, so the 32 products of a tile are spread
// over three threads; Sc has two buffers in tensor memory (by tile parity), which lets the Sc product and the mask of the
// next tile run while the readout of this one is still being issued.
#pragma once
#include "hla_tc_causal.cuh"

namespace hla {
namespace tc {

template <int DV> struct CgCfg {
    static constexpr int kVB = DV / 64;
    static constexpr int kOffW = kVB * kBlk;                 // operand-row tile: directly after the Y blocks
    static constexpr int kOffX = kOffW + kBlk;
    static constexpr int kStageBytes = kOffX + kVB * kBlk;
    static constexpr int kB3Block = 64 * 128;
    static constexpr int kB3Bytes = (kVB + 1) * kB3Block;
    static constexpr int kOffB3 = 2 * kStageBytes;
    static constexpr int kOffZ = kOffB3 + 2 * kB3Bytes;       // float [2][64]: column d of the state behind each image
    static constexpr int kOffDv = kOffZ + 2 * 64 * 4;         // float [2][128]: delta of the tile's tokens (DIR 1)
    static constexpr int kOffBars = kOffDv + 2 * 128 * 4;
    static constexpr int kSmem = 1024 + kOffBars + 256;
    static constexpr int kNState = DV + 8;
    static constexpr int kColAcc = 0, kColState = 64, kColS = 256;      // Sc of tile it at kColS + 128 (it & 1)
    static_assert(kColState + kNState <= kColS, "tensor memory");
    static_assert(kSmem <= 227 * 1024, "shared memory");
};

// Seven groups of four warps: 0..3 one thread each (TMA, three MMA issuers), 4..7 operand rows, 8..15 mask, 16..19 state
// image, 20..23 and 24..27 the two epilogue groups.  The epilogue holds 56 monomial gradients, 18 features and 18 feature
// gradients per thread, which does not fit the 72 registers a thread gets at 896 threads: the other groups hand registers
// over (setmaxnreg), 4 x 32 x (40 + 4 x 64 + 2 x 104) = the 64512 the launch was given.
constexpr int kCgThreads = 28 * 32;
constexpr int kCgScMmaWarp = 2, kCgStMmaWarp = 3, kCgRowWarp0 = 4, kCgMaskWarp0 = 8, kCgConvWarp0 = 16, kCgEpiWarp0 = 20;
constexpr int kCgIssueRegs = 40, kCgWorkRegs = 64, kCgEpiRegs = 104;
static_assert(4 * 32 * (kCgIssueRegs + 4 * kCgWorkRegs + 2 * kCgEpiRegs) == kCgThreads * 72, "register budget");

template <int DV, int DIR>
__global__ void __launch_bounds__(kCgThreads, 1) tc_causal_grad_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapY,
                                                                       const float* __restrict__ qf, const float* __restrict__ kf,
                                                                       const float* __restrict__ eta, const float* __restrict__ delta,
                                                                       const float* __restrict__ init, float* __restrict__ out, int N, int BH, int S, int ld,
                                                                       float eps, int* status) {
    using Cfg = CgCfg<DV>;
    constexpr int kStageBytes = Cfg::kStageBytes;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    float* zvec = reinterpret_cast<float*>(smem + Cfg::kOffZ);
    float* dvec = reinterpret_cast<float*>(smem + Cfg::kOffDv);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::kOffBars);
    uint64_t* stage_ready = bars;         // [2] 128 arrivals + the TMA transaction
    uint64_t* stage_free = bars + 2;      // [2] 2 MMA commits
    uint64_t* p_full = bars + 11;         // [2] MMA commit, barrier it & 1: Sc is complete
    uint64_t* pm_ready = bars + 13;       // [2] 256 arrivals, barrier it & 1: Sm is in tensor memory
    uint64_t* state_full = bars + 7;      // MMA commit
    uint64_t* acc_full = bars + 19;       // [2] MMA commit, barrier it & 1 (each epilogue group waits on its own)
    uint64_t* state_read = bars + 9;      // 128 arrivals
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 10);
    uint64_t* acc_free = bars + 17;       // [2] 128 arrivals, barrier it & 1: accumulator and state-column vector of tile it have been read
    uint64_t* b3_ready = bars + 15;       // [2] 128 arrivals, barrier it & 1

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int T = (N + kTileTokens - 1) / kTileTokens;
    const CaWork cw = causal_work(T, BH, S, 0);
    const int w0 = cw.w0, nwork = cw.w1 - cw.w0;
    const int bh = blockIdx.y;
    auto tile_of = [&](int it) { return (DIR == 0 ? w0 + it : w0 + nwork - 1 - it) - bh * T; };
    grid_launch_dependents();

    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(&stage_ready[i], 129);
            mbar_init(&stage_free[i], 2);
            mbar_init(&b3_ready[i], 128);
            mbar_init(&acc_free[i], 128);
            mbar_init(&acc_full[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&p_full[i], 1);
            mbar_init(&pm_ready[i], 256);
        }
        mbar_init(state_full, 1);
        mbar_init(state_read, 128);
        fence_mbar_init();
        prefetch_tmap(&mapX);
        prefetch_tmap(&mapY);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    for (int i = tid; i < 2 * Cfg::kB3Bytes / 16; i += kCgThreads) reinterpret_cast<uint4*>(smem + Cfg::kOffB3)[i] = make_uint4(0, 0, 0, 0);
    if (tid < 128) zvec[tid] = 0.f;
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    grid_dependency_wait();
    bool ok = true;

    if (warp >= kCgEpiWarp0) {
        reg_inc<kCgEpiRegs>();
        // epilogue: thread = row x of the accumulator (DIR 0: query token, DIR 1: key token).  Two groups (warps 20..23 and
        // 24..27) take the tiles in turn: a group releases the accumulator as soon as it has read it and then has two tile
        // times for the gradient arithmetic of its rows.
        const int qt = warp & 3, row = qt * 32 + lane, grp = (warp - kCgEpiWarp0) >> 2;
        const uint32_t aa = tmem + Cfg::kColAcc + ((uint32_t)(qt * 32) << 16);
        float fn[DIR == 0 ? 6 : 18], en = 0.f, dn = 0.f;
        auto prefetch = [&](int it) {
            const int tok = min(tile_of(it) * kTileTokens + row, N - 1);
            if (DIR == 0) {
                load_feat<6>(fn, qf + ((size_t)bh * N + tok) * 6);
                en = __ldg(eta + (size_t)bh * N + tok);
                dn = __ldg(delta + (size_t)bh * N + tok);
            } else {
#pragma unroll
                for (int f = 0; f < 3; ++f) load_feat<6>(fn + 6 * f, kf + (((size_t)bh * 3 + f) * N + tok) * 6);
            }
        };
        if (nwork > grp) prefetch(grp);
        for (int it = grp; it < nwork; it += 2) {
            const int tok = tile_of(it) * kTileTokens + row;
            float f[DIR == 0 ? 6 : 18];
#pragma unroll
            for (int i = 0; i < (DIR == 0 ? 6 : 18); ++i) f[i] = fn[i];
            const float r = 1.f / (en + eps), dl = dn;
            if (it + 2 < nwork) prefetch(it + 2);
            if (ok && !mbar_wait(&acc_full[grp], (it >> 1) & 1)) { ok = false; report_timeout(status, 934); }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            float g[kMono];
            {
                uint32_t a[64];
#pragma unroll
                for (int c = 0; c < 4; ++c) tmem_ld16(aa + 16 * c, *reinterpret_cast<uint32_t(*)[16]>(a + 16 * c));
                tmem_ld_wait();
                tc_fence_before();
                const float* zv = zvec + (it & 1) * 64 + kCaRowPad;
#pragma unroll
                for (int m = 0; m < kMono; ++m) {
                    const float z = zv[m];
                    g[m] = DIR == 0 ? r * fmaf(-dl, z, __uint_as_float(a[kCaRowPad + m])) : __uint_as_float(a[kCaRowPad + m]) + z;
                }
                mbar_arrive(&acc_free[it & 1]);      // the accumulator and this item's vector have been read
            }
            if (DIR == 0) {
                float q[6], dq[6];
#pragma unroll
                for (int i = 0; i < 6; ++i) q[i] = f[i];
                query_monomials_grad_t<3>(q, g, dq);
                if (tok < N) store_feat<6>(out + ((size_t)bh * N + tok) * 6, dq);
            } else {
                float k[18], dk[18];
#pragma unroll
                for (int i = 0; i < 18; ++i) k[i] = f[i];
                key_folded_grad_t<3>(k, g, dk);
                if (tok < N) {
#pragma unroll
                    for (int ff = 0; ff < 3; ++ff) store_feat<6>(out + (((size_t)bh * 3 + ff) * N + tok) * 6, dk + 6 * ff);
                }
            }
        }
    } else if (warp < kCgRowWarp0) {
        reg_dec<kCgIssueRegs>();
        if (warp == 0) {
            if (lane == 0) {
                for (int it = 0; it < nwork; ++it) {
                    const int st = it & 1, u = it >> 1, tile = tile_of(it);
                    if (!mbar_wait(&stage_free[st], (u & 1) ^ 1)) { report_timeout(status, 921); break; }
                    mbar_arrive_expect_tx(&stage_ready[st], 2 * DV * kTileTokens * 2);
                    for (int b = 0; b < Cfg::kVB; ++b) {
                        tma_load_3d(smem + st * kStageBytes + b * kBlk, &mapY, &stage_ready[st], b * 64, tile * kTileTokens, bh);
                        tma_load_3d(smem + st * kStageBytes + Cfg::kOffX + b * kBlk, &mapX, &stage_ready[st], b * 64, tile * kTileTokens, bh);
                    }
                }
            }
        } else if (warp == 1) {
            if (lane == 0) {
                const uint32_t id_r = idesc_bf16(128, 64, false, false);
                const uint32_t id_w = idesc_bf16(128, 64, false, true);
                const uint32_t b3base = smem_u32(smem + Cfg::kOffB3);
                for (int it = 0; it < nwork; ++it) {
                    const int st = it & 1, u = it >> 1;
                    const uint32_t ya = smem_u32(smem + st * kStageBytes), wa = ya + Cfg::kOffW, xa = ya + Cfg::kOffX;
                    if (!mbar_wait(&stage_ready[st], u & 1)) { report_timeout(status, 922); break; }
                    if (!(mbar_wait(&b3_ready[it & 1], (it >> 1) & 1) && (it == 0 || mbar_wait(&acc_free[(it - 1) & 1], ((it - 1) >> 1) & 1)))) {
                        report_timeout(status, 923);
                        break;
                    }
                    tc_fence_after();
                    const uint32_t b3a = b3base + (it & 1) * Cfg::kB3Bytes;
                    {      // acc = X * image^T: one column per state row, value channels as K
                        uint64_t da = smem_desc_sw128(xa, 16, 1024), db = smem_desc_sw128(b3a, 16, 1024);
                        uint32_t acc = 0u;
#pragma unroll 1
                        for (int blk = 0; blk < Cfg::kVB; ++blk, da += (kBlk >> 4) - 8, db += (Cfg::kB3Block >> 4) - 8)
#pragma unroll 1
                            for (int k = 0; k < 4; ++k, da += 2, db += 2, acc = 1u) umma_bf16(tmem + Cfg::kColAcc, da, db, id_r, acc);
                    }
                    if (!mbar_wait(&pm_ready[it & 1], (it >> 1) & 1)) { report_timeout(status, 925); break; }
                    tc_fence_after();
                    {      // acc += Sm * W; the two packed halves of Sm sit at columns 0..31 and 64..95 of the block
                        uint64_t db = smem_desc_sw128(wa, kBlk, 1024);
                        const uint32_t sm = tmem + Cfg::kColS + 128 * (it & 1);
#pragma unroll 1
                        for (int ks = 0; ks < kTileTokens / 16; ++ks, db += 128) umma_bf16_ta(tmem + Cfg::kColAcc, sm + 8 * ks + (ks >= 4 ? 32 : 0), db, id_w, 1u);
                    }
                    umma_commit(&acc_full[it & 1]);
                    umma_commit(&stage_free[st]);
                }
            }
        } else if (warp == kCgScMmaWarp) {
            if (lane == 0) {
                const uint32_t id_s = idesc_bf16(128, 128, false, false);
                for (int it = 0; it < nwork; ++it) {
                    const int st = it & 1, u = it >> 1;
                    const uint32_t ya = smem_u32(smem + st * kStageBytes), xa = ya + Cfg::kOffX;
                    if (!mbar_wait(&stage_ready[st], u & 1)) { report_timeout(status, 935); break; }
                    // the buffer last held Sm of tile it - 2: free once that tile's Sm * W products have completed
                    if (it >= 2 && !mbar_wait(&acc_full[it & 1], ((it - 2) >> 1) & 1)) { report_timeout(status, 936); break; }
                    tc_fence_after();
                    {      // Sc = X Y^T: four K steps per 64-column block, 32 bytes apart inside a 128-byte row
                        uint64_t da = smem_desc_sw128(xa, 16, 1024), db = smem_desc_sw128(ya, 16, 1024);
                        uint32_t acc = 0u;
#pragma unroll 1
                        for (int blk = 0; blk < Cfg::kVB; ++blk, da += (kBlk >> 4) - 8, db += (kBlk >> 4) - 8)
#pragma unroll 1
                            for (int k = 0; k < 4; ++k, da += 2, db += 2, acc = 1u) umma_bf16(tmem + Cfg::kColS + 128 * (it & 1), da, db, id_s, acc);
                    }
                    umma_commit(&p_full[it & 1]);
                }
            }
        } else {
            if (lane == 0) {
                const uint32_t id_st = idesc_bf16(64, Cfg::kNState, true, true);
                for (int it = 0; it < nwork; ++it) {
                    const int st = it & 1, u = it >> 1;
                    const uint32_t ya = smem_u32(smem + st * kStageBytes), wa = ya + Cfg::kOffW;
                    if (it > 0 && !mbar_wait(state_read, (it - 1) & 1)) { report_timeout(status, 926); break; }
                    if (it == 0 && !mbar_wait(&b3_ready[0], 0)) { report_timeout(status, 927); break; }
                    if (!mbar_wait(&stage_ready[st], u & 1)) { report_timeout(status, 928); break; }
                    tc_fence_after();
                    {      // state += W^T [Y | W]
                        uint64_t da = smem_desc_sw128(wa, kBlk, 1024), db = smem_desc_sw128(ya, kBlk, 1024);
#pragma unroll 1
                        for (int ks = 0; ks < kTileTokens / 16; ++ks, da += 128, db += 128) umma_bf16(tmem + Cfg::kColState, da, db, id_st, 1u);
                    }
                    umma_commit(state_full);
                    umma_commit(&stage_free[st]);
                }
            }
        }
    } else {
        reg_dec<kCgWorkRegs>();
        if (warp < kCgMaskWarp0) {
            // operand rows W: thread = token row of the tile
            const int row = tid - kCgRowWarp0 * 32;
            if (DIR == 0) {
                float kn[18];
                auto prefetch = [&](int it) {
                    const int tok = min(tile_of(it) * kTileTokens + row, N - 1);
#pragma unroll
                    for (int f = 0; f < 3; ++f) load_feat<6>(kn + 6 * f, kf + (((size_t)bh * 3 + f) * N + tok) * 6);
                };
                if (nwork > 0) prefetch(0);
                for (int it = 0; it < nwork; ++it) {
                    const int st = it & 1, u = it >> 1;
                    const bool valid = tile_of(it) * kTileTokens + row < N;
                    float k[18];
#pragma unroll
                    for (int i = 0; i < 18; ++i) k[i] = valid ? kn[i] : 0.f;
                    if (ok && !mbar_wait(&stage_free[st], (u & 1) ^ 1)) { ok = false; report_timeout(status, 929); }
                    if (!ok) continue;
                    float s12[6][6], k3[6];
#pragma unroll
                    for (int x = 0; x < 6; ++x) {
                        k3[x] = k[12 + x];
#pragma unroll
                        for (int y = x; y < 6; ++y) s12[x][y] = (x == y) ? k[x] * k[6 + x] : fmaf(k[x], k[6 + y], k[y] * k[6 + x]);
                    }
                    shifted_key_row(smem_u32(smem + st * kStageBytes) + Cfg::kOffW, row, valid ? 1.f : 0.f, s12, k3, std::make_integer_sequence<int, 7>{});
                    fence_proxy_async();
                    mbar_arrive(&stage_ready[st]);
                    if (it + 1 < nwork) prefetch(it + 1);
                }
            } else {
                float qn[6], en = 0.f, dn = 0.f;
                auto prefetch = [&](int it) {
                    const int tok = min(tile_of(it) * kTileTokens + row, N - 1);
                    load_feat<6>(qn, qf + ((size_t)bh * N + tok) * 6);
                    en = __ldg(eta + (size_t)bh * N + tok);
                    dn = __ldg(delta + (size_t)bh * N + tok);
                };
                if (nwork > 0) prefetch(0);
                for (int it = 0; it < nwork; ++it) {
                    const int st = it & 1, u = it >> 1;
                    const bool valid = tile_of(it) * kTileTokens + row < N;
                    float q[6], qs[6];
                    const float r = valid ? 1.f / (en + eps) : 0.f, dl = valid ? dn : 0.f;
#pragma unroll
                    for (int i = 0; i < 6; ++i) {
                        q[i] = valid ? qn[i] : 0.f;
                        qs[i] = r * q[i];
                    }
                    if (ok && !mbar_wait(&stage_free[st], (u & 1) ^ 1)) { ok = false; report_timeout(status, 930); }
                    if (!ok) continue;
                    shifted_mono_row(smem_u32(smem + st * kStageBytes) + Cfg::kOffW, row, -dl, qs, q, std::make_integer_sequence<int, 7>{});
                    dvec[st * 128 + row] = dl;
                    fence_proxy_async();
                    mbar_arrive(&stage_ready[st]);
                    if (it + 1 < nwork) prefetch(it + 1);
                }
            }
        } else if (warp < kCgConvWarp0) {
            // mask: thread = row x of Sc (DIR 0: query token i; DIR 1: key token j), two warps per 32 rows, 64 columns each.
            // DIR 0 keeps the columns y <= x and subtracts the row's own delta; DIR 1 keeps y >= x and subtracts the delta of
            // the column's token.
            const int qt = warp & 3, half = (warp - kCgMaskWarp0) >> 2;
            const uint32_t pa0 = tmem + Cfg::kColS + 64 * half + ((uint32_t)(qt * 32) << 16);
            float dn = 0.f;
            auto prefetch = [&](int it) {
                const int tok = min(tile_of(it) * kTileTokens + qt * 32 + lane, N - 1);
                dn = __ldg(delta + (size_t)bh * N + tok);
            };
            if (DIR == 0 && nwork > 0) prefetch(0);
            for (int it = 0; it < nwork; ++it) {
                const float dl = dn;
                if (DIR == 0 && it + 1 < nwork) prefetch(it + 1);
                if (ok && !mbar_wait(&p_full[it & 1], (it >> 1) & 1)) { ok = false; report_timeout(status, 931); }
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                const uint32_t pa = pa0 + 128 * (it & 1);
                const float* dv = dvec + (it & 1) * 128;      // written before stage_ready of this item, which p_full follows
#pragma unroll 1
                for (int bb = 0; bb < 2; ++bb) {
                    const int b = 2 * half + bb;
                    const bool whole = DIR == 0 ? b < qt : b > qt;
                    uint32_t w[16];
                    if (whole || b == qt) {
                        uint32_t r[32];
                        tmem_ld16(pa + 32 * bb, *reinterpret_cast<uint32_t(*)[16]>(r));
                        tmem_ld16(pa + 32 * bb + 16, *reinterpret_cast<uint32_t(*)[16]>(r + 16));
                        tmem_ld_wait();
#pragma unroll
                        for (int e = 0; e < 16; ++e) {
                            float d0 = dl, d1 = dl;
                            if (DIR == 1) {
                                const float2 dd = *reinterpret_cast<const float2*>(dv + 32 * b + 2 * e);
                                d0 = dd.x;
                                d1 = dd.y;
                            }
                            float v0 = __uint_as_float(r[2 * e]) - d0, v1 = __uint_as_float(r[2 * e + 1]) - d1;
                            if (!whole) {
                                if (DIR == 0 ? 2 * e > lane : 2 * e < lane) v0 = 0.f;
                                if (DIR == 0 ? 2 * e + 1 > lane : 2 * e + 1 < lane) v1 = 0.f;
                            }
                            w[e] = pack_bf16(v0, v1);
                        }
                    } else {
#pragma unroll
                        for (int e = 0; e < 16; ++e) w[e] = 0u;
                    }
                    tmem_st8(pa + 16 * bb, w[0], w[1], w[2], w[3], w[4], w[5], w[6], w[7]);
                    tmem_st8(pa + 16 * bb + 8, w[8], w[9], w[10], w[11], w[12], w[13], w[14], w[15]);
                }
                tmem_st_wait();
                tc_fence_before();
                mbar_arrive(&pm_ready[it & 1]);
            }
        } else {
            // state image (rows as in the forward sweep) and, beside it, column d of the state in fp32
            const int qt = warp & 3, R = qt * 16 + lane, m = R - kCaRowPad;
            const bool active = lane < 16, mine = active && m >= 0 && m < kMono;
            const uint32_t sa = tmem + Cfg::kColState + ((uint32_t)(qt * 32) << 16);
            const uint32_t b3base = smem_u32(smem + Cfg::kOffB3);
            for (int it = 0; it < nwork; ++it) {
                if (it == 0) {
                    const float* src = init + ((size_t)(bh * S + blockIdx.x) * kMono + (mine ? m : 0)) * ld;
#pragma unroll 1
                    for (int c = 0; c < (DV + 8) / 8; ++c) {
                        float v[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) v[e] = 0.f;
                        if (mine && 8 * c < ld) {
                            const float4 a = *reinterpret_cast<const float4*>(src + 8 * c);
                            v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
                            if (8 * c + 4 < ld) {
                                const float4 b = *reinterpret_cast<const float4*>(src + 8 * c + 4);
                                v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
                            }
                        }
                        tmem_st8(sa + 8 * c, __float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]), __float_as_uint(v[3]), __float_as_uint(v[4]),
                                 __float_as_uint(v[5]), __float_as_uint(v[6]), __float_as_uint(v[7]));
                        if (mine) {
                            if (8 * c < DV)
                                st_shared_v4(b3base + (c >> 3) * Cfg::kB3Block + sw128_off(R, c & 7), pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]),
                                             pack_bf16(v[6], v[7]));
                            else
                                zvec[R] = v[0];
                        }
                    }
                    tmem_st_wait();
                    tc_fence_before();
                    fence_proxy_async();
                    mbar_arrive(&b3_ready[0]);
                }
                if (ok && !mbar_wait(state_full, it & 1)) { ok = false; report_timeout(status, 932); }
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                if (it + 1 < nwork) {
                    // the image and the vector written now were last read for the previous tile: its epilogue must have read the
                    // vector, which also means that every product of that tile has completed
                    if (it > 0 && ok && !mbar_wait(&acc_free[(it - 1) & 1], ((it - 1) >> 1) & 1)) { ok = false; report_timeout(status, 933); }
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t img = b3base + ((it + 1) & 1) * Cfg::kB3Bytes;
#pragma unroll 1
                    for (int h = 0; h < DV / 32; ++h) {
                        uint32_t r[32], rz[8];
                        tmem_ld16(sa + 32 * h, *reinterpret_cast<uint32_t(*)[16]>(r));
                        tmem_ld16(sa + 32 * h + 16, *reinterpret_cast<uint32_t(*)[16]>(r + 16));
                        if (h == DV / 32 - 1) tmem_ld8(sa + DV, rz);
                        tmem_ld_wait();
                        if (h == DV / 32 - 1) {
                            tc_fence_before();
                            mbar_arrive(state_read);
                        }
                        if (mine) {
#pragma unroll
                            for (int c = 0; c < 4; ++c) {
                                const int cc = 4 * h + c;
                                st_shared_v4(img + (cc >> 3) * Cfg::kB3Block + sw128_off(R, cc & 7), pack_bf16(__uint_as_float(r[8 * c]), __uint_as_float(r[8 * c + 1])),
                                             pack_bf16(__uint_as_float(r[8 * c + 2]), __uint_as_float(r[8 * c + 3])),
                                             pack_bf16(__uint_as_float(r[8 * c + 4]), __uint_as_float(r[8 * c + 5])),
                                             pack_bf16(__uint_as_float(r[8 * c + 6]), __uint_as_float(r[8 * c + 7])));
                            }
                            if (h == DV / 32 - 1) zvec[((it + 1) & 1) * 64 + R] = __uint_as_float(rz[0]);
                        }
                    }
                    tc_fence_before();
                    fence_proxy_async();
                    mbar_arrive(&b3_ready[(it + 1) & 1]);
                } else {
                    mbar_arrive(state_read);
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, 512);
}

// Feature gradients of the causal operator: the state of every piece and its prefix scan (as in the forward), the forward
// sweep for dq; then, on the gradient states the value-gradient pass left in `part` (suffix sums), the backward sweep for dk.
template <int DV>
inline hla_status launch_causal_backward_features(const Dims& D, int BH, const float* qf, const float* kf, const void* V, const void* dO, float* dqf, float* dkf,
                                                  char* ws, const hla_ws_layout& L, size_t off_part, size_t off_delta, bool second, LaunchRec& rec) {
    CUtensorMap mapV, mapdO;
    if (!make_map_bhnd(&mapV, V, BH, D.N, DV, kTileTokens) || !make_map_bhnd(&mapdO, dO, BH, D.N, DV, kTileTokens)) return HLA_ERR_CUDA;
    int* status = reinterpret_cast<int*>(ws + L.status);
    float* part = reinterpret_cast<float*>(ws + off_part);
    float* state = reinterpret_cast<float*>(ws + L.state);
    const float* eta = reinterpret_cast<const float*>(ws + L.eta);
    const float* delta = reinterpret_cast<const float*>(ws + off_delta);
    const int T = (D.N + kTileTokens - 1) / kTileTokens;
    if (!second) {
        if (!set_smem(tc_state_build_kernel<DV, 3>, SbCfg<3>::kSmem) || !set_smem(tc_causal_grad_kernel<DV, 0>, CgCfg<DV>::kSmem)) return HLA_ERR_CUDA;
        rec.begin("tc_state_build");
        launch_pdl(tc_state_build_kernel<DV, 3>, dim3(D.S, BH), dim3(kSbThreads), SbCfg<3>::kSmem, rec.st, mapV, kf, part, D.N, D.S, D.ld, status,
                   (const float*)nullptr, (const float*)nullptr, 0.f);
        if (!rec.end()) return HLA_ERR_CUDA;
        rec.begin("tc_scan_pieces");
        launch_pdl(tc_scan_pieces_kernel<3>, dim3((kMono * D.ld + 255) / 256, BH), dim3(256), 0, rec.st, part, state, D.S, D.ld, 0, T, 0);
        if (!rec.end()) return HLA_ERR_CUDA;
        rec.begin("tc_causal_dq");
        launch_pdl(tc_causal_grad_kernel<DV, 0>, dim3(D.S, BH), dim3(kCgThreads), CgCfg<DV>::kSmem, rec.st, mapdO, mapV, qf, kf, eta, delta, (const float*)part, dqf,
                   D.N, BH, D.S, D.ld, D.eps, status);
        return rec.end() ? HLA_OK : HLA_ERR_CUDA;
    }
    if (!set_smem(tc_causal_grad_kernel<DV, 1>, CgCfg<DV>::kSmem)) return HLA_ERR_CUDA;
    rec.begin("tc_causal_dk");
    launch_pdl(tc_causal_grad_kernel<DV, 1>, dim3(D.S, BH), dim3(kCgThreads), CgCfg<DV>::kSmem, rec.st, mapV, mapdO, qf, kf, eta, delta, (const float*)part, dkf, D.N,
               BH, D.S, D.ld, D.eps, status);
    return rec.end() ? HLA_OK : HLA_ERR_CUDA;
}

// dO . o, then dq on the forward states, then the gradient states, dV and dk on them.
inline hla_status causal_backward(const Dims& D, int BH, const float* qf, const float* kf, const void* V, const void* O, const void* dO, float* dqf, float* dkf,
                                  void* dV, char* ws, const hla_ws_layout& L, size_t off_part, size_t off_delta, LaunchRec& rec) {
    if (D.F != 3) return HLA_ERR_UNSUPPORTED;
    hla_status s;
    // the value-gradient pass computes delta first; the forward sweep for dq needs it, so the order is: delta (inside the
    // first call below), dq, then the gradient states with dV, then dk
    if (D.d == 128) {
        s = launch_causal_delta<128>(D, BH, O, dO, ws, off_delta, rec);
        if (s == HLA_OK) s = launch_causal_backward_features<128>(D, BH, qf, kf, V, dO, dqf, dkf, ws, L, off_part, off_delta, false, rec);
        if (s == HLA_OK) s = launch_causal_backward_values<128>(D, BH, qf, kf, dO, dV, ws, L, off_part, off_delta, rec);
        if (s == HLA_OK) s = launch_causal_backward_features<128>(D, BH, qf, kf, V, dO, dqf, dkf, ws, L, off_part, off_delta, true, rec);
    } else {
        s = launch_causal_delta<64>(D, BH, O, dO, ws, off_delta, rec);
        if (s == HLA_OK) s = launch_causal_backward_features<64>(D, BH, qf, kf, V, dO, dqf, dkf, ws, L, off_part, off_delta, false, rec);
        if (s == HLA_OK) s = launch_causal_backward_values<64>(D, BH, qf, kf, dO, dV, ws, L, off_part, off_delta, rec);
        if (s == HLA_OK) s = launch_causal_backward_features<64>(D, BH, qf, kf, V, dO, dqf, dkf, ws, L, off_part, off_delta, true, rec);
    }
    return s;
}

}  // namespace tc
}  // namespace hla
