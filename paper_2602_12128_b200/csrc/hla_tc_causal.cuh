// Causal HLA (Section 4.4 "Causal Attention, Decay Factors and Sequential Updates", Eq. "seq.updates") on the tensor
// cores, F = 3 factors with d_phi = 6, at the level of the folded monomial features.
//
// Token i sees the tokens j <= i.  With the context tensor carried along the sequence (C^i = C^{i-1} + T_{k_i} (x) v_i),
// the output of a 128-token tile splits into what the tokens before the tile contribute and what the tile's own tokens do:
//     [num | eta]_i = mono_i . [Csym | zsym](tokens before the tile)  +  sum_{j in tile, j <= i} (mono_i . Tsym_j) [v_j | 1]
// The first term is the readout of the non-causal path against the state *before* the tile; the second is a 128 x 128
// block of the masked attention matrix times the value tile.  The sequence of a head is cut into pieces (one per CTA that
// touches the head); a first pass builds the state of every piece, a fixed-order exclusive scan over the pieces of a head
// gives each piece its initial state, and the kernel below sweeps a piece tile by tile:
//
//     P      = mono tile * Tsym tile^T                    (MMA, K = 64)      P[i][j] = prod_f (q_i . k^f_j)
//     acc    = mono tile * [Csym | zsym]                  (MMA, K = 64)      state before the tile, bf16 image in shared memory
//     state += Tsym tile^T * [V | 1]                      (MMA, K = 128 tokens, 64 rows)   fp32 in tensor memory
//     Pm     = bf16(P) where j <= i, else 0               (threads; written back to tensor memory as the next A operand)
//     acc   += Pm * [V | 1]                               (MMA, K = 128 tokens)
//     o_i    = acc_i[0..d) / (acc_i[d] + eps)             (threads; TMA store)
//     state -> bf16 image for the next tile               (threads)
//
// Operand rows are shifted by 8 columns, as in the query pass of the backward: a row of the folded key tile is
// [1, 0 x 7, Tsym_0..55] and a row of the monomial tile is [0 x 8, mono_0..55].  Read as the block that follows the
// value blocks, the key tile therefore supplies the "ones" column d of [V | 1], so the normaliser and the key-side sum
// zsym come out of the same products as the numerator and the state (column d), and no product of their own is needed.
// State row 8 + m holds [Csym[m][0..d), zsym[m], 0 ...]; rows 0..7 are kept zero in the bf16 image.  The image is
// double-buffered: the image for tile t + 1 is written while the products of tile t still read theirs.
//
// Warp roles: 0 TMA (value tiles), 1 MMA issue (P, readout, Pm * V), 26 MMA issue (state), 2..5 monomial rows of q, 6..9 folded key rows, 10..17 mask (two warps
// per 32 rows, 64 columns each), 18..21 state image, 22..25 epilogue.  A role is one warp per scheduler running a
// straight instruction stream per tile, so what bounds a tile is the longest of these streams: they are kept short
// (selects only where the mask cuts a 32 x 32 block, conversions 32 columns at a time, out-of-line waits, rolled loops).
#pragma once
#include "hla_tc.cuh"
#include "hla_tc_fused_k.cuh"

namespace hla {
namespace tc {

constexpr int kCaThreads = 27 * 32;
constexpr int kCaStateMmaWarp = 26;
constexpr int kCaGenQWarp0 = 2, kCaGenKWarp0 = 6, kCaMaskWarp0 = 10, kCaConvWarp0 = 18, kCaEpiWarp0 = 22;
constexpr int kCaRowPad = 8;      // operand column / state row of monomial 0

template <int DV> struct CaCfg {
    static constexpr int kVB = DV / 64;                     // 64-column blocks of a value tile
    static constexpr int kStages = 2;
    static constexpr int kOffT = kVB * kBlk;                // folded key tile: directly after the value blocks
    static constexpr int kOffM = kOffT + kBlk;              // query monomial tile
    static constexpr int kStageBytes = kOffM + kBlk;
    static constexpr int kB3Block = 64 * 128;               // 64 state rows x 64 columns
    static constexpr int kB3Bytes = (kVB + 1) * kB3Block;   // one bf16 image of the state
    static constexpr int kOffB3 = kStages * kStageBytes;    // two images: the sweep writes the next one while the current one is read
    static constexpr int kOffO = kOffB3 + 2 * kB3Bytes;
    static constexpr int kOffBars = kOffO + kVB * kBlk;
    static constexpr int kSmem = 1024 + kOffBars + 256;
    static constexpr int kNAcc = DV + 16, kNState = DV + 8;
    static constexpr int kColAcc = 0, kColState = DV + 16, kColP = 2 * DV + 32;      // tensor-memory columns
    static_assert(kColP + 128 <= 512, "tensor memory");
    static_assert(kSmem <= 227 * 1024, "shared memory");
};

// Work items are (head, tile), w = bh * T + tile.  G == 0: grid (S, heads), CTA (s, bh) owns the tiles
// [s * ceil(T / S), (s + 1) * ceil(T / S)) of its head and piece slot (bh, s).  G > 0: G CTAs own contiguous runs of
// work items, CTA c the items [total c / G, total (c + 1) / G); a run inside one head is piece c - (first CTA of the head).
struct CaWork {
    int w0, w1;
};
__device__ __forceinline__ CaWork causal_work(int T, int BH, int S, int G) {
    CaWork w;
    if (G == 0) {
        const int tiles_per = (T + S - 1) / S;
        const int bh = blockIdx.y, s = blockIdx.x;
        w.w0 = bh * T + min(T, s * tiles_per);
        w.w1 = bh * T + min(T, (s + 1) * tiles_per);
    } else {
        const long long total = (long long)BH * T;
        w.w0 = (int)(total * blockIdx.x / G);
        w.w1 = (int)(total * (blockIdx.x + 1) / G);
    }
    return w;
}
__device__ __forceinline__ int causal_slot(int bh, int T, int BH, int S, int G) {
    if (G == 0) return bh * S + blockIdx.x;
    return bh * S + ((int)blockIdx.x - owner_of_work((long long)bh * T, (long long)BH * T, G));
}

// [first, 0 x 7, v_0..55] as one 128-byte operand row
__device__ __forceinline__ void store_shifted_row(uint32_t blk, uint32_t row, float first, const float (&v)[kMono]) {
    st_shared_v4(blk + sw128_off(row, 0), pack_bf16(first, 0.f), 0u, 0u, 0u);
#pragma unroll
    for (int c = 1; c < 8; ++c)
        st_shared_v4(blk + sw128_off(row, c), pack_bf16(v[8 * c - 8], v[8 * c - 7]), pack_bf16(v[8 * c - 6], v[8 * c - 5]),
                     pack_bf16(v[8 * c - 4], v[8 * c - 3]), pack_bf16(v[8 * c - 2], v[8 * c - 1]));
}

// The same rows formed 16 bytes at a time, so that only a few values are live at once.  Chunk C (1..7) holds the
// monomials 8 C - 8 .. 8 C - 1.
template <int M> __device__ __forceinline__ float mono_value(const float (&qs)[6], const float (&q)[6]) {
    constexpr int abc = mono_abc(M), a = abc / 36, b = (abc / 6) % 6, c = abc % 6;
    return qs[a] * q[b] * q[c];
}
template <int C, int... E>
__device__ __forceinline__ void shifted_mono_chunk(uint32_t blk, uint32_t row, const float (&qs)[6], const float (&q)[6], std::integer_sequence<int, E...>) {
    const float v[8] = {mono_value<8 * (C - 1) + E>(qs, q)...};
    st_shared_v4(blk + sw128_off(row, C), pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
}
// [first, 0 x 7, qs_a q_b q_c ...]: qs = q gives the monomials, qs = r q the monomials scaled by r
template <int... C>
__device__ __forceinline__ void shifted_mono_row(uint32_t blk, uint32_t row, float first, const float (&qs)[6], const float (&q)[6],
                                                 std::integer_sequence<int, C...>) {
    st_shared_v4(blk + sw128_off(row, 0), pack_bf16(first, 0.f), 0u, 0u, 0u);
    (shifted_mono_chunk<C + 1>(blk, row, qs, q, std::make_integer_sequence<int, 8>{}), ...);
}
template <int C, int... E>
__device__ __forceinline__ void shifted_key_chunk(uint32_t blk, uint32_t row, const float (&s12)[6][6], const float (&k3)[6], std::integer_sequence<int, E...>) {
    const float v[8] = {folded_value<8 * (C - 1) + E>(s12, k3)...};
    st_shared_v4(blk + sw128_off(row, C), pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
}
template <int... C>
__device__ __forceinline__ void shifted_key_row(uint32_t blk, uint32_t row, float first, const float (&s12)[6][6], const float (&k3)[6],
                                                std::integer_sequence<int, C...>) {
    st_shared_v4(blk + sw128_off(row, 0), pack_bf16(first, 0.f), 0u, 0u, 0u);
    (shifted_key_chunk<C + 1>(blk, row, s12, k3, std::make_integer_sequence<int, 8>{}), ...);
}

// In-place exclusive scan of the piece states of every head, in piece order (bit-reproducible); the sum of all pieces,
// i.e. the state after the last token, goes to `state`.  REVERSE: the scan runs from the last piece to the first (every
// piece gets the sum of the pieces after it).  carry != 0: the scan starts from what `state` holds (the state an earlier
// call left there: Eq. "seq.updates" continued across calls) instead of zero.
template <int F, bool REVERSE = false>
__global__ void __launch_bounds__(256) tc_scan_pieces_kernel(float* __restrict__ part, float* __restrict__ state, int S, int ld, int G, int T, int carry) {
    constexpr int kN = MT<F>::kN;
    const int bh = blockIdx.y;
    grid_launch_dependents();
    grid_dependency_wait();
    const size_t n_per = (size_t)kN * ld;
    int count = S;
    if (G > 0) {
        const long long total = (long long)gridDim.y * T;
        count = owner_of_work((long long)bh * T + T - 1, total, G) - owner_of_work((long long)bh * T, total, G) + 1;
    }
    const size_t e = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (e >= n_per) return;
    float* p = part + (size_t)bh * S * n_per + e;
    float run = carry ? state[(size_t)bh * n_per + e] : 0.f;
    for (int s0 = 0; s0 < count; s0 += 8) {      // eight independent loads in flight, then the scan in piece order
        float t[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) t[k] = s0 + k < count ? p[(size_t)(REVERSE ? count - 1 - s0 - k : s0 + k) * n_per] : 0.f;
#pragma unroll
        for (int k = 0; k < 8; ++k)
            if (s0 + k < count) {
                p[(size_t)(REVERSE ? count - 1 - s0 - k : s0 + k) * n_per] = run;
                run += t[k];
            }
    }
    state[(size_t)bh * n_per + e] = run;
}

// MODE 0: the forward sweep described above.
// MODE 1: the same sweep run backwards over the tokens with the two operand-row tiles exchanged, for the gradient of the
// values: dV_j = sum_{i >= j} (Tsym_j . r_i mono_i) dO_i.  The "query" rows are the folded keys, the "key" rows are the
// scaled monomials [-delta_i, 0 x 7, r_i mono_i] (delta_i = dO_i . o_i, so the carried state is [dCsym | dzsym]), the value
// tile is dO, a CTA walks its piece from the last tile to the first (grid (S, heads) only), the mask keeps i >= j, and
// the result leaves without a normaliser.
template <int DV, int MODE>
__global__ void __launch_bounds__(kCaThreads, 1) tc_causal_forward_kernel(const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapO,
                                                                          const float* __restrict__ qf, const float* __restrict__ kf,
                                                                          const float* __restrict__ init, float* __restrict__ eta_out,
                                                                          const float* __restrict__ eta_in, const float* __restrict__ delta, int N, int BH,
                                                                          int S, int ld, int G, float eps, int* status) {
    using Cfg = CaCfg<DV>;
    constexpr int kStageBytes = Cfg::kStageBytes;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::kOffBars);
    uint64_t* stage_ready = bars;         // [2] 256 arrivals + the TMA transaction: operand-row tiles written, value tile landed
    uint64_t* stage_free = bars + 2;      // [2] 2 MMA commits (one per issuing thread): every product that reads the stage has finished
    uint64_t* p_full = bars + 4;          // MMA commit
    uint64_t* pm_ready = bars + 5;        // 256 arrivals: masked bf16 block is in tensor memory
    uint64_t* b3_ready = bars + 15;       // [2] 128 arrivals, barrier it & 1: state image of tile it (at the start of a piece also the
                                          // state) is in place; two barriers because the image of tile it + 1 can be ready before
                                          // the readout of tile it has waited
    uint64_t* acc_free = bars + 12;       // 128 arrivals: the accumulator has been drained
    uint64_t* rd_done = bars + 13;        // [2] MMA commit after the readout of tile it, on barrier it & 1 (a waiter may lag two
                                          // tiles behind the issuing thread, which one barrier's phase parity cannot tell apart)
    uint64_t* state_full = bars + 7;      // MMA commit
    uint64_t* acc_full = bars + 8;        // MMA commit
    uint64_t* state_read = bars + 9;      // 128 arrivals: the state after a tile has been read out of tensor memory
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 10);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 11);      // (bars + 12: acc_free)

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int T = (N + kTileTokens - 1) / kTileTokens;
    const CaWork cw = causal_work(T, BH, S, G);
    const int w0 = cw.w0, nwork = cw.w1 - cw.w0;
    auto work_of = [&](int it) { return MODE == 0 ? w0 + it : w0 + nwork - 1 - it; };                 // (head, tile) of the CTA's it-th item
    auto starts = [&](int it) { return it == 0 || (MODE == 0 && (w0 + it) % T == 0); };          // a piece begins with this item
    grid_launch_dependents();

    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(&stage_ready[i], 257);
            mbar_init(&stage_free[i], 2);
        }
        mbar_init(p_full, 1);
        mbar_init(pm_ready, 256);
        mbar_init(&b3_ready[0], 128);
        mbar_init(&b3_ready[1], 128);
        mbar_init(acc_free, 128);
        mbar_init(&rd_done[0], 1);
        mbar_init(&rd_done[1], 1);
        mbar_init(state_full, 1);
        mbar_init(acc_full, 1);
        mbar_init(state_read, 128);
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tmap(&mapV);
        prefetch_tmap(&mapO);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    // rows 0..7 of the state images (and their padding columns) are never written again: zero both images once
    for (int i = tid; i < 2 * Cfg::kB3Bytes / 16; i += kCaThreads) reinterpret_cast<uint4*>(smem + Cfg::kOffB3)[i] = make_uint4(0, 0, 0, 0);
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    grid_dependency_wait();
    bool ok = true;

    if (warp == 0) {
        if (lane == 0) {
            for (int it = 0; it < nwork; ++it) {
                const int st = it & 1, u = it >> 1, work = work_of(it);
                if (!mbar_wait_c(&stage_free[st], (u & 1) ^ 1)) { report_timeout(status, 901); break; }
                mbar_arrive_expect_tx(&stage_ready[st], DV * kTileTokens * 2);
                for (int b = 0; b < Cfg::kVB; ++b) tma_load_3d(smem + st * kStageBytes + b * kBlk, &mapV, &stage_ready[st], b * 64, (work % T) * kTileTokens, work / T);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t id_p = idesc_bf16(128, 128, false, false);
            const uint32_t id_r = idesc_bf16(128, Cfg::kNAcc, false, true);
            const uint32_t b3base = smem_u32(smem + Cfg::kOffB3);
            for (int it = 0; it < nwork; ++it) {
                const int st = it & 1, u = it >> 1;
                const uint32_t sa = smem_u32(smem + st * kStageBytes), ta = sa + Cfg::kOffT, ma = sa + Cfg::kOffM;
                if (!mbar_wait_c(&stage_ready[st], u & 1)) { report_timeout(status, 902); break; }
                tc_fence_after();
                {      // P = mono * Tsym^T
                    uint64_t da = smem_desc_sw128(ma, 16, 1024), db = smem_desc_sw128(ta, 16, 1024);
#pragma unroll 1
                    for (int ks = 0; ks < 4; ++ks, da += 2, db += 2) umma_bf16(tmem + Cfg::kColP, da, db, id_p, ks > 0 ? 1u : 0u);
                }
                umma_commit(p_full);
                if (!(mbar_wait_c(&b3_ready[it & 1], (it >> 1) & 1) && mbar_wait_c(acc_free, (it & 1) ^ 1))) { report_timeout(status, 903); break; }
                tc_fence_after();
                const uint32_t b3a = b3base + (it & 1) * Cfg::kB3Bytes;
                {      // acc = mono * [Csym | zsym] of the tokens before the tile
                    uint64_t da = smem_desc_sw128(ma, 16, 1024), db = smem_desc_sw128(b3a, Cfg::kB3Block, 1024);
#pragma unroll 1
                    for (int ks = 0; ks < 4; ++ks, da += 2, db += 128) umma_bf16(tmem + Cfg::kColAcc, da, db, id_r, ks > 0 ? 1u : 0u);
                }
                umma_commit(&rd_done[it & 1]);
                if (!mbar_wait_c(pm_ready, it & 1)) { report_timeout(status, 905); break; }
                tc_fence_after();
                {      // acc += Pm * [V | 1]; the two packed halves of Pm sit at columns 0..31 and 64..95 of the block
                    uint64_t db = smem_desc_sw128(sa, kBlk, 1024);
#pragma unroll 1
                    for (int ks = 0; ks < kTileTokens / 16; ++ks, db += 128) umma_bf16_ta(tmem + Cfg::kColAcc, tmem + Cfg::kColP + 8 * ks + (ks >= 4 ? 32 : 0), db, id_r, 1u);
                }
                umma_commit(acc_full);
                umma_commit(&stage_free[st]);
            }
        }
    } else if (warp == kCaStateMmaWarp) {
        // The state products are issued by a thread of their own: they depend on nothing the other products make, and the
        // chain state -> image -> readout of consecutive tiles is the long one.
        if (lane == 0) {
            const uint32_t id_s = idesc_bf16(64, Cfg::kNState, true, true);
            for (int it = 0; it < nwork; ++it) {
                const int st = it & 1, u = it >> 1;
                const uint32_t sa = smem_u32(smem + st * kStageBytes), ta = sa + Cfg::kOffT;
                // the state after the previous tile must have been read out of tensor memory; the first tile of a piece
                // waits for the initial state
                if (it > 0 && !mbar_wait_c(state_read, (it - 1) & 1)) { report_timeout(status, 911); break; }
                if (starts(it) && !mbar_wait_c(&b3_ready[it & 1], (it >> 1) & 1)) { report_timeout(status, 912); break; }
                if (!mbar_wait_c(&stage_ready[st], u & 1)) { report_timeout(status, 904); break; }
                tc_fence_after();
                {      // state += Tsym^T * [V | 1]
                    uint64_t da = smem_desc_sw128(ta, kBlk, 1024), db = smem_desc_sw128(sa, kBlk, 1024);
#pragma unroll 1
                    for (int ks = 0; ks < kTileTokens / 16; ++ks, da += 128, db += 128) umma_bf16(tmem + Cfg::kColState, da, db, id_s, 1u);
                }
                umma_commit(state_full);
                umma_commit(&stage_free[st]);
            }
        }
    } else if (warp < kCaMaskWarp0) {
        // operand rows: thread = token row of the tile.  Warps 2..5 write the tile the attention block and the readout take as
        // their A operand (MODE 0: monomials of q; MODE 1: folded keys), warps 6..9 the tile that sits behind the value blocks
        // (MODE 0: folded keys with the ones column; MODE 1: scaled monomials with -delta in that column).
        const bool first_group = warp < kCaGenKWarp0;
        const int row = (tid - kCaGenQWarp0 * 32) & 127;
        const bool from_q = first_group == (MODE == 0);
        const int dst_off = first_group ? Cfg::kOffM : Cfg::kOffT;
        if (from_q) {
            float qn[6], en = 0.f, dn = 0.f;
            auto prefetch = [&](int it) {
                const int work = work_of(it), bh = work / T, tok = min((work % T) * kTileTokens + row, N - 1);
                load_feat<6>(qn, qf + ((size_t)bh * N + tok) * 6);
                if (MODE == 1) {
                    en = __ldg(eta_in + (size_t)bh * N + tok);
                    dn = __ldg(delta + (size_t)bh * N + tok);
                }
            };
            if (nwork > 0) prefetch(0);
            for (int it = 0; it < nwork; ++it) {
                const int st = it & 1, u = it >> 1, work = work_of(it);
                const bool valid = (work % T) * kTileTokens + row < N;
                float q[6], qs[6], first = 0.f;
#pragma unroll
                for (int i = 0; i < 6; ++i) q[i] = valid ? qn[i] : 0.f;
                if (MODE == 1) {
                    const float r = valid ? 1.f / (en + eps) : 0.f;
#pragma unroll
                    for (int i = 0; i < 6; ++i) qs[i] = r * q[i];
                    first = valid ? -dn : 0.f;
                } else {
#pragma unroll
                    for (int i = 0; i < 6; ++i) qs[i] = q[i];
                }
                if (ok && !mbar_wait_c(&stage_free[st], (u & 1) ^ 1)) { ok = false; report_timeout(status, 906); }
                if (!ok) continue;
                shifted_mono_row(smem_u32(smem + st * kStageBytes) + dst_off, row, first, qs, q, std::make_integer_sequence<int, 7>{});
                fence_proxy_async();
                mbar_arrive(&stage_ready[st]);
                if (it + 1 < nwork) prefetch(it + 1);      // after the fence: a fence waits for the loads in flight
            }
        } else {
            float kn[18];
            auto prefetch = [&](int it) {
                const int work = work_of(it), bh = work / T, tok = min((work % T) * kTileTokens + row, N - 1);
#pragma unroll
                for (int f = 0; f < 3; ++f) load_feat<6>(kn + 6 * f, kf + (((size_t)bh * 3 + f) * N + tok) * 6);
            };
            if (nwork > 0) prefetch(0);
            for (int it = 0; it < nwork; ++it) {
                const int st = it & 1, u = it >> 1, work = work_of(it);
                const bool valid = (work % T) * kTileTokens + row < N;
                float k[18];
#pragma unroll
                for (int i = 0; i < 18; ++i) k[i] = valid ? kn[i] : 0.f;
                if (ok && !mbar_wait_c(&stage_free[st], (u & 1) ^ 1)) { ok = false; report_timeout(status, 910); }
                if (!ok) continue;
                float s12[6][6], k3[6];      // [x][y], x < y: k1[x] k2[y] + k1[y] k2[x];  [x][x]: k1[x] k2[x]
#pragma unroll
                for (int x = 0; x < 6; ++x) {
                    k3[x] = k[12 + x];
#pragma unroll
                    for (int y = x; y < 6; ++y) s12[x][y] = (x == y) ? k[x] * k[6 + x] : fmaf(k[x], k[6 + y], k[y] * k[6 + x]);
                }
                shifted_key_row(smem_u32(smem + st * kStageBytes) + dst_off, row, (MODE == 0 && valid) ? 1.f : 0.f, s12, k3, std::make_integer_sequence<int, 7>{});
                fence_proxy_async();
                mbar_arrive(&stage_ready[st]);
                if (it + 1 < nwork) prefetch(it + 1);
            }
        }
    } else if (warp < kCaConvWarp0) {
        // mask: thread = query row i of the block, two warps per 32 rows: warp (qt, half) owns the columns 64 half .. 64 half
        // + 63 of the rows 32 qt .. 32 qt + 31.  A 32 x 32 sub-block left of the diagonal is kept whole, right of it dropped;
        // only the diagonal one is cut element by element.  Each warp packs its 64 columns over the first 32 of them.
        const int qt = warp & 3, half = (warp - kCaMaskWarp0) >> 2;
        const uint32_t pa = tmem + Cfg::kColP + 64 * half + ((uint32_t)(qt * 32) << 16);
        for (int it = 0; it < nwork; ++it) {
            if (ok && !mbar_wait_c(p_full, it & 1)) { ok = false; report_timeout(status, 907); }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
#pragma unroll 1
            for (int bb = 0; bb < 2; ++bb) {      // sub-block column 2 half + bb against sub-block row qt
                const int b = 2 * half + bb;
                uint32_t w[16];
                const bool whole = MODE == 0 ? b < qt : b > qt;      // sub-block entirely on the kept side of the diagonal
                if (whole || b == qt) {
                    uint32_t r[32];
                    tmem_ld16(pa + 32 * bb, *reinterpret_cast<uint32_t(*)[16]>(r));
                    tmem_ld16(pa + 32 * bb + 16, *reinterpret_cast<uint32_t(*)[16]>(r + 16));
                    tmem_ld_wait();
                    if (whole) {
#pragma unroll
                        for (int e = 0; e < 16; ++e) w[e] = pack_bf16(__uint_as_float(r[2 * e]), __uint_as_float(r[2 * e + 1]));
                    } else if (MODE == 0) {
#pragma unroll
                        for (int e = 0; e < 16; ++e)
                            w[e] = pack_bf16(2 * e <= lane ? __uint_as_float(r[2 * e]) : 0.f, 2 * e + 1 <= lane ? __uint_as_float(r[2 * e + 1]) : 0.f);
                    } else {
#pragma unroll
                        for (int e = 0; e < 16; ++e)
                            w[e] = pack_bf16(2 * e >= lane ? __uint_as_float(r[2 * e]) : 0.f, 2 * e + 1 >= lane ? __uint_as_float(r[2 * e + 1]) : 0.f);
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
            mbar_arrive(pm_ready);
        }
    } else if (warp < kCaEpiWarp0) {
        // state image.  A 64-row accumulator keeps row R in lane 32 (R / 16) + R % 16: lanes 0..15 of each warp's quarter.
        const int qt = warp & 3, R = qt * 16 + lane, m = R - kCaRowPad;
        const bool active = lane < 16, mine = active && m >= 0 && m < kMono;
        const uint32_t sa = tmem + Cfg::kColState + ((uint32_t)(qt * 32) << 16);
        const uint32_t b3base = smem_u32(smem + Cfg::kOffB3);
        constexpr int kChunks = Cfg::kNAcc / 8;      // 16-byte chunks of an image row
        auto store_chunk = [&](int img, int c, const float (&v)[8]) {      // image `img` is the one item `img` (mod 2) reads
            if (active)
                st_shared_v4(b3base + (img & 1) * Cfg::kB3Bytes + (c >> 3) * Cfg::kB3Block + sw128_off(R, c & 7), pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]),
                             pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
        };
        for (int it = 0; it < nwork; ++it) {
            const int work = work_of(it), bh = work / T;
            if (starts(it)) {
                // a piece begins: its initial state goes to tensor memory (fp32) and to the image (bf16)
                const float* src = init + ((size_t)causal_slot(bh, T, BH, S, G) * kMono + (mine ? m : 0)) * ld;
#pragma unroll 1
                for (int c = 0; c < kChunks; ++c) {
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
                    if (8 * c < Cfg::kNState)
                        tmem_st8(sa + 8 * c, __float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]), __float_as_uint(v[3]), __float_as_uint(v[4]),
                                 __float_as_uint(v[5]), __float_as_uint(v[6]), __float_as_uint(v[7]));
                    store_chunk(it, c, v);
                }
                tmem_st_wait();
                tc_fence_before();
                fence_proxy_async();
                mbar_arrive(&b3_ready[it & 1]);
            }
            if (ok && !mbar_wait_c(state_full, it & 1)) { ok = false; report_timeout(status, 908); }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            if (it + 1 < nwork && !starts(it + 1)) {
                // the image written now was last read by the readout of the previous tile (issued by the other thread)
                if (it > 0 && ok && !mbar_wait_c(&rd_done[(it - 1) & 1], ((it - 1) >> 1) & 1)) { ok = false; report_timeout(status, 913); }
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                // 32 columns per batch of loads; column d (zsym) rides with the last batch.  The state product of the next tile
                // may run as soon as the last load has completed.  Rows that hold no monomial stay zero.
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
                            const int cc = 4 * h + c;      // 16-byte chunk of the image row
                            st_shared_v4(img + (cc >> 3) * Cfg::kB3Block + sw128_off(R, cc & 7), pack_bf16(__uint_as_float(r[8 * c]), __uint_as_float(r[8 * c + 1])),
                                         pack_bf16(__uint_as_float(r[8 * c + 2]), __uint_as_float(r[8 * c + 3])),
                                         pack_bf16(__uint_as_float(r[8 * c + 4]), __uint_as_float(r[8 * c + 5])),
                                         pack_bf16(__uint_as_float(r[8 * c + 6]), __uint_as_float(r[8 * c + 7])));
                        }
                        if (h == DV / 32 - 1)
                            st_shared_v4(img + (DV / 64) * Cfg::kB3Block + sw128_off(R, 0), pack_bf16(__uint_as_float(rz[0]), 0.f), 0u, 0u, 0u);
                    }
                }
                tc_fence_before();
                fence_proxy_async();
                mbar_arrive(&b3_ready[(it + 1) & 1]);
            } else {
                mbar_arrive(state_read);      // nothing is read: the next tile (if any) starts a piece with a state of its own
            }
        }
    } else {
        // epilogue: thread = token row
        const int qt = warp & 3, row = qt * 32 + lane, etid = tid - kCaEpiWarp0 * 32;
        const uint32_t aa = tmem + Cfg::kColAcc + ((uint32_t)(qt * 32) << 16);
        const uint32_t os = smem_u32(smem + Cfg::kOffO);
        for (int it = 0; it < nwork; ++it) {
            const int work = work_of(it), bh = work / T, tile = work % T;
            if (!mbar_wait_c(acc_full, it & 1)) {
                report_timeout(status, 909);
                *abort_flag = 1;
            }
            if (etid == 0) tma_store_wait_read0();      // the staging tile has been read by the previous store
            named_barrier(1, 128);
            if (*abort_flag) break;
            tc_fence_after();
            uint32_t re[8];
            tmem_ld8(aa + DV, re);
            tmem_ld_wait();
            const float eta = __uint_as_float(re[0]);
            const float rinv = MODE == 0 ? 1.f / (eta + eps) : 1.f;
#pragma unroll 1
            for (int h = 0; h < DV / 32; ++h) {
                uint32_t r[32];
                tmem_ld16(aa + 32 * h, *reinterpret_cast<uint32_t(*)[16]>(r));
                tmem_ld16(aa + 32 * h + 16, *reinterpret_cast<uint32_t(*)[16]>(r + 16));
                tmem_ld_wait();
                if (h == DV / 32 - 1) {
                    tc_fence_before();
                    mbar_arrive(acc_free);
                }
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    st_shared_v4(os + (h >> 1) * kBlk + sw128_off(row, 4 * (h & 1) + c), pack_bf16(__uint_as_float(r[8 * c]) * rinv, __uint_as_float(r[8 * c + 1]) * rinv),
                                 pack_bf16(__uint_as_float(r[8 * c + 2]) * rinv, __uint_as_float(r[8 * c + 3]) * rinv),
                                 pack_bf16(__uint_as_float(r[8 * c + 4]) * rinv, __uint_as_float(r[8 * c + 5]) * rinv),
                                 pack_bf16(__uint_as_float(r[8 * c + 6]) * rinv, __uint_as_float(r[8 * c + 7]) * rinv));
            }
            fence_proxy_async();
            named_barrier(1, 128);
            if (etid == 0) {
                for (int b = 0; b < Cfg::kVB; ++b) tma_store_3d(&mapO, smem + Cfg::kOffO + b * kBlk, b * 64, tile * kTileTokens, bh);
                tma_store_commit();
            }
            const int tok = tile * kTileTokens + row;
            if (MODE == 0 && tok < N) eta_out[(size_t)bh * N + tok] = eta;
        }
        if (etid == 0) tma_store_wait_all0();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, 512);
}

// Exclusive scan of the piece states, then the causal sweep.  The pieces are those of the kernel that built them:
// G == 0: S pieces per head from a (S, heads) grid; G > 0: the pieces of a persistent kernel of G CTAs (at most S per head).
template <int DV>
inline hla_status launch_causal_sweep(const Dims& D, int BH, const float* qf, const float* kf, const void* V, void* O, char* ws, const hla_ws_layout& L,
                                      size_t off_part, int S, int G, bool carry, LaunchRec& rec) {
    CUtensorMap mapV, mapO;
    if (!make_map_bhnd(&mapV, V, BH, D.N, DV, kTileTokens) || !make_map_bhnd(&mapO, O, BH, D.N, DV, kTileTokens)) return HLA_ERR_CUDA;
    int* status = reinterpret_cast<int*>(ws + L.status);
    float* part = reinterpret_cast<float*>(ws + off_part);
    float* state = reinterpret_cast<float*>(ws + L.state);
    float* eta = reinterpret_cast<float*>(ws + L.eta);
    if (!set_smem(tc_causal_forward_kernel<DV, 0>, CaCfg<DV>::kSmem)) return HLA_ERR_CUDA;
    const int T = (D.N + kTileTokens - 1) / kTileTokens;
    rec.begin("tc_scan_pieces");
    launch_pdl(tc_scan_pieces_kernel<3>, dim3((kMono * D.ld + 255) / 256, BH), dim3(256), 0, rec.st, part, state, S, D.ld, G, T, carry ? 1 : 0);
    if (!rec.end()) return HLA_ERR_CUDA;
    rec.begin("tc_causal_forward");
    launch_pdl(tc_causal_forward_kernel<DV, 0>, G > 0 ? dim3(G) : dim3(S, BH), dim3(kCaThreads), CaCfg<DV>::kSmem, rec.st, mapV, mapO, qf, kf,
               (const float*)part, eta, (const float*)nullptr, (const float*)nullptr, D.N, BH, S, D.ld, G, D.eps, status);
    return rec.end() ? HLA_OK : HLA_ERR_CUDA;
}

inline hla_status causal_sweep(const Dims& D, int BH, const float* qf, const float* kf, const void* V, void* O, char* ws, const hla_ws_layout& L,
                               size_t off_part, int S, int G, bool carry, LaunchRec& rec) {
    if (D.F != 3) return HLA_ERR_UNSUPPORTED;
    if (D.d == 128) return launch_causal_sweep<128>(D, BH, qf, kf, V, O, ws, L, off_part, S, G, carry, rec);
    return launch_causal_sweep<64>(D, BH, qf, kf, V, O, ws, L, off_part, S, G, carry, rec);
}

// Feature-level causal forward: state of every piece (the non-causal state build, one piece per split) -> scan -> sweep.
template <int DV>
inline hla_status launch_causal_state_build(const Dims& D, int BH, const float* kf, const void* V, char* ws, const hla_ws_layout& L, size_t off_part,
                                            LaunchRec& rec) {
    CUtensorMap mapV;
    if (!make_map_bhnd(&mapV, V, BH, D.N, DV, kTileTokens)) return HLA_ERR_CUDA;
    if (!set_smem(tc_state_build_kernel<DV, 3>, SbCfg<3>::kSmem)) return HLA_ERR_CUDA;
    rec.begin("tc_state_build");
    launch_pdl(tc_state_build_kernel<DV, 3>, dim3(D.S, BH), dim3(kSbThreads), SbCfg<3>::kSmem, rec.st, mapV, kf, reinterpret_cast<float*>(ws + off_part), D.N, D.S,
               D.ld, reinterpret_cast<int*>(ws + L.status), (const float*)nullptr, (const float*)nullptr, 0.f);
    return rec.end() ? HLA_OK : HLA_ERR_CUDA;
}

inline hla_status causal_forward(const Dims& D, int BH, const float* qf, const float* kf, const void* V, void* O, char* ws, const hla_ws_layout& L,
                                 size_t off_part, bool carry, LaunchRec& rec) {
    if (D.F != 3) return HLA_ERR_UNSUPPORTED;
    const hla_status s = D.d == 128 ? launch_causal_state_build<128>(D, BH, kf, V, ws, L, off_part, rec)
                                    : launch_causal_state_build<64>(D, BH, kf, V, ws, L, off_part, rec);
    if (s != HLA_OK) return s;
    return causal_sweep(D, BH, qf, kf, V, O, ws, L, off_part, D.S, 0, carry, rec);
}

// delta_i = dO_i . o_i for every token row (bf16 rows of d values, fp32 sum): d / 8 lanes per row, 16 bytes per lane.
template <int DV>
__global__ void __launch_bounds__(256) tc_delta_kernel(const __nv_bfloat16* __restrict__ O, const __nv_bfloat16* __restrict__ dO, float* __restrict__ delta,
                                                       long long rows) {
    constexpr int LPR = DV / 8;                 // lanes per row
    grid_launch_dependents();
    grid_dependency_wait();
    const long long t = (long long)blockIdx.x * 256 + threadIdx.x;
    const long long row = t / LPR;
    const int part = (int)(t % LPR);
    float a = 0.f;
    if (row < rows) {
        const uint4 x = *reinterpret_cast<const uint4*>(O + row * DV + 8 * part);
        const uint4 y = *reinterpret_cast<const uint4*>(dO + row * DV + 8 * part);
        const uint32_t xs[4] = {x.x, x.y, x.z, x.w}, ys[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            a = fmaf(__uint_as_float(xs[e] << 16), __uint_as_float(ys[e] << 16), a);
            a = fmaf(__uint_as_float(xs[e] & 0xffff0000u), __uint_as_float(ys[e] & 0xffff0000u), a);
        }
    }
#pragma unroll
    for (int o = LPR / 2; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
    if (row < rows && part == 0) delta[row] = a;
}

template <int DV>
inline hla_status launch_causal_delta(const Dims& D, int BH, const void* O, const void* dO, char* ws, size_t off_delta, LaunchRec& rec) {
    const long long rows = (long long)BH * D.N;
    rec.begin("tc_delta");
    launch_pdl(tc_delta_kernel<DV>, dim3((unsigned)((rows * (DV / 8) + 255) / 256)), dim3(256), 0, rec.st, static_cast<const __nv_bfloat16*>(O),
               static_cast<const __nv_bfloat16*>(dO), reinterpret_cast<float*>(ws + off_delta), rows);
    return rec.end() ? HLA_OK : HLA_ERR_CUDA;
}

// Backward of the causal operator at the feature level, value side: the gradient state of every piece, its suffix scan,
// and the sweep that gives dV (delta must have been computed).
template <int DV>
inline hla_status launch_causal_backward_values(const Dims& D, int BH, const float* qf, const float* kf, const void* dO, void* dV, char* ws,
                                                const hla_ws_layout& L, size_t off_part, size_t off_delta, LaunchRec& rec) {
    CUtensorMap mapdO, mapdV;
    if (!make_map_bhnd(&mapdO, dO, BH, D.N, DV, kTileTokens) || !make_map_bhnd(&mapdV, dV, BH, D.N, DV, kTileTokens)) return HLA_ERR_CUDA;
    int* status = reinterpret_cast<int*>(ws + L.status);
    float* part = reinterpret_cast<float*>(ws + off_part);
    float* dstate = reinterpret_cast<float*>(ws + L.dstate);
    float* eta = reinterpret_cast<float*>(ws + L.eta);
    float* delta = reinterpret_cast<float*>(ws + off_delta);
    if (!set_smem(tc_state_build_kernel<DV, 3, true>, SbCfg<3>::kSmem) || !set_smem(tc_causal_forward_kernel<DV, 1>, CaCfg<DV>::kSmem)) return HLA_ERR_CUDA;
    const int T = (D.N + kTileTokens - 1) / kTileTokens;
    rec.begin("tc_dstate_build");
    launch_pdl(tc_state_build_kernel<DV, 3, true>, dim3(D.S, BH), dim3(kSbThreads), SbCfg<3>::kSmem, rec.st, mapdO, qf, part, D.N, D.S, D.ld, status,
               (const float*)eta, (const float*)delta, D.eps);
    if (!rec.end()) return HLA_ERR_CUDA;
    rec.begin("tc_scan_pieces");
    launch_pdl(tc_scan_pieces_kernel<3, true>, dim3((kMono * D.ld + 255) / 256, BH), dim3(256), 0, rec.st, part, dstate, D.S, D.ld, 0, T, 0);
    if (!rec.end()) return HLA_ERR_CUDA;
    rec.begin("tc_causal_dv");
    launch_pdl(tc_causal_forward_kernel<DV, 1>, dim3(D.S, BH), dim3(kCaThreads), CaCfg<DV>::kSmem, rec.st, mapdO, mapdV, qf, kf, (const float*)part,
               (float*)nullptr, (const float*)eta, (const float*)delta, D.N, BH, D.S, D.ld, 0, D.eps, status);
    return rec.end() ? HLA_OK : HLA_ERR_CUDA;
}

}  // namespace tc
}  // namespace hla
