// Tensor-core (tcgen05 / TMEM / TMA) kernels of the HLA core for bf16, F = 3
// factors with d_phi = 6 (P = 216 features), d in {64, 128}.
//
// Symmetry folding.  The query tensor T_q[i] = q_i (x) q_i (x) q_i is symmetric, so the
// readout sum_p T_q[i][p] C[p] only sees C summed over index permutations:
//     sum_p T_q[i][p] C[p][g] = sum_m mono_i[m] Csym[m][g],   m = (a <= b <= c), 56 monomials,
//     mono_i[m] = q_a q_b q_c,   Csym[m] = sum over the distinct permutations (x,y,z) of (a,b,c) of C[xyz].
// Because C = sum_j T_k[j] v_j^T (Theorem 4.2), Csym = sum_j Tsym_k[j] v_j^T with the folded key
// feature Tsym_k[j][m] = sum over distinct permutations of k1_j[x] k2_j[y] k3_j[z].  So every
// contraction of the path runs over 56 (padded to 64) features instead of 216, with identical
// results up to rounding order; the kept state is the folded one, [56][d] (+ the folded z).
//
//   state build : Csym^T[d x 64] += V_tile^T[d x 128 tok] * Tsym_k tile[128 tok x 64]; zsym in fp32 registers
//   reduce/emit : fixed-order sum of the split partials; emits the bf16 MMA operands of the state
//   readout     : [num | eta][128 tok x (d+16)] = mono tile[128 x 64] * [Csym | zsym]; o = num / (eta + eps)
//   bwd (query) : D2 = dO * Csym^T -> delta, dmono, dq on the ALUs;  dCsym^T += dO^T * (r mono);  dzsym on the ALUs
//   bwd (key)   : dV = Tsym_k * dCsym;  G = V * dCsym^T + dzsym -> dk1, dk2, dk3 on the ALUs
//
// Operand tiles are formed in registers, rounded once to bf16 and written straight into the
// 128-byte-swizzled shared-memory layout the MMA descriptors describe; T_q / T_k never exist in global memory.
#pragma once
#include "../../include/hla.h"
#include "hla_common.cuh"
#include <utility>
#include "hla_tc_prim.cuh"

namespace hla {
namespace tc {

constexpr int kTileTokens = 128;
constexpr int kMono = 56;        // distinct monomials of degree 3 in 6 variables
constexpr int kMonoPad = 64;
constexpr int kBlk = 16384;      // one 128-row x 128-byte swizzled block

// index of the monomial (a <= b <= c) in lexicographic order
__host__ __device__ constexpr int mono_idx(int a, int b, int c) { return a * (a * a - 21 * a + 146) / 6 + (b - a) * (13 - a - b) / 2 + (c - b); }
__host__ __device__ constexpr int imin(int a, int b) { return a < b ? a : b; }
__host__ __device__ constexpr int imax(int a, int b) { return a > b ? a : b; }
__host__ __device__ constexpr int mono_of(int x, int y, int z) {
    return mono_idx(imin(imin(x, y), z), x + y + z - imin(imin(x, y), z) - imax(imax(x, y), z), imax(imax(x, y), z));
}

// The two monomial geometries of the tensor-core path.  F factors of d_phi features each: the query tensor q (x) ... (x) q
// has kN distinct monomials; every operand tile over the monomials is kPad columns wide, in kBlocks swizzled blocks of 64.
//   F = 3, d_phi = 6  (the paper's main model): 56 monomials q_a q_b q_c, a <= b <= c
//   F = 2, d_phi = 12 (its 2-factor variant):   78 monomials q_a q_b,     a <= b
template <int F> struct MT;
template <> struct MT<3> { static constexpr int kDphi = 6, kN = 56, kPad = 64, kBlocks = 1, kKf = 18, kMaps = 3; };
template <> struct MT<2> { static constexpr int kDphi = 12, kN = 78, kPad = 80, kBlocks = 2, kKf = 24, kMaps = 2; };
// index of the monomial (a <= b) of the 2-factor geometry in lexicographic order
__host__ __device__ constexpr int mono_idx2(int a, int b) { return a * (25 - a) / 2 + (b - a); }

struct Plan {
    size_t b3;    // bf16 [BH][d+16][kPad]  rows g < d: Csym[.][g] (K-major over m); row d: zsym; rest 0
    size_t bq;    // bf16 [BH][kPad][d]     Csym[m][.]
    size_t bd3;   // the same two operands of the gradient state (dCsym | dzsym)
    size_t bdq;
    size_t end;
};

inline bool supported(bool bf16, int d, int F, int dphi) { return bf16 && (d == 64 || d == 128) && ((F == 3 && dphi == 6) || (F == 2 && dphi == 12)); }
inline int n_mono(int F) { return F == 3 ? MT<3>::kN : MT<2>::kN; }
inline int mono_pad(int F) { return F == 3 ? MT<3>::kPad : MT<2>::kPad; }

inline size_t plan(Plan& p, const Dims& D, int BH, size_t off) {
    auto up = [](size_t x) { return (x + 255) / 256 * 256; };
    const int pad = mono_pad(D.F);
    const size_t n3 = (size_t)BH * (D.d + 16) * pad * 2, nq = (size_t)BH * pad * D.d * 2;
    p.b3 = off; off = up(off + n3);
    p.bq = off; off = up(off + nq);
    p.bd3 = off; off = up(off + n3);
    p.bdq = off; off = up(off + nq);
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

// Per-context memo of what a call would otherwise redo on the host every time: encoded tensor maps (keyed by base
// pointer and geometry; a caller that passes the same buffers again pays a 128-byte copy instead of a driver call) and
// the kernels whose dynamic shared-memory limit has already been raised.  hla_forward / hla_backward make their
// context's memo current for the calling thread while they run.
struct HostCache {
    struct MapEntry { const void* ptr; uint64_t k0, k1; CUtensorMap map; };
    static constexpr int kMaps = 32, kFuncs = 24;
    MapEntry maps[kMaps];
    int nmaps = 0, next = 0;
    const void* funcs[kFuncs];
    int nfuncs = 0;
    const CUtensorMap* find(const void* ptr, uint64_t k0, uint64_t k1) const {
        for (int i = 0; i < nmaps; ++i)
            if (maps[i].ptr == ptr && maps[i].k0 == k0 && maps[i].k1 == k1) return &maps[i].map;
        return nullptr;
    }
    void insert(const void* ptr, uint64_t k0, uint64_t k1, const CUtensorMap& m) {
        MapEntry& e = maps[nmaps < kMaps ? nmaps++ : (next++ % kMaps)];
        e.ptr = ptr; e.k0 = k0; e.k1 = k1; e.map = m;
    }
};
inline thread_local HostCache* t_host_cache = nullptr;
struct HostCacheScope {
    explicit HostCacheScope(HostCache* c) { t_host_cache = c; }
    ~HostCacheScope() { t_host_cache = nullptr; }
};

// bf16 tensor [BH][N][d] (d innermost), box = 64 columns x box_rows tokens of one head, 128-byte swizzle.
inline bool make_map_bhnd(CUtensorMap* m, const void* ptr, int BH, int N, int d, int box_rows) {
    const uint64_t k0 = (1ull << 63) | ((uint64_t)(uint32_t)BH << 32) | (uint32_t)N, k1 = ((uint64_t)(uint32_t)d << 32) | (uint32_t)box_rows;
    if (t_host_cache)
        if (const CUtensorMap* hit = t_host_cache->find(ptr, k0, k1)) { *m = *hit; return true; }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)N, (cuuint64_t)BH};
    cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)N * d * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
    cuuint32_t es[3] = {1, 1, 1};
    if (fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
           CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    if (t_host_cache) t_host_cache->insert(ptr, k0, k1, *m);
    return true;
}

// bf16 matrix [rows][cols], box = 64 columns x box_rows, 128-byte swizzle.
inline bool make_map_2d(CUtensorMap* m, const void* ptr, size_t rows, int cols, int box_rows) {
    const uint64_t k0 = (uint64_t)rows, k1 = ((uint64_t)(uint32_t)cols << 32) | (uint32_t)box_rows;
    if (t_host_cache)
        if (const CUtensorMap* hit = t_host_cache->find(ptr, k0, k1)) { *m = *hit; return true; }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    cuuint32_t es[2] = {1, 1};
    if (fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
           CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    if (t_host_cache) t_host_cache->insert(ptr, k0, k1, *m);
    return true;
}

// Launch with programmatic stream serialization (see grid_dependency_wait): the kernel's blocks may start while the
// previous kernel of the stream drains; every kernel launched this way waits for its predecessor before it touches
// global memory that the library's kernels write or read.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}
// The same without the attribute, for a kernel that reads caller-provided memory (the phi weights) before its wait and
// may directly follow a kernel of the caller that wrote it: it starts only after everything before it has completed.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_serial(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// ---- small device helpers ----------------------------------------------------------------
__device__ __forceinline__ void report_timeout(int* status, int where) {
    atomicExch(status + kStatusTimeout, 1);
    atomicExch(status + kStatusWhere, where);
}
__device__ __forceinline__ void named_barrier(int id, int nthreads) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory"); }
__device__ __forceinline__ void st_shared_b16(uint32_t addr, unsigned short v) { asm volatile("st.shared.b16 [%0], %1;" ::"r"(addr), "h"(v) : "memory"); }
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ void load6(float* dst, const float* __restrict__ src) {
    const float2* s = reinterpret_cast<const float2*>(src);
    const float2 a = __ldg(s), b = __ldg(s + 1), c = __ldg(s + 2);
    dst[0] = a.x; dst[1] = a.y; dst[2] = b.x; dst[3] = b.y; dst[4] = c.x; dst[5] = c.y;
}
__device__ __forceinline__ void store6(float* dst, const float* v) {
    float2* d = reinterpret_cast<float2*>(dst);
    d[0] = make_float2(v[0], v[1]); d[1] = make_float2(v[2], v[3]); d[2] = make_float2(v[4], v[5]);
}

// d_phi consecutive fp32 features of one token
template <int DP> __device__ __forceinline__ void load_feat(float* dst, const float* __restrict__ src) {
    const float2* s = reinterpret_cast<const float2*>(src);
#pragma unroll
    for (int i = 0; i < DP / 2; ++i) {
        const float2 a = __ldg(s + i);
        dst[2 * i] = a.x;
        dst[2 * i + 1] = a.y;
    }
}
template <int DP> __device__ __forceinline__ void store_feat(float* dst, const float* v) {
    float2* d = reinterpret_cast<float2*>(dst);
#pragma unroll
    for (int i = 0; i < DP / 2; ++i) d[i] = make_float2(v[2 * i], v[2 * i + 1]);
}

// One operand row of kPad bf16 (kN values * scale, then zeros) into row `row` of a tile of kBlocks swizzled 128-row blocks.
template <int F> __device__ __forceinline__ void store_mono_row_t(uint32_t tile, uint32_t row, const float (&m)[MT<F>::kN], float scale) {
    constexpr int N = MT<F>::kN;
#pragma unroll
    for (int c = 0; c < MT<F>::kPad / 8; ++c) {
        float v[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] = 8 * c + e < N ? m[8 * c + e < N ? 8 * c + e : 0] * scale : 0.f;
        st_shared_v4(tile + (c >> 3) * kBlk + sw128_off(row, c & 7), pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
    }
}

// One operand row of 64 bf16 (56 values * scale, 8 zeros) into row `row` of a swizzled 128-row block.
__device__ __forceinline__ void store_mono_row(uint32_t blk, uint32_t row, const float (&m)[kMono], float scale) {
#pragma unroll
    for (int c = 0; c < 7; ++c)
        st_shared_v4(blk + sw128_off(row, c), pack_bf16(m[8 * c] * scale, m[8 * c + 1] * scale), pack_bf16(m[8 * c + 2] * scale, m[8 * c + 3] * scale),
                     pack_bf16(m[8 * c + 4] * scale, m[8 * c + 5] * scale), pack_bf16(m[8 * c + 6] * scale, m[8 * c + 7] * scale));
    st_shared_v4(blk + sw128_off(row, 7), 0u, 0u, 0u, 0u);
}

// mono[m] = q_a q_b q_c for a <= b <= c.
__device__ __forceinline__ void query_monomials(const float (&q)[6], float (&mono)[kMono]) {
#pragma unroll
    for (int a = 0; a < 6; ++a)
#pragma unroll
        for (int b = a; b < 6; ++b) {
            const float qab = q[a] * q[b];
#pragma unroll
            for (int c = b; c < 6; ++c) mono[mono_idx(a, b, c)] = qab * q[c];
        }
}

// dq[x] = sum_m dmono[m] * d(q_a q_b q_c)/dq_x.
__device__ __forceinline__ void query_monomials_grad(const float (&q)[6], const float (&dm)[kMono], float (&dq)[6]) {
    float qq[6][6];
#pragma unroll
    for (int a = 0; a < 6; ++a)
#pragma unroll
        for (int b = a; b < 6; ++b) qq[a][b] = q[a] * q[b];
#pragma unroll
    for (int a = 0; a < 6; ++a) dq[a] = 0.f;
#pragma unroll
    for (int a = 0; a < 6; ++a)
#pragma unroll
        for (int b = a; b < 6; ++b)
#pragma unroll
            for (int c = b; c < 6; ++c) {
                const float g = dm[mono_idx(a, b, c)];
                dq[a] = fmaf(g, qq[b][c], dq[a]);
                dq[b] = fmaf(g, qq[a][c], dq[b]);
                dq[c] = fmaf(g, qq[a][b], dq[c]);
            }
}

// Folded key features: ts[m] = sum over the distinct permutations (x,y,z) of m = (a,b,c) of k1[x] k2[y] k3[z].
// k = (k1[0..5], k2[0..5], k3[0..5]).
__device__ __forceinline__ void key_folded(const float (&k)[18], float (&ts)[kMono]) {
    float s12[6][6];   // [x][y], x < y: k1[x]k2[y] + k1[y]k2[x];  [x][x]: k1[x]k2[x]
#pragma unroll
    for (int x = 0; x < 6; ++x)
#pragma unroll
        for (int y = x; y < 6; ++y) s12[x][y] = (x == y) ? k[x] * k[6 + x] : fmaf(k[x], k[6 + y], k[y] * k[6 + x]);
#pragma unroll
    for (int a = 0; a < 6; ++a)
#pragma unroll
        for (int b = a; b < 6; ++b)
#pragma unroll
            for (int c = b; c < 6; ++c) {
                float v;
                if (a == b && b == c) v = s12[a][a] * k[12 + a];
                else if (a == b) v = fmaf(s12[a][a], k[12 + c], s12[a][c] * k[12 + a]);
                else if (b == c) v = fmaf(s12[a][c], k[12 + c], s12[c][c] * k[12 + a]);
                else v = fmaf(s12[a][b], k[12 + c], fmaf(s12[a][c], k[12 + b], s12[b][c] * k[12 + a]));
                ts[mono_idx(a, b, c)] = v;
            }
}

// Gradients of L = sum_{x,y,z} G[sort(x,y,z)] k1[x] k2[y] k3[z] with respect to k1, k2, k3.
__device__ __forceinline__ void key_folded_grad(const float (&k)[18], const float (&G)[kMono], float (&dk)[18]) {
    float s12[6][6];
#pragma unroll
    for (int x = 0; x < 6; ++x)
#pragma unroll
        for (int y = x; y < 6; ++y) s12[x][y] = (x == y) ? k[x] * k[6 + x] : fmaf(k[x], k[6 + y], k[y] * k[6 + x]);
#pragma unroll
    for (int i = 0; i < 18; ++i) dk[i] = 0.f;
#pragma unroll
    for (int z = 0; z < 6; ++z)
#pragma unroll
        for (int x = 0; x < 6; ++x)
#pragma unroll
            for (int y = x; y < 6; ++y) dk[12 + z] = fmaf(G[mono_of(x, y, z)], s12[x][y], dk[12 + z]);
#pragma unroll
    for (int x = 0; x < 6; ++x)
#pragma unroll
        for (int y = x; y < 6; ++y) {
            float h = 0.f;   // H[x][y] = sum_z G[sort(x,y,z)] k3[z], symmetric in (x, y)
#pragma unroll
            for (int z = 0; z < 6; ++z) h = fmaf(G[mono_of(x, y, z)], k[12 + z], h);
            dk[x] = fmaf(h, k[6 + y], dk[x]);
            dk[6 + y] = fmaf(h, k[x], dk[6 + y]);
            if (x != y) {
                dk[y] = fmaf(h, k[6 + x], dk[y]);
                dk[6 + x] = fmaf(h, k[y], dk[6 + x]);
            }
        }
}

// ---- the same generators for either geometry -----------------------------------------------------------------------------
template <int F> __device__ __forceinline__ void query_monomials_t(const float (&q)[MT<F>::kDphi], float (&mono)[MT<F>::kN]) {
    if constexpr (F == 3) {
        query_monomials(q, mono);
    } else {
#pragma unroll
        for (int a = 0; a < 12; ++a)
#pragma unroll
            for (int b = a; b < 12; ++b) mono[mono_idx2(a, b)] = q[a] * q[b];
    }
}
// dq[x] = sum_m dmono[m] d(monomial m) / dq_x
template <int F> __device__ __forceinline__ void query_monomials_grad_t(const float (&q)[MT<F>::kDphi], const float (&dm)[MT<F>::kN], float (&dq)[MT<F>::kDphi]) {
    if constexpr (F == 3) {
        query_monomials_grad(q, dm, dq);
    } else {
#pragma unroll
        for (int a = 0; a < 12; ++a) dq[a] = 0.f;
#pragma unroll
        for (int a = 0; a < 12; ++a)
#pragma unroll
            for (int b = a; b < 12; ++b) {
                const float g = dm[mono_idx2(a, b)];
                dq[a] = fmaf(g, q[b], dq[a]);
                dq[b] = fmaf(g, q[a], dq[b]);
            }
    }
}
// Folded key features.  F = 2: k = (k1[0..11], k2[0..11]), ts[(a <= b)] = k1[a] k2[b] + k1[b] k2[a]  (a < b),  k1[a] k2[a]  (a == b).
template <int F> __device__ __forceinline__ void key_folded_t(const float (&k)[MT<F>::kKf], float (&ts)[MT<F>::kN]) {
    if constexpr (F == 3) {
        key_folded(k, ts);
    } else {
#pragma unroll
        for (int a = 0; a < 12; ++a)
#pragma unroll
            for (int b = a; b < 12; ++b) ts[mono_idx2(a, b)] = a == b ? k[a] * k[12 + a] : fmaf(k[a], k[12 + b], k[b] * k[12 + a]);
    }
}
// Gradients of L = sum_{x,y} G[sort(x,y)] k1[x] k2[y] (F = 2) with respect to k1, k2.
template <int F> __device__ __forceinline__ void key_folded_grad_t(const float (&k)[MT<F>::kKf], const float (&G)[MT<F>::kN], float (&dk)[MT<F>::kKf]) {
    if constexpr (F == 3) {
        key_folded_grad(k, G, dk);
    } else {
#pragma unroll
        for (int i = 0; i < 24; ++i) dk[i] = 0.f;
#pragma unroll
        for (int x = 0; x < 12; ++x)
#pragma unroll
            for (int y = 0; y < 12; ++y) {
                const float g = G[mono_idx2(x < y ? x : y, x < y ? y : x)];
                dk[x] = fmaf(g, k[12 + y], dk[x]);
                dk[12 + y] = fmaf(g, k[x], dk[12 + y]);
            }
    }
}

// =======================================================================================
// State build
// =======================================================================================
constexpr int kSbThreads = 320;            // warp 0: TMA, warp 1: MMA, warps 2..9: two generator groups of 128 threads
template <int F> struct SbCfg {
    static constexpr int kStages = F == 3 ? 4 : 3;
    static constexpr int kStageBytes = 2 * kBlk + MT<F>::kBlocks * kBlk;   // V (two 64-column blocks) + folded key tile
    static constexpr int kOffZ = kStages * kStageBytes;                    // zred [8 warps][kPad] floats
    static constexpr int kOffBars = kOffZ + 8 * MT<F>::kPad * 4;
    static constexpr int kSmem = 1024 + kOffBars + 256;
    static constexpr int kTmemCols = F == 3 ? 64 : 128;
};

// GRAD = false: the state of Theorem 4.2, rows = folded key features of `kf`, values = V.
// GRAD = true (3 factors only): the gradient of that state when every token sees only the tokens up to itself,
// [dCsym | dzsym] = sum_i r_i mono_i (x) [dO_i | -delta_i]: `kf` points to the query features, the value map to dO,
// r_i = 1 / (eta_i + eps) and delta_i = dO_i . o_i come from `eta` and `delta`.
template <int DV, int F, bool GRAD = false>
__global__ void __launch_bounds__(kSbThreads, 1) tc_state_build_kernel(const __grid_constant__ CUtensorMap mapV, const float* __restrict__ kf,
                                                                       float* __restrict__ part, int N, int S, int ld, int* status,
                                                                       const float* __restrict__ eta = nullptr, const float* __restrict__ delta = nullptr,
                                                                       float eps = 0.f) {
    using M = MT<F>;
    using Cfg = SbCfg<F>;
    constexpr int kStages = Cfg::kStages, kStageBytes = Cfg::kStageBytes;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    float* zred = reinterpret_cast<float*>(smem + Cfg::kOffZ);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::kOffBars);
    uint64_t* full_v = bars;                  // [stages]
    uint64_t* full_t = bars + kStages;        // [stages]
    uint64_t* empty = bars + 2 * kStages;     // [stages]
    uint64_t* acc_done = bars + 3 * kStages;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 3 * kStages + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int s = blockIdx.x, bh = blockIdx.y;
    const int tiles = (N + kTileTokens - 1) / kTileTokens;
    const int tiles_per = (tiles + S - 1) / S;
    const int tile0 = s * tiles_per;
    const int ntiles = max(0, min(tiles, tile0 + tiles_per) - tile0);
    float* out = part + ((size_t)bh * S + s) * M::kN * ld;

    grid_launch_dependents();
    if (ntiles == 0) {   // an empty split contributes zeros
        grid_dependency_wait();
        for (int i = tid; i < M::kN * ld; i += kSbThreads) out[i] = 0.f;
        return;
    }
    if (DV == 64) {      // rows 64..127 of the MMA's M dimension read a second V block: keep it zero
        for (int st = 0; st < kStages; ++st) {
            uint4* vz = reinterpret_cast<uint4*>(smem + st * kStageBytes + kBlk);
            for (int i = tid; i < kBlk / 16; i += kSbThreads) vz[i] = make_uint4(0, 0, 0, 0);
        }
        fence_proxy_async();
    }
    if (tid == 0) {
        for (int i = 0; i < kStages; ++i) {
            mbar_init(&full_v[i], 1);
            mbar_init(&full_t[i], 128);
            mbar_init(&empty[i], 1);
        }
        mbar_init(acc_done, 1);
        fence_mbar_init();
        prefetch_tmap(&mapV);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, Cfg::kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    grid_dependency_wait();
    bool ok = true;

    if (warp == 0) {
        if (lane == 0) {
            for (int it = 0; it < ntiles; ++it) {
                const int st = it % kStages, u = it / kStages;
                if (!mbar_wait(&empty[st], (u & 1) ^ 1)) { report_timeout(status, 101); break; }
                uint8_t* vs = smem + st * kStageBytes;
                mbar_arrive_expect_tx(&full_v[st], DV * kTileTokens * 2);
                for (int b = 0; b < DV / 64; ++b) tma_load_3d(vs + b * kBlk, &mapV, &full_v[st], b * 64, (tile0 + it) * kTileTokens, bh);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = idesc_bf16(128, M::kPad, true, true);
            for (int it = 0; it < ntiles; ++it) {
                const int st = it % kStages, u = it / kStages;
                if (!(mbar_wait(&full_v[st], u & 1) && mbar_wait(&full_t[st], u & 1))) { report_timeout(status, 102); break; }
                tc_fence_after();
                const uint32_t va = smem_u32(smem + st * kStageBytes), ta = va + 2 * kBlk;
#pragma unroll
                for (int ks = 0; ks < kTileTokens / 16; ++ks)
                    umma_bf16(tmem, smem_desc_sw128(va + ks * 2048, kBlk, 1024), smem_desc_sw128(ta + ks * 2048, kBlk, 1024), idesc,
                              (it > 0 || ks > 0) ? 1u : 0u);
                umma_commit(&empty[st]);
            }
            umma_commit(acc_done);
        }
    } else {
        const int grp = (warp - 2) >> 2;
        const int row = ((warp - 2) & 3) * 32 + lane;
        float zacc[M::kN];
#pragma unroll
        for (int i = 0; i < M::kN; ++i) zacc[i] = 0.f;
        // The key features of the group's next tile are loaded while the current one is processed (row index clamped:
        // the loads are unconditional, out-of-range rows are zeroed when used).
        float k[M::kKf], kn[M::kKf], en = 0.f, dn = 0.f;
        auto prefetch = [&](int it) {
            const int tok = min((tile0 + it) * kTileTokens + row, N - 1);
            if constexpr (GRAD) {
                load_feat<M::kDphi>(kn, kf + ((size_t)bh * N + tok) * M::kDphi);
                en = __ldg(eta + (size_t)bh * N + tok);
                dn = __ldg(delta + (size_t)bh * N + tok);
            } else {
#pragma unroll
                for (int f = 0; f < F; ++f) load_feat<M::kDphi>(kn + M::kDphi * f, kf + (((size_t)bh * F + f) * N + tok) * M::kDphi);
            }
        };
        if (grp < ntiles) prefetch(grp);
        for (int it = grp; it < ntiles; it += 2) {
            const int st = it % kStages, u = it / kStages;
            const int tok = (tile0 + it) * kTileTokens + row;
#pragma unroll
            for (int i = 0; i < (GRAD ? M::kDphi : M::kKf); ++i) k[i] = tok < N ? kn[i] : 0.f;
            const float rr = GRAD && tok < N ? 1.f / (en + eps) : 0.f, nd = -dn;
            if (it + 2 < ntiles) prefetch(it + 2);
            float ts[M::kN];
            if constexpr (GRAD) {
                float q[M::kDphi];
#pragma unroll
                for (int i = 0; i < M::kDphi; ++i) q[i] = k[i];
                query_monomials_t<F>(q, ts);
#pragma unroll
                for (int i = 0; i < M::kN; ++i) {
                    ts[i] *= rr;
                    zacc[i] = fmaf(nd, ts[i], zacc[i]);
                }
            } else {
                key_folded_t<F>(k, ts);
#pragma unroll
                for (int i = 0; i < M::kN; ++i) zacc[i] += ts[i];
            }
            if (ok && !mbar_wait(&empty[st], (u & 1) ^ 1)) { ok = false; report_timeout(status, 103); }
            if (ok) {
                store_mono_row_t<F>(smem_u32(smem + st * kStageBytes + 2 * kBlk), row, ts, 1.f);
                fence_proxy_async();
                mbar_arrive(&full_t[st]);
            }
        }
        // zsym: sum the per-token-slot accumulators over the 256 generator threads
#pragma unroll
        for (int i = 0; i < M::kN; ++i) {
            const float v = warp_sum(zacc[i]);
            if (lane == 0) zred[(warp - 2) * M::kPad + i] = v;
        }
        named_barrier(1, 256);
        const int gi = tid - 64;
        if (gi < M::kN) {
            float z = 0.f;
#pragma unroll
            for (int w = 0; w < 8; ++w) z += zred[w * M::kPad + gi];
            out[(size_t)gi * ld + DV] = z;
            for (int c = DV + 1; c < ld; ++c) out[(size_t)gi * ld + c] = 0.f;
        }
        if (warp < 6) {   // warps 2..5 cover the four TMEM lane quarters (lane = value channel g)
            const int quarter = warp & 3;
            if (ok && !mbar_wait(acc_done, 0)) { ok = false; report_timeout(status, 104); }
            ok = __all_sync(0xffffffffu, ok);
            tc_fence_after();
            const int g = quarter * 32 + lane;
            if (ok && quarter * 32 < DV) {
#pragma unroll
                for (int c = 0; c < M::kPad / 8; ++c) {
                    uint32_t r[8];
                    tmem_ld8(tmem + ((uint32_t)(quarter * 32) << 16) + 8 * c, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        if (8 * c + e < M::kN) out[(size_t)(8 * c + e) * ld + g] = __uint_as_float(r[e]);
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, Cfg::kTmemCols);
}

// =======================================================================================
// Reduce the split partials [BH][S][56][ld] in a fixed order -> fp32 folded state [BH][56][ld]
// (column d = folded z) and the two bf16 MMA operands of that state.
// =======================================================================================
// grid = (8, heads): block c of a head owns the monomials 8c .. 8c+7 (block 7 owns only the zero padding 56..63).
// The partials of head bh are the slots [bh * S, bh * S + count).  With G == 0 every head has count = S slots (kernels
// whose grid is splits x heads); with G > 0 the producer was a persistent kernel of G CTAs over heads x T work items and
// the head's slots are its pieces, one per CTA that touched it (see owner_of_work).
__host__ __device__ inline int owner_of_work(long long w, long long total, int G) { return (int)(((w + 1) * G - 1) / total); }

template <int DV, int F>
__global__ void __launch_bounds__(256) tc_reduce_emit_kernel(const float* __restrict__ part, float* __restrict__ state,
                                                             __nv_bfloat16* __restrict__ b3, __nv_bfloat16* __restrict__ bq, int S, int ld, int G, int T) {
    constexpr int kN = MT<F>::kN, kPad = MT<F>::kPad;
    __shared__ float sm[8][kMaxD + 8];
    const int m0 = 8 * blockIdx.x, bh = blockIdx.y, tid = threadIdx.x;      // gridDim.x = kPad / 8
    grid_launch_dependents();
    grid_dependency_wait();
    const size_t n_per = (size_t)kN * ld;
    int count = S;
    if (G > 0) {
        const long long total = (long long)gridDim.y * T;
        count = owner_of_work((long long)bh * T + T - 1, total, G) - owner_of_work((long long)bh * T, total, G) + 1;
    }
    for (int i = tid; i < 8 * ld; i += 256) {
        const int mm = i / ld, col = i - mm * ld, m = m0 + mm;
        float a = 0.f;
        if (m < kN) {
            const float* src = part + (size_t)bh * S * n_per + (size_t)m * ld + col;
            for (int s = 0; s < count; ++s) a += src[(size_t)s * n_per];      // fixed order: bit-reproducible
            state[(size_t)bh * n_per + (size_t)m * ld + col] = a;
        }
        sm[mm][col] = a;
    }
    __syncthreads();
    __nv_bfloat16* o3 = b3 + (size_t)bh * (DV + 16) * kPad;
    for (int row = tid; row < DV + 16; row += 256) {       // row <= DV: column `row` of the state (row == DV is z); rest zero
        uint32_t w[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) w[e] = row <= DV ? pack_bf16(sm[2 * e][row], sm[2 * e + 1][row]) : 0u;
        *reinterpret_cast<uint4*>(o3 + (size_t)row * kPad + m0) = make_uint4(w[0], w[1], w[2], w[3]);
    }
    __nv_bfloat16* oq = bq + (size_t)bh * kPad * DV;
    for (int i = tid; i < 8 * DV; i += 256) {
        const int mm = i / DV, g = i - mm * DV;
        oq[(size_t)(m0 + mm) * DV + g] = __float2bfloat16_rn(sm[mm][g]);
    }
}

// =======================================================================================
// Readout + normaliser
// =======================================================================================
// warps 0..7: epilogue (thread = token row x half of the value channels; one warp per scheduler could not keep up with
// the tile rate), warps 8..11: monomial generators, warp 12: TMA + MMA
constexpr int kRoThreads = 416;
constexpr int kRoGenWarp0 = 8, kRoMmaWarp = 12;
template <int DV, int F> struct RoCfg {
    static constexpr int kNmma = DV + 16;
    static constexpr int kABytes = MT<F>::kBlocks * kBlk;                       // one monomial tile
    static constexpr int kB3Block = ((kNmma * 128 + 1023) / 1024) * 1024;       // one 64-monomial block of the state operand: [kNmma rows][128 B]
    static constexpr int kB3Bytes = MT<F>::kBlocks * kNmma * 128;               // bytes the TMA loads deliver
    static constexpr int kOBytes = kTileTokens * DV * 2;
    static constexpr int kOffA = 0;                       // 2 monomial tiles
    static constexpr int kOffB3 = 2 * kABytes;
    static constexpr int kOffO = kOffB3 + MT<F>::kBlocks * kB3Block;   // 2 staging tiles
    static constexpr int kOffBars = kOffO + 2 * kOBytes;
    static constexpr int kSmemUsed = 1024 + kOffBars + 256;
    static constexpr int kSmem = kSmemUsed > 120 * 1024 ? kSmemUsed : 120 * 1024;   // one CTA per SM (it owns all of TMEM)
};

template <int DV, int F>
__global__ void __launch_bounds__(kRoThreads, 1) tc_readout_kernel(const __grid_constant__ CUtensorMap mapB3, const __grid_constant__ CUtensorMap mapO,
                                                                   const float* __restrict__ qf, float* __restrict__ eta_out, int N, int BH,
                                                                   float eps, int* status) {
    using Cfg = RoCfg<DV, F>;
    using M = MT<F>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::kOffBars);
    uint64_t* a_full = bars;          // [2] 128 generator arrivals
    uint64_t* a_empty = bars + 2;     // [2] MMA commit
    uint64_t* acc_full = bars + 4;    // [2] MMA commit
    uint64_t* acc_empty = bars + 6;   // [2] 256 epilogue arrivals
    uint64_t* b3_full = bars + 8;
    uint64_t* b3_free = bars + 9;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 10);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 11);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tiles_per_head = (N + kTileTokens - 1) / kTileTokens;
    const long long total = (long long)BH * tiles_per_head;
    const int w0 = (int)(total * blockIdx.x / gridDim.x), w1 = (int)(total * (blockIdx.x + 1) / gridDim.x);
    const int nwork = w1 - w0;
    grid_launch_dependents();

    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(&a_full[i], 128);
            mbar_init(&a_empty[i], 1);
            mbar_init(&acc_full[i], 1);
            mbar_init(&acc_empty[i], 256);
        }
        mbar_init(b3_full, 1);
        mbar_init(b3_free, 1);
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tmap(&mapB3);
        prefetch_tmap(&mapO);
    }
    if (warp == kRoMmaWarp) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    grid_dependency_wait();
    bool ok = true;

    if (warp == kRoMmaWarp) {
        if (lane == 0) {
            const uint32_t idesc = idesc_bf16(128, Cfg::kNmma, false, false);
            const uint32_t b3a = smem_u32(smem + Cfg::kOffB3);
            int cur_bh = -1, nload = 0;
            for (int it = 0; it < nwork; ++it) {
                const int work = w0 + it, bh = work / tiles_per_head;
                const int ab = it & 1, u = it >> 1;
                if (bh != cur_bh) {
                    if (cur_bh >= 0) {   // every MMA that reads the old state operand must have finished
                        umma_commit(b3_free);
                        if (!mbar_wait(b3_free, (nload - 1) & 1)) { report_timeout(status, 201); break; }
                    }
                    mbar_arrive_expect_tx(b3_full, Cfg::kB3Bytes);
                    for (int b = 0; b < M::kBlocks; ++b) tma_load_2d(smem + Cfg::kOffB3 + b * Cfg::kB3Block, &mapB3, b3_full, b * 64, bh * Cfg::kNmma);
                    if (!mbar_wait(b3_full, nload & 1)) { report_timeout(status, 202); break; }
                    ++nload;
                    cur_bh = bh;
                }
                if (!(mbar_wait(&a_full[ab], u & 1) && mbar_wait(&acc_empty[ab], (u & 1) ^ 1))) { report_timeout(status, 203); break; }
                tc_fence_after();
                const uint32_t aa = smem_u32(smem + Cfg::kOffA + ab * Cfg::kABytes);
#pragma unroll
                for (int ks = 0; ks < M::kPad / 16; ++ks)
                    umma_bf16(tmem + ab * 256, smem_desc_sw128(aa + (ks >> 2) * kBlk + (ks & 3) * 32, 16, 1024),
                              smem_desc_sw128(b3a + (ks >> 2) * Cfg::kB3Block + (ks & 3) * 32, 16, 1024), idesc, ks > 0 ? 1u : 0u);
                umma_commit(&a_empty[ab]);
                umma_commit(&acc_full[ab]);
            }
        }
    } else if (warp >= kRoGenWarp0) {
        const int row = tid - kRoGenWarp0 * 32;
        float qn[M::kDphi];      // query features of the next tile, loaded one tile ahead (row index clamped)
        auto prefetch = [&](int it) {
            const int work = w0 + it, bh = work / tiles_per_head, tok = min((work % tiles_per_head) * kTileTokens + row, N - 1);
            load_feat<M::kDphi>(qn, qf + ((size_t)bh * N + tok) * M::kDphi);
        };
        if (nwork > 0) prefetch(0);
        for (int it = 0; it < nwork; ++it) {
            const int work = w0 + it, tok = (work % tiles_per_head) * kTileTokens + row;
            const int ab = it & 1, u = it >> 1;
            float q[M::kDphi];
#pragma unroll
            for (int i = 0; i < M::kDphi; ++i) q[i] = tok < N ? qn[i] : 0.f;
            if (it + 1 < nwork) prefetch(it + 1);
            float mono[M::kN];
            query_monomials_t<F>(q, mono);
            if (ok && !mbar_wait(&a_empty[ab], (u & 1) ^ 1)) { ok = false; report_timeout(status, 204); }
            if (!ok) continue;
            store_mono_row_t<F>(smem_u32(smem + Cfg::kOffA + ab * Cfg::kABytes), row, mono, 1.f);
            fence_proxy_async();
            mbar_arrive(&a_full[ab]);
        }
    } else {
        const int row = tid & 127, half = tid >> 7;   // TMEM lane = token row of the tile; columns half * DV/2 ...
        constexpr int HC = DV / 2;
        for (int it = 0; it < nwork; ++it) {
            const int work = w0 + it, bh = work / tiles_per_head, tile = work % tiles_per_head;
            const int ab = it & 1, u = it >> 1;
            if (!mbar_wait(&acc_full[ab], u & 1)) {
                report_timeout(status, 205);
                *abort_flag = 1;
            }
            if (tid == 0) tma_store_wait_read1();      // the staging tile of two tiles ago has been read by its store
            named_barrier(3, 256);                     // every epilogue thread arrives, timed out or not
            if (*abort_flag) break;                    // uniform across the eight warps
            tc_fence_after();
            const uint32_t ta = tmem + ab * 256 + ((uint32_t)((warp & 3) * 32) << 16);
            // the whole accumulator row (numerator and normaliser) in one batch of TMEM loads, then the buffer is released
            uint32_t re[8], r[HC];
            tmem_ld8(ta + DV, re);
#pragma unroll
            for (int c = 0; c < HC / 16; ++c) tmem_ld16(ta + half * HC + 16 * c, *reinterpret_cast<uint32_t(*)[16]>(r + 16 * c));
            tmem_ld_wait();
            tc_fence_before();
            mbar_arrive(&acc_empty[ab]);
            const float eta = __uint_as_float(re[0]);
            const float rinv = 1.f / (eta + eps);
            const uint32_t os = smem_u32(smem + Cfg::kOffO + ab * Cfg::kOBytes);
#pragma unroll
            for (int c = 0; c < HC / 16; ++c) {
                uint32_t w[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) w[e] = pack_bf16(__uint_as_float(r[16 * c + 2 * e]) * rinv, __uint_as_float(r[16 * c + 2 * e + 1]) * rinv);
                const int cc = half * (HC / 16) + c;      // 16-column chunk of the row
                const uint32_t blk = os + (cc >> 2) * kBlk;
                st_shared_v4(blk + sw128_off(row, (2 * cc) & 7), w[0], w[1], w[2], w[3]);
                st_shared_v4(blk + sw128_off(row, (2 * cc + 1) & 7), w[4], w[5], w[6], w[7]);
            }
            fence_proxy_async();
            named_barrier(2, 256);
            if (tid == 0) {
                for (int b = 0; b < DV / 64; ++b) tma_store_3d(&mapO, smem + Cfg::kOffO + ab * Cfg::kOBytes + b * kBlk, b * 64, tile * kTileTokens, bh);
                tma_store_commit();
            }
            const int tok = tile * kTileTokens + row;
            if (half == 0 && tok < N) eta_out[(size_t)bh * N + tok] = eta;
        }
        if (tid == 0) tma_store_wait_all0();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kRoMmaWarp) tmem_dealloc(tmem, 512);
}

// =======================================================================================
// Backward, pass over the queries (split over tokens like the state build):
//   D2[i][m]  = sum_g dO_i[g] Csym[m][g]                                   (MMA, K = d)
//   s_i       = sum_m mono_i[m] D2[i][m] ;  delta_i = dO_i . o_i = r_i s_i ;  deta_i = -r_i delta_i
//   dmono_i[m]= r_i D2[i][m] + deta_i zsym[m]  ->  dq_i                     (ALUs)
//   [dCsym | dzsym][m][:] += (r_i mono_i[m]) * [dO_i | deta_i / r_i]         (MMA, K = tokens)
// O itself is not read: dO . o is recovered from D2.
//
// The second product has the monomials on the M side (64 rows) and d + 8 columns: the operand row that a generator
// thread writes for its token is [deta/r, 0 x 7, r mono_0..55], so the same 128-byte row serves as row of the A operand
// (rows 8..63 = monomials) and, read as the block that follows the dO blocks, as columns d..d+7 of the B operand
// (column d = deta/r, the rest zero).  Accumulator row 8+m then holds dCsym[m][0..d-1], dzsym[m], 0, 0, 0: one row of
// the partial state, and dz costs no product of its own.  Rows 0..7 of the accumulator are not used.
//
// The tensor pipe needs ~100 cycles per MMA of this size (set by the operand bytes it reads from shared memory, not by
// the arithmetic), so the MMAs per tile are kept at 16 and are issued by two threads (D2: warp 1, dC: warp 2).
// =======================================================================================
constexpr int kBqGroups = 3;                            // generator groups of 128 threads; tile `it` belongs to group it % 3
constexpr int kBqThreads = 128 + 128 * kBqGroups;       // warp 0: TMA, warp 1: D2 MMAs, warp 2: dC MMAs, warp 3 idle, warps 4..: generators
constexpr int kBqRowPad = 8;                            // accumulator row of monomial 0
// F = 2: the operand row is [deta/r, 0 x 7, r mono_0..77, 0 x 42] = 128 columns in two blocks, the dC product has M = 128
// (accumulator lane = row) and three stages fit; F = 3: 64 columns, M = 64 (row R in lane 32 (R / 16) + R % 16), four stages.
template <int F> struct BqCfg {
    static constexpr int kStages = F == 3 ? 4 : 3;
    static constexpr int kStageBytes = (2 + MT<F>::kBlocks) * kBlk;      // dO tile (d/64 blocks of 64 columns) directly followed by the operand-row tile
    static constexpr int kOpBlock = MT<F>::kPad * 128;                   // Csym operand [kPad][d] bf16: one block per 64 value channels
    static constexpr int kOffOp = kStages * kStageBytes;
    static constexpr int kOffZ = kOffOp + ((2 * kOpBlock + 1023) / 1024) * 1024;      // zsym (kPad floats)
    static constexpr int kOffBars = kOffZ + MT<F>::kPad * 4;
    static constexpr int kSmem = 1024 + kOffBars + 256;
    static constexpr int kColD2 = F == 3 ? 256 : 160;                    // TMEM columns of the D2 buffers (one per group)
    static constexpr int kD2Stride = F == 3 ? 64 : 96;
    static constexpr int kM = F == 3 ? 64 : 128;                         // rows of the dC product
    static_assert((4 * kStages + 2 * kBqGroups + 3) * 8 <= 256, "barrier block");
};

template <int DV, int F>
__global__ void __launch_bounds__(kBqThreads, 1) tc_bwd_query_kernel(const __grid_constant__ CUtensorMap mapdO, const __grid_constant__ CUtensorMap mapBq,
                                                                     const float* __restrict__ qf, const float* __restrict__ eta,
                                                                     const float* __restrict__ state, float* __restrict__ dqf,
                                                                     float* __restrict__ part, int N, int S, int ld, float eps, int* status) {
    using M = MT<F>;
    using Cfg = BqCfg<F>;
    constexpr int kStages = Cfg::kStages, kStageBytes = Cfg::kStageBytes;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    float* zsym = reinterpret_cast<float*>(smem + Cfg::kOffZ);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::kOffBars);
    uint64_t* full_do = bars;                     // [stages] TMA
    uint64_t* full_rm = bars + kStages;           // [stages] 128 arrivals: the operand rows of the tile are complete
    uint64_t* empty_rm = bars + 2 * kStages;      // [stages] MMA commit (dC): the operand-row tile is free
    uint64_t* empty_do = bars + 3 * kStages;      // [stages] MMA commits (D2 and dC): the dO tile is free
    uint64_t* d2_full = bars + 4 * kStages;       // [groups] MMA commit
    uint64_t* d2_empty = d2_full + kBqGroups;     // [groups] 128 arrivals
    uint64_t* op_full = d2_empty + kBqGroups;
    uint64_t* acc_done = op_full + 1;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_done + 1);
    constexpr int kRmOff = (DV / 64) * kBlk;        // operand-row tile inside a stage
    constexpr int kNC = DV + 8;                     // columns of the dC product

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int s = blockIdx.x, bh = blockIdx.y;
    const int tiles = (N + kTileTokens - 1) / kTileTokens;
    const int tiles_per = (tiles + S - 1) / S;
    const int tile0 = s * tiles_per;
    const int ntiles = max(0, min(tiles, tile0 + tiles_per) - tile0);
    float* out = part + ((size_t)bh * S + s) * M::kN * ld;
    grid_launch_dependents();
    if (ntiles == 0) {
        grid_dependency_wait();
        for (int i = tid; i < M::kN * ld; i += kBqThreads) out[i] = 0.f;
        return;
    }
    if (F == 2) {      // operand-row columns 86..127 are read by the M = 128 product and never written: keep them zero
        for (int st = 0; st < kStages; ++st) {
            uint4* z = reinterpret_cast<uint4*>(smem + st * kStageBytes + kRmOff + kBlk);
            for (int i = tid; i < kBlk / 16; i += kBqThreads) z[i] = make_uint4(0, 0, 0, 0);
        }
        fence_proxy_async();
    }
    if (tid == 0) {
        for (int i = 0; i < kStages; ++i) {
            mbar_init(&full_do[i], 1);
            mbar_init(&full_rm[i], 128);
            mbar_init(&empty_rm[i], 1);
            mbar_init(&empty_do[i], 2);
        }
        for (int i = 0; i < kBqGroups; ++i) {
            mbar_init(&d2_full[i], 1);
            mbar_init(&d2_empty[i], 128);
        }
        mbar_init(op_full, 1);
        mbar_init(acc_done, 1);
        fence_mbar_init();
        prefetch_tmap(&mapdO);
        prefetch_tmap(&mapBq);
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
    // (zsym is read by the generator warps only; the named barrier keeps the other warps out of it)
    if (warp >= 4) {
        if (tid - 128 < M::kPad) zsym[tid - 128] = tid - 128 < M::kN ? state[((size_t)bh * M::kN + tid - 128) * ld + DV] : 0.f;
        named_barrier(1, 128 * kBqGroups);
    }
    bool ok = true;

    if (warp == 0) {
        if (elect_one()) {
            mbar_arrive_expect_tx(op_full, M::kPad * DV * 2);
            for (int b = 0; b < DV / 64; ++b) tma_load_2d(smem + Cfg::kOffOp + b * Cfg::kOpBlock, &mapBq, op_full, b * 64, bh * M::kPad);
            for (int it = 0; it < ntiles; ++it) {
                const int st = it % kStages, u = it / kStages;
                if (!mbar_wait(&empty_do[st], (u & 1) ^ 1)) { report_timeout(status, 301); break; }
                uint8_t* ds = smem + st * kStageBytes;
                mbar_arrive_expect_tx(&full_do[st], DV * kTileTokens * 2);
                for (int b = 0; b < DV / 64; ++b) tma_load_3d(ds + b * kBlk, &mapdO, &full_do[st], b * 64, (tile0 + it) * kTileTokens, bh);
            }
        }
    } else if (warp == 1) {
        if (elect_one()) {
            // D2 = dO (K-major over g) * Csym (K-major over g); tile `it` is issued as soon as its dO tile has landed
            // and the group that owns the tile has read its previous D2, which is long before the group asks for it.
            const uint32_t idesc2 = idesc_bf16(128, M::kPad, false, false);
            const uint32_t opa = smem_u32(smem + Cfg::kOffOp);
            if (!mbar_wait(op_full, 0)) report_timeout(status, 302);
            else
                for (int it = 0; it < ntiles; ++it) {
                    const int st = it % kStages, u = it / kStages, buf = it % kBqGroups, ub = it / kBqGroups;
                    if (!(mbar_wait(&full_do[st], u & 1) && mbar_wait(&d2_empty[buf], (ub & 1) ^ 1))) { report_timeout(status, 303); break; }
                    tc_fence_after();
                    const uint32_t da = smem_u32(smem + st * kStageBytes);
#pragma unroll
                    for (int ks = 0; ks < DV / 16; ++ks)
                        umma_bf16(tmem + Cfg::kColD2 + Cfg::kD2Stride * buf, smem_desc_sw128(da + (ks >> 2) * kBlk + (ks & 3) * 32, 16, 1024),
                                  smem_desc_sw128(opa + (ks >> 2) * Cfg::kOpBlock + (ks & 3) * 32, 16, 1024), idesc2, ks > 0 ? 1u : 0u);
                    umma_commit(&d2_full[buf]);
                    umma_commit(&empty_do[st]);
                }
        }
    } else if (warp == 2) {
        if (elect_one()) {
            // [dCsym | dzsym] += (operand rows)^T (MN-major, M rows) * [dO | operand rows' first 8 columns] (MN-major, N = d + 8)
            const uint32_t idesc1 = idesc_bf16(Cfg::kM, kNC, true, true);
            for (int it = 0; it < ntiles; ++it) {
                const int st = it % kStages, u = it / kStages;
                if (!(mbar_wait(&full_do[st], u & 1) && mbar_wait(&full_rm[st], u & 1))) { report_timeout(status, 304); break; }
                tc_fence_after();
                const uint32_t da = smem_u32(smem + st * kStageBytes), ra = da + kRmOff;
#pragma unroll
                for (int ks = 0; ks < kTileTokens / 16; ++ks)
                    umma_bf16(tmem, smem_desc_sw128(ra + ks * 2048, kBlk, 1024), smem_desc_sw128(da + ks * 2048, kBlk, 1024), idesc1,
                              (it > 0 || ks > 0) ? 1u : 0u);
                umma_commit(&empty_do[st]);
                umma_commit(&empty_rm[st]);
            }
            umma_commit(acc_done);
        }
    } else if (warp >= 4) {
        const int grp = (warp - 4) >> 2, quarter = warp & 3;
        const int row = quarter * 32 + lane;    // token row of the tile == TMEM lane this thread can read
        // The features and the normaliser of the group's next tile are loaded while the current one is processed
        // (row index clamped: the loads are unconditional, out-of-range rows are zeroed when used).
        float qn[M::kDphi], etan;
        auto prefetch = [&](int it) {
            const int tok = min((tile0 + it) * kTileTokens + row, N - 1);
            load_feat<M::kDphi>(qn, qf + ((size_t)bh * N + tok) * M::kDphi);
            etan = __ldg(eta + (size_t)bh * N + tok);
        };
        if (grp < ntiles) prefetch(grp);
        for (int it = grp; it < ntiles; it += kBqGroups) {
            const int st = it % kStages, u = it / kStages, buf = grp, ub = it / kBqGroups;
            const int tok = (tile0 + it) * kTileTokens + row;
            const uint32_t rblk = smem_u32(smem + st * kStageBytes + kRmOff);
            float q[M::kDphi], r = 0.f;
#pragma unroll
            for (int i = 0; i < M::kDphi; ++i) q[i] = tok < N ? qn[i] : 0.f;
            if (tok < N) r = 1.f / (etan + eps);
            {   // columns 8.. of the operand row: r_i * mono_i, formed from the scaled features so that no monomial stays live
                // across the wait below
                float qs[M::kDphi], rmono[M::kN];
#pragma unroll
                for (int i = 0; i < M::kDphi; ++i) qs[i] = r * q[i];
                if constexpr (F == 3) {
#pragma unroll
                    for (int a = 0; a < 6; ++a)
#pragma unroll
                        for (int b = a; b < 6; ++b) {
                            const float qab = qs[a] * q[b];
#pragma unroll
                            for (int c = b; c < 6; ++c) rmono[mono_idx(a, b, c)] = qab * q[c];
                        }
                } else {
#pragma unroll
                    for (int a = 0; a < 12; ++a)
#pragma unroll
                        for (int b = a; b < 12; ++b) rmono[mono_idx2(a, b)] = qs[a] * q[b];
                }
                if (ok && !mbar_wait(&empty_rm[st], (u & 1) ^ 1)) { ok = false; report_timeout(status, 305); }
                if (ok) {
#pragma unroll
                    for (int c = 1; c < (kBqRowPad + M::kN + 7) / 8; ++c) {      // 16-byte chunk c holds the monomials 8 c - 8 .. 8 c - 1
                        float v[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) v[e] = 8 * c - 8 + e < M::kN ? rmono[8 * c - 8 + e < M::kN ? 8 * c - 8 + e : 0] : 0.f;
                        st_shared_v4(rblk + (c >> 3) * kBlk + sw128_off(row, c & 7), pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]),
                                     pack_bf16(v[6], v[7]));
                    }
                }
            }
            if (ok && !mbar_wait(&d2_full[buf], ub & 1)) { ok = false; report_timeout(status, 306); }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) continue;
            tc_fence_after();
            constexpr int kD2Chunks = (M::kN + 7) / 8;
            uint32_t d2[8 * kD2Chunks];
            const uint32_t ta = tmem + Cfg::kColD2 + Cfg::kD2Stride * buf + ((uint32_t)(quarter * 32) << 16);
#pragma unroll
            for (int c = 0; c < kD2Chunks; ++c) tmem_ld8(ta + 8 * c, *reinterpret_cast<uint32_t(*)[8]>(d2 + 8 * c));
            tmem_ld_wait();
            tc_fence_before();
            mbar_arrive(&d2_empty[buf]);
            float dq[M::kDphi];
            float sdot, deta;
            if constexpr (F == 3) {
                // The monomials are recomputed where they are used (two multiplies each) instead of being kept in 56 registers.
                float qq[6][6];
#pragma unroll
                for (int a = 0; a < 6; ++a)
#pragma unroll
                    for (int b = a; b < 6; ++b) qq[a][b] = q[a] * q[b];
                float sd[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int a = 0; a < 6; ++a)
#pragma unroll
                    for (int b = a; b < 6; ++b)
#pragma unroll
                        for (int c = b; c < 6; ++c) {
                            const int m = mono_idx(a, b, c);
                            sd[m & 3] = fmaf(qq[a][b] * q[c], __uint_as_float(d2[m]), sd[m & 3]);
                        }
                sdot = (sd[0] + sd[1]) + (sd[2] + sd[3]);
                deta = -r * r * sdot;
                // columns 0..7 of the operand row: deta / r, then zeros; one proxy fence covers the whole row
                st_shared_v4(rblk + sw128_off(row, 0), pack_bf16(-r * sdot, 0.f), 0u, 0u, 0u);
                fence_proxy_async();
                mbar_arrive(&full_rm[st]);
                if (it + kBqGroups < ntiles) prefetch(it + kBqGroups);
#pragma unroll
                for (int a = 0; a < 6; ++a) dq[a] = 0.f;
#pragma unroll
                for (int a = 0; a < 6; ++a)
#pragma unroll
                    for (int b = a; b < 6; ++b)
#pragma unroll
                        for (int c = b; c < 6; ++c) {
                            const int m = mono_idx(a, b, c);
                            const float g = fmaf(r, __uint_as_float(d2[m]), deta * zsym[m]);      // dmono_i[m]
                            dq[a] = fmaf(g, qq[b][c], dq[a]);
                            dq[b] = fmaf(g, qq[a][c], dq[b]);
                            dq[c] = fmaf(g, qq[a][b], dq[c]);
                        }
            } else {
                float sd[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int a = 0; a < 12; ++a)
#pragma unroll
                    for (int b = a; b < 12; ++b) {
                        const int m = mono_idx2(a, b);
                        sd[m & 3] = fmaf(q[a] * q[b], __uint_as_float(d2[m]), sd[m & 3]);
                    }
                sdot = (sd[0] + sd[1]) + (sd[2] + sd[3]);
                deta = -r * r * sdot;
                st_shared_v4(rblk + sw128_off(row, 0), pack_bf16(-r * sdot, 0.f), 0u, 0u, 0u);
                fence_proxy_async();
                mbar_arrive(&full_rm[st]);
                if (it + kBqGroups < ntiles) prefetch(it + kBqGroups);
#pragma unroll
                for (int a = 0; a < 12; ++a) dq[a] = 0.f;
#pragma unroll
                for (int a = 0; a < 12; ++a)
#pragma unroll
                    for (int b = a; b < 12; ++b) {
                        const int m = mono_idx2(a, b);
                        const float g = fmaf(r, __uint_as_float(d2[m]), deta * zsym[m]);          // dmono_i[m]
                        dq[a] = fmaf(g, q[b], dq[a]);
                        dq[b] = fmaf(g, q[a], dq[b]);
                    }
            }
            if (tok < N) store_feat<M::kDphi>(dqf + ((size_t)bh * N + tok) * M::kDphi, dq);
        }
        if (grp == 0) {
            if (ok && !mbar_wait(acc_done, 0)) { ok = false; report_timeout(status, 307); }
            ok = __all_sync(0xffffffffu, ok);
            tc_fence_after();
            // F = 3: a 64-row accumulator keeps row R in TMEM lane 32 * (R / 16) + R % 16 (lanes 0..15 of each warp's quarter);
            // F = 2: a 128-row accumulator keeps row R in lane R
            const int m = (F == 3 ? quarter * 16 + lane : quarter * 32 + lane) - kBqRowPad;
            const bool mine = (F == 3 ? lane < 16 : true) && m >= 0 && m < M::kN;
            if (ok) {
#pragma unroll 1
                for (int c = 0; c < kNC / 8; ++c) {
                    uint32_t rr[8];
                    tmem_ld8(tmem + ((uint32_t)(quarter * 32) << 16) + 8 * c, rr);
                    tmem_ld_wait();
                    if (mine) {
                        float4* dst = reinterpret_cast<float4*>(out + (size_t)m * ld + 8 * c);
                        dst[0] = make_float4(__uint_as_float(rr[0]), __uint_as_float(rr[1]), __uint_as_float(rr[2]), __uint_as_float(rr[3]));
                        if (8 * c + 4 < ld) dst[1] = make_float4(__uint_as_float(rr[4]), __uint_as_float(rr[5]), __uint_as_float(rr[6]), __uint_as_float(rr[7]));
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, 512);
}

// =======================================================================================
// Backward, pass over the keys (persistent over (head, tile) like the readout):
//   dV_j      = sum_m Tsym_k[j][m] dCsym[m][:]                               (MMA, K = 64)
//   G_j[m]    = sum_g v_j[g] dCsym[m][g] + dzsym[m]                          (MMA, K = d; + on the ALUs)
//   dk1, dk2, dk3 from G_j and the key features                              (ALUs)
// =======================================================================================
constexpr int kBkThreads = 320;   // warp 0: TMA loads, warp 1: MMA, warps 2..9: two worker groups of 128 threads
template <int DV, int F> struct BkCfg {
    static constexpr int kVBytes = 2 * kBlk;                              // V stage (two 64-column blocks; d = 64 uses one)
    static constexpr int kABytes = MT<F>::kBlocks * kBlk;                 // one folded key tile
    static constexpr int kOffV = 0;                                       // 2 stages
    static constexpr int kOffA = 2 * kVBytes;                             // 2 folded key tiles (one per group)
    static constexpr int kOffB3 = kOffA + 2 * kABytes;                    // dCsym operand [d+16][kPad], one block per 64 monomials
    static constexpr int kB3Block = (((DV + 16) * 128 + 1023) / 1024) * 1024;
    static constexpr int kB3Bytes = MT<F>::kBlocks * (DV + 16) * 128;
    static constexpr int kBqBlock = MT<F>::kPad * 128;                    // dCsym operand [kPad][d], one block per 64 value channels
    static constexpr int kOffBq = kOffB3 + MT<F>::kBlocks * kB3Block;
    // dV staging tiles (one per group) for a TMA store; with the wider tiles of F = 2 they do not fit and dV leaves
    // straight from registers (32-byte stores)
    static constexpr bool kStagedOut = F == 3;
    static constexpr int kOffO = kOffBq + ((2 * kBqBlock + 1023) / 1024) * 1024;
    static constexpr int kOBytes = kTileTokens * DV * 2;
    static constexpr int kOffBars = kOffO + (kStagedOut ? 2 * kOBytes : 0);
    static constexpr int kOffDz = kOffBars + 256;                         // float [2 groups][128]: dzsym of the group's current head
    static constexpr int kSmemUsed = 1024 + kOffDz + 1024;
    static_assert(kSmemUsed <= 227 * 1024, "shared memory");
    static constexpr int kSmem = kSmemUsed > 120 * 1024 ? kSmemUsed : 120 * 1024;
    static constexpr int kColD4 = 256, kD4Stride = F == 3 ? 64 : 96;      // TMEM: D3[grp] at 128 grp, D4[grp] at 256 + stride grp
};

template <int DV, int F>
__global__ void __launch_bounds__(kBkThreads, 1) tc_bwd_key_kernel(const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapB3,
                                                                   const __grid_constant__ CUtensorMap mapBq, const __grid_constant__ CUtensorMap mapdV,
                                                                   const float* __restrict__ kf, const float* __restrict__ dstate,
                                                                   float* __restrict__ dkf, __nv_bfloat16* __restrict__ dV, int N, int BH, int ld, int* status) {
    using Cfg = BkCfg<DV, F>;
    using M = MT<F>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::kOffBars);
    uint64_t* full_v = bars;            // [2]
    uint64_t* empty_v = bars + 2;       // [2] MMA commit
    uint64_t* a_full = bars + 4;        // [2] 128 arrivals (per group)
    uint64_t* d4_full = bars + 6;       // [2] MMA commit
    uint64_t* d3_full = bars + 8;       // [2] MMA commit
    uint64_t* acc_empty = bars + 10;    // [2] 128 arrivals
    uint64_t* op_full = bars + 12;
    uint64_t* op_free = bars + 13;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 14);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tiles_per_head = (N + kTileTokens - 1) / kTileTokens;
    const long long total = (long long)BH * tiles_per_head;
    const int w0 = (int)(total * blockIdx.x / gridDim.x), w1 = (int)(total * (blockIdx.x + 1) / gridDim.x);
    const int nwork = w1 - w0;
    grid_launch_dependents();

    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(&full_v[i], 1);
            mbar_init(&empty_v[i], 1);
            mbar_init(&a_full[i], 128);
            mbar_init(&d4_full[i], 1);
            mbar_init(&d3_full[i], 1);
            mbar_init(&acc_empty[i], 128);
        }
        mbar_init(op_full, 1);
        mbar_init(op_free, 1);
        fence_mbar_init();
        prefetch_tmap(&mapV);
        prefetch_tmap(&mapB3);
        prefetch_tmap(&mapBq);
        prefetch_tmap(&mapdV);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;     // D3[grp] at columns 128*grp, D4[grp] at columns 256 + kD4Stride*grp
    grid_dependency_wait();
    bool ok = true;

    if (warp == 0) {
        if (lane == 0) {
            for (int it = 0; it < nwork; ++it) {
                const int work = w0 + it, bh = work / tiles_per_head, tile = work % tiles_per_head;
                const int st = it & 1, u = it >> 1;
                if (!mbar_wait(&empty_v[st], (u & 1) ^ 1)) { report_timeout(status, 401); break; }
                uint8_t* vs = smem + Cfg::kOffV + st * Cfg::kVBytes;
                mbar_arrive_expect_tx(&full_v[st], DV * kTileTokens * 2);
                for (int b = 0; b < DV / 64; ++b) tma_load_3d(vs + b * kBlk, &mapV, &full_v[st], b * 64, tile * kTileTokens, bh);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc4 = idesc_bf16(128, M::kPad, false, false);    // G  = V (K-major over g) * dCsym (K-major over g)
            const uint32_t idesc3 = idesc_bf16(128, DV, false, false);         // dV = Tsym_k (K-major over m) * dCsym^T (K-major over m)
            const uint32_t b3a = smem_u32(smem + Cfg::kOffB3), bqa = smem_u32(smem + Cfg::kOffBq);
            int cur_bh = -1, nload = 0;
            for (int it = 0; it < nwork; ++it) {
                const int work = w0 + it, bh = work / tiles_per_head;
                const int st = it & 1, u = it >> 1, grp = it & 1;
                if (bh != cur_bh) {
                    if (cur_bh >= 0) {
                        umma_commit(op_free);
                        if (!mbar_wait(op_free, (nload - 1) & 1)) { report_timeout(status, 402); break; }
                    }
                    mbar_arrive_expect_tx(op_full, Cfg::kB3Bytes + M::kPad * DV * 2);
                    for (int b = 0; b < M::kBlocks; ++b) tma_load_2d(smem + Cfg::kOffB3 + b * Cfg::kB3Block, &mapB3, op_full, b * 64, bh * (DV + 16));
                    for (int b = 0; b < DV / 64; ++b) tma_load_2d(smem + Cfg::kOffBq + b * Cfg::kBqBlock, &mapBq, op_full, b * 64, bh * M::kPad);
                    if (!mbar_wait(op_full, nload & 1)) { report_timeout(status, 403); break; }
                    ++nload;
                    cur_bh = bh;
                }
                if (!(mbar_wait(&full_v[st], u & 1) && mbar_wait(&acc_empty[grp], (u & 1) ^ 1))) { report_timeout(status, 404); break; }
                tc_fence_after();
                const uint32_t va = smem_u32(smem + Cfg::kOffV + st * Cfg::kVBytes);
#pragma unroll
                for (int ks = 0; ks < DV / 16; ++ks)
                    umma_bf16(tmem + Cfg::kColD4 + Cfg::kD4Stride * grp, smem_desc_sw128(va + (ks >> 2) * kBlk + (ks & 3) * 32, 16, 1024),
                              smem_desc_sw128(bqa + (ks >> 2) * Cfg::kBqBlock + (ks & 3) * 32, 16, 1024), idesc4, ks > 0 ? 1u : 0u);
                umma_commit(&d4_full[grp]);
                umma_commit(&empty_v[st]);
                if (!mbar_wait(&a_full[grp], u & 1)) { report_timeout(status, 405); break; }
                tc_fence_after();
                const uint32_t aa = smem_u32(smem + Cfg::kOffA + grp * Cfg::kABytes);
#pragma unroll
                for (int ks = 0; ks < M::kPad / 16; ++ks)
                    umma_bf16(tmem + 128 * grp, smem_desc_sw128(aa + (ks >> 2) * kBlk + (ks & 3) * 32, 16, 1024),
                              smem_desc_sw128(b3a + (ks >> 2) * Cfg::kB3Block + (ks & 3) * 32, 16, 1024), idesc3, ks > 0 ? 1u : 0u);
                umma_commit(&d3_full[grp]);
            }
        }
    } else {
        const int grp = (warp - 2) >> 2, quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const bool leader = (warp - 2) == 4 * grp && lane == 0;
        float kn[M::kKf];     // key features of the group's next tile, loaded one tile ahead (row index clamped)
        auto prefetch = [&](int it) {
            const int work = w0 + it, bh = work / tiles_per_head, tok = min((work % tiles_per_head) * kTileTokens + row, N - 1);
#pragma unroll
            for (int f = 0; f < F; ++f) load_feat<M::kDphi>(kn + M::kDphi * f, kf + (((size_t)bh * F + f) * N + tok) * M::kDphi);
        };
        if (grp < nwork) prefetch(grp);
        float* dzs = reinterpret_cast<float*>(smem + Cfg::kOffDz) + grp * 128;
        int cur_bh = -1;
        for (int it = grp; it < nwork; it += 2) {
            const int work = w0 + it, bh = work / tiles_per_head, tile = work % tiles_per_head;
            const int u = it >> 1;
            const int tok = tile * kTileTokens + row;
            if (bh != cur_bh) {      // dzsym of the head, once per head and group instead of 56 global loads per thread and tile
                named_barrier(1 + grp, 128);
                if (row < M::kN) dzs[row] = __ldg(dstate + (size_t)bh * M::kN * ld + DV + (size_t)row * ld);
                named_barrier(1 + grp, 128);
                cur_bh = bh;
            }
            float k[M::kKf];
#pragma unroll
            for (int i = 0; i < M::kKf; ++i) k[i] = tok < N ? kn[i] : 0.f;
            if (it + 2 < nwork) prefetch(it + 2);
            {
                float ts[M::kN];
                key_folded_t<F>(k, ts);
                // the folded key tile of this group is free: its last reader (the dV MMA two tiles ago) was waited for below
                store_mono_row_t<F>(smem_u32(smem + Cfg::kOffA + grp * Cfg::kABytes), row, ts, 1.f);
                fence_proxy_async();
                mbar_arrive(&a_full[grp]);
            }
            // ---- G -> dk
            if (ok && !mbar_wait(&d4_full[grp], u & 1)) { ok = false; report_timeout(status, 406); }
            ok = __all_sync(0xffffffffu, ok);
            if (ok) {
                tc_fence_after();
                float G[M::kN];
                const uint32_t ta = tmem + Cfg::kColD4 + Cfg::kD4Stride * grp + ((uint32_t)(quarter * 32) << 16);
#pragma unroll
                for (int c = 0; c < (M::kN + 7) / 8; ++c) {
                    uint32_t rr[8];
                    tmem_ld8(ta + 8 * c, rr);
                    tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        if (8 * c + e < M::kN) G[8 * c + e] = __uint_as_float(rr[e]) + dzs[8 * c + e];
                }
                float dk[M::kKf];
                key_folded_grad_t<F>(k, G, dk);
                if (tok < N) {
#pragma unroll
                    for (int f = 0; f < F; ++f) store_feat<M::kDphi>(dkf + (((size_t)bh * F + f) * N + tok) * M::kDphi, dk + M::kDphi * f);
                }
            }
            // ---- dV
            if (ok && !mbar_wait(&d3_full[grp], u & 1)) { ok = false; report_timeout(status, 407); }
            ok = __all_sync(0xffffffffu, ok);
            if constexpr (Cfg::kStagedOut) {
                if (leader) tma_store_wait_read0();          // this group's staging tile has been read by its previous store
                named_barrier(1 + grp, 128);
                if (ok) {
                    tc_fence_after();
                    const uint32_t ta = tmem + 128 * grp + ((uint32_t)(quarter * 32) << 16);
                    const uint32_t os = smem_u32(smem + Cfg::kOffO + grp * Cfg::kOBytes);
#pragma unroll
                    for (int h = 0; h < DV / 64; ++h) {      // 64 columns per batch of TMEM loads
                        uint32_t r[64];
#pragma unroll
                        for (int c = 0; c < 4; ++c) tmem_ld16(ta + 64 * h + 16 * c, *reinterpret_cast<uint32_t(*)[16]>(r + 16 * c));
                        tmem_ld_wait();
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            uint32_t w[8];
#pragma unroll
                            for (int e = 0; e < 8; ++e) w[e] = pack_bf16(__uint_as_float(r[16 * c + 2 * e]), __uint_as_float(r[16 * c + 2 * e + 1]));
                            const uint32_t blk = os + h * kBlk;
                            st_shared_v4(blk + sw128_off(row, 2 * c), w[0], w[1], w[2], w[3]);
                            st_shared_v4(blk + sw128_off(row, 2 * c + 1), w[4], w[5], w[6], w[7]);
                        }
                    }
                    tc_fence_before();
                    mbar_arrive(&acc_empty[grp]);
                    fence_proxy_async();
                }
                named_barrier(1 + grp, 128);
                if (ok && leader) {
                    for (int b = 0; b < DV / 64; ++b) tma_store_3d(&mapdV, smem + Cfg::kOffO + grp * Cfg::kOBytes + b * kBlk, b * 64, tile * kTileTokens, bh);
                    tma_store_commit();
                }
            } else {
                if (ok) {
                    tc_fence_after();
                    const uint32_t ta = tmem + 128 * grp + ((uint32_t)(quarter * 32) << 16);
                    __nv_bfloat16* dst = dV + ((size_t)bh * N + (tok < N ? tok : 0)) * DV;
#pragma unroll 2
                    for (int c = 0; c < DV / 16; ++c) {
                        uint32_t r[16], w[8];
                        tmem_ld16(ta + 16 * c, r);
                        tmem_ld_wait();
#pragma unroll
                        for (int e = 0; e < 8; ++e) w[e] = pack_bf16(__uint_as_float(r[2 * e]), __uint_as_float(r[2 * e + 1]));
                        if (tok < N) st_global_v8(dst + 16 * c, w);      // one full 32-byte sector per store
                    }
                    tc_fence_before();
                    mbar_arrive(&acc_empty[grp]);
                }
            }
        }
        if (Cfg::kStagedOut && leader) tma_store_wait_all0();
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, 512);
}

// Self-test of the bounded waits: one CTA waits on a barrier that nothing ever arrives at, with a limit of
// `limit_ns`; the wait must run out, record the time-out in the status words and let the kernel return normally.
__global__ void tc_wait_selftest_kernel(int* status, unsigned long long limit_ns) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        fence_mbar_init();
    }
    __syncthreads();
    if (threadIdx.x == 0 && !mbar_wait(&bar, 0, limit_ns)) report_timeout(status, 901);
}

// ---- host launch helpers ---------------------------------------------------------------
template <typename K>
inline bool set_smem(K kernel, int bytes) {
    const void* key = reinterpret_cast<const void*>(kernel);
    HostCache* hc = t_host_cache;
    if (hc)
        for (int i = 0; i < hc->nfuncs; ++i)
            if (hc->funcs[i] == key) return true;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
    if (hc && hc->nfuncs < HostCache::kFuncs) hc->funcs[hc->nfuncs++] = key;
    return true;
}

template <int DV, int F>
inline hla_status launch_core_forward(const Plan& P, const Dims& D, int BH, const float* qf, const float* kf, const void* V, void* O, char* ws,
                                      const hla_ws_layout& L, size_t off_part, int sm_count, LaunchRec& rec, bool readout) {
    constexpr int kPad = MT<F>::kPad;
    CUtensorMap mapV, mapO, mapB3;
    __nv_bfloat16* b3 = reinterpret_cast<__nv_bfloat16*>(ws + P.b3);
    __nv_bfloat16* bq = reinterpret_cast<__nv_bfloat16*>(ws + P.bq);
    if (!make_map_bhnd(&mapV, V, BH, D.N, DV, kTileTokens) || !make_map_bhnd(&mapO, O, BH, D.N, DV, kTileTokens) ||
        !make_map_2d(&mapB3, b3, (size_t)BH * (DV + 16), kPad, DV + 16))
        return HLA_ERR_CUDA;
    int* status = reinterpret_cast<int*>(ws + L.status);
    float* part = reinterpret_cast<float*>(ws + off_part);
    float* state = reinterpret_cast<float*>(ws + L.state);
    float* eta = reinterpret_cast<float*>(ws + L.eta);
    if (!set_smem(tc_state_build_kernel<DV, F>, SbCfg<F>::kSmem) || !set_smem(tc_readout_kernel<DV, F>, RoCfg<DV, F>::kSmem)) return HLA_ERR_CUDA;
    cudaStream_t st = rec.st;
    rec.begin("tc_state_build");
    launch_pdl(tc_state_build_kernel<DV, F>, dim3(D.S, BH), dim3(kSbThreads), SbCfg<F>::kSmem, st, mapV, kf, part, D.N, D.S, D.ld, status, (const float*)nullptr, (const float*)nullptr, 0.f);
    if (!rec.end()) return HLA_ERR_CUDA;
    rec.begin("tc_reduce_emit");
    launch_pdl(tc_reduce_emit_kernel<DV, F>, dim3(kPad / 8, BH), dim3(256), 0, st, part, state, b3, bq, D.S, D.ld, 0, 0);
    if (!rec.end()) return HLA_ERR_CUDA;
    if (!readout) return HLA_OK;
    const int tiles = (D.N + kTileTokens - 1) / kTileTokens;
    const long long total = (long long)BH * tiles;
    const int grid = (int)(total < sm_count ? total : sm_count);
    rec.begin("tc_readout");
    launch_pdl(tc_readout_kernel<DV, F>, grid, dim3(kRoThreads), RoCfg<DV, F>::kSmem, st, mapB3, mapO, qf, eta, D.N, BH, D.eps, status);
    return rec.end() ? HLA_OK : HLA_ERR_CUDA;
}

// Reduction of the pieces the fused key-side kernel (G CTAs over heads x T tiles, at most `smax` pieces per head) left.
// scratch_state: the fp32 sum goes to the gradient-state region instead of the state region (the causal forward keeps
// the state region for the state it carries from call to call).
template <int F>
inline hla_status reduce_pieces_f(const Plan& P, const Dims& D, int BH, char* ws, const hla_ws_layout& L, size_t off_part, int smax, int G, LaunchRec& rec,
                                  bool scratch_state) {
    __nv_bfloat16* b3 = reinterpret_cast<__nv_bfloat16*>(ws + P.b3);
    __nv_bfloat16* bq = reinterpret_cast<__nv_bfloat16*>(ws + P.bq);
    float* part = reinterpret_cast<float*>(ws + off_part);
    float* state = reinterpret_cast<float*>(ws + (scratch_state ? L.dstate : L.state));
    const int T = (D.N + kTileTokens - 1) / kTileTokens;
    rec.begin("tc_reduce_emit");
    if (D.d == 128) launch_pdl(tc_reduce_emit_kernel<128, F>, dim3(MT<F>::kPad / 8, BH), dim3(256), 0, rec.st, part, state, b3, bq, smax, D.ld, G, T);
    else launch_pdl(tc_reduce_emit_kernel<64, F>, dim3(MT<F>::kPad / 8, BH), dim3(256), 0, rec.st, part, state, b3, bq, smax, D.ld, G, T);
    return rec.end() ? HLA_OK : HLA_ERR_CUDA;
}
inline hla_status reduce_pieces(const Plan& P, const Dims& D, int BH, char* ws, const hla_ws_layout& L, size_t off_part, int smax, int G, LaunchRec& rec,
                                bool scratch_state = false) {
    return D.F == 3 ? reduce_pieces_f<3>(P, D, BH, ws, L, off_part, smax, G, rec, scratch_state)
                    : reduce_pieces_f<2>(P, D, BH, ws, L, off_part, smax, G, rec, scratch_state);
}

// The two bf16 operand images of a state that already sits, summed, in the workspace (the state region, or with
// gradient = true the gradient-state region): what the reduction emits, from one "piece" that is the state itself.  Used
// when the caller has added the states of several sequence shards between the key side and the query side of a pass.
template <int DV, int F>
inline hla_status launch_emit_from_state(const Plan& P, const Dims& D, int BH, char* ws, const hla_ws_layout& L, bool gradient, LaunchRec& rec) {
    float* st = reinterpret_cast<float*>(ws + (gradient ? L.dstate : L.state));
    __nv_bfloat16* b3 = reinterpret_cast<__nv_bfloat16*>(ws + (gradient ? P.bd3 : P.b3));
    __nv_bfloat16* bq = reinterpret_cast<__nv_bfloat16*>(ws + (gradient ? P.bdq : P.bq));
    rec.begin("tc_reduce_emit");
    launch_pdl(tc_reduce_emit_kernel<DV, F>, dim3(MT<F>::kPad / 8, BH), dim3(256), 0, rec.st, (const float*)st, st, b3, bq, 1, D.ld, 0, 0);
    return rec.end() ? HLA_OK : HLA_ERR_CUDA;
}
inline hla_status emit_from_state(const Plan& P, const Dims& D, int BH, char* ws, const hla_ws_layout& L, bool gradient, LaunchRec& rec) {
    if (D.F == 3) return D.d == 128 ? launch_emit_from_state<128, 3>(P, D, BH, ws, L, gradient, rec) : launch_emit_from_state<64, 3>(P, D, BH, ws, L, gradient, rec);
    return D.d == 128 ? launch_emit_from_state<128, 2>(P, D, BH, ws, L, gradient, rec) : launch_emit_from_state<64, 2>(P, D, BH, ws, L, gradient, rec);
}

// The readout alone (feature-level entry), on the operand image in the workspace.
template <int DV, int F>
inline hla_status launch_readout_only(const Plan& P, const Dims& D, int BH, const float* qf, void* O, char* ws, const hla_ws_layout& L, int sm_count,
                                      LaunchRec& rec) {
    CUtensorMap mapO, mapB3;
    __nv_bfloat16* b3 = reinterpret_cast<__nv_bfloat16*>(ws + P.b3);
    if (!make_map_bhnd(&mapO, O, BH, D.N, DV, kTileTokens) || !make_map_2d(&mapB3, b3, (size_t)BH * (DV + 16), MT<F>::kPad, DV + 16)) return HLA_ERR_CUDA;
    if (!set_smem(tc_readout_kernel<DV, F>, RoCfg<DV, F>::kSmem)) return HLA_ERR_CUDA;
    const int tiles = (D.N + kTileTokens - 1) / kTileTokens;
    const long long total = (long long)BH * tiles;
    const int grid = (int)(total < sm_count ? total : sm_count);
    rec.begin("tc_readout");
    launch_pdl(tc_readout_kernel<DV, F>, grid, dim3(kRoThreads), RoCfg<DV, F>::kSmem, rec.st, mapB3, mapO, qf, reinterpret_cast<float*>(ws + L.eta), D.N, BH,
               D.eps, reinterpret_cast<int*>(ws + L.status));
    return rec.end() ? HLA_OK : HLA_ERR_CUDA;
}
inline hla_status readout_only(const Plan& P, const Dims& D, int BH, const float* qf, void* O, char* ws, const hla_ws_layout& L, int sm_count, LaunchRec& rec) {
    if (D.F == 3) return D.d == 128 ? launch_readout_only<128, 3>(P, D, BH, qf, O, ws, L, sm_count, rec) : launch_readout_only<64, 3>(P, D, BH, qf, O, ws, L, sm_count, rec);
    return D.d == 128 ? launch_readout_only<128, 2>(P, D, BH, qf, O, ws, L, sm_count, rec) : launch_readout_only<64, 2>(P, D, BH, qf, O, ws, L, sm_count, rec);
}

// readout = false stops after the state has been built and reduced (the fused query-side kernel reads it out).
inline hla_status core_forward(const Plan& P, const Dims& D, int BH, const float* qf, const float* kf, const void* V, void* O, char* ws,
                               const hla_ws_layout& L, size_t off_part, int sm_count, LaunchRec& rec, bool readout = true) {
    if (D.F == 3) {
        if (D.d == 128) return launch_core_forward<128, 3>(P, D, BH, qf, kf, V, O, ws, L, off_part, sm_count, rec, readout);
        return launch_core_forward<64, 3>(P, D, BH, qf, kf, V, O, ws, L, off_part, sm_count, rec, readout);
    }
    if (D.d == 128) return launch_core_forward<128, 2>(P, D, BH, qf, kf, V, O, ws, L, off_part, sm_count, rec, readout);
    return launch_core_forward<64, 2>(P, D, BH, qf, kf, V, O, ws, L, off_part, sm_count, rec, readout);
}

template <int DV, int F>
inline hla_status launch_core_backward(const Plan& P, const Dims& D, int BH, const float* qf, const float* kf, const void* V, const void* dO,
                                       float* dqf, float* dkf, void* dV, char* ws, const hla_ws_layout& L, size_t off_part, int sm_count,
                                       LaunchRec& rec, int phase) {
    // phase 0: the whole backward; 1: query pass and reduction only (leaves the gradient state in the workspace);
    // 2: key pass only, on the gradient state in the workspace (its operand images are formed first)
    constexpr int kPad = MT<F>::kPad;
    CUtensorMap mapV, mapdO, mapdV, mapBq, mapBd3, mapBdq;
    __nv_bfloat16* bq = reinterpret_cast<__nv_bfloat16*>(ws + P.bq);
    __nv_bfloat16* bd3 = reinterpret_cast<__nv_bfloat16*>(ws + P.bd3);
    __nv_bfloat16* bdq = reinterpret_cast<__nv_bfloat16*>(ws + P.bdq);
    if (!make_map_bhnd(&mapV, V, BH, D.N, DV, kTileTokens) || !make_map_bhnd(&mapdO, dO, BH, D.N, DV, kTileTokens) ||
        !make_map_bhnd(&mapdV, dV, BH, D.N, DV, kTileTokens) || !make_map_2d(&mapBq, bq, (size_t)BH * kPad, DV, kPad) ||
        !make_map_2d(&mapBd3, bd3, (size_t)BH * (DV + 16), kPad, DV + 16) || !make_map_2d(&mapBdq, bdq, (size_t)BH * kPad, DV, kPad))
        return HLA_ERR_CUDA;
    int* status = reinterpret_cast<int*>(ws + L.status);
    float* part = reinterpret_cast<float*>(ws + off_part);
    const float* state = reinterpret_cast<const float*>(ws + L.state);
    float* dstate = reinterpret_cast<float*>(ws + L.dstate);
    const float* eta = reinterpret_cast<const float*>(ws + L.eta);
    if (!set_smem(tc_bwd_query_kernel<DV, F>, BqCfg<F>::kSmem) || !set_smem(tc_bwd_key_kernel<DV, F>, BkCfg<DV, F>::kSmem)) return HLA_ERR_CUDA;
    cudaStream_t st = rec.st;
    if (phase != 2) {
        rec.begin("tc_bwd_query");
        launch_pdl(tc_bwd_query_kernel<DV, F>, dim3(D.S, BH), dim3(kBqThreads), BqCfg<F>::kSmem, st, mapdO, mapBq, qf, eta, state, dqf, part, D.N, D.S, D.ld, D.eps,
                   status);
        if (!rec.end()) return HLA_ERR_CUDA;
        rec.begin("tc_reduce_emit");
        launch_pdl(tc_reduce_emit_kernel<DV, F>, dim3(kPad / 8, BH), dim3(256), 0, st, part, dstate, bd3, bdq, D.S, D.ld, 0, 0);
        if (!rec.end()) return HLA_ERR_CUDA;
        if (phase == 1) return HLA_OK;
    } else {
        const hla_status e = launch_emit_from_state<DV, F>(P, D, BH, ws, L, true, rec);
        if (e != HLA_OK) return e;
    }
    const int tiles = (D.N + kTileTokens - 1) / kTileTokens;
    const long long total = (long long)BH * tiles;
    const int grid = (int)(total < sm_count ? total : sm_count);
    rec.begin("tc_bwd_key");
    launch_pdl(tc_bwd_key_kernel<DV, F>, grid, dim3(kBkThreads), BkCfg<DV, F>::kSmem, st, mapV, mapBd3, mapBdq, mapdV, kf, dstate, dkf,
               static_cast<__nv_bfloat16*>(dV), D.N, BH, D.ld, status);
    return rec.end() ? HLA_OK : HLA_ERR_CUDA;
}

inline hla_status core_backward(const Plan& P, const Dims& D, int BH, const float* qf, const float* kf, const void* V, const void* dO,
                                float* dqf, float* dkf, void* dV, char* ws, const hla_ws_layout& L, size_t off_part, int sm_count, LaunchRec& rec,
                                int phase = 0) {
    if (D.F == 3) {
        if (D.d == 128) return launch_core_backward<128, 3>(P, D, BH, qf, kf, V, dO, dqf, dkf, dV, ws, L, off_part, sm_count, rec, phase);
        return launch_core_backward<64, 3>(P, D, BH, qf, kf, V, dO, dqf, dkf, dV, ws, L, off_part, sm_count, rec, phase);
    }
    if (D.d == 128) return launch_core_backward<128, 2>(P, D, BH, qf, kf, V, dO, dqf, dkf, dV, ws, L, off_part, sm_count, rec, phase);
    return launch_core_backward<64, 2>(P, D, BH, qf, kf, V, dO, dqf, dkf, dV, ws, L, off_part, sm_count, rec, phase);
}

}  // namespace tc
}  // namespace hla
