// fp32 SIMT kernels for the whole HLA path (feature maps, state build, split
// reduction, readout + normaliser, and the backward passes).  They follow the
// factored scheme of Theorem 4.2 literally - T_k and T_q are formed per token
// tile in shared memory, never in global memory - and serve the fp32 data type
// and every configuration outside the tensor-core kernels' set.
#pragma once
#include "hla_common.cuh"

namespace hla {
namespace simt {

constexpr int kTok = 16;          // tokens per shared-memory tile
constexpr int kThreads = 256;
constexpr int kPld = kMaxP + 1;   // row stride of a T tile (odd: no bank conflicts on column reads)

// Features of one tile into shared memory as featS[f][t][dphi]; the query side
// puts the same vector into every slot.  Tokens past N get zeros.
template <bool QSIDE>
__device__ __forceinline__ void stage_features(float* featS, const float* __restrict__ feat, const Dims& D, int bh, int tok0) {
    const int n = D.F * kTok * D.dphi;
    for (int idx = threadIdx.x; idx < n; idx += blockDim.x) {
        const int i = idx % D.dphi;
        const int t = (idx / D.dphi) % kTok;
        const int f = idx / (D.dphi * kTok);
        const int tok = tok0 + t;
        float v = 0.f;
        if (tok < D.N) {
            v = QSIDE ? feat[((size_t)bh * D.N + tok) * D.dphi + i]
                      : feat[(((size_t)bh * D.F + f) * D.N + tok) * D.dphi + i];
        }
        featS[idx] = v;
    }
}

// T[t][p] = prod_f featS[f][t][i_f(p)], p = ((i_0 * dphi + i_1) * dphi + ...) (first factor slowest).
__device__ __forceinline__ void build_T_tile(float* Tt, const float* featS, const Dims& D) {
    for (int idx = threadIdx.x; idx < kTok * D.P; idx += blockDim.x) {
        const int t = idx / D.P, p = idx - t * D.P;
        float prod = 1.f;
        int rem = p;
        for (int f = D.F - 1; f >= 0; --f) {
            const int i = rem % D.dphi;
            rem /= D.dphi;
            prod *= featS[(f * kTok + t) * D.dphi + i];
        }
        Tt[t * kPld + p] = prod;
    }
}

// The value-side tile X [kTok][d] and its extra column xz [kTok]:
//   forward  : X = V,          xz = 1                       (contract with V and with ones)
//   backward : X = r * dO,     xz = -r * (dO . O),  r = 1 / (eta + eps)
template <typename T, bool BWD>
__device__ __forceinline__ void load_x_tile(float* Xs, float* xz, float* rS, const T* __restrict__ X, const T* __restrict__ O,
                                            const float* __restrict__ eta, const Dims& D, int bh, int tok0) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarp = blockDim.x >> 5;
    if (BWD) {
        for (int t = warp; t < kTok; t += nwarp) {
            const int tok = tok0 + t;
            float s = 0.f;
            if (tok < D.N) {
                const size_t base = ((size_t)bh * D.N + tok) * D.d;
                for (int g = lane; g < D.d; g += 32) s += ldf(X + base + g) * ldf(O + base + g);
            }
            s = warp_sum(s);
            if (lane == 0) {
                const float r = tok < D.N ? 1.f / (eta[(size_t)bh * D.N + tok] + D.eps) : 0.f;
                rS[t] = r;
                xz[t] = -r * s;
            }
        }
        __syncthreads();
    } else {
        if (threadIdx.x < kTok) xz[threadIdx.x] = (tok0 + threadIdx.x < D.N) ? 1.f : 0.f;
    }
    for (int idx = threadIdx.x; idx < kTok * D.d; idx += blockDim.x) {
        const int t = idx / D.d, g = idx - t * D.d;
        const int tok = tok0 + t;
        float v = 0.f;
        if (tok < D.N) {
            v = ldf(X + ((size_t)bh * D.N + tok) * D.d + g);
            if (BWD) v *= rS[t];
        }
        Xs[t * kMaxD + g] = v;
    }
}

// Partial state of one token split:  part[bh][s][p][0..d-1] = sum_t T[t][p] X[t][:],  column d = sum_t T[t][p] xz[t].
// Forward (QSIDE = false, BWD = false): T = T_k, X = V            -> C, z       (Theorem 4.2: C = T_k (x)_1 V)
// Backward (QSIDE = true,  BWD = true ): T = T_q, X = dnum | deta -> dC, dz
template <typename T, bool BWD>
__global__ void __launch_bounds__(kThreads) state_build_kernel(Dims D, const float* __restrict__ feat, const T* __restrict__ X,
                                                               const T* __restrict__ O, const float* __restrict__ eta,
                                                               float* __restrict__ part) {
    __shared__ float featS[kTok * kMaxP];
    __shared__ float Tt[kTok * kPld];
    __shared__ __align__(16) float Xs[kTok * kMaxD];
    __shared__ float xz[kTok], rS[kTok];
    const int s = blockIdx.x, bh = blockIdx.y;
    const int gx = threadIdx.x & 31, py = threadIdx.x >> 5;
    const int tiles = (D.N + kTok - 1) / kTok;
    const int tiles_per = (tiles + D.S - 1) / D.S;
    const int tile0 = s * tiles_per, tile1 = min(tiles, tile0 + tiles_per);

    float acc[32][4];
#pragma unroll
    for (int k = 0; k < 32; ++k) acc[k][0] = acc[k][1] = acc[k][2] = acc[k][3] = 0.f;
    float zacc = 0.f;

    for (int tile = tile0; tile < tile1; ++tile) {
        const int tok0 = tile * kTok;
        __syncthreads();
        stage_features<BWD>(featS, feat, D, bh, tok0);
        load_x_tile<T, BWD>(Xs, xz, rS, X, O, eta, D, bh, tok0);
        __syncthreads();
        build_T_tile(Tt, featS, D);
        __syncthreads();
        const bool colok = 4 * gx < D.d;
        for (int t = 0; t < kTok; ++t) {
            float4 x = colok ? *reinterpret_cast<const float4*>(&Xs[t * kMaxD + 4 * gx]) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int k = 0; k < 32; ++k) {
                const int p = py + 8 * k;
                if (p < D.P) {
                    const float tv = Tt[t * kPld + p];
                    acc[k][0] = fmaf(tv, x.x, acc[k][0]);
                    acc[k][1] = fmaf(tv, x.y, acc[k][1]);
                    acc[k][2] = fmaf(tv, x.z, acc[k][2]);
                    acc[k][3] = fmaf(tv, x.w, acc[k][3]);
                }
            }
            if (threadIdx.x < D.P) zacc = fmaf(Tt[t * kPld + threadIdx.x], xz[t], zacc);
        }
    }
    float* out = part + ((size_t)bh * D.S + s) * D.P * D.ld;
    if (4 * gx < D.d) {
#pragma unroll
        for (int k = 0; k < 32; ++k) {
            const int p = py + 8 * k;
            if (p < D.P) *reinterpret_cast<float4*>(&out[(size_t)p * D.ld + 4 * gx]) = make_float4(acc[k][0], acc[k][1], acc[k][2], acc[k][3]);
        }
    }
    if (threadIdx.x < D.P) {
        out[(size_t)threadIdx.x * D.ld + D.d] = zacc;
        for (int c = D.d + 1; c < D.ld; ++c) out[(size_t)threadIdx.x * D.ld + c] = 0.f;
    }
}

// out[bh][i] = sum_s part[bh][s][i] in a fixed order (no atomics: bitwise reproducible).
__global__ void reduce_partials_kernel(float* __restrict__ out, const float* __restrict__ part, int BH, int S, size_t n_per) {
    const size_t total = (size_t)BH * n_per;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const size_t bh = i / n_per, j = i - bh * n_per;
        float a = 0.f;
        for (int s = 0; s < S; ++s) a += part[(bh * S + s) * n_per + j];
        out[i] = a;
    }
}

// Readout  Y[t][:] = T[t] . state[:, 0..d-1];  NORMALISE: eta_t = T[t] . state[:, d], Y /= (eta + eps), eta saved
// (Eq. "hla.la.form" and the normaliser).  Without NORMALISE it is the key-side pass dV = T_k dC.
template <typename T, bool NORMALISE>
__global__ void __launch_bounds__(kThreads) readout_kernel(Dims D, const float* __restrict__ feat, const float* __restrict__ state,
                                                           T* __restrict__ Y, float* __restrict__ eta_out) {
    __shared__ float featS[kTok * kMaxP];
    __shared__ float Tt[kTok * kPld];
    __shared__ float etaS[kTok];
    const int bh = blockIdx.y, tok0 = blockIdx.x * kTok;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    stage_features<NORMALISE>(featS, feat, D, bh, tok0);
    __syncthreads();
    build_T_tile(Tt, featS, D);
    __syncthreads();
    const float* st = state + (size_t)bh * D.P * D.ld;
    if (NORMALISE && threadIdx.x < kTok) {
        float e = 0.f;
        for (int p = 0; p < D.P; ++p) e = fmaf(Tt[threadIdx.x * kPld + p], st[(size_t)p * D.ld + D.d], e);
        etaS[threadIdx.x] = e;
        if (tok0 + threadIdx.x < D.N) eta_out[(size_t)bh * D.N + tok0 + threadIdx.x] = e;
    }
    float a0[4] = {0.f, 0.f, 0.f, 0.f}, a1[4] = {0.f, 0.f, 0.f, 0.f};
    const int t0 = 2 * warp, t1 = 2 * warp + 1;
    if (4 * lane < D.d) {
        for (int p = 0; p < D.P; ++p) {
            const float4 s = *reinterpret_cast<const float4*>(&st[(size_t)p * D.ld + 4 * lane]);
            const float u = Tt[t0 * kPld + p], w = Tt[t1 * kPld + p];
            a0[0] = fmaf(u, s.x, a0[0]); a0[1] = fmaf(u, s.y, a0[1]); a0[2] = fmaf(u, s.z, a0[2]); a0[3] = fmaf(u, s.w, a0[3]);
            a1[0] = fmaf(w, s.x, a1[0]); a1[1] = fmaf(w, s.y, a1[1]); a1[2] = fmaf(w, s.z, a1[2]); a1[3] = fmaf(w, s.w, a1[3]);
        }
    }
    __syncthreads();
    if (4 * lane < D.d) {
        const float r0 = NORMALISE ? 1.f / (etaS[t0] + D.eps) : 1.f;
        const float r1 = NORMALISE ? 1.f / (etaS[t1] + D.eps) : 1.f;
        if (tok0 + t0 < D.N) {
            T* y = Y + ((size_t)bh * D.N + tok0 + t0) * D.d + 4 * lane;
            for (int c = 0; c < 4; ++c) stf(y + c, a0[c] * r0);
        }
        if (tok0 + t1 < D.N) {
            T* y = Y + ((size_t)bh * D.N + tok0 + t1) * D.d + 4 * lane;
            for (int c = 0; c < 4; ++c) stf(y + c, a1[c] * r1);
        }
    }
}

// Gradient with respect to the feature vectors:
//   G[t][p] = sum_g X[t][g] S[p][g] + xz[t] S[p][d]           (= dT_q or dT_k)
//   dfeat^f[t][a] = sum over p with i_f(p) = a of G[t][p] * prod_{f' != f} feat^{f'}[t][i_f'(p)]
// QSIDE: X = dnum, xz = deta, S = (C|z), every slot holds q, the slots' gradients are summed.
// key side: X = V, xz = 1, S = (dC|dz), one gradient per factor.
template <typename T, bool QSIDE>
__global__ void __launch_bounds__(kThreads) feature_grad_kernel(Dims D, const float* __restrict__ feat, const T* __restrict__ X,
                                                                const T* __restrict__ O, const float* __restrict__ eta,
                                                                const float* __restrict__ S, float* __restrict__ dfeat) {
    __shared__ float featS[kTok * kMaxP];
    __shared__ float G[kTok * kPld];
    __shared__ __align__(16) float Xs[kTok * kMaxD];
    __shared__ float xz[kTok], rS[kTok];
    const int bh = blockIdx.y, tok0 = blockIdx.x * kTok;
    stage_features<QSIDE>(featS, feat, D, bh, tok0);
    load_x_tile<T, QSIDE>(Xs, xz, rS, X, O, eta, D, bh, tok0);
    __syncthreads();
    if (threadIdx.x < D.P) {
        const int p = threadIdx.x;
        const float* srow = S + ((size_t)bh * D.P + p) * D.ld;
        float acc[kTok];
#pragma unroll
        for (int t = 0; t < kTok; ++t) acc[t] = 0.f;
        for (int g = 0; g < D.d; g += 4) {
            const float4 s = *reinterpret_cast<const float4*>(srow + g);
#pragma unroll
            for (int t = 0; t < kTok; ++t) {
                const float4 x = *reinterpret_cast<const float4*>(&Xs[t * kMaxD + g]);
                acc[t] = fmaf(x.x, s.x, fmaf(x.y, s.y, fmaf(x.z, s.z, fmaf(x.w, s.w, acc[t]))));
            }
        }
        const float sz = srow[D.d];
#pragma unroll
        for (int t = 0; t < kTok; ++t) G[t * kPld + p] = fmaf(xz[t], sz, acc[t]);
    }
    __syncthreads();
    const int per = D.P / D.dphi;
    const int items = QSIDE ? kTok * D.dphi : kTok * D.F * D.dphi;
    for (int idx = threadIdx.x; idx < items; idx += blockDim.x) {
        const int a = idx % D.dphi;
        const int t = QSIDE ? idx / D.dphi : idx / (D.F * D.dphi);
        const int fsel = QSIDE ? 0 : (idx / D.dphi) % D.F;
        float total = 0.f;
        for (int f = QSIDE ? 0 : fsel; f < (QSIDE ? D.F : fsel + 1); ++f) {
            int stride = 1;
            for (int e = f + 1; e < D.F; ++e) stride *= D.dphi;
            for (int pp = 0; pp < per; ++pp) {
                const int lo = pp % stride, hi = pp / stride;
                const int p = (hi * D.dphi + a) * stride + lo;
                float prod = 1.f;
                int rem = p;
                for (int f2 = D.F - 1; f2 >= 0; --f2) {
                    const int i = rem % D.dphi;
                    rem /= D.dphi;
                    if (f2 != f) prod *= featS[(f2 * kTok + t) * D.dphi + i];
                }
                total = fmaf(G[t * kPld + p], prod, total);
            }
        }
        const int tok = tok0 + t;
        if (tok < D.N) {
            if (QSIDE) dfeat[((size_t)bh * D.N + tok) * D.dphi + a] = total;
            else dfeat[(((size_t)bh * D.F + fsel) * D.N + tok) * D.dphi + a] = total;
        }
    }
}

// ---------------------------------------------------------------------------
// Feature networks (appendix "Defining phi"): feat = ReLU(W2^T GELU(W1^T x + b1) + b2)
// ---------------------------------------------------------------------------
template <typename T>
struct PhiWeights {
    const T* W1[kMaxF];
    const T* b1[kMaxF];
    const T* W2[kMaxF];
    const T* b2[kMaxF];
    int nmaps;
};

constexpr int kPhiThreads = 128;
constexpr int kGld = kMaxD + 1;

// rows = B*H*N tokens of X [rows][d].  KSIDE: nmaps = F, output kf[bh][f][n][dphi]; else output qf[row][dphi].
template <typename T, bool KSIDE>
__global__ void __launch_bounds__(kPhiThreads) phi_forward_kernel(const T* __restrict__ X, PhiWeights<T> W, float* __restrict__ out,
                                                                  size_t rows, int N, int d, int dphi) {
    __shared__ __align__(16) float xs[kTok * kMaxD];
    __shared__ float gs[kTok * kGld];
    const size_t row0 = (size_t)blockIdx.x * kTok;
    const int j = threadIdx.x;
    for (int idx = threadIdx.x; idx < kTok * d; idx += blockDim.x) {
        const int t = idx / d, i = idx - t * d;
        xs[t * kMaxD + i] = (row0 + t < rows) ? ldf(X + (row0 + t) * d + i) : 0.f;
    }
    __syncthreads();
    for (int m = 0; m < W.nmaps; ++m) {
        if (j < d) {
            float acc[kTok];
#pragma unroll
            for (int t = 0; t < kTok; ++t) acc[t] = 0.f;
            for (int i = 0; i < d; i += 4) {
                const float w0 = ldf(W.W1[m] + (size_t)(i + 0) * d + j), w1 = ldf(W.W1[m] + (size_t)(i + 1) * d + j);
                const float w2 = ldf(W.W1[m] + (size_t)(i + 2) * d + j), w3 = ldf(W.W1[m] + (size_t)(i + 3) * d + j);
#pragma unroll
                for (int t = 0; t < kTok; ++t) {
                    const float4 x = *reinterpret_cast<const float4*>(&xs[t * kMaxD + i]);
                    acc[t] = fmaf(x.x, w0, fmaf(x.y, w1, fmaf(x.z, w2, fmaf(x.w, w3, acc[t]))));
                }
            }
            const float b = ldf(W.b1[m] + j);
#pragma unroll
            for (int t = 0; t < kTok; ++t) gs[t * kGld + j] = gelu_erf(acc[t] + b);
        }
        __syncthreads();
        for (int idx = threadIdx.x; idx < kTok * dphi; idx += blockDim.x) {
            const int t = idx / dphi, o = idx - t * dphi;
            float p = ldf(W.b2[m] + o);
            for (int jj = 0; jj < d; ++jj) p = fmaf(gs[t * kGld + jj], ldf(W.W2[m] + (size_t)jj * dphi + o), p);
            const size_t row = row0 + t;
            if (row < rows) {
                const float v = fmaxf(p, 0.f);
                if (KSIDE) {
                    const size_t bh = row / N, n = row - bh * N;
                    out[((bh * W.nmaps + m) * N + n) * dphi + o] = v;
                } else {
                    out[row * dphi + o] = v;
                }
            }
        }
        __syncthreads();
    }
}

// dX[row][:] = sum over maps of W1 (GELU'(h) * (W2 (dfeat * [pre > 0]))), h and pre recomputed.
template <typename T, bool KSIDE>
__global__ void __launch_bounds__(kPhiThreads) phi_backward_kernel(const T* __restrict__ X, PhiWeights<T> W, const float* __restrict__ dfeat,
                                                                   T* __restrict__ dX, size_t rows, int N, int d, int dphi) {
    __shared__ __align__(16) float xs[kTok * kMaxD];
    __shared__ float gs[kTok * kGld];
    __shared__ float dps[kTok * kMaxP];
    const size_t row0 = (size_t)blockIdx.x * kTok;
    const int j = threadIdx.x;
    for (int idx = threadIdx.x; idx < kTok * d; idx += blockDim.x) {
        const int t = idx / d, i = idx - t * d;
        xs[t * kMaxD + i] = (row0 + t < rows) ? ldf(X + (row0 + t) * d + i) : 0.f;
    }
    float dxacc[kTok];
#pragma unroll
    for (int t = 0; t < kTok; ++t) dxacc[t] = 0.f;
    __syncthreads();
    for (int m = 0; m < W.nmaps; ++m) {
        float h[kTok];
        if (j < d) {
#pragma unroll
            for (int t = 0; t < kTok; ++t) h[t] = 0.f;
            for (int i = 0; i < d; i += 4) {
                const float w0 = ldf(W.W1[m] + (size_t)(i + 0) * d + j), w1 = ldf(W.W1[m] + (size_t)(i + 1) * d + j);
                const float w2 = ldf(W.W1[m] + (size_t)(i + 2) * d + j), w3 = ldf(W.W1[m] + (size_t)(i + 3) * d + j);
#pragma unroll
                for (int t = 0; t < kTok; ++t) {
                    const float4 x = *reinterpret_cast<const float4*>(&xs[t * kMaxD + i]);
                    h[t] = fmaf(x.x, w0, fmaf(x.y, w1, fmaf(x.z, w2, fmaf(x.w, w3, h[t]))));
                }
            }
            const float b = ldf(W.b1[m] + j);
#pragma unroll
            for (int t = 0; t < kTok; ++t) {
                h[t] += b;
                gs[t * kGld + j] = gelu_erf(h[t]);
            }
        }
        __syncthreads();
        for (int idx = threadIdx.x; idx < kTok * dphi; idx += blockDim.x) {
            const int t = idx / dphi, o = idx - t * dphi;
            float p = ldf(W.b2[m] + o);
            for (int jj = 0; jj < d; ++jj) p = fmaf(gs[t * kGld + jj], ldf(W.W2[m] + (size_t)jj * dphi + o), p);
            const size_t row = row0 + t;
            float g = 0.f;
            if (row < rows && p > 0.f) {
                if (KSIDE) {
                    const size_t bh = row / N, n = row - bh * N;
                    g = dfeat[((bh * W.nmaps + m) * N + n) * dphi + o];
                } else {
                    g = dfeat[row * dphi + o];
                }
            }
            dps[t * dphi + o] = g;
        }
        __syncthreads();
        if (j < d) {
#pragma unroll
            for (int t = 0; t < kTok; ++t) {
                float dg = 0.f;
                for (int o = 0; o < dphi; ++o) dg = fmaf(dps[t * dphi + o], ldf(W.W2[m] + (size_t)j * dphi + o), dg);
                gs[t * kGld + j] = dg * gelu_erf_grad(h[t]);   // dh; gs is free: every read of GELU(h) finished before the last barrier
            }
        }
        __syncthreads();
        if (j < d) {
            const T* wrow = W.W1[m] + (size_t)j * d;   // here thread j plays the input index i
            for (int jj = 0; jj < d; ++jj) {
                const float w = ldf(wrow + jj);
#pragma unroll
                for (int t = 0; t < kTok; ++t) dxacc[t] = fmaf(gs[t * kGld + jj], w, dxacc[t]);
            }
        }
        __syncthreads();
    }
    if (j < d) {
#pragma unroll
        for (int t = 0; t < kTok; ++t)
            if (row0 + t < rows) stf(dX + (row0 + t) * d + j, dxacc[t]);
    }
}

}  // namespace simt
}  // namespace hla
