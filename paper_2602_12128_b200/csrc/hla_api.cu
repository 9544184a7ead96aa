// C ABI of the HLA library: context, validation, workspace layout and the
// launch sequences of forward and backward.  See include/hla.h for the contract.
#include "../../include/hla.h"

#include <mutex>
#include <new>
#include <string.h>

#include "hla_common.cuh"
#include "hla_simt.cuh"
#include "hla_tc.cuh"
#include "hla_tc_phi.cuh"
#include "hla_tc_fused.cuh"
#include "hla_tc_fused_k.cuh"
#include "hla_tc_wgrad.cuh"
#include "hla_tc_vmod.cuh"
#include "hla_tc_causal.cuh"
#include "hla_tc_causal_grad.cuh"

using namespace hla;

struct hla_ctx {
    hla_config cfg;
    Dims D;
    int BH;
    bool tc;            // tensor-core kernels in use
    bool phi_set;
    hla_mlp phi_q;
    hla_mlp phi_k[kMaxF];
    hla_ws_layout L;
    size_t off_part;    // split partials (scratch)
    int k_pieces;       // most pieces a head has in the fused key-side kernel of the forward
    bool vmod, phi_v_set;   // value modulation enabled at creation; its weights given
    hla_vmlp phi_v[2];
    tc::VmodPlan vmp;   // scratch of the value modulation inside the workspace
    size_t off_delta;   // dO . o per token (scratch of the causal backward)
    bool carry;         // causal forward starts from the state the previous call left in the workspace
    size_t off_wpart;   // per-CTA partials of the weight gradients (scratch; tensor-core path with the phi maps)
    tc::Plan tcp;       // tensor-core operand buffers inside the workspace
    size_t ws_bytes;
    int sm_count;
    LaunchRec rec;      // launch counter and optional per-kernel event timing
    tc::HostCache hc;   // tensor maps and kernel attributes already set up by earlier calls
    int device;         // device the context was created on (the kernel attributes above are per device)
};

namespace {

constexpr size_t kNone = (size_t)-1;

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Carver {
    size_t off = 0;
    size_t take(size_t bytes) {
        const size_t o = off;
        off = align_up(off + bytes, 256);
        return o;
    }
};

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int ipow(int b, int e) {
    long long r = 1;
    for (int i = 0; i < e; ++i) {
        r *= b;
        if (r > (1 << 20)) return 1 << 20;
    }
    return (int)r;
}

template <typename T>
simt::PhiWeights<T> pack_weights(const hla_mlp* m, int n) {
    simt::PhiWeights<T> w{};
    w.nmaps = n;
    for (int i = 0; i < n; ++i) {
        w.W1[i] = static_cast<const T*>(m[i].W1);
        w.b1[i] = static_cast<const T*>(m[i].b1);
        w.W2[i] = static_cast<const T*>(m[i].W2);
        w.b2[i] = static_cast<const T*>(m[i].b2);
    }
    return w;
}

int reduce_blocks(size_t total) {
    size_t b = (total + 255) / 256;
    return (int)(b > 4096 ? 4096 : (b < 1 ? 1 : b));
}

// ---- fp32 SIMT path --------------------------------------------------------
template <typename T>
hla_status simt_phi_forward(hla_ctx* c, const void* Q, const void* K, char* ws, cudaStream_t st) {
    const Dims& D = c->D;
    const size_t rows = (size_t)c->BH * D.N;
    const int blocks = (int)((rows + simt::kTok - 1) / simt::kTok);
    c->rec.begin("simt_phi_forward");
    simt::phi_forward_kernel<T, false><<<blocks, simt::kPhiThreads, 0, st>>>(
        static_cast<const T*>(Q), pack_weights<T>(&c->phi_q, 1), reinterpret_cast<float*>(ws + c->L.qf), rows, D.N, D.d, D.dphi);
    if (!c->rec.end()) return HLA_ERR_CUDA;
    c->rec.begin("simt_phi_forward");
    simt::phi_forward_kernel<T, true><<<blocks, simt::kPhiThreads, 0, st>>>(
        static_cast<const T*>(K), pack_weights<T>(c->phi_k, D.F), reinterpret_cast<float*>(ws + c->L.kf), rows, D.N, D.d, D.dphi);
    if (!c->rec.end()) return HLA_ERR_CUDA;
    return HLA_OK;
}

template <typename T>
hla_status simt_core_forward(hla_ctx* c, const float* qf, const float* kf, const void* V, void* O, char* ws, cudaStream_t st) {
    const Dims& D = c->D;
    float* part = reinterpret_cast<float*>(ws + c->off_part);
    float* state = reinterpret_cast<float*>(ws + c->L.state);
    float* eta = reinterpret_cast<float*>(ws + c->L.eta);
    c->rec.begin("simt_state_build");
    simt::state_build_kernel<T, false><<<dim3(D.S, c->BH), simt::kThreads, 0, st>>>(D, kf, static_cast<const T*>(V), nullptr, nullptr, part);
    if (!c->rec.end()) return HLA_ERR_CUDA;
    const size_t n_per = (size_t)D.P * D.ld;
    c->rec.begin("simt_reduce_partials");
    simt::reduce_partials_kernel<<<reduce_blocks(n_per * c->BH), 256, 0, st>>>(state, part, c->BH, D.S, n_per);
    if (!c->rec.end()) return HLA_ERR_CUDA;
    const int tiles = (D.N + simt::kTok - 1) / simt::kTok;
    c->rec.begin("simt_readout");
    simt::readout_kernel<T, true><<<dim3(tiles, c->BH), simt::kThreads, 0, st>>>(D, qf, state, static_cast<T*>(O), eta);
    if (!c->rec.end()) return HLA_ERR_CUDA;
    return HLA_OK;
}

template <typename T>
hla_status simt_core_backward(hla_ctx* c, const float* qf, const float* kf, const void* V, const void* O, const void* dO,
                              float* dqf, float* dkf, void* dV, char* ws, cudaStream_t st) {
    const Dims& D = c->D;
    float* part = reinterpret_cast<float*>(ws + c->off_part);
    const float* state = reinterpret_cast<const float*>(ws + c->L.state);
    float* dstate = reinterpret_cast<float*>(ws + c->L.dstate);
    const float* eta = reinterpret_cast<const float*>(ws + c->L.eta);
    const int tiles = (D.N + simt::kTok - 1) / simt::kTok;
    const size_t n_per = (size_t)D.P * D.ld;
    // pass over the queries: dC, dz, then dq
    c->rec.begin("simt_state_build");
    simt::state_build_kernel<T, true><<<dim3(D.S, c->BH), simt::kThreads, 0, st>>>(D, qf, static_cast<const T*>(dO), static_cast<const T*>(O), eta, part);
    if (!c->rec.end()) return HLA_ERR_CUDA;
    c->rec.begin("simt_reduce_partials");
    simt::reduce_partials_kernel<<<reduce_blocks(n_per * c->BH), 256, 0, st>>>(dstate, part, c->BH, D.S, n_per);
    if (!c->rec.end()) return HLA_ERR_CUDA;
    c->rec.begin("simt_feature_grad");
    simt::feature_grad_kernel<T, true><<<dim3(tiles, c->BH), simt::kThreads, 0, st>>>(D, qf, static_cast<const T*>(dO), static_cast<const T*>(O), eta, state, dqf);
    if (!c->rec.end()) return HLA_ERR_CUDA;
    // pass over the keys: dV, dk^f
    c->rec.begin("simt_readout");
    simt::readout_kernel<T, false><<<dim3(tiles, c->BH), simt::kThreads, 0, st>>>(D, kf, dstate, static_cast<T*>(dV), nullptr);
    if (!c->rec.end()) return HLA_ERR_CUDA;
    c->rec.begin("simt_feature_grad");
    simt::feature_grad_kernel<T, false><<<dim3(tiles, c->BH), simt::kThreads, 0, st>>>(D, kf, static_cast<const T*>(V), nullptr, nullptr, dstate, dkf);
    if (!c->rec.end()) return HLA_ERR_CUDA;
    return HLA_OK;
}

template <typename T>
hla_status simt_phi_backward(hla_ctx* c, const void* Q, const void* K, void* dQ, void* dK, char* ws, cudaStream_t st) {
    const Dims& D = c->D;
    const size_t rows = (size_t)c->BH * D.N;
    const int blocks = (int)((rows + simt::kTok - 1) / simt::kTok);
    c->rec.begin("simt_phi_backward");
    simt::phi_backward_kernel<T, false><<<blocks, simt::kPhiThreads, 0, st>>>(
        static_cast<const T*>(Q), pack_weights<T>(&c->phi_q, 1), reinterpret_cast<const float*>(ws + c->L.dqf), static_cast<T*>(dQ), rows, D.N, D.d, D.dphi);
    if (!c->rec.end()) return HLA_ERR_CUDA;
    c->rec.begin("simt_phi_backward");
    simt::phi_backward_kernel<T, true><<<blocks, simt::kPhiThreads, 0, st>>>(
        static_cast<const T*>(K), pack_weights<T>(c->phi_k, D.F), reinterpret_cast<const float*>(ws + c->L.dkf), static_cast<T*>(dK), rows, D.N, D.d, D.dphi);
    if (!c->rec.end()) return HLA_ERR_CUDA;
    return HLA_OK;
}

template <typename T>
hla_status forward_simt(hla_ctx* c, const void* Q, const void* K, const void* V, void* O, char* ws, cudaStream_t st) {
    const float *qf, *kf;
    if (c->cfg.phi == HLA_PHI_MLP) {
        hla_status s = simt_phi_forward<T>(c, Q, K, ws, st);
        if (s != HLA_OK) return s;
        qf = reinterpret_cast<const float*>(ws + c->L.qf);
        kf = reinterpret_cast<const float*>(ws + c->L.kf);
    } else {
        qf = static_cast<const float*>(Q);
        kf = static_cast<const float*>(K);
    }
    return simt_core_forward<T>(c, qf, kf, V, O, ws, st);
}

template <typename T>
hla_status backward_simt(hla_ctx* c, const void* Q, const void* K, const void* V, const void* O, const void* dO, void* dQ,
                         void* dK, void* dV, char* ws, cudaStream_t st) {
    const bool mlp = c->cfg.phi == HLA_PHI_MLP;
    const float* qf = mlp ? reinterpret_cast<const float*>(ws + c->L.qf) : static_cast<const float*>(Q);
    const float* kf = mlp ? reinterpret_cast<const float*>(ws + c->L.kf) : static_cast<const float*>(K);
    float* dqf = mlp ? reinterpret_cast<float*>(ws + c->L.dqf) : static_cast<float*>(dQ);
    float* dkf = mlp ? reinterpret_cast<float*>(ws + c->L.dkf) : static_cast<float*>(dK);
    hla_status s = simt_core_backward<T>(c, qf, kf, V, O, dO, dqf, dkf, dV, ws, st);
    if (s != HLA_OK || !mlp) return s;
    return simt_phi_backward<T>(c, Q, K, dQ, dK, ws, st);
}

hla_status check_call(const hla_ctx* c, const void* const* ptrs, int n, const void* ws, size_t ws_bytes) {
    if (!c) return HLA_ERR_INVALID_ARG;
    for (int i = 0; i < n; ++i)
        if (!ptrs[i] || !aligned16(ptrs[i])) return HLA_ERR_INVALID_ARG;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u)) return HLA_ERR_INVALID_ARG;
    if (ws_bytes < c->ws_bytes) return HLA_ERR_WORKSPACE;
    if (c->cfg.phi == HLA_PHI_MLP && !c->phi_set) return HLA_ERR_INVALID_ARG;
    return HLA_OK;
}

// The kernel attributes a context has set belong to the device that was current then.
void follow_device(hla_ctx* ctx) {
    int dev = ctx->device;
    if (cudaGetDevice(&dev) == cudaSuccess && dev != ctx->device) {
        ctx->hc.nfuncs = 0;
        ctx->device = dev;
    }
}

}  // namespace

extern "C" {

hla_status hla_create(const hla_config* cfg, hla_ctx** out) {
    if (out) *out = nullptr;
    if (!cfg || !out) return HLA_ERR_INVALID_ARG;
    hla_config c = *cfg;
    if (c.B <= 0 || c.H <= 0 || c.N <= 0 || c.d <= 0) return HLA_ERR_INVALID_ARG;
    if (c.F < 0 || c.d_phi < 0 || c.n_splits < 0) return HLA_ERR_INVALID_ARG;
    if (c.phi != HLA_PHI_MLP && c.phi != HLA_PHI_NONE) return HLA_ERR_INVALID_ARG;
    if (c.dtype != HLA_BF16 && c.dtype != HLA_F32) return HLA_ERR_INVALID_ARG;
    if (c.F == 0) c.F = 3;
    if (c.d_phi == 0) {
        if (c.F == 3) c.d_phi = 6;
        else if (c.F == 2) c.d_phi = 12;
        else return HLA_ERR_INVALID_ARG;
    }
    if (!(c.eps > 0.f)) c.eps = 1e-6f;
    if (c.causal != 0 && c.causal != 1) return HLA_ERR_INVALID_ARG;
    if (c.value_mod != 0 && c.value_mod != 1) return HLA_ERR_INVALID_ARG;
    if (c.value_mod && !(c.dtype == HLA_BF16 && (c.d == 64 || c.d == 128) && (long long)c.B * c.H * c.N < (1ll << 31))) return HLA_ERR_UNSUPPORTED;
    if (c.F > kMaxF) return HLA_ERR_UNSUPPORTED;
    const int P = ipow(c.d_phi, c.F);
    if (P > kMaxP) return HLA_ERR_UNSUPPORTED;
    if (c.d > kMaxD || (c.d % 4) != 0) return HLA_ERR_UNSUPPORTED;
    if ((long long)c.B * c.H > 65535) return HLA_ERR_UNSUPPORTED;
    if (c.dtype == HLA_BF16 && (c.d % 8) != 0) return HLA_ERR_UNSUPPORTED;   // 16-byte rows

    hla_ctx* x = new (std::nothrow) hla_ctx();
    if (!x) return HLA_ERR_NO_MEMORY;
    x->cfg = c;
    x->BH = c.B * c.H;
    x->phi_set = false;
    x->sm_count = 148;
    int dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0) x->sm_count = n;
    }
    (void)cudaGetLastError();
    x->device = dev;
    Dims& D = x->D;
    D.B = c.B; D.H = c.H; D.N = c.N; D.d = c.d; D.F = c.F; D.dphi = c.d_phi; D.P = P;
    D.ld = c.d + 4;
    D.eps = c.eps;
    x->tc = tc::supported(c.dtype == HLA_BF16, c.d, c.F, c.d_phi) && (long long)c.B * c.H * c.N < (1ll << 31);   // the tensor-core kernels index tokens in 32 bits
    if (c.causal && !(x->tc && c.F == 3)) {      // the causal sweep exists for the 3-factor tensor-core set only
        delete x;
        return HLA_ERR_UNSUPPORTED;
    }
    const int tile = x->tc ? tc::kTileTokens : simt::kTok;
    const int tiles = (c.N + tile - 1) / tile;
    int S = c.n_splits;
    if (S == 0) {
        if (x->tc) {
            // One CTA per SM: S * heads CTAs run in ceil(S * heads / SMs) waves.  Take the split count that fills its
            // waves best (each extra wave is charged 2 % for its start-up and drain), with at least 8 tiles per CTA.
            const int smax = tiles / 8 > 1 ? (tiles / 8 < 64 ? tiles / 8 : 64) : 1;
            double best = -1.0;
            for (int cand = 1; cand <= smax; ++cand) {
                const long long ctas = (long long)cand * x->BH;
                const long long waves = (ctas + x->sm_count - 1) / x->sm_count;
                const double score = (double)ctas / (double)(waves * x->sm_count) - 0.02 * (double)(waves - 1);
                if (score > best + 1e-9) { best = score; S = cand; }
            }
        } else {
            S = (2 * x->sm_count + x->BH - 1) / x->BH;
        }
    }
    if (S > tiles) S = tiles;
    if (S < 1) S = 1;
    D.S = S;

    const bool mlp = c.phi == HLA_PHI_MLP;
    const size_t tok = (size_t)x->BH * c.N;
    Carver cv;
    hla_ws_layout& L = x->L;
    L.status = cv.take(64);
    L.qf = mlp ? cv.take(tok * c.d_phi * 4) : kNone;
    L.kf = mlp ? cv.take(tok * c.F * c.d_phi * 4) : kNone;
    L.state = cv.take((size_t)x->BH * P * D.ld * 4);
    L.eta = cv.take(tok * 4);
    L.dstate = cv.take((size_t)x->BH * P * D.ld * 4);
    L.dqf = mlp ? cv.take(tok * c.d_phi * 4) : kNone;
    L.dkf = mlp ? cv.take(tok * c.F * c.d_phi * 4) : kNone;
    L.state_ld = D.ld;
    L.state_rows = x->tc ? tc::n_mono(c.F) : P;
    L.n_splits = S;
    L.tensor_core = x->tc ? 1 : 0;
    // partial states: S per head from the split kernels, or the pieces of the fused key-side kernel (folded rows)
    x->k_pieces = 0;
    size_t part_bytes = (size_t)x->BH * S * P * D.ld * 4;
    if (x->tc && mlp) {
        x->k_pieces = tc::fused_key_max_pieces(x->BH, tiles, tc::fused_key_grid(x->BH, c.N, x->sm_count));
        const size_t need = (size_t)x->BH * x->k_pieces * tc::n_mono(c.F) * D.ld * 4;
        if (need > part_bytes) part_bytes = need;
    }
    x->off_part = cv.take(part_bytes);
    x->off_wpart = (x->tc && mlp) ? cv.take(tc::wgrad_part_bytes(c.d, (long long)x->BH * c.N, x->sm_count)) : kNone;
    if (x->tc) cv.off = tc::plan(x->tcp, D, x->BH, cv.off);
    x->off_delta = c.causal ? cv.take(tok * 4) : kNone;      // dO . o per token (causal backward)
    x->carry = false;
    x->vmod = c.value_mod != 0;
    x->phi_v_set = false;
    if (x->vmod) cv.off = tc::vmod_plan(x->vmp, c.d, (long long)x->BH * c.N, cv.off);
    x->ws_bytes = cv.off;
    *out = x;
    return HLA_OK;
}

hla_status hla_set_phi(hla_ctx* ctx, const hla_mlp* phi_q, const hla_mlp* phi_k) {
    if (!ctx || !phi_q || !phi_k) return HLA_ERR_INVALID_ARG;
    if (ctx->cfg.phi != HLA_PHI_MLP) return HLA_ERR_INVALID_ARG;
    const hla_mlp* all[1 + kMaxF];
    all[0] = phi_q;
    for (int f = 0; f < ctx->D.F; ++f) all[1 + f] = phi_k + f;
    for (int i = 0; i < 1 + ctx->D.F; ++i) {
        const void* p[4] = {all[i]->W1, all[i]->b1, all[i]->W2, all[i]->b2};
        for (int j = 0; j < 4; ++j)
            if (!p[j]) return HLA_ERR_INVALID_ARG;
        if (!aligned16(all[i]->W1) || !aligned16(all[i]->W2)) return HLA_ERR_INVALID_ARG;
    }
    ctx->phi_q = *phi_q;
    for (int f = 0; f < ctx->D.F; ++f) ctx->phi_k[f] = phi_k[f];
    ctx->phi_set = true;
    return HLA_OK;
}

hla_status hla_set_carry(hla_ctx* ctx, int carry) {
    if (!ctx || (carry != 0 && carry != 1)) return HLA_ERR_INVALID_ARG;
    if (!ctx->cfg.causal) return HLA_ERR_INVALID_ARG;
    ctx->carry = carry != 0;
    return HLA_OK;
}

size_t hla_workspace_bytes(const hla_ctx* ctx) { return ctx ? ctx->ws_bytes : 0; }

hla_status hla_workspace_layout(const hla_ctx* ctx, hla_ws_layout* out) {
    if (!ctx || !out) return HLA_ERR_INVALID_ARG;
    *out = ctx->L;
    return HLA_OK;
}

}  // extern "C"

namespace {
// phase 0: the whole forward; 1: key side only (state left in the workspace); 2: query side only, on the state in the workspace
hla_status forward_impl(hla_ctx* ctx, const void* Q, const void* K, const void* V, void* O, void* workspace, size_t workspace_bytes, void* cuda_stream,
                        int phase) {
    hla_status s;
    if (phase == 1) {
        const void* ptrs[2] = {K, V};
        s = check_call(ctx, ptrs, 2, workspace, workspace_bytes);
    } else if (phase == 2) {
        const void* ptrs[2] = {Q, O};
        s = check_call(ctx, ptrs, 2, workspace, workspace_bytes);
    } else {
        const void* ptrs[4] = {Q, K, V, O};
        s = check_call(ctx, ptrs, 4, workspace, workspace_bytes);
    }
    if (s != HLA_OK) return s;
    if (phase != 0 && (!ctx->tc || ctx->cfg.causal)) return HLA_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char* ws = static_cast<char*>(workspace);
    ctx->rec.start_call(st);
    (void)cudaGetLastError();
    if (phase != 2 && cudaMemsetAsync(ws + ctx->L.status, 0, 64, st) != cudaSuccess) return HLA_ERR_CUDA;
    follow_device(ctx);
    tc::HostCacheScope scope(&ctx->hc);
    if (ctx->tc) {
        const float *qf, *kf;
        if (ctx->cfg.phi == HLA_PHI_MLP) {
            // one kernel for the key maps and the state build -> reduction of its pieces -> one kernel for phi_q, readout
            // and normaliser
            if (phase != 2) {
                s = tc::phik_state(ctx->D, ctx->BH, ctx->phi_k, K, V, ws, ctx->L, ctx->off_part, ctx->k_pieces, ctx->sm_count, ctx->rec);
                if (s != HLA_OK) return s;
                s = tc::reduce_pieces(ctx->tcp, ctx->D, ctx->BH, ws, ctx->L, ctx->off_part, ctx->k_pieces,
                                      tc::fused_key_grid(ctx->BH, ctx->D.N, ctx->sm_count), ctx->rec, ctx->cfg.causal != 0);
                if (s != HLA_OK || phase == 1) return s;
            } else {
                s = tc::emit_from_state(ctx->tcp, ctx->D, ctx->BH, ws, ctx->L, false, ctx->rec);
                if (s != HLA_OK) return s;
            }
            // causal: only the feature map of the query side runs (no readout), which leaves the features of both sides in the
            // workspace; the pieces of the key-side kernel become the pieces of the sweep
            s = tc::phiq_readout(ctx->tcp, ctx->D, ctx->BH, &ctx->phi_q, Q, O, ws, ctx->L, ctx->sm_count, ctx->rec, !ctx->cfg.causal);
            if (s != HLA_OK || !ctx->cfg.causal) return s;
            return tc::causal_sweep(ctx->D, ctx->BH, reinterpret_cast<const float*>(ws + ctx->L.qf), reinterpret_cast<const float*>(ws + ctx->L.kf), V, O,
                                    ws, ctx->L, ctx->off_part, ctx->k_pieces, tc::fused_key_grid(ctx->BH, ctx->D.N, ctx->sm_count), ctx->carry, ctx->rec);
        } else {
            qf = static_cast<const float*>(Q);
            kf = static_cast<const float*>(K);
        }
        if (ctx->cfg.causal) return tc::causal_forward(ctx->D, ctx->BH, qf, kf, V, O, ws, ctx->L, ctx->off_part, ctx->carry, ctx->rec);
        if (phase == 2) {
            s = tc::emit_from_state(ctx->tcp, ctx->D, ctx->BH, ws, ctx->L, false, ctx->rec);
            if (s != HLA_OK) return s;
            return tc::readout_only(ctx->tcp, ctx->D, ctx->BH, qf, O, ws, ctx->L, ctx->sm_count, ctx->rec);
        }
        return tc::core_forward(ctx->tcp, ctx->D, ctx->BH, qf, kf, V, O, ws, ctx->L, ctx->off_part, ctx->sm_count, ctx->rec, phase == 0);
    }
    if (ctx->cfg.dtype == HLA_F32) return forward_simt<float>(ctx, Q, K, V, O, ws, st);
    return forward_simt<__nv_bfloat16>(ctx, Q, K, V, O, ws, st);
}
}  // namespace

extern "C" {

hla_status hla_forward(hla_ctx* ctx, const void* Q, const void* K, const void* V, void* O, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return forward_impl(ctx, Q, K, V, O, workspace, workspace_bytes, cuda_stream, 0);
}
hla_status hla_forward_keys(hla_ctx* ctx, const void* K, const void* V, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return forward_impl(ctx, nullptr, K, V, nullptr, workspace, workspace_bytes, cuda_stream, 1);
}
hla_status hla_forward_queries(hla_ctx* ctx, const void* Q, void* O, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return forward_impl(ctx, Q, nullptr, nullptr, O, workspace, workspace_bytes, cuda_stream, 2);
}

}  // extern "C"

namespace {
hla_status backward_impl(hla_ctx* ctx, const void* Q, const void* K, const void* V, const void* O, const void* dO, void* dQ, void* dK, void* dV,
                         void* workspace, size_t workspace_bytes, void* cuda_stream, int phase) {
    const void* ptrs[8] = {Q, K, V, O, dO, dQ, dK, dV};
    hla_status s = check_call(ctx, ptrs, 8, workspace, workspace_bytes);
    if (s != HLA_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char* ws = static_cast<char*>(workspace);
    ctx->rec.start_call(st);
    (void)cudaGetLastError();
    follow_device(ctx);
    tc::HostCacheScope scope(&ctx->hc);
    if (phase != 0 && (!ctx->tc || ctx->cfg.causal)) return HLA_ERR_UNSUPPORTED;
    if (ctx->tc) {
        const bool mlp = ctx->cfg.phi == HLA_PHI_MLP;
        // the phi backward writes rows of dQ, dK with 32-byte stores; so does the 2-factor key pass with dV
        if (mlp && ((reinterpret_cast<uintptr_t>(dQ) | reinterpret_cast<uintptr_t>(dK)) & 31u)) return HLA_ERR_INVALID_ARG;
        if (ctx->D.F == 2 && (reinterpret_cast<uintptr_t>(dV) & 31u)) return HLA_ERR_INVALID_ARG;
        const float* qf = mlp ? reinterpret_cast<const float*>(ws + ctx->L.qf) : static_cast<const float*>(Q);
        const float* kf = mlp ? reinterpret_cast<const float*>(ws + ctx->L.kf) : static_cast<const float*>(K);
        float* dqf = mlp ? reinterpret_cast<float*>(ws + ctx->L.dqf) : static_cast<float*>(dQ);
        float* dkf = mlp ? reinterpret_cast<float*>(ws + ctx->L.dkf) : static_cast<float*>(dK);
        if (ctx->cfg.causal) {
            if (ctx->carry) return HLA_ERR_UNSUPPORTED;      // a chunk that started from a carried state has no backward here
            s = tc::causal_backward(ctx->D, ctx->BH, qf, kf, V, O, dO, dqf, dkf, dV, ws, ctx->L, ctx->off_part, ctx->off_delta, ctx->rec);
        } else {
            s = tc::core_backward(ctx->tcp, ctx->D, ctx->BH, qf, kf, V, dO, dqf, dkf, dV, ws, ctx->L, ctx->off_part, ctx->sm_count, ctx->rec, phase);
        }
        if (s != HLA_OK || !mlp || phase == 1) return s;
        return tc::phi_backward(ctx->D, ctx->BH, &ctx->phi_q, ctx->phi_k, Q, K, dQ, dK, ws, ctx->L, ctx->sm_count, ctx->rec);
    }
    if (ctx->cfg.dtype == HLA_F32) return backward_simt<float>(ctx, Q, K, V, O, dO, dQ, dK, dV, ws, st);
    return backward_simt<__nv_bfloat16>(ctx, Q, K, V, O, dO, dQ, dK, dV, ws, st);
}
}  // namespace

extern "C" {

hla_status hla_backward(hla_ctx* ctx, const void* Q, const void* K, const void* V, const void* O, const void* dO, void* dQ, void* dK, void* dV,
                        void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return backward_impl(ctx, Q, K, V, O, dO, dQ, dK, dV, workspace, workspace_bytes, cuda_stream, 0);
}
hla_status hla_backward_queries(hla_ctx* ctx, const void* Q, const void* K, const void* V, const void* O, const void* dO, void* dQ, void* dK, void* dV,
                                void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return backward_impl(ctx, Q, K, V, O, dO, dQ, dK, dV, workspace, workspace_bytes, cuda_stream, 1);
}
hla_status hla_backward_keys(hla_ctx* ctx, const void* Q, const void* K, const void* V, const void* O, const void* dO, void* dQ, void* dK, void* dV,
                             void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return backward_impl(ctx, Q, K, V, O, dO, dQ, dK, dV, workspace, workspace_bytes, cuda_stream, 2);
}

hla_status hla_backward_weights(hla_ctx* ctx, const void* Q, const void* K, const hla_mlp_grad* dphi_q, const hla_mlp_grad* dphi_k, void* workspace,
                                size_t workspace_bytes, void* cuda_stream) {
    const void* ptrs[2] = {Q, K};
    hla_status s = check_call(ctx, ptrs, 2, workspace, workspace_bytes);
    if (s != HLA_OK) return s;
    if (ctx->cfg.phi != HLA_PHI_MLP) return HLA_ERR_INVALID_ARG;
    if (!ctx->tc) return HLA_ERR_UNSUPPORTED;
    const hla_mlp_grad* all[1 + kMaxF];
    int n = 0;
    if (dphi_q) all[n++] = dphi_q;
    if (dphi_k)
        for (int f = 0; f < ctx->D.F; ++f) all[n++] = dphi_k + f;
    for (int i = 0; i < n; ++i) {
        const void* p[4] = {all[i]->dW1, all[i]->db1, all[i]->dW2, all[i]->db2};
        for (int j = 0; j < 4; ++j)
            if (!p[j] || !aligned16(p[j])) return HLA_ERR_INVALID_ARG;
    }
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    ctx->rec.start_call(st);
    (void)cudaGetLastError();
    follow_device(ctx);
    tc::HostCacheScope scope(&ctx->hc);
    return tc::phi_wgrad(ctx->D, ctx->BH, &ctx->phi_q, ctx->phi_k, Q, K, dphi_q, dphi_k, static_cast<char*>(workspace), ctx->L, ctx->off_wpart,
                         ctx->sm_count, ctx->rec);
}

hla_status hla_set_phi_v(hla_ctx* ctx, const hla_vmlp* v1, const hla_vmlp* v2) {
    if (!ctx || !v1 || !v2) return HLA_ERR_INVALID_ARG;
    if (!ctx->vmod) return HLA_ERR_INVALID_ARG;
    const hla_vmlp* all[2] = {v1, v2};
    for (int i = 0; i < 2; ++i) {
        const void* p[6] = {all[i]->ln_g, all[i]->ln_b, all[i]->W1, all[i]->b1, all[i]->W2, all[i]->b2};
        for (int j = 0; j < 6; ++j)
            if (!p[j]) return HLA_ERR_INVALID_ARG;
        if (!aligned16(all[i]->W1) || !aligned16(all[i]->W2)) return HLA_ERR_INVALID_ARG;
    }
    ctx->phi_v[0] = *v1;
    ctx->phi_v[1] = *v2;
    ctx->phi_v_set = true;
    return HLA_OK;
}

namespace {
hla_status value_mod_call(hla_ctx* ctx, const void* T, const void* V, const void* dOut, void* Out, void* dT, void* dV, int accumulate, bool backward,
                          void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!ctx) return HLA_ERR_INVALID_ARG;
    if (!ctx->vmod || !ctx->phi_v_set) return HLA_ERR_INVALID_ARG;
    const void* in[3] = {T, V, backward ? dOut : T};
    for (int i = 0; i < 3; ++i)
        if (!in[i] || !aligned16(in[i])) return HLA_ERR_INVALID_ARG;
    const void* out[2] = {backward ? dT : Out, backward ? dV : Out};
    for (int i = 0; i < 2; ++i)
        if (!out[i] || (reinterpret_cast<uintptr_t>(out[i]) & 31u)) return HLA_ERR_INVALID_ARG;
    if (!backward && (Out == T || Out == V)) return HLA_ERR_INVALID_ARG;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return HLA_ERR_INVALID_ARG;
    if (workspace_bytes < ctx->ws_bytes) return HLA_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char* ws = static_cast<char*>(workspace);
    ctx->rec.start_call(st);
    (void)cudaGetLastError();
    follow_device(ctx);
    tc::HostCacheScope scope(&ctx->hc);
    const long long rows = (long long)ctx->BH * ctx->D.N;
    int* status = reinterpret_cast<int*>(ws + ctx->L.status);
    // like hla_forward, the forward starts a new record of device-side time-outs
    if (!backward && cudaMemsetAsync(ws + ctx->L.status, 0, 64, st) != cudaSuccess) return HLA_ERR_CUDA;
    if (ctx->D.d == 128)
        return tc::launch_vmod<128>(ctx->vmp, rows, ctx->phi_v, T, V, dOut, Out, dT, dV, accumulate, backward, ws, status, ctx->sm_count, ctx->rec);
    return tc::launch_vmod<64>(ctx->vmp, rows, ctx->phi_v, T, V, dOut, Out, dT, dV, accumulate, backward, ws, status, ctx->sm_count, ctx->rec);
}
}  // namespace

hla_status hla_value_mod_forward(hla_ctx* ctx, const void* T, const void* V, void* Out, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return value_mod_call(ctx, T, V, nullptr, Out, nullptr, nullptr, 0, false, workspace, workspace_bytes, cuda_stream);
}

hla_status hla_value_mod_backward(hla_ctx* ctx, const void* T, const void* V, const void* dOut, void* dT, void* dV, int32_t accumulate_dV, void* workspace,
                                  size_t workspace_bytes, void* cuda_stream) {
    return value_mod_call(ctx, T, V, dOut, nullptr, dT, dV, accumulate_dV != 0, true, workspace, workspace_bytes, cuda_stream);
}

// ---- forward on the library's own scratch array ---------------------------------------------
// The scratch of hla_forward_static.  In host code `g_static_ws` only names the symbol: it is not a
// device address, and a kernel handed it would read the wrong memory.  The address each device has
// for it is looked up once per device with cudaGetSymbolAddress and cached below.
static __device__ __align__(256) unsigned char g_static_ws[HLA_STATIC_WS_BYTES];

namespace {
constexpr int kMaxDevices = 64;
void* g_static_ws_addr[kMaxDevices] = {};
std::mutex g_static_ws_mutex;

// Device address of g_static_ws on the current device (looked up on the first call per device).
hla_status static_ws_address(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        (void)cudaGetLastError();
        return HLA_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(g_static_ws_mutex);
    if (!g_static_ws_addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_ws) != cudaSuccess || !p) {
            (void)cudaGetLastError();
            return HLA_ERR_CUDA;
        }
        g_static_ws_addr[dev] = p;
    }
    *out = g_static_ws_addr[dev];
    return HLA_OK;
}
}  // namespace

hla_status hla_forward_static(hla_ctx* ctx, const void* Q, const void* K, const void* V, void* O, void* cuda_stream, void** scratch_out) {
    if (scratch_out) *scratch_out = nullptr;
    if (!ctx) return HLA_ERR_INVALID_ARG;
    if (ctx->ws_bytes > (size_t)HLA_STATIC_WS_BYTES) return HLA_ERR_WORKSPACE;    // this shape needs more scratch than the library carries
    void* ws = nullptr;
    const hla_status s = static_ws_address(&ws);
    if (s != HLA_OK) return s;
    if (scratch_out) *scratch_out = ws;
    // hla_forward clears the status words and writes every other region before reading it, so nothing
    // left by an earlier call is used.
    return hla_forward(ctx, Q, K, V, O, ws, (size_t)HLA_STATIC_WS_BYTES, cuda_stream);
}

hla_status hla_last_device_status(hla_ctx* ctx, const void* workspace, void* cuda_stream) {
    if (!ctx || !workspace) return HLA_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int32_t words[16] = {0};
    if (cudaMemcpyAsync(words, static_cast<const char*>(workspace) + ctx->L.status, sizeof(words), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return HLA_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return HLA_ERR_CUDA;
    return words[kStatusTimeout] != 0 ? HLA_ERR_DEVICE_TIMEOUT : HLA_OK;
}

hla_status hla_selftest_bounded_wait(hla_ctx* ctx, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!ctx || !workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return HLA_ERR_INVALID_ARG;
    if (workspace_bytes < ctx->ws_bytes) return HLA_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char* ws = static_cast<char*>(workspace);
    (void)cudaGetLastError();
    if (cudaMemsetAsync(ws + ctx->L.status, 0, 64, st) != cudaSuccess) return HLA_ERR_CUDA;
    tc::tc_wait_selftest_kernel<<<1, 32, 0, st>>>(reinterpret_cast<int*>(ws + ctx->L.status), 1000000ull);   // gives up after 1 ms
    return cudaPeekAtLastError() == cudaSuccess ? HLA_OK : HLA_ERR_CUDA;
}

int32_t hla_last_launch_count(const hla_ctx* ctx) { return ctx ? ctx->rec.launches : 0; }

hla_status hla_timing_enable(hla_ctx* ctx, int32_t on) {
    if (!ctx) return HLA_ERR_INVALID_ARG;
    ctx->rec.timing = on != 0;
    return HLA_OK;
}

int32_t hla_timing_collect(hla_ctx* ctx) { return ctx ? ctx->rec.collect() : 0; }

hla_status hla_timing_get(const hla_ctx* ctx, int32_t i, const char** name, double* total_ms, int64_t* launches) {
    if (!ctx || i < 0 || i >= (int32_t)ctx->rec.acc.size() || !name || !total_ms || !launches) return HLA_ERR_INVALID_ARG;
    *name = ctx->rec.acc[i].name;
    *total_ms = ctx->rec.acc[i].ms;
    *launches = ctx->rec.acc[i].n;
    return HLA_OK;
}

hla_status hla_destroy(hla_ctx* ctx) {
    if (!ctx) return HLA_ERR_INVALID_ARG;
    delete ctx;
    return HLA_OK;
}

const char* hla_status_string(hla_status s) {
    switch (s) {
        case HLA_OK: return "ok";
        case HLA_ERR_INVALID_ARG: return "invalid argument";
        case HLA_ERR_UNSUPPORTED: return "unsupported configuration";
        case HLA_ERR_WORKSPACE: return "workspace too small";
        case HLA_ERR_CUDA: return "CUDA error";
        case HLA_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
        case HLA_ERR_NO_MEMORY: return "out of host memory";
    }
    return "unknown status";
}

}  // extern "C"
