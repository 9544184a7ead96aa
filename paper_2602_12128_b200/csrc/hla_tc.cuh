// Tensor-core (tcgen05 / TMEM / TMA) kernels of the HLA path.
#pragma once
#include "../../include/hla.h"
#include "hla_common.cuh"

namespace hla {
namespace tc {

constexpr int kTileTokens = 128;

struct Plan {
    size_t end;
};

inline bool supported(bool bf16, int d, int F, int dphi) {
    (void)bf16; (void)d; (void)F; (void)dphi;
    return false;
}

inline size_t plan(Plan& p, const Dims&, int, size_t off) {
    p.end = off;
    return off;
}

inline hla_status forward(const Plan&, const Dims&, int, bool, const hla_mlp*, const hla_mlp*, const void*, const void*, const void*,
                          void*, char*, const hla_ws_layout&, size_t, int, cudaStream_t, int*) {
    return HLA_ERR_UNSUPPORTED;
}

inline hla_status backward(const Plan&, const Dims&, int, bool, const hla_mlp*, const hla_mlp*, const void*, const void*, const void*,
                           const void*, const void*, void*, void*, void*, char*, const hla_ws_layout&, size_t, int, cudaStream_t, int*) {
    return HLA_ERR_UNSUPPORTED;
}

}  // namespace tc
}  // namespace hla
