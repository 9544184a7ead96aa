"""Algorithmic work model of the HLA operator (FLOPs = 2 x multiply-adds, bytes
= tensors that must cross HBM once).

The counts are those of the paper's factored scheme (Theorem 4.2 and the
complexity paragraph of Section 4.3): per token and head, each contraction of a
P = d_phi**F feature vector against a [P, d+1] state (d value channels plus the
normaliser column) is 2*P*(d+1) FLOPs.  Work a particular kernel saves by
exploiting symmetry is NOT subtracted: throughput is always quoted on these
algorithmic counts.
"""
from __future__ import annotations


def n_features(F: int, d_phi: int) -> int:
    return d_phi ** F


def n_monomials(F: int, d_phi: int) -> int:
    """Distinct monomials of degree F in d_phi variables: what is left of the P features of the symmetric query
    tensor q (x) ... (x) q once equal index permutations are merged (56 of 216 for F = 3, d_phi = 6)."""
    from math import comb
    return comb(d_phi + F - 1, F)


def core_fwd_flops_per_token(d: int, F: int, d_phi: int) -> int:
    """State build + readout, each 2*P*(d+1)."""
    return 2 * 2 * n_features(F, d_phi) * (d + 1)


def core_bwd_flops_per_token(d: int, F: int, d_phi: int) -> int:
    """Four contractions of the same shape: dC/dz, dT_q, dV, dT_k."""
    return 4 * 2 * n_features(F, d_phi) * (d + 1)


def phi_fwd_flops_per_token(d: int, F: int, d_phi: int) -> int:
    """(1+F) feature maps, each Linear(d,d) + Linear(d,d_phi)."""
    return (1 + F) * 2 * d * (d + d_phi)


def phi_bwd_flops_per_token(d: int, F: int, d_phi: int) -> int:
    """Recompute the hidden layer, then the two transposed products (input gradient only)."""
    return (1 + F) * (2 * d * d + 2 * d * d_phi + 2 * d * d)


def fwd_flops_per_token(d, F, d_phi, with_phi=True):
    return core_fwd_flops_per_token(d, F, d_phi) + (phi_fwd_flops_per_token(d, F, d_phi) if with_phi else 0)


def bwd_flops_per_token(d, F, d_phi, with_phi=True):
    return core_bwd_flops_per_token(d, F, d_phi) + (phi_bwd_flops_per_token(d, F, d_phi) if with_phi else 0)


def fwd_bytes_per_token(d, F, d_phi, elt=2, with_phi=True):
    """V read + O write (+ Q, K read with phi); features only cross HBM when they are an input."""
    core = 2 * d * elt
    return core + 2 * d * elt if with_phi else core + (1 + F) * d_phi * 4


def bwd_bytes_per_token(d, F, d_phi, elt=2, with_phi=True):
    """dO, O, V read + dV write (+ Q, K read and dQ, dK write with phi)."""
    core = 4 * d * elt
    return core + 4 * d * elt if with_phi else core + 2 * (1 + F) * d_phi * 4


def paper_layer_flops(N: int, heads: int, d: int, F: int, d_phi: int) -> dict:
    """FLOPs of one whole HLA attention block as the paper's Table 3 counts them:
    q/k/v/o projections on D = heads*d channels, the six per-head MLPs (phi_q,
    F key maps, two value-modulation maps; first layers d->d, second layers
    d->d_phi for q/k and d->d for the value maps), and the operator core with
    P*d multiply-adds per contraction."""
    D = heads * d
    proj = 4 * 2 * N * D * D
    first = (1 + F + 2) * 2 * N * d * d * heads
    second = (1 + F) * 2 * N * d * d_phi * heads + 2 * 2 * N * d * d * heads
    core = 2 * 2 * N * n_features(F, d_phi) * d * heads
    return {"proj": proj, "mlp": first + second, "core": core, "total": proj + first + second + core}


def quadratic_layer_flops(N: int, heads: int, d: int) -> int:
    """Softmax-attention block as Table 3 counts it: projections + QK^T + AV."""
    D = heads * d
    return 4 * 2 * N * D * D + 4 * N * N * d * heads


def folded_flops_per_token(d: int, F: int, d_phi: int, backward: bool, with_phi: bool = True) -> int:
    """FLOPs the symmetry-folded scheme has to execute: every core contraction runs over the n_monomials(F, d_phi)
    merged features instead of P; the phi maps are unchanged.  Used for the roofline (what the hardware must do),
    never for the reported throughput (which stays on the algorithmic counts above)."""
    m = n_monomials(F, d_phi)
    core = 2 * 2 * m * (d + 1) + (4 * 2 * m * (d + 1) if backward else 0)
    phi = 0
    if with_phi:
        phi = phi_fwd_flops_per_token(d, F, d_phi) + (phi_bwd_flops_per_token(d, F, d_phi) if backward else 0)
    return core + phi


def value_mod_flops_per_token(d: int, backward: bool) -> int:
    """Value modulation T + phi_v1(T) (.) phi_v2(V): two maps of two d x d Linear layers each (Table 3 counts them in
    the layer total).  The backward adds the two transposed products per map; the recomputed forward is not counted."""
    fwd = 2 * (2 * d * d + 2 * d * d)
    return fwd + (2 * (2 * d * d + 2 * d * d) if backward else 0)
