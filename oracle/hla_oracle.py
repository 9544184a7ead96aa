"""fp64 CPU oracle for Hadamard Linear Attention (HLA).

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain reference the CUDA
library is checked against.  Only the tests, the smoke check and the CPU-baseline
leg of the benchmark may import it; the product path never does.  It shares no
code, tables or helpers with the CUDA sources and imports nothing from the
package.

Everything is numpy float64 and works on ONE head at a time:

    q      [N, d_phi]      query features  phi_q(q_i)            (>= 0 for the normaliser)
    ks     list of F arrays [N, d_phi]     key features phi_{k_f}(k_j)
    v      [N, d]          values
    o      [N, d]          attention output

Two independent forms of the same operator are implemented:

  * the literal quadratic definition (paper Eq. "hla", Section 4.1): the F
    similarity matrices are multiplied elementwise, rows are normalised, and the
    result multiplies V;
  * the factored linear-time scheme (Lemma 4.1, Theorem 4.2, the normaliser
    paragraph after it, and the 2-/3-factor einsum listings of the appendix):
    per-token outer-product tensors T_k, T_q, the context tensor C = T_k (x)_1 V,
    the key-side sum z, eta = T_q . z, and the readout T_q (x) C;

plus the sequential-update recurrence (Eq. "seq.updates") for the state, causal HLA
(Section 4.4) as the masked quadratic definition and as the sequential recurrence
with one output per token, analytic gradients in every form, and the feature networks phi of the appendix
("Defining phi": Linear - GELU - Linear - optional ReLU).

Readings of points the paper leaves open (the same readings the CUDA library
takes):
  * eps is added to the normaliser before dividing: o = num / (eta + eps)
    (the listings write `eta + eps`; the value of eps is not given - it is an argument here).
  * The division is applied to the contracted numerator; the listings divide the
    query outer products first, which is the same up to rounding.
  * eta_i = sum_j A_ij = T_q[i] . sum_j T_k[j]  (the listings' `sum_over_k`); the
    displayed formula for eta in the text is garbled.
  * In the theorem's proof the summed token index is the key/value index j.
  * The P = d_phi**F features of a token are flattened with the FIRST factor's
    index slowest (the listings' `bhsdef -> view(dp**3)`).
  * Causal HLA (Section 4.4): the text speaks of multiplying an n x n {0,1} matrix M "to the keys"; the sequential
    form it then gives (C^i holds tokens 1..i and is read by T_q^i) fixes the meaning: A_ij is kept for j <= i, the
    diagonal included, and the normaliser sums the kept entries.  Decay factors (a non-binary M) are cited, not
    defined, and are not implemented.
  * Value modulation (Section 4.5; appendix "Defining phi"): the text fixes T + phi_v1(T) (.) phi_v2(V), two
    Linear layers of width d with a GELU in between, no final activation, and says only that phi_v1, phi_v2 "use a
    LayerNorm".  Reading taken here: the LayerNorm acts on the input of each map (over the d channels of a
    token, biased variance, eps_ln = 1e-5, learnable scale and shift), i.e. phi_v(x) = W2^T GELU(W1^T LN(x) + b1) + b2.
    Where the LayerNorm sits is PARITY UNPINNED by the paper; the functions are pinned against pure-Python loops,
    closed forms and finite differences.
  * phi: exact (erf) GELU, both Linear layers have a bias, hidden width = d,
    ReLU applied at the end for phi_q and phi_k.  The figure defining phi is
    missing from the text, so the phi functions here are PARITY UNPINNED by the
    paper beyond that verbal description; they are pinned only against
    math.erf, a pure-Python loop version and finite differences.
"""
from __future__ import annotations

import numpy as np
from scipy.special import erf as _erf

F64 = np.float64


# --------------------------------------------------------------------------- #
# Feature networks phi (appendix "Defining phi"; Algorithm 1 step 4)
# --------------------------------------------------------------------------- #
def gelu_erf(x):
    """GELU(x) = x * Phi(x) with the exact normal CDF Phi(x) = (1 + erf(x / sqrt 2)) / 2."""
    x = np.asarray(x, dtype=F64)
    return 0.5 * x * (1.0 + _erf(x / np.sqrt(2.0)))


def gelu_erf_grad(x):
    """d/dx GELU(x) = Phi(x) + x * pdf(x)."""
    x = np.asarray(x, dtype=F64)
    cdf = 0.5 * (1.0 + _erf(x / np.sqrt(2.0)))
    pdf = np.exp(-0.5 * x * x) / np.sqrt(2.0 * np.pi)
    return cdf + x * pdf


def phi_mlp(x, W1, b1, W2, b2, relu=True):
    """Feature map of the appendix: two Linear layers with a GELU in between and
    a final ReLU (which the normaliser's non-negativity requirement needs).

    x [N, d];  W1 [d, d_hidden] (input index first), b1 [d_hidden];
    W2 [d_hidden, d_phi], b2 [d_phi].  Returns features [N, d_phi].
    """
    x = np.asarray(x, F64)
    h = x @ np.asarray(W1, F64) + np.asarray(b1, F64)       # first Linear
    g = gelu_erf(h)                                          # GELU
    p = g @ np.asarray(W2, F64) + np.asarray(b2, F64)       # second Linear
    return np.maximum(p, 0.0) if relu else p


def phi_mlp_backward(x, W1, b1, W2, b2, dfeat, relu=True):
    """Gradient of sum(dfeat * phi_mlp(x)) with respect to x (weights held fixed)."""
    x = np.asarray(x, F64)
    W1 = np.asarray(W1, F64)
    W2 = np.asarray(W2, F64)
    h = x @ W1 + np.asarray(b1, F64)
    g = gelu_erf(h)
    p = g @ W2 + np.asarray(b2, F64)
    dp = np.asarray(dfeat, F64) * (p > 0.0) if relu else np.asarray(dfeat, F64)
    dg = dp @ W2.T
    dh = dg * gelu_erf_grad(h)
    return dh @ W1.T


def phi_mlp_backward_weights(x, W1, b1, W2, b2, dfeat, relu=True):
    """Gradients of sum(dfeat * phi_mlp(x)) with respect to the weights of the map, summed over the
    tokens (Section 5, "Training Details": the phi networks are trained).  Returns (dW1, db1, dW2, db2)
    with the shapes of W1, b1, W2, b2."""
    x = np.asarray(x, F64)
    W1 = np.asarray(W1, F64)
    W2 = np.asarray(W2, F64)
    h = x @ W1 + np.asarray(b1, F64)
    g = gelu_erf(h)
    p = g @ W2 + np.asarray(b2, F64)
    dp = np.asarray(dfeat, F64) * (p > 0.0) if relu else np.asarray(dfeat, F64)
    dW2 = g.T @ dp                          # second Linear: p = g W2 + b2
    db2 = dp.sum(axis=0)
    dh = (dp @ W2.T) * gelu_erf_grad(h)
    dW1 = x.T @ dh                          # first Linear: h = x W1 + b1
    db1 = dh.sum(axis=0)
    return dW1, db1, dW2, db2


# --------------------------------------------------------------------------- #
# Outer-product tensors T_q, T_k (paragraph before Theorem 4.2)
# --------------------------------------------------------------------------- #
def outer_features(vectors):
    """[T]_j = vectors[0][j] (x) vectors[1][j] (x) ... flattened to [N, d_phi**F],
    first factor's index slowest."""
    t = np.asarray(vectors[0], F64)
    n = t.shape[0]
    for r in vectors[1:]:
        r = np.asarray(r, F64)
        t = np.einsum("np,ne->npe", t, r).reshape(n, -1)
    return t


# --------------------------------------------------------------------------- #
# Form 1: the literal quadratic definition (Eq. "hla")
# --------------------------------------------------------------------------- #
def similarity_matrices(q, ks):
    """s^f = phi_q(Q) phi_{k_f}(K)^T, one N x N matrix per factor."""
    q = np.asarray(q, F64)
    return [q @ np.asarray(k, F64).T for k in ks]


def attention_matrix(q, ks):
    """A = s^1 (.) s^2 (.) ... : the Hadamard product of the F similarity matrices."""
    s = similarity_matrices(q, ks)
    A = s[0].copy()
    for sf in s[1:]:
        A = A * sf
    return A


def hla_quadratic(q, ks, v, eps):
    """o_i = (sum_j A_ij v_j) / (sum_j A_ij + eps).  Returns (o, eta)."""
    A = attention_matrix(q, ks)
    eta = A.sum(axis=1)
    num = A @ np.asarray(v, F64)
    return num / (eta + eps)[:, None], eta


def hla_quadratic_rows(q_rows, ks, v, eps):
    """The definition evaluated for a subset of query rows only (the definition is
    separable over query rows).  q_rows [m, d_phi]."""
    return hla_quadratic(q_rows, ks, v, eps)


# --------------------------------------------------------------------------- #
# Form 2: the factored linear-time scheme (Theorem 4.2 + listings)
# --------------------------------------------------------------------------- #
def context_state(ks, v):
    """C = T_k (x)_1 V  in  R^{P x d}  and  z = sum_j [T_k]_j  in R^P."""
    Tk = outer_features(ks)
    C = np.einsum("jp,jg->pg", Tk, np.asarray(v, F64))
    z = Tk.sum(axis=0)
    return C, z


def context_state_streaming(ks, v):
    """The same state by the sequential update C^i = C^{i-1} + T_{k_i} (x) v_i."""
    Tk = outer_features(ks)
    v = np.asarray(v, F64)
    C = np.zeros((Tk.shape[1], v.shape[1]), F64)
    z = np.zeros(Tk.shape[1], F64)
    for i in range(Tk.shape[0]):
        C = C + np.multiply.outer(Tk[i], v[i])
        z = z + Tk[i]
    return C, z


def readout(q, F, C, z, eps):
    """o = (T_q (x) C) / (T_q . z + eps).  Returns (o, eta)."""
    Tq = outer_features([q] * F)
    eta = Tq @ z
    num = Tq @ C
    return num / (eta + eps)[:, None], eta


def hla_factored(q, ks, v, eps):
    """Linear-time HLA: state build then query readout.  Returns (o, eta, C, z)."""
    C, z = context_state(ks, v)
    o, eta = readout(q, len(ks), C, z, eps)
    return o, eta, C, z


# --------------------------------------------------------------------------- #
# Gradients (the paper trains through the operator; the formulas below are the
# derivatives of the two forms above)
# --------------------------------------------------------------------------- #
def hla_quadratic_backward(q, ks, v, do, eps):
    """Gradients of L = sum(do * o) through the quadratic form.
    Returns (dq [N,d_phi], dks list of [N,d_phi], dv [N,d])."""
    q = np.asarray(q, F64)
    ks = [np.asarray(k, F64) for k in ks]
    v = np.asarray(v, F64)
    do = np.asarray(do, F64)
    s = similarity_matrices(q, ks)
    A = attention_matrix(q, ks)
    eta = A.sum(axis=1)
    r = 1.0 / (eta + eps)
    o = (A @ v) * r[:, None]
    # dL/dA_ij = r_i * do_i . (v_j - o_i)
    dA = r[:, None] * (do @ v.T - np.sum(do * o, axis=1)[:, None])
    dv = (A * r[:, None]).T @ do
    dq = np.zeros_like(q)
    dks = []
    for f in range(len(ks)):
        others = np.ones_like(A)
        for f2 in range(len(ks)):
            if f2 != f:
                others = others * s[f2]
        ds = dA * others                      # dL/ds^f_ij
        dq += ds @ ks[f]
        dks.append(ds.T @ q)
    return dq, dks, dv


def _slot_contract(dT, vectors, slot):
    """sum over all tensor indices except `slot` of dT[j, i_1..i_F] * prod_{f != slot} vectors[f][j, i_f].
    dT is [N, d_phi**F] (first factor slowest); returns [N, d_phi]."""
    Fn = len(vectors)
    n, dphi = vectors[0].shape
    letters = "abcdefgh"[:Fn]
    t = dT.reshape((n,) + (dphi,) * Fn)
    operands = [t]
    subs = ["n" + letters]
    for f in range(Fn):
        if f != slot:
            operands.append(np.asarray(vectors[f], F64))
            subs.append("n" + letters[f])
    return np.einsum(",".join(subs) + "->n" + letters[slot], *operands)


def hla_factored_backward(q, ks, v, do, eps):
    """Gradients of L = sum(do * o) through the factored form (two passes:
    one over the queries that also reduces dC, dz; one over the keys).
    Returns (dq, dks, dv)."""
    q = np.asarray(q, F64)
    ks = [np.asarray(k, F64) for k in ks]
    v = np.asarray(v, F64)
    do = np.asarray(do, F64)
    Fn = len(ks)
    Tk = outer_features(ks)
    Tq = outer_features([q] * Fn)
    C = Tk.T @ v
    z = Tk.sum(axis=0)
    eta = Tq @ z
    r = 1.0 / (eta + eps)
    o = (Tq @ C) * r[:, None]
    dnum = do * r[:, None]
    deta = -r * np.sum(do * o, axis=1)
    # pass over the queries
    dC = Tq.T @ dnum
    dz = Tq.T @ deta
    dTq = dnum @ C.T + np.multiply.outer(deta, z)
    dq = np.zeros_like(q)
    for slot in range(Fn):                    # the same vector sits in every slot of T_q
        dq += _slot_contract(dTq, [q] * Fn, slot)
    # pass over the keys
    dv = Tk @ dC
    dTk = v @ dC.T + dz[None, :]
    dks = [_slot_contract(dTk, ks, f) for f in range(Fn)]
    return dq, dks, dv


# --------------------------------------------------------------------------- #
# Causal HLA (Section 4.4 "Causal Attention, Decay Factors and Sequential
# Updates", Eq. "seq.updates")
# --------------------------------------------------------------------------- #
def causal_mask(n):
    """M in {0,1}^{n x n}: token i sees tokens j <= i (itself included)."""
    return np.tril(np.ones((n, n), F64))


def hla_quadratic_causal(q, ks, v, eps):
    """The definition with the {0,1} mask applied to the Hadamard product:
    A_ij = M_ij prod_f s^f_ij,  o_i = (sum_j A_ij v_j) / (sum_j A_ij + eps).  Returns (o, eta)."""
    A = attention_matrix(q, ks) * causal_mask(np.asarray(q).shape[0])
    eta = A.sum(axis=1)
    num = A @ np.asarray(v, F64)
    return num / (eta + eps)[:, None], eta


def hla_streaming(q, ks, v, eps):
    """Sequential updates: at token i the context tensor takes C^i = C^{i-1} + T_{k_i} (x) v_i (and the key-side sum
    z^i = z^{i-1} + T_{k_i}), and the output of that token is the product of T_q^i with C^i, normalised by
    T_q^i . z^i + eps.  Returns (o, eta)."""
    Fn = len(ks)
    Tk = outer_features(ks)
    Tq = outer_features([q] * Fn)
    v = np.asarray(v, F64)
    n = Tk.shape[0]
    C = np.zeros((Tk.shape[1], v.shape[1]), F64)
    z = np.zeros(Tk.shape[1], F64)
    o = np.empty((n, v.shape[1]), F64)
    eta = np.empty(n, F64)
    for i in range(n):
        C = C + np.multiply.outer(Tk[i], v[i])
        z = z + Tk[i]
        eta[i] = Tq[i] @ z
        o[i] = (Tq[i] @ C) / (eta[i] + eps)
    return o, eta


def hla_quadratic_causal_backward(q, ks, v, do, eps):
    """Gradients of L = sum(do * o) through the masked quadratic form.  Returns (dq, dks, dv)."""
    q = np.asarray(q, F64)
    ks = [np.asarray(k, F64) for k in ks]
    v = np.asarray(v, F64)
    do = np.asarray(do, F64)
    M = causal_mask(q.shape[0])
    s = similarity_matrices(q, ks)
    A = attention_matrix(q, ks) * M
    eta = A.sum(axis=1)
    r = 1.0 / (eta + eps)
    o = (A @ v) * r[:, None]
    # dL/dA_ij = r_i * do_i . (v_j - o_i) where the mask lets A_ij vary, 0 elsewhere
    dA = M * (r[:, None] * (do @ v.T - np.sum(do * o, axis=1)[:, None]))
    dv = (A * r[:, None]).T @ do
    dq = np.zeros_like(q)
    dks = []
    for f in range(len(ks)):
        others = np.ones_like(A)
        for f2 in range(len(ks)):
            if f2 != f:
                others = others * s[f2]
        ds = dA * others
        dq += ds @ ks[f]
        dks.append(ds.T @ q)
    return dq, dks, dv


def hla_streaming_backward(q, ks, v, do, eps):
    """Gradients of L = sum(do * o) through the sequential form: a forward sweep that carries C^i, z^i for the
    query-side gradients, and a reverse sweep that carries the gradient of the state (token j's key tensor enters
    every C^i with i >= j, so it collects dC^j = sum_{i >= j} T_q^i (x) dnum_i).  Returns (dq, dks, dv)."""
    q = np.asarray(q, F64)
    ks = [np.asarray(k, F64) for k in ks]
    v = np.asarray(v, F64)
    do = np.asarray(do, F64)
    Fn = len(ks)
    Tk = outer_features(ks)
    Tq = outer_features([q] * Fn)
    n, P = Tk.shape
    C = np.zeros((P, v.shape[1]), F64)
    z = np.zeros(P, F64)
    dTq = np.empty((n, P), F64)
    dnum = np.empty_like(v)
    deta = np.empty(n, F64)
    for i in range(n):
        C = C + np.multiply.outer(Tk[i], v[i])
        z = z + Tk[i]
        r = 1.0 / (Tq[i] @ z + eps)
        o = (Tq[i] @ C) * r
        dnum[i] = do[i] * r
        deta[i] = -r * (do[i] @ o)
        dTq[i] = C @ dnum[i] + deta[i] * z
    dC = np.zeros_like(C)
    dz = np.zeros(P, F64)
    dTk = np.empty((n, P), F64)
    dv = np.empty_like(v)
    for i in range(n - 1, -1, -1):
        dC = dC + np.multiply.outer(Tq[i], dnum[i])
        dz = dz + deta[i] * Tq[i]
        dv[i] = Tk[i] @ dC
        dTk[i] = dC @ v[i] + dz
    dq = np.zeros_like(q)
    for slot in range(Fn):
        dq += _slot_contract(dTq, [q] * Fn, slot)
    dks = [_slot_contract(dTk, ks, f) for f in range(Fn)]
    return dq, dks, dv


_FORWARD_FORMS = {
    "quadratic": lambda q, ks, v, eps: hla_quadratic(q, ks, v, eps),
    "factored": lambda q, ks, v, eps: hla_factored(q, ks, v, eps)[:2],
    "causal_quadratic": lambda q, ks, v, eps: hla_quadratic_causal(q, ks, v, eps),
    "causal_streaming": lambda q, ks, v, eps: hla_streaming(q, ks, v, eps),
}


def _backward_form(form):
    return {"quadratic": hla_quadratic_backward, "factored": hla_factored_backward,
            "causal_quadratic": hla_quadratic_causal_backward,
            "causal_streaming": hla_streaming_backward}[form]


# --------------------------------------------------------------------------- #
# Whole-operator wrappers over [B, H, N, *] tensors (Algorithm 1 steps 4-5)
# --------------------------------------------------------------------------- #
def hla_core_forward(qf, kf, V, eps, form="factored"):
    """qf [B,H,N,d_phi], kf [B,H,F,N,d_phi], V [B,H,N,d] -> (O [B,H,N,d], eta [B,H,N]).
    form: "factored" | "quadratic" (all tokens see all tokens), "causal_quadratic" | "causal_streaming"."""
    B, H, N, _ = qf.shape
    Fn = kf.shape[2]
    O = np.empty(V.shape, F64)
    ETA = np.empty((B, H, N), F64)
    for b in range(B):
        for h in range(H):
            ks = [kf[b, h, f] for f in range(Fn)]
            o, eta = _FORWARD_FORMS[form](qf[b, h], ks, V[b, h], eps)
            O[b, h] = o
            ETA[b, h] = eta
    return O, ETA


def hla_core_backward(qf, kf, V, dO, eps, form="factored"):
    """Gradients of sum(dO * O) w.r.t. qf, kf, V (same shapes as the inputs)."""
    B, H, N, _ = qf.shape
    Fn = kf.shape[2]
    dqf = np.empty(qf.shape, F64)
    dkf = np.empty(kf.shape, F64)
    dV = np.empty(V.shape, F64)
    fn = _backward_form(form)
    for b in range(B):
        for h in range(H):
            ks = [kf[b, h, f] for f in range(Fn)]
            dq, dks, dv = fn(qf[b, h], ks, V[b, h], dO[b, h], eps)
            dqf[b, h] = dq
            for f in range(Fn):
                dkf[b, h, f] = dks[f]
            dV[b, h] = dv
    return dqf, dkf, dV


def phi_features(Q, K, phi_q, phi_k):
    """Algorithm 1 step 4: q <- hla_to_q(q); k_f <- hla_to_k_f(k), one weight set
    per map shared by all batches and heads.  phi_q = (W1,b1,W2,b2); phi_k = list of F such tuples.
    Q, K [B,H,N,d] -> qf [B,H,N,d_phi], kf [B,H,F,N,d_phi]."""
    B, H, N, d = Q.shape
    qf = phi_mlp(Q.reshape(-1, d), *phi_q).reshape(B, H, N, -1)
    kfs = [phi_mlp(K.reshape(-1, d), *w).reshape(B, H, N, -1) for w in phi_k]
    return qf, np.stack(kfs, axis=2)


def hla_forward(Q, K, V, phi_q, phi_k, eps, form="factored"):
    """Steps 4-5 of Algorithm 1 on raw per-head Q, K, V [B,H,N,d].
    Returns (O, eta, qf, kf)."""
    qf, kf = phi_features(Q, K, phi_q, phi_k)
    O, eta = hla_core_forward(qf, kf, V, eps, form)
    return O, eta, qf, kf


def hla_backward(Q, K, V, dO, phi_q, phi_k, eps, form="factored"):
    """Gradients of sum(dO * O) w.r.t. raw Q, K, V through phi and the core.
    Returns (dQ, dK, dV, dqf, dkf)."""
    B, H, N, d = Q.shape
    qf, kf = phi_features(Q, K, phi_q, phi_k)
    dqf, dkf, dV = hla_core_backward(qf, kf, V, dO, eps, form)
    dQ = phi_mlp_backward(Q.reshape(-1, d), *phi_q, dqf.reshape(-1, dqf.shape[-1])).reshape(Q.shape)
    dK = np.zeros(K.shape, F64)
    for f, w in enumerate(phi_k):             # the same K feeds every key map
        dK += phi_mlp_backward(K.reshape(-1, d), *w, dkf[:, :, f].reshape(-1, dkf.shape[-1])).reshape(K.shape)
    return dQ, dK, dV, dqf, dkf


def hla_backward_weights(Q, K, V, dO, phi_q, phi_k, eps, form="factored"):
    """Gradients of sum(dO * O) w.r.t. the weights of phi_q and of every phi_{k_f} (one weight set per
    map, shared by all batches and heads, so the per-token gradients are summed over B, H and N).
    Returns (gq, [gk_1, ...]), each a tuple (dW1, db1, dW2, db2)."""
    B, H, N, d = Q.shape
    qf, kf = phi_features(Q, K, phi_q, phi_k)
    dqf, dkf, _ = hla_core_backward(qf, kf, V, dO, eps, form)
    gq = phi_mlp_backward_weights(Q.reshape(-1, d), *phi_q, dqf.reshape(-1, dqf.shape[-1]))
    gk = [phi_mlp_backward_weights(K.reshape(-1, d), *w, dkf[:, :, f].reshape(-1, dkf.shape[-1])) for f, w in enumerate(phi_k)]
    return gq, gk


# --------------------------------------------------------------------------- #
# Value modulation (Section 4.5 "Value Modulation"; appendix "Defining phi")
# --------------------------------------------------------------------------- #
LN_EPS = 1e-5


def layer_norm(x, gamma, beta, eps=LN_EPS):
    """LayerNorm over the last axis: (x - mean) / sqrt(var + eps) * gamma + beta, biased variance."""
    x = np.asarray(x, F64)
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    return (x - mu) / np.sqrt(var + eps) * np.asarray(gamma, F64) + np.asarray(beta, F64)


def phi_v_mlp(x, ln_g, ln_b, W1, b1, W2, b2):
    """One value-modulation map: LayerNorm, Linear(d, d), GELU, Linear(d, d); no final activation.
    x [N, d]; W1, W2 [d, d] (input index first)."""
    xn = layer_norm(x, ln_g, ln_b)
    return gelu_erf(xn @ np.asarray(W1, F64) + np.asarray(b1, F64)) @ np.asarray(W2, F64) + np.asarray(b2, F64)


def phi_v_mlp_backward(x, ln_g, ln_b, W1, b1, W2, b2, dy):
    """Gradient of sum(dy * phi_v_mlp(x)) with respect to x (weights held fixed)."""
    x = np.asarray(x, F64)
    W1 = np.asarray(W1, F64)
    W2 = np.asarray(W2, F64)
    g_ = np.asarray(ln_g, F64)
    d = x.shape[-1]
    mu = x.mean(axis=-1, keepdims=True)
    rstd = 1.0 / np.sqrt(((x - mu) ** 2).mean(axis=-1, keepdims=True) + LN_EPS)
    xhat = (x - mu) * rstd
    h = (xhat * g_ + np.asarray(ln_b, F64)) @ W1 + np.asarray(b1, F64)
    dh = (np.asarray(dy, F64) @ W2.T) * gelu_erf_grad(h)
    dxhat = (dh @ W1.T) * g_
    # LayerNorm: xhat depends on every channel of its token through the mean and the variance
    return rstd * (dxhat - dxhat.mean(axis=-1, keepdims=True) - xhat * (dxhat * xhat).mean(axis=-1, keepdims=True))


def value_modulation(T, V, v1, v2):
    """T + phi_v1(T) (.) phi_v2(V) for one head: T (the attention result A V), V [N, d]; v1, v2 = (ln_g, ln_b, W1, b1, W2, b2)."""
    return np.asarray(T, F64) + phi_v_mlp(T, *v1) * phi_v_mlp(V, *v2)


def value_modulation_backward(T, V, dOut, v1, v2):
    """Gradients of sum(dOut * value_modulation(T, V)) with respect to T and V."""
    dOut = np.asarray(dOut, F64)
    y1, y2 = phi_v_mlp(T, *v1), phi_v_mlp(V, *v2)
    dT = dOut + phi_v_mlp_backward(T, *v1, dOut * y2)
    dV = phi_v_mlp_backward(V, *v2, dOut * y1)
    return dT, dV
