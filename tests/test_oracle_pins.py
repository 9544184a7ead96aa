"""Pins for the fp64 oracle: every check compares it with something other than
itself - the paper's identities, closed forms, brute force in pure Python,
textbook special cases, finite differences, and the FLOP counts the paper prints."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import hla_oracle as orc
from paper_2602_12128_b200 import flops

RNG = np.random.default_rng(1234)


def feats(n, dphi, F, rng=RNG):
    q = np.abs(rng.standard_normal((n, dphi)))
    ks = [np.abs(rng.standard_normal((n, dphi))) for _ in range(F)]
    return q, ks


# ---- Lemma 4.1 --------------------------------------------------------------
@pytest.mark.parametrize("F", [1, 2, 3, 4])
def test_lemma_4_1_outer_products(F):
    """prod_f (q . r^f) == sum over all entries of (q x..x q) (.) (r^1 x..x r^F)."""
    dphi = 5
    q = RNG.standard_normal((7, dphi))
    rs = [RNG.standard_normal((7, dphi)) for _ in range(F)]
    lhs = np.ones(7)
    for r in rs:
        lhs *= np.sum(q * r, axis=1)
    rhs = np.sum(orc.outer_features([q] * F) * orc.outer_features(rs), axis=1)
    np.testing.assert_allclose(rhs, lhs, rtol=1e-12, atol=1e-13)


def test_outer_features_index_order():
    """First factor's index is the slowest one in the flattened feature axis."""
    a = np.array([[1.0, 10.0]])
    b = np.array([[2.0, 3.0]])
    c = np.array([[5.0, 7.0]])
    t = orc.outer_features([a, b, c])[0]
    want = [a[0, i] * b[0, j] * c[0, k] for i in range(2) for j in range(2) for k in range(2)]
    np.testing.assert_allclose(t, want)


# ---- equality of the forms (Theorem 4.2, sequential updates) ------------------
@pytest.mark.parametrize("F,dphi", [(1, 8), (2, 12), (3, 6), (2, 3)])
def test_quadratic_equals_factored_equals_streaming(F, dphi):
    n, d = 37, 9
    q, ks = feats(n, dphi, F)
    v = RNG.standard_normal((n, d))
    eps = 1e-6
    o1, eta1 = orc.hla_quadratic(q, ks, v, eps)
    o2, eta2, C, z = orc.hla_factored(q, ks, v, eps)
    Cs, zs = orc.context_state_streaming(ks, v)
    np.testing.assert_allclose(o2, o1, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(eta2, eta1, rtol=1e-12)
    np.testing.assert_allclose(Cs, C, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(zs, z, rtol=1e-12)
    assert C.shape == (dphi ** F, d)


# ---- brute force in pure Python -----------------------------------------------
def brute_force(q, ks, v, eps):
    n, d = len(v), len(v[0])
    out = [[0.0] * d for _ in range(n)]
    for i in range(n):
        w = []
        for j in range(n):
            a = 1.0
            for k in ks:
                a *= sum(q[i][t] * k[j][t] for t in range(len(q[i])))
            w.append(a)
        eta = sum(w)
        for g in range(d):
            out[i][g] = sum(w[j] * v[j][g] for j in range(n)) / (eta + eps)
    return np.array(out)


@pytest.mark.parametrize("F", [2, 3])
def test_brute_force_tiny(F):
    n, dphi, d = 6, 3, 4
    q, ks = feats(n, dphi, F)
    v = RNG.standard_normal((n, d))
    want = brute_force(q.tolist(), [k.tolist() for k in ks], v.tolist(), 1e-3)
    np.testing.assert_allclose(orc.hla_quadratic(q, ks, v, 1e-3)[0], want, rtol=1e-12)
    np.testing.assert_allclose(orc.hla_factored(q, ks, v, 1e-3)[0], want, rtol=1e-11)


def test_brute_force_state_entries():
    """C[(a,b,c), g] = sum_j k1_j[a] k2_j[b] k3_j[c] v_j[g] by explicit loops."""
    n, dphi, d = 5, 3, 2
    _, ks = feats(n, dphi, 3)
    v = RNG.standard_normal((n, d))
    C, z = orc.context_state(ks, v)
    for a, b, c in itertools.product(range(dphi), repeat=3):
        p = (a * dphi + b) * dphi + c
        zz = sum(ks[0][j, a] * ks[1][j, b] * ks[2][j, c] for j in range(n))
        assert abs(z[p] - zz) < 1e-12
        for g in range(d):
            cc = sum(ks[0][j, a] * ks[1][j, b] * ks[2][j, c] * v[j, g] for j in range(n))
            assert abs(C[p, g] - cc) < 1e-12


def test_one_hot_features_group_mean():
    """With one-hot features A is a 0/1 matrix and o_i is the mean of V over the
    keys that share the query's class in every factor."""
    n, dphi, d = 12, 3, 5
    cls_q = RNG.integers(0, dphi, n)
    cls_k = [RNG.integers(0, dphi, n) for _ in range(3)]
    eye = np.eye(dphi)
    q = eye[cls_q]
    ks = [eye[c] for c in cls_k]
    v = RNG.standard_normal((n, d))
    o, eta = orc.hla_factored(q, ks, v, 0.0 + 1e-300)[:2]
    for i in range(n):
        members = [j for j in range(n) if all(c[j] == cls_q[i] for c in cls_k)]
        assert eta[i] == len(members)
        if members:
            np.testing.assert_allclose(o[i], v[members].mean(axis=0), rtol=1e-12, atol=1e-14)


# ---- special cases ---------------------------------------------------------------
def test_F1_is_normalised_linear_attention():
    n, dphi, d = 50, 8, 6
    q, ks = feats(n, dphi, 1)
    v = RNG.standard_normal((n, d))
    want = (q @ (ks[0].T @ v)) / (q @ ks[0].sum(axis=0))[:, None]       # phi(Q)(phi(K)^T V) / (phi(Q) . sum phi(K))
    np.testing.assert_allclose(orc.hla_factored(q, ks, v, 0.0)[0], want, rtol=1e-12)
    np.testing.assert_allclose(orc.hla_quadratic(q, ks, v, 0.0)[0], want, rtol=1e-12)


@pytest.mark.parametrize("F", [2, 3])
def test_equal_key_maps_give_elementwise_power(F):
    n, dphi = 20, 4
    q, ks = feats(n, dphi, 1)
    A = orc.attention_matrix(q, ks * F)
    np.testing.assert_allclose(A, (q @ ks[0].T) ** F, rtol=1e-12)


def test_rank_bound():
    """rank(A) <= min(N, d_phi^F) (rank relaxation paragraph)."""
    n, dphi, F = 40, 2, 3
    q, ks = feats(n, dphi, F)
    A = orc.attention_matrix(q, ks)
    assert np.linalg.matrix_rank(A, tol=1e-9) <= dphi ** F


# ---- normaliser invariants ----------------------------------------------------------
def test_rows_sum_to_one_and_convexity():
    n, dphi, d, F = 33, 6, 7, 3
    q, ks = feats(n, dphi, F)
    eps = 1e-6
    ones = np.ones((n, d))
    o, eta = orc.hla_factored(q, ks, ones, eps)[:2]
    np.testing.assert_allclose(o, np.repeat((eta / (eta + eps))[:, None], d, 1), rtol=1e-12)
    v = RNG.standard_normal((n, d))
    o = orc.hla_factored(q, ks, v, 0.0)[0]
    assert np.all(o <= v.max(axis=0) + 1e-12) and np.all(o >= v.min(axis=0) - 1e-12)
    W = orc.attention_matrix(q, ks)
    W = W / W.sum(axis=1, keepdims=True)
    np.testing.assert_allclose(W.sum(axis=1), 1.0, rtol=1e-13)
    np.testing.assert_allclose(W @ v, o, rtol=1e-10, atol=1e-13)


def test_symmetries():
    n, dphi, d, F = 21, 4, 5, 3
    q, ks = feats(n, dphi, F)
    v = RNG.standard_normal((n, d))
    o = orc.hla_factored(q, ks, v, 0.0)[0]
    perm = RNG.permutation(n)
    np.testing.assert_allclose(orc.hla_factored(q, [k[perm] for k in ks], v[perm], 0.0)[0], o, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(orc.hla_factored(q[perm], ks, v, 0.0)[0], o[perm], rtol=1e-12)
    scale = np.abs(RNG.standard_normal((n, 1))) + 0.5
    np.testing.assert_allclose(orc.hla_factored(q * scale, ks, v, 0.0)[0], o, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(orc.hla_factored(q, [ks[0], 3.0 * ks[1], ks[2]], v, 0.0)[0], o, rtol=1e-11, atol=1e-13)


# ---- gradients -------------------------------------------------------------------------
def fd_grad(fun, x, h=1e-6):
    g = np.zeros_like(x)
    it = np.nditer(x, flags=["multi_index"])
    for _ in it:
        idx = it.multi_index
        xp = x.copy(); xp[idx] += h
        xm = x.copy(); xm[idx] -= h
        g[idx] = (fun(xp) - fun(xm)) / (2 * h)
    return g


@pytest.mark.parametrize("F,dphi", [(2, 3), (3, 3), (3, 2)])
@pytest.mark.parametrize("form", ["quadratic", "factored"])
def test_core_gradients_finite_differences(F, dphi, form):
    n, d = 9, 4
    rng = np.random.default_rng(7)
    q = np.abs(rng.standard_normal((n, dphi))) + 0.1
    ks = [np.abs(rng.standard_normal((n, dphi))) + 0.1 for _ in range(F)]
    v = rng.standard_normal((n, d))
    do = rng.standard_normal((n, d))
    eps = 1e-2
    bw = orc.hla_quadratic_backward if form == "quadratic" else orc.hla_factored_backward
    dq, dks, dv = bw(q, ks, v, do, eps)

    def loss(q_=q, ks_=ks, v_=v):
        return float(np.sum(do * orc.hla_quadratic(q_, ks_, v_, eps)[0]))

    np.testing.assert_allclose(dq, fd_grad(lambda x: loss(q_=x), q), rtol=1e-6, atol=1e-8)
    np.testing.assert_allclose(dv, fd_grad(lambda x: loss(v_=x), v), rtol=1e-6, atol=1e-8)
    for f in range(F):
        def lf(x, f=f):
            kk = list(ks); kk[f] = x
            return loss(ks_=kk)
        np.testing.assert_allclose(dks[f], fd_grad(lf, ks[f]), rtol=1e-6, atol=1e-8)


def test_backward_forms_agree_and_scale_identities():
    n, dphi, d, F = 40, 6, 8, 3
    q, ks = feats(n, dphi, F)
    v = RNG.standard_normal((n, d))
    do = RNG.standard_normal((n, d))
    g1 = orc.hla_quadratic_backward(q, ks, v, do, 0.0)
    g2 = orc.hla_factored_backward(q, ks, v, do, 0.0)
    np.testing.assert_allclose(g2[0], g1[0], rtol=1e-9, atol=1e-12)
    np.testing.assert_allclose(g2[2], g1[2], rtol=1e-9, atol=1e-12)
    for f in range(F):
        np.testing.assert_allclose(g2[1][f], g1[1][f], rtol=1e-9, atol=1e-12)
    # o is invariant to rescaling a query or a whole key map (eps = 0) -> Euler identities
    np.testing.assert_allclose(np.sum(q * g1[0], axis=1), 0.0, atol=1e-10)
    for f in range(F):
        assert abs(np.sum(ks[f] * g1[1][f])) < 1e-9
    # rows of the normalised weights sum to one -> sum_j dV_j = sum_i dO_i
    np.testing.assert_allclose(g1[2].sum(axis=0), do.sum(axis=0), rtol=1e-10)


# ---- causal HLA (Section 4.4, Eq. "seq.updates") -------------------------------------------
def brute_force_causal(q, ks, v, eps):
    """Token i averages the values of tokens 0..i with weights prod_f (q_i . k^f_j): plain loops."""
    n, d = len(v), len(v[0])
    out = [[0.0] * d for _ in range(n)]
    etas = [0.0] * n
    for i in range(n):
        w = []
        for j in range(i + 1):
            a = 1.0
            for k in ks:
                a *= sum(q[i][t] * k[j][t] for t in range(len(q[i])))
            w.append(a)
        etas[i] = sum(w)
        for g in range(d):
            out[i][g] = sum(w[j] * v[j][g] for j in range(i + 1)) / (etas[i] + eps)
    return np.array(out), np.array(etas)


@pytest.mark.parametrize("F,dphi", [(1, 5), (2, 4), (3, 3), (2, 12), (3, 6)])
def test_causal_quadratic_equals_streaming_equals_brute_force(F, dphi):
    n, d = 11, 5
    rng = np.random.default_rng(100 + F)
    q, ks = feats(n, dphi, F, rng)
    v = rng.standard_normal((n, d))
    want_o, want_eta = brute_force_causal(q.tolist(), [k.tolist() for k in ks], v.tolist(), 1e-3)
    oq, eq = orc.hla_quadratic_causal(q, ks, v, 1e-3)
    os_, es = orc.hla_streaming(q, ks, v, 1e-3)
    np.testing.assert_allclose(oq, want_o, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(eq, want_eta, rtol=1e-12)
    np.testing.assert_allclose(os_, want_o, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(es, want_eta, rtol=1e-11)


def test_causal_special_cases():
    """What the mask fixes without any arithmetic of the oracle's own: the first token returns its own value,
    the last token's output is the unmasked operator's last row, a prefix of the sequence gives a prefix of the
    output (no token sees the future), and F = 1 is causal normalised linear attention by cumulative sums."""
    n, dphi, d, F = 17, 4, 6, 3
    rng = np.random.default_rng(5)
    q, ks = feats(n, dphi, F, rng)
    v = rng.standard_normal((n, d))
    for fn in (orc.hla_quadratic_causal, orc.hla_streaming):
        o, eta = fn(q, ks, v, 0.0)
        np.testing.assert_allclose(o[0], v[0], rtol=1e-12)
        np.testing.assert_allclose(o[-1], orc.hla_quadratic(q, ks, v, 0.0)[0][-1], rtol=1e-11)
        o_pre, eta_pre = fn(q[:9], [k[:9] for k in ks], v[:9], 0.0)
        np.testing.assert_allclose(o[:9], o_pre, rtol=1e-12)
        np.testing.assert_allclose(eta[:9], eta_pre, rtol=1e-12)
        # changing a later token leaves earlier outputs alone
        v2 = v.copy(); v2[12] += 3.0
        k2 = [k.copy() for k in ks]; k2[1][12] *= 2.0
        o2, _ = fn(q, k2, v2, 0.0)
        np.testing.assert_array_equal(o2[:12], o[:12])
        assert np.abs(o2[12:] - o[12:]).max() > 1e-3
    # F = 1: o_i = q_i . cumsum_j (k_j v_j^T) / q_i . cumsum_j k_j
    S = np.cumsum(ks[0][:, :, None] * v[:, None, :], axis=0)
    zc = np.cumsum(ks[0], axis=0)
    want = np.einsum("np,npg->ng", q, S) / np.einsum("np,np->n", q, zc)[:, None]
    np.testing.assert_allclose(orc.hla_quadratic_causal(q, ks[:1], v, 0.0)[0], want, rtol=1e-11)
    np.testing.assert_allclose(orc.hla_streaming(q, ks[:1], v, 0.0)[0], want, rtol=1e-11)
    # constant values: every (causal) convex combination returns the constant
    vc = np.tile(rng.standard_normal(d), (n, 1))
    np.testing.assert_allclose(orc.hla_streaming(q, ks, vc, 0.0)[0], vc, rtol=1e-11)


@pytest.mark.parametrize("F,dphi", [(1, 4), (2, 3), (3, 3)])
@pytest.mark.parametrize("form", ["causal_quadratic", "causal_streaming"])
def test_causal_gradients_finite_differences(F, dphi, form):
    n, d = 8, 3
    rng = np.random.default_rng(11)
    q = np.abs(rng.standard_normal((n, dphi))) + 0.1
    ks = [np.abs(rng.standard_normal((n, dphi))) + 0.1 for _ in range(F)]
    v = rng.standard_normal((n, d))
    do = rng.standard_normal((n, d))
    eps = 1e-2
    bw = orc.hla_quadratic_causal_backward if form == "causal_quadratic" else orc.hla_streaming_backward
    dq, dks, dv = bw(q, ks, v, do, eps)

    def loss(q_=q, ks_=ks, v_=v):
        # the loss is evaluated by the pure-Python loops, not by the function under test
        o, _ = brute_force_causal(q_.tolist(), [k.tolist() for k in ks_], v_.tolist(), eps)
        return float(np.sum(do * o))

    np.testing.assert_allclose(dq, fd_grad(lambda x: loss(q_=x), q), rtol=1e-6, atol=1e-8)
    np.testing.assert_allclose(dv, fd_grad(lambda x: loss(v_=x), v), rtol=1e-6, atol=1e-8)
    for f in range(F):
        def lf(x, f=f):
            kk = list(ks); kk[f] = x
            return loss(ks_=kk)
        np.testing.assert_allclose(dks[f], fd_grad(lf, ks[f]), rtol=1e-6, atol=1e-8)


def test_causal_backward_forms_agree_and_identities():
    n, dphi, d, F = 37, 6, 8, 3
    rng = np.random.default_rng(12)
    q, ks = feats(n, dphi, F, rng)
    v = rng.standard_normal((n, d))
    do = rng.standard_normal((n, d))
    g1 = orc.hla_quadratic_causal_backward(q, ks, v, do, 0.0)
    g2 = orc.hla_streaming_backward(q, ks, v, do, 0.0)
    np.testing.assert_allclose(g2[0], g1[0], rtol=1e-9, atol=1e-12)
    np.testing.assert_allclose(g2[2], g1[2], rtol=1e-9, atol=1e-12)
    for f in range(F):
        np.testing.assert_allclose(g2[1][f], g1[1][f], rtol=1e-9, atol=1e-12)
    # scale invariance of every row (eps = 0) and rows summing to one, as without the mask
    np.testing.assert_allclose(np.sum(q * g1[0], axis=1), 0.0, atol=1e-10)
    for f in range(F):
        assert abs(np.sum(ks[f] * g1[1][f])) < 1e-9
    np.testing.assert_allclose(g1[2].sum(axis=0), do.sum(axis=0), rtol=1e-10)
    # the last token is seen only by itself: dv_last = do_last (its own weight is 1 after normalisation
    # only if it were alone; in general dv_last = A_nn / eta_n * do_n)
    A = orc.attention_matrix(q, ks)
    np.testing.assert_allclose(g1[2][-1], A[-1, -1] / np.tril(A)[-1].sum() * do[-1], rtol=1e-10)
    # the first query sees one token: o_0 = v_0 whatever q_0 is -> dq_0 = 0
    np.testing.assert_allclose(g1[0][0], 0.0, atol=1e-12)


def test_causal_wrappers_dispatch_per_head():
    rng = np.random.default_rng(13)
    B, H, N, dphi, d, F = 2, 2, 7, 3, 4, 3
    qf = np.abs(rng.standard_normal((B, H, N, dphi)))
    kf = np.abs(rng.standard_normal((B, H, F, N, dphi)))
    V = rng.standard_normal((B, H, N, d))
    dO = rng.standard_normal((B, H, N, d))
    O, eta = orc.hla_core_forward(qf, kf, V, 1e-3, "causal_streaming")
    dq, dk, dV = orc.hla_core_backward(qf, kf, V, dO, 1e-3, "causal_quadratic")
    for b in range(B):
        for h in range(H):
            ks = [kf[b, h, f] for f in range(F)]
            want, weta = brute_force_causal(qf[b, h].tolist(), [k.tolist() for k in ks], V[b, h].tolist(), 1e-3)
            np.testing.assert_allclose(O[b, h], want, rtol=1e-11)
            np.testing.assert_allclose(eta[b, h], weta, rtol=1e-11)
            g = orc.hla_streaming_backward(qf[b, h], ks, V[b, h], dO[b, h], 1e-3)
            np.testing.assert_allclose(dq[b, h], g[0], rtol=1e-9, atol=1e-12)
            np.testing.assert_allclose(dV[b, h], g[2], rtol=1e-9, atol=1e-12)
            for f in range(F):
                np.testing.assert_allclose(dk[b, h, f], g[1][f], rtol=1e-9, atol=1e-12)

# ---- phi networks ------------------------------------------------------------------------
def test_gelu_against_math_erf_and_known_values():
    xs = np.linspace(-6, 6, 97)
    want = [0.5 * x * (1.0 + math.erf(x / math.sqrt(2.0))) for x in xs]
    np.testing.assert_allclose(orc.gelu_erf(xs), want, rtol=1e-14, atol=1e-16)
    assert orc.gelu_erf(0.0) == 0.0
    assert abs(orc.gelu_erf(1.0) - 0.8413447460685429) < 1e-15      # Phi(1)
    assert abs(orc.gelu_erf(-1.0) + 0.15865525393145707) < 1e-15    # -Phi(-1)
    assert abs(orc.gelu_erf(10.0) - 10.0) < 1e-12


def test_phi_mlp_against_python_loops_and_fd():
    rng = np.random.default_rng(3)
    n, d, dphi = 4, 5, 3
    x = rng.standard_normal((n, d))
    W1 = rng.standard_normal((d, d)); b1 = rng.standard_normal(d)
    W2 = rng.standard_normal((d, dphi)); b2 = rng.standard_normal(dphi)
    got = orc.phi_mlp(x, W1, b1, W2, b2)
    for t in range(n):
        h = [sum(x[t, i] * W1[i, j] for i in range(d)) + b1[j] for j in range(d)]
        g = [0.5 * a * (1.0 + math.erf(a / math.sqrt(2.0))) for a in h]
        p = [sum(g[j] * W2[j, o] for j in range(d)) + b2[o] for o in range(dphi)]
        np.testing.assert_allclose(got[t], [max(a, 0.0) for a in p], rtol=1e-13, atol=1e-15)
    assert np.all(got >= 0) and np.any(got == 0) and np.any(got > 0)
    dfeat = rng.standard_normal((n, dphi))
    dx = orc.phi_mlp_backward(x, W1, b1, W2, b2, dfeat)
    fd = fd_grad(lambda xx: float(np.sum(dfeat * orc.phi_mlp(xx, W1, b1, W2, b2))), x)
    np.testing.assert_allclose(dx, fd, rtol=1e-6, atol=1e-8)


def test_full_operator_gradients_fd():
    """dQ, dK, dV through phi and the core against central differences (tiny sizes;
    the seed keeps every ReLU pre-activation away from its kink)."""
    rng = np.random.default_rng(11)
    B, H, N, d, dphi, F = 1, 2, 6, 4, 2, 3
    Q = rng.standard_normal((B, H, N, d)); K = rng.standard_normal((B, H, N, d))
    V = rng.standard_normal((B, H, N, d)); dO = rng.standard_normal((B, H, N, d))
    mk = lambda: (rng.standard_normal((d, d)), rng.standard_normal(d), rng.standard_normal((d, dphi)), rng.standard_normal(dphi) + 0.5)
    phi_q, phi_k = mk(), [mk() for _ in range(F)]
    eps = 1e-3
    dQ, dK, dV, _, _ = orc.hla_backward(Q, K, V, dO, phi_q, phi_k, eps)
    loss = lambda Q_=Q, K_=K, V_=V: float(np.sum(dO * orc.hla_forward(Q_, K_, V_, phi_q, phi_k, eps, "quadratic")[0]))
    np.testing.assert_allclose(dQ, fd_grad(lambda x: loss(Q_=x), Q, 1e-6), rtol=2e-5, atol=1e-8)
    np.testing.assert_allclose(dK, fd_grad(lambda x: loss(K_=x), K, 1e-6), rtol=2e-5, atol=1e-8)
    np.testing.assert_allclose(dV, fd_grad(lambda x: loss(V_=x), V, 1e-6), rtol=2e-5, atol=1e-8)


def test_phi_weight_gradients_fd():
    """dW1, db1, dW2, db2 of one map against central differences of sum(dfeat * phi(x))."""
    rng = np.random.default_rng(5)
    n, d, dphi = 7, 4, 3
    x = rng.standard_normal((n, d))
    W = [rng.standard_normal((d, d)), rng.standard_normal(d), rng.standard_normal((d, dphi)), rng.standard_normal(dphi) + 0.3]
    dfeat = rng.standard_normal((n, dphi))
    got = orc.phi_mlp_backward_weights(x, *W, dfeat)
    assert [g.shape for g in got] == [w.shape for w in W]
    pre = orc.phi_mlp(x, *W, relu=False)
    assert np.abs(pre).min() > 1e-3 and np.any(pre < 0) and np.any(pre > 0)      # away from the ReLU kink, both sides present
    for i in range(4):
        def loss(w, i=i):
            Wv = list(W)
            Wv[i] = w
            return float(np.sum(dfeat * orc.phi_mlp(x, *Wv)))
        np.testing.assert_allclose(got[i], fd_grad(loss, W[i]), rtol=1e-6, atol=1e-8)
    # a dropped ReLU mask or a transposed product would also break these closed forms
    mask = pre > 0
    np.testing.assert_allclose(got[3], (dfeat * mask).sum(axis=0), rtol=1e-13)
    g = orc.gelu_erf(x @ W[0] + W[1])
    want_dW2 = sum(np.multiply.outer(g[t], (dfeat * mask)[t]) for t in range(n))
    np.testing.assert_allclose(got[2], want_dW2, rtol=1e-12, atol=1e-14)


def test_full_operator_weight_gradients_fd():
    """Weight gradients of every map through the core, summed over batches, heads and tokens."""
    rng = np.random.default_rng(12)
    B, H, N, d, dphi, F = 2, 2, 5, 3, 2, 3
    Q = rng.standard_normal((B, H, N, d)); K = rng.standard_normal((B, H, N, d))
    V = rng.standard_normal((B, H, N, d)); dO = rng.standard_normal((B, H, N, d))
    mk = lambda: [rng.standard_normal((d, d)), rng.standard_normal(d), rng.standard_normal((d, dphi)), rng.standard_normal(dphi) + 0.7]
    phi_q, phi_k = mk(), [mk() for _ in range(F)]
    eps = 1e-3
    gq, gk = orc.hla_backward_weights(Q, K, V, dO, phi_q, phi_k, eps)

    def loss(pq, pk):
        return float(np.sum(dO * orc.hla_forward(Q, K, V, pq, pk, eps, "quadratic")[0]))

    for i in range(4):
        def lq(w, i=i):
            pq = list(phi_q)
            pq[i] = w
            return loss(pq, phi_k)
        np.testing.assert_allclose(gq[i], fd_grad(lq, phi_q[i], 1e-6), rtol=5e-5, atol=1e-8)
        for f in range(F):
            def lk(w, i=i, f=f):
                pk = [list(m) for m in phi_k]
                pk[f][i] = w
                return loss(phi_q, pk)
            np.testing.assert_allclose(gk[f][i], fd_grad(lk, phi_k[f][i], 1e-6), rtol=5e-5, atol=1e-8)


def test_whole_operator_wrappers_against_per_head_per_token_loops():
    """The [B,H,N,*] wrappers (phi_features, hla_core_forward, hla_forward, hla_core_backward) against explicit loops
    over batches, heads and tokens that call the per-token map and the per-head definition: a wrong stack axis,
    a reshape that mixes heads, or key maps applied in the wrong order fails here.  Every map has its own weights."""
    rng = np.random.default_rng(21)
    B, H, N, d, dphi, F = 2, 3, 5, 4, 2, 3
    Q = rng.standard_normal((B, H, N, d)); K = rng.standard_normal((B, H, N, d)); V = rng.standard_normal((B, H, N, d))
    dO = rng.standard_normal((B, H, N, d))
    mk = lambda: (rng.standard_normal((d, d)), rng.standard_normal(d), rng.standard_normal((d, dphi)), rng.standard_normal(dphi) + 0.5)
    phi_q, phi_k = mk(), [mk() for _ in range(F)]
    eps = 1e-4
    qf, kf = orc.phi_features(Q, K, phi_q, phi_k)
    assert qf.shape == (B, H, N, dphi) and kf.shape == (B, H, F, N, dphi)
    O, eta, qf2, kf2 = orc.hla_forward(Q, K, V, phi_q, phi_k, eps, "factored")
    assert np.array_equal(qf, qf2) and np.array_equal(kf, kf2)
    dqf, dkf, dV = orc.hla_core_backward(qf, kf, V, dO, eps, "factored")
    for b in range(B):
        for h in range(H):
            q_loop = np.stack([orc.phi_mlp(Q[b, h, n][None, :], *phi_q)[0] for n in range(N)])
            np.testing.assert_allclose(qf[b, h], q_loop, rtol=1e-13, atol=1e-15)
            ks_loop = []
            for f in range(F):
                k_loop = np.stack([orc.phi_mlp(K[b, h, n][None, :], *phi_k[f])[0] for n in range(N)])
                np.testing.assert_allclose(kf[b, h, f], k_loop, rtol=1e-13, atol=1e-15)
                ks_loop.append(k_loop)
            want = brute_force(q_loop.tolist(), [k.tolist() for k in ks_loop], V[b, h].tolist(), eps)
            np.testing.assert_allclose(O[b, h], want, rtol=1e-10, atol=1e-13)
            o_def, eta_def = orc.hla_quadratic(q_loop, ks_loop, V[b, h], eps)
            np.testing.assert_allclose(eta[b, h], eta_def, rtol=1e-12)
            dq, dks, dv = orc.hla_quadratic_backward(q_loop, ks_loop, V[b, h], dO[b, h], eps)
            np.testing.assert_allclose(dqf[b, h], dq, rtol=1e-9, atol=1e-12)
            np.testing.assert_allclose(dV[b, h], dv, rtol=1e-9, atol=1e-12)
            for f in range(F):
                np.testing.assert_allclose(dkf[b, h, f], dks[f], rtol=1e-9, atol=1e-12)


# ---- value modulation (Section 4.5) -------------------------------------------------------------
def vm_weights(rng, d):
    return (rng.standard_normal(d) * 0.3 + 1.0, rng.standard_normal(d) * 0.2, rng.standard_normal((d, d)) / np.sqrt(d), rng.standard_normal(d) * 0.1,
            rng.standard_normal((d, d)) / np.sqrt(d), rng.standard_normal(d) * 0.1)


def test_layer_norm_closed_forms_and_python_loops():
    rng = np.random.default_rng(31)
    x = rng.standard_normal((5, 7)) * 3.0 + 2.0
    y = orc.layer_norm(x, np.ones(7), np.zeros(7), eps=0.0)
    np.testing.assert_allclose(y.mean(axis=1), 0.0, atol=1e-14)
    np.testing.assert_allclose((y ** 2).mean(axis=1), 1.0, rtol=1e-13)           # biased variance: exactly one
    np.testing.assert_allclose(orc.layer_norm(4.0 * x + 9.0, np.ones(7), np.zeros(7), eps=0.0), y, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(orc.layer_norm(np.array([[1.0, 3.0]]), [1.0, 1.0], [0.0, 0.0], eps=0.0), [[-1.0, 1.0]], rtol=1e-15)
    g, b = rng.standard_normal(7), rng.standard_normal(7)
    got = orc.layer_norm(x, g, b)
    for t in range(5):
        mu = sum(x[t]) / 7
        var = sum((a - mu) ** 2 for a in x[t]) / 7
        want = [(x[t, i] - mu) / math.sqrt(var + 1e-5) * g[i] + b[i] for i in range(7)]
        np.testing.assert_allclose(got[t], want, rtol=1e-13, atol=1e-15)


def test_phi_v_mlp_against_python_loops():
    rng = np.random.default_rng(32)
    n, d = 3, 5
    x = rng.standard_normal((n, d))
    ln_g, ln_b, W1, b1, W2, b2 = vm_weights(rng, d)
    got = orc.phi_v_mlp(x, ln_g, ln_b, W1, b1, W2, b2)
    assert got.shape == (n, d) and np.any(got < 0)                 # no ReLU at the end
    for t in range(n):
        mu = sum(x[t]) / d
        var = sum((a - mu) ** 2 for a in x[t]) / d
        xn = [(x[t, i] - mu) / math.sqrt(var + 1e-5) * ln_g[i] + ln_b[i] for i in range(d)]
        h = [sum(xn[i] * W1[i, j] for i in range(d)) + b1[j] for j in range(d)]
        g = [0.5 * a * (1.0 + math.erf(a / math.sqrt(2.0))) for a in h]
        y = [sum(g[j] * W2[j, o] for j in range(d)) + b2[o] for o in range(d)]
        np.testing.assert_allclose(got[t], y, rtol=1e-12, atol=1e-14)


def test_value_modulation_special_cases_and_gradients():
    rng = np.random.default_rng(33)
    n, d = 6, 4
    T, V, dOut = rng.standard_normal((n, d)), rng.standard_normal((n, d)), rng.standard_normal((n, d))
    v1, v2 = vm_weights(rng, d), vm_weights(rng, d)
    out = orc.value_modulation(T, V, v1, v2)
    np.testing.assert_allclose(out, T + orc.phi_v_mlp(T, *v1) * orc.phi_v_mlp(V, *v2), rtol=1e-14)
    # phi_v2 == 1 (zero second layer, unit bias): the update is phi_v1(T) itself; phi_v2 == 0: the identity
    one = v2[:4] + (np.zeros((d, d)), np.ones(d))
    zero = v2[:4] + (np.zeros((d, d)), np.zeros(d))
    np.testing.assert_allclose(orc.value_modulation(T, V, v1, one), T + orc.phi_v_mlp(T, *v1), rtol=1e-14)
    np.testing.assert_allclose(orc.value_modulation(T, V, v1, zero), T, rtol=0, atol=0)
    # the LayerNorm makes each map blind to a shift and (up to eps) a positive rescaling of its input token
    np.testing.assert_allclose(orc.phi_v_mlp(3.0 * V + 5.0, *v2), orc.phi_v_mlp(V, *v2), rtol=1e-4, atol=1e-6)
    dT, dV = orc.value_modulation_backward(T, V, dOut, v1, v2)
    loss = lambda T_=T, V_=V: float(np.sum(dOut * orc.value_modulation(T_, V_, v1, v2)))
    np.testing.assert_allclose(dT, fd_grad(lambda x: loss(T_=x), T, 1e-6), rtol=2e-6, atol=1e-8)
    np.testing.assert_allclose(dV, fd_grad(lambda x: loss(V_=x), V, 1e-6), rtol=2e-6, atol=1e-8)
    dx = orc.phi_v_mlp_backward(V, *v2, dOut)
    np.testing.assert_allclose(dx, fd_grad(lambda x: float(np.sum(dOut * orc.phi_v_mlp(x, *v2))), V, 1e-6), rtol=2e-6, atol=1e-8)
    # a gradient through a LayerNorm has no component along the all-ones direction and (eps -> 0) none along the input's
    # own centred direction: shifting or rescaling the token does not change the output
    np.testing.assert_allclose(dx.sum(axis=1), 0.0, atol=1e-12)


# ---- FLOP model against the paper's tables ---------------------------------------------------
def load_golden():
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_flop_tables.txt")
    out = {}
    for line in open(path):
        if line.strip() and not line.startswith("#"):
            k, val = line.split()[:2]
            out[k] = float(val)
    return out


def test_flop_model_matches_paper_tables():
    gold = load_golden()
    T = 1e12
    H, d = 12, 128
    l3 = {n: flops.paper_layer_flops(n, H, d, 3, 6)["total"] / T for n in (12600, 32760)}
    l2 = flops.paper_layer_flops(32760, H, d, 2, 12)["total"] / T
    qd = {n: flops.quadratic_layer_flops(n, H, d) / T for n in (12600, 32760)}
    assert abs(qd[12600] - gold["quadratic_layer_12600"]) < 0.006
    assert abs(qd[32760] - gold["quadratic_layer_32760"]) < 0.006
    assert abs(l3[12600] - gold["hla3f_layer_12600"]) < 0.006
    assert abs(l3[32760] - gold["hla3f_layer_32760"]) < 0.006
    # whole model = quadratic model - (#HLA blocks) * (quadratic layer - HLA layer)
    assert abs(gold["wan_model_32760"] - 21 * (qd[32760] - l3[32760]) - gold["hla3f_r1_21_model"]) < 0.05
    assert abs(gold["wan_model_32760"] - 10 * (qd[32760] - l3[32760]) - gold["hla3f_r1_10_model"]) < 0.05
    assert abs(gold["wan_model_12600"] - 15 * (qd[12600] - l3[12600]) - gold["hla3f_r2_15_model"]) < 0.05
    assert abs(gold["wan_model_32760"] - 21 * (qd[32760] - l2) - gold["hla2f_r1_21_model"]) < 0.05
    # the operator core is d_phi^F features against d channels
    assert flops.n_features(3, 6) == 216 and flops.n_features(2, 12) == 144
    assert flops.core_fwd_flops_per_token(128, 3, 6) == 111456
