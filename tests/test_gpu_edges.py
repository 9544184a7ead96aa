"""Edge cases of the tensor-core path through the C ABI: degenerate sizes (a single token, one ragged tile,
exact tile multiples), many heads (persistent CTAs crossing head boundaries, more heads than SMs), queries
whose features are all zero, a large eps, the narrower head width with the phi maps, and run-to-run
reproducibility of the backward."""
import numpy as np
import pytest
import torch

from oracle import hla_oracle as orc
from paper_2602_12128_b200 import binding, synth
from hla_testlib import DeviceRun, TOL, relerr, l2err, dev_weights, to_dev

pytestmark = pytest.mark.gpu
EPS = 1e-6
f64 = lambda a: np.asarray(a, np.float64)


def _inputs(s, vscale=True, seed=0):
    _, _, V = synth.make_qkv(s, seed)
    if vscale:
        V = synth.bf16_round(V * np.float32(np.sqrt(s.d)))
    qf, kf = synth.make_features(s, seed + 3)
    return qf, kf, V, synth.make_dO(s, seed + 2)


@pytest.mark.parametrize("d,N,B,H", [(128, 1, 1, 1), (128, 5, 1, 2), (64, 1, 2, 1), (128, 128, 1, 1), (128, 129, 1, 1), (64, 256, 1, 3),
                                     (128, 255, 1, 2)])
def test_degenerate_token_counts_forward_backward(d, N, B, H):
    s = synth.HlaShape("t", B, H, N, d, "bf16", "inv_sqrt_d")
    qf, kf, V, dO = _inputs(s)
    run = DeviceRun(s, "none", EPS)
    assert run.op.layout.tensor_core == 1
    O = run.forward(qf, kf, V)
    dq, dk, dv = run.backward(dO)
    Oq, eta = orc.hla_core_forward(f64(qf), f64(kf), f64(V), EPS, "quadratic")
    rq, rk, rv = orc.hla_core_backward(f64(qf), f64(kf), f64(V), f64(dO), EPS, "quadratic")
    assert relerr(O, Oq) < TOL["bf16"] and relerr(run.eta(), eta) < TOL["bf16"]
    assert relerr(dv, rv) < TOL["bf16"]
    # dq and dk are differences of terms of size |dO_i . o_i| (with a single key they cancel completely: every weight
    # is 1, o = v, dq = dk = 0 up to eps), so the error is measured against that term size when the result is smaller.
    term = np.abs((f64(dO) * Oq).sum(-1)).max()
    assert np.abs(dq - rq).max() < TOL["bf16"] * max(np.abs(rq).max(), term)
    assert np.abs(dk - rk).max() < TOL["bf16"] * max(np.abs(rk).max(), term)


@pytest.mark.parametrize("d,N,B,H", [(128, 130, 10, 20), (64, 300, 1, 37)])
def test_many_heads(d, N, B, H):
    """More heads than SMs (the persistent kernels walk several heads per CTA, one split per head) and a head
    count that does not divide the SM count."""
    s = synth.HlaShape("t", B, H, N, d, "bf16", "inv_sqrt_d")
    qf, kf, V, dO = _inputs(s)
    run = DeviceRun(s, "none", EPS)
    O = run.forward(qf, kf, V)
    dq, dk, dv = run.backward(dO)
    Oq, eta = orc.hla_core_forward(f64(qf), f64(kf), f64(V), EPS, "quadratic")
    rq, rk, rv = orc.hla_core_backward(f64(qf), f64(kf), f64(V), f64(dO), EPS, "quadratic")
    assert relerr(O, Oq) < TOL["bf16"]
    assert relerr(dv, rv) < TOL["bf16"] and relerr(dq, rq) < TOL["bf16"] and relerr(dk, rk) < TOL["bf16"]


def test_queries_with_all_zero_features_and_large_eps():
    """A query whose features are all zero has eta = 0: its output is 0 / eps = 0 and its gradients stay finite.
    A large eps (1e-2) changes the normalisation visibly and must match the oracle too."""
    s = synth.HlaShape("t", 1, 2, 700, 128, "bf16", "inv_sqrt_d")
    qf, kf, V, dO = _inputs(s)
    qf[0, :, ::7, :] = 0.0
    for eps in (1e-6, 1e-2):
        run = DeviceRun(s, "none", eps)
        O = run.forward(qf, kf, V)
        dq, dk, dv = run.backward(dO)
        assert np.all(O[0, :, ::7, :] == 0.0)
        Oq, eta = orc.hla_core_forward(f64(qf), f64(kf), f64(V), eps, "quadratic")
        rq, rk, rv = orc.hla_core_backward(f64(qf), f64(kf), f64(V), f64(dO), eps, "quadratic")
        assert np.all(np.isfinite(dq)) and np.all(np.isfinite(dk)) and np.all(np.isfinite(dv))
        assert relerr(O, Oq) < TOL["bf16"]
        assert relerr(dv, rv) < TOL["bf16"] and relerr(dk, rk) < TOL["bf16"]
        live = np.ones(qf.shape[2], bool)
        live[::7] = False
        assert relerr(dq[:, :, live], rq[:, :, live]) < TOL["bf16"]


def test_backward_bitwise_reproducible():
    s = synth.HlaShape("t", 1, 3, 3000, 128, "bf16", "rms_qk", backward=True)
    Q, K, V = synth.make_qkv(s)
    dO = synth.make_dO(s)
    pq, pk = synth.make_phi_weights(s.d, s.d_phi, s.F, s.dtype)
    run = DeviceRun(s, "mlp", EPS, n_splits=4)
    run.set_weights(pq, pk)
    run.forward(Q, K, V)
    a = run.backward(dO)
    run.forward(Q, K, V)
    b = run.backward(dO)
    for x, y in zip(a, b):
        assert np.array_equal(x, y)


@pytest.mark.parametrize("shape", [synth.CONFIGS["small_bf16"], synth.HlaShape("ragged64", 1, 3, 777, 64, "bf16", "rms_qk"),
                                   synth.HlaShape("ragged128", 2, 1, 131, 128, "bf16", "inv_sqrt_d")], ids=lambda s: s.name)
def test_forward_backward_with_phi_stage_by_stage(shape):
    """The small benchmark shape (B=2, H=12, N=4096, d=64) and two ragged shapes with the phi maps (fused query side,
    key maps, both phi backward kernels), forward and backward, stage by stage."""
    s = shape
    Q, K, V = synth.make_qkv(s)
    dO = synth.make_dO(s)
    pq, pk = synth.make_phi_weights(s.d, s.d_phi, s.F, s.dtype)
    run = DeviceRun(s, "mlp", EPS)
    run.set_weights(pq, pk)
    O = run.forward(Q, K, V)
    dQ, dK, dV = run.backward(dO)
    gq, gk = run.features()
    nq = s.B * s.H * s.N * s.d_phi
    dqf = run.region("dqf", nq, (s.B, s.H, s.N, s.d_phi))
    dkf = run.region("dkf", nq * s.F, (s.B, s.H, s.F, s.N, s.d_phi))
    Oc, _ = orc.hla_core_forward(gq, gk, f64(V), EPS, "factored")
    assert relerr(O, Oc) < TOL["bf16"]
    rq, rk, rv = orc.hla_core_backward(gq, gk, f64(V), f64(dO), EPS, "factored")
    assert relerr(dV, rv) < TOL["bf16"] and relerr(dqf, rq) < TOL["bf16"] and relerr(dkf, rk) < TOL["bf16"]
    d = s.d
    pre_q = orc.phi_mlp(f64(Q).reshape(-1, d), *pq, relu=False).reshape(gq.shape)
    pre_k = np.stack([orc.phi_mlp(f64(K).reshape(-1, d), *w, relu=False).reshape(gq.shape) for w in pk], axis=2)
    flip_q, flip_k = (gq > 0) != (pre_q > 0), (gk > 0) != (pre_k > 0)
    assert flip_q.mean() < 5e-3 and flip_k.mean() < 5e-3
    rQ = orc.phi_mlp_backward(f64(Q).reshape(-1, d), *pq, dqf.reshape(-1, s.d_phi)).reshape(Q.shape)
    rK = sum(orc.phi_mlp_backward(f64(K).reshape(-1, d), *pk[f], dkf[:, :, f].reshape(-1, s.d_phi)).reshape(K.shape) for f in range(s.F))
    same_q, same_k = ~flip_q.any(axis=-1), ~flip_k.any(axis=(2, 4))
    assert relerr(dQ[same_q], rQ[same_q]) < TOL["bf16"]
    assert relerr(dK[same_k], rK[same_k]) < TOL["bf16"]


@pytest.mark.parametrize("d", [64, 128])
def test_phi_with_large_biases(d):
    """First-layer biases of the size of the pre-activations themselves (the kernels add b1 inside the first-layer
    product): features against the oracle's phi, and the phi backward at the feature gradients the GPU produced."""
    s = synth.HlaShape(f"bias{d}", 1, 2, 300, d, "bf16", "rms_qk")
    Q, K, V = synth.make_qkv(s)
    dO = synth.make_dO(s)
    pq, pk = synth.make_phi_weights(s.d, s.d_phi, s.F, s.dtype)
    rng = np.random.default_rng(5)
    bf = lambda a: torch.from_numpy(a.astype(np.float32)).to(torch.bfloat16).float().numpy()

    def with_bias(w):
        W1, b1, W2, b2 = w
        return W1, bf(rng.standard_normal(b1.shape)), W2, bf(0.5 * rng.standard_normal(b2.shape))

    pq, pk = with_bias(pq), [with_bias(w) for w in pk]
    run = DeviceRun(s, "mlp", EPS)
    run.set_weights(pq, pk)
    run.forward(Q, K, V)
    dQ, dK, dV = run.backward(dO)
    gq, gk = run.features()
    ref_q = orc.phi_mlp(f64(Q).reshape(-1, d), *pq).reshape(gq.shape)
    assert relerr(gq, ref_q) < TOL["bf16"]
    for f in range(s.F):
        ref_k = orc.phi_mlp(f64(K).reshape(-1, d), *pk[f]).reshape(gq.shape)
        assert relerr(gk[:, :, f], ref_k) < TOL["bf16"]
    nq = s.B * s.H * s.N * s.d_phi
    dqf = run.region("dqf", nq, (s.B, s.H, s.N, s.d_phi))
    dkf = run.region("dkf", nq * s.F, (s.B, s.H, s.F, s.N, s.d_phi))
    pre_q = orc.phi_mlp(f64(Q).reshape(-1, d), *pq, relu=False).reshape(gq.shape)
    pre_k = np.stack([orc.phi_mlp(f64(K).reshape(-1, d), *w, relu=False).reshape(gq.shape) for w in pk], axis=2)
    same_q = ~((gq > 0) != (pre_q > 0)).any(axis=-1)
    same_k = ~((gk > 0) != (pre_k > 0)).any(axis=(2, 4))
    assert same_q.mean() > 0.95 and same_k.mean() > 0.9
    rQ = orc.phi_mlp_backward(f64(Q).reshape(-1, d), *pq, dqf.reshape(-1, s.d_phi)).reshape(Q.shape)
    rK = sum(orc.phi_mlp_backward(f64(K).reshape(-1, d), *pk[f], dkf[:, :, f].reshape(-1, s.d_phi)).reshape(K.shape) for f in range(s.F))
    assert relerr(dQ[same_q], rQ[same_q]) < TOL["bf16"]
    assert relerr(dK[same_k], rK[same_k]) < TOL["bf16"]


def test_back_to_back_steps_without_host_sync():
    """Twelve training steps enqueued back to back on one stream, alternating between two sets of inputs and output
    buffers, with no host synchronisation in between (each kernel's set-up overlaps the drain of the previous one):
    every step's O, dQ, dK, dV must be bit-identical to the same step run alone."""
    s = synth.HlaShape("b2b", 1, 6, 5000, 128, "bf16", "rms_qk", backward=True)
    pq, pk = synth.make_phi_weights(s.d, s.d_phi, s.F, s.dtype)
    op = binding.Hla(s.B, s.H, s.N, s.d, dtype=s.dtype, phi="mlp", F=s.F, d_phi=s.d_phi, eps=EPS)
    op.set_phi(*dev_weights(pq, pk, s.dtype))
    sets = []
    for seed in (0, 7):
        Q, K, V = synth.make_qkv(s, seed=seed)
        dO = synth.make_dO(s)
        sets.append(tuple(to_dev(a, s.dtype) for a in (Q, K, V, dO)))
    ref = []
    for Q, K, V, dO in sets:           # each set alone, synchronised
        O = op.forward(Q, K, V)
        dQ, dK, dV = op.backward(Q, K, V, O, dO)
        torch.cuda.synchronize()
        assert op.device_status() == binding.HLA_OK
        ref.append([t.clone() for t in (O, dQ, dK, dV)])
    outs = []
    for step in range(12):             # enqueued back to back
        Q, K, V, dO = sets[step & 1]
        O = op.forward(Q, K, V)
        dQ, dK, dV = op.backward(Q, K, V, O, dO)
        outs.append((O, dQ, dK, dV))
    torch.cuda.synchronize()
    assert op.device_status() == binding.HLA_OK
    for step, got in enumerate(outs):
        for a, b in zip(got, ref[step & 1]):
            assert torch.equal(a, b), step
