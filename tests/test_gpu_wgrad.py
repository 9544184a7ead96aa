"""GPU parity of hla_backward_weights (gradients of the phi weights) against the fp64 oracle, through the C ABI.

Graded stage-wise like the rest of the backward: the library's weight gradients are compared with the oracle's
phi_mlp_backward_weights evaluated on the inputs that stage actually had - the feature gradients the GPU's core backward
produced, masked by the ReLU mask of the features the GPU's forward kept - and then end to end against the oracle's own
chain (its own features and masks), where the few tokens whose mask differs are part of the error."""
import numpy as np
import pytest
import torch

from oracle import hla_oracle as orc
from paper_2602_12128_b200 import binding, synth
from hla_testlib import DeviceRun, TOL, relerr, report, to_np

pytestmark = pytest.mark.gpu
EPS = 1e-6
f64 = lambda a: np.asarray(a, np.float64)


def oracle_stagewise(X, w, feat, dfeat):
    """Sum over heads of the oracle's weight gradients of one map at the masked feature gradients the GPU used.
    X [B,H,N,d]; feat, dfeat [B,H,N,d_phi]."""
    acc = None
    B, H = X.shape[:2]
    for b in range(B):
        for h in range(H):
            dp = f64(dfeat[b, h]) * (feat[b, h] > 0)
            g = orc.phi_mlp_backward_weights(f64(X[b, h]), *w, dp, relu=False)
            acc = g if acc is None else tuple(a + c for a, c in zip(acc, g))
    return acc


def run_training_step(s, weights_twice=False):
    Q, K, V = synth.make_qkv(s)
    dO = synth.make_dO(s)
    pq, pk = synth.make_phi_weights(s.d, s.d_phi, s.F, s.dtype)
    run = DeviceRun(s, "mlp", EPS)
    run.set_weights(pq, pk)
    run.forward(Q, K, V)
    run.backward(dO)
    gq, gk = run.op.backward_weights(run.Q, run.K)
    torch.cuda.synchronize()
    assert run.op.device_status() == binding.HLA_OK
    assert run.op.launches() == 4          # one pass + one reduction per side
    got_q = [to_np(t) for t in gq]
    got_k = [[to_np(t) for t in g] for g in gk]
    return run, (Q, K, V, dO, pq, pk), got_q, got_k


@pytest.mark.parametrize("d,N,B,H", [(128, 1500, 2, 3), (64, 777, 1, 2), (128, 100, 1, 1)])
def test_weight_gradients_stagewise_and_end_to_end(d, N, B, H):
    s = synth.HlaShape("t", B, H, N, d, "bf16", "rms_qk", backward=True)
    run, (Q, K, V, dO, pq, pk), got_q, got_k = run_training_step(s)
    gqf, gkf = run.features()
    nq = s.B * s.H * s.N * s.d_phi
    dqf = run.region("dqf", nq, (s.B, s.H, s.N, s.d_phi))
    dkf = run.region("dkf", nq * s.F, (s.B, s.H, s.F, s.N, s.d_phi))
    names = ("dW1", "db1", "dW2", "db2")
    ref_q = oracle_stagewise(Q, pq, gqf, dqf)
    for name, got, ref in zip(names, got_q, ref_q):
        assert got.shape == ref.shape
        assert relerr(got, ref) < TOL["bf16"], ("phi_q", name, relerr(got, ref))
    for f in range(s.F):
        ref_k = oracle_stagewise(K, pk[f], gkf[:, :, f], dkf[:, :, f])
        for name, got, ref in zip(names, got_k[f], ref_k):
            assert relerr(got, ref) < TOL["bf16"], (f"phi_k{f + 1}", name, relerr(got, ref))
    # end to end against the oracle's own chain from Q, K, V, dO: reported, not bounded, for these weights - the final ReLU
    # makes the chain discontinuous and dq grows like 1 / |phi_q(q)|, so a few tokens dominate the difference of the sums
    eq, ek = orc.hla_backward_weights(f64(Q), f64(K), f64(V), f64(dO), pq, pk, EPS, "factored")
    worst = {}
    for name, got, ref in zip(names, got_q, eq):
        worst["q_" + name] = relerr(got, ref)
    for f in range(s.F):
        for name, got, ref in zip(names, got_k[f], ek[f]):
            worst[f"k{f + 1}_" + name] = relerr(got, ref)
    report(f"weight gradients end to end d={d} N={N}", **worst)


def test_weight_gradients_end_to_end_where_the_chain_is_smooth():
    """With second-layer biases that keep every feature well above zero no ReLU clips (the chain from Q, K, V, dO to the
    weight gradients is smooth) and no query has tiny features: there the whole chain is bounded end to end."""
    s = synth.HlaShape("t", 1, 3, 1200, 128, "bf16", "rms_qk", backward=True)
    Q, K, V = synth.make_qkv(s)
    dO = synth.make_dO(s)
    pq, pk = synth.make_phi_weights(s.d, s.d_phi, s.F, s.dtype)
    lift = lambda w: (w[0], w[1], synth.bf16_round(w[2] * np.float32(0.25)), synth.bf16_round(np.abs(w[3]) + np.float32(1.5)))
    pq, pk = lift(pq), [lift(w) for w in pk]
    run = DeviceRun(s, "mlp", EPS)
    run.set_weights(pq, pk)
    run.forward(Q, K, V)
    run.backward(dO)
    gq, gk = run.op.backward_weights(run.Q, run.K)
    torch.cuda.synchronize()
    assert run.op.device_status() == binding.HLA_OK
    gqf, gkf = run.features()
    assert gqf.min() > 0.1 and gkf.min() > 0.1
    eq, ek = orc.hla_backward_weights(f64(Q), f64(K), f64(V), f64(dO), pq, pk, EPS, "factored")
    worst = {}
    for name, got, ref in zip(("dW1", "db1", "dW2", "db2"), gq, eq):
        worst["q_" + name] = relerr(to_np(got), ref)
    for f in range(s.F):
        for name, got, ref in zip(("dW1", "db1", "dW2", "db2"), gk[f], ek[f]):
            worst[f"k{f + 1}_" + name] = relerr(to_np(got), ref)
    # db2 of a key map is sum_t dk^f_t, and the scale invariance of the operator (sum_t k^f_t . dk^f_t = 0, exact for
    # eps = 0) makes that sum cancel when the features are nearly constant, as they are here: it is bounded relative
    # to the sum of the magnitudes of its terms, like any sum with cancellation
    _, _, _, _, dkf_o = orc.hla_backward(f64(Q), f64(K), f64(V), f64(dO), pq, pk, EPS, "factored")
    for f in range(s.F):
        scale = np.abs(dkf_o[:, :, f]).sum(axis=(0, 1, 2)).max()
        worst[f"k{f + 1}_db2"] = float(np.abs(to_np(gk[f][3]) - ek[f][3]).max() / scale)
    report("weight gradients end to end, smooth chain", **worst)
    assert max(worst.values()) < TOL["bf16"], worst


def test_weight_gradients_bitwise_reproducible_and_optional_sides():
    s = synth.HlaShape("t", 1, 2, 900, 128, "bf16", "inv_sqrt_d", backward=True)
    run, _, got_q, got_k = run_training_step(s)
    op = run.op
    gq2, gk2 = op.backward_weights(run.Q, run.K)
    torch.cuda.synchronize()
    for a, b in zip(got_q, gq2):
        assert np.array_equal(a, to_np(b))
    for ga, gb in zip(got_k, gk2):
        for a, b in zip(ga, gb):
            assert np.array_equal(a, to_np(b))
    # one side only: the other side's buffers are not touched
    mk = lambda: tuple(torch.full(sh, 7.0, dtype=torch.float32, device="cuda") for sh in ((s.d, s.d), (s.d,), (s.d, s.d_phi), (s.d_phi,)))
    only_q = mk()
    binding.hla_backward_weights(op.ctx, run.Q, run.K, only_q, None, op.workspace)
    torch.cuda.synchronize()
    assert op.launches() == 2
    for a, b in zip(got_q, only_q):
        assert np.array_equal(a, to_np(b))
    only_k = [mk() for _ in range(s.F)]
    binding.hla_backward_weights(op.ctx, run.Q, run.K, None, only_k, op.workspace)
    torch.cuda.synchronize()
    for ga, gb in zip(got_k, only_k):
        for a, b in zip(ga, gb):
            assert np.array_equal(a, to_np(b))
    assert op.device_status() == binding.HLA_OK


def test_weight_gradients_refused_outside_the_supported_set():
    lib = binding.load_library()
    none = binding.Hla(1, 2, 300, 128, dtype="bf16", phi="none", eps=EPS)
    p = none.workspace.data_ptr()
    n = none.workspace.numel()
    assert lib.hla_backward_weights(none.ctx, p, p, None, None, p, n, None) == binding.HLA_ERR_INVALID_ARG
    f32 = binding.Hla(1, 2, 300, 16, dtype="f32", phi="mlp", eps=EPS)
    w = tuple(torch.zeros(sh, dtype=torch.float32, device="cuda") for sh in ((16, 16), (16,), (16, 6), (6,)))
    f32.set_phi(w, [w, w, w])
    p = f32.workspace.data_ptr()
    assert lib.hla_backward_weights(f32.ctx, p, p, None, None, p, f32.workspace.numel(), None) == binding.HLA_ERR_UNSUPPORTED
