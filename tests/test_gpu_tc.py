"""GPU parity of the bf16 tensor-core kernels (tcgen05 state build, reduce/emit,
readout) against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import hla_oracle as orc
from paper_2602_12128_b200 import binding, synth
from hla_testlib import DeviceRun, TOL, fold_symmetric, oracle_state, relerr, l2err, report

pytestmark = pytest.mark.gpu
EPS = 1e-6


@pytest.mark.parametrize("d,N,B,H,splits", [(128, 1000, 1, 2, 0), (128, 128, 1, 1, 1), (128, 77, 1, 3, 0), (64, 1500, 2, 2, 5),
                                            (128, 4096 + 40, 1, 2, 7), (64, 129, 1, 1, 4)])
def test_core_forward_bf16_features(d, N, B, H, splits):
    """Feature-level entry point: the features are fp32 inputs, V is bf16; spans several
    128-token tiles, ragged tails, more splits than tiles, and both head widths."""
    s = synth.HlaShape("t", B, H, N, d, "bf16", "inv_sqrt_d")
    _, _, V = synth.make_qkv(s)
    V = synth.bf16_round(V * np.float32(np.sqrt(d)))          # V ~ N(0,1)
    qf, kf = synth.make_features(s)
    run = DeviceRun(s, "none", EPS, splits)
    assert run.op.layout.tensor_core == 1
    O = run.forward(qf, kf, V)
    f64 = lambda a: a.astype(np.float64)
    Oq, eta = orc.hla_core_forward(f64(qf), f64(kf), f64(V), EPS, "factored")
    C, z = run.state()                               # folded over the permutation symmetry: 56 rows
    Co, zo = oracle_state(f64(kf), f64(V))
    Co, zo = fold_symmetric(Co), fold_symmetric(zo[..., None])[..., 0]
    assert C.shape[2] == 56
    assert relerr(z, zo) < 1e-5                      # fp32 accumulation of unrounded products
    assert relerr(C, Co) < TOL["bf16"] / 4           # folded key features rounded to bf16 once
    assert relerr(run.eta(), eta) < TOL["bf16"] / 4
    assert relerr(O, Oq) < TOL["bf16"], (relerr(O, Oq), l2err(O, Oq))
    assert run.op.launches() == 3


@pytest.mark.parametrize("d,N,B,H,splits", [(128, 1000, 1, 2, 0), (64, 1500, 2, 2, 5), (128, 77, 1, 3, 0), (128, 4096 + 40, 1, 2, 7), (64, 129, 1, 1, 4)])
def test_core_forward_and_backward_two_factors(d, N, B, H, splits):
    """The paper's 2-factor variant (d_phi = 12: 78 monomials q_a q_b, a <= b, in two operand blocks) at the feature level:
    state (folded over the symmetry of q (x) q), normaliser, output and all three gradients against the oracle."""
    s = synth.HlaShape("t", B, H, N, d, "bf16", "inv_sqrt_d", False, 2, 12)
    _, _, V = synth.make_qkv(s)
    V = synth.bf16_round(V * np.float32(np.sqrt(d)))
    qf, kf = synth.make_features(s)
    dO = synth.make_dO(s)
    run = DeviceRun(s, "none", EPS, splits)
    assert run.op.layout.tensor_core == 1 and run.op.layout.state_rows == 78
    O = run.forward(qf, kf, V)
    assert run.op.launches() == 3
    f64 = lambda a: a.astype(np.float64)
    Oq, eta = orc.hla_core_forward(f64(qf), f64(kf), f64(V), EPS, "quadratic" if N <= 1500 else "factored")
    C, z = run.state()
    Co, zo = oracle_state(f64(kf), f64(V))
    Co, zo = fold_symmetric(Co, 12, 2), fold_symmetric(zo[..., None], 12, 2)[..., 0]
    assert relerr(z, zo) < 1e-5
    assert relerr(C, Co) < TOL["bf16"] / 4
    assert relerr(run.eta(), eta) < TOL["bf16"] / 4
    assert relerr(O, Oq) < TOL["bf16"], relerr(O, Oq)
    dq, dk, dv = run.backward(dO)
    assert run.op.launches() == 3
    rq, rk, rv = orc.hla_core_backward(f64(qf), f64(kf), f64(V), f64(dO), EPS, "quadratic" if N <= 1000 else "factored")
    assert relerr(dv, rv) < TOL["bf16"], relerr(dv, rv)
    assert relerr(dq, rq) < TOL["bf16"], relerr(dq, rq)
    assert relerr(dk, rk) < TOL["bf16"], relerr(dk, rk)
    again = run.forward(qf, kf, V)
    assert np.array_equal(O, again)


def test_config2_small_bf16_forward_stagewise():
    """B=2,H=12,N=4096,d=64 bf16 with the phi maps: features against the oracle's,
    then the core against the oracle core run on the features the GPU produced,
    then end to end on rows whose normaliser is not tiny."""
    s = synth.CONFIGS["small_bf16"]
    Q, K, V = synth.make_qkv(s)
    pq, pk = synth.make_phi_weights(s.d, s.d_phi, s.F, s.dtype)
    run = DeviceRun(s, "mlp", EPS)
    run.set_weights(pq, pk)
    O = run.forward(Q, K, V)
    f64 = lambda a: a.astype(np.float64)
    Oq, eta, qf, kf = orc.hla_forward(f64(Q), f64(K), f64(V), pq, pk, EPS, "factored")
    gq, gk = run.features()
    assert relerr(gq, qf) < TOL["bf16"] and relerr(gk, kf) < TOL["bf16"]
    Oc, _ = orc.hla_core_forward(gq, gk, f64(V), EPS, "factored")
    assert relerr(O, Oc) < TOL["bf16"]
    # End to end the max-norm is ill-conditioned: a query whose features are all small compared with the
    # bf16-level error of the features has an output that swings between class averages (and ReLU makes it
    # discontinuous).  So end to end the bound is on the relative L2 error, over rows whose normaliser is not tiny.
    keep = eta >= 1e-3 * np.median(eta)
    report("config2 end to end", kept_fraction=keep.mean(), l2_kept=l2err(O[keep], Oq[keep]), maxnorm_kept=relerr(O[keep], Oq[keep]),
           maxnorm_all=relerr(O, Oq))
    assert keep.mean() > 0.5
    assert l2err(O[keep], Oq[keep]) < TOL["bf16"], l2err(O[keep], Oq[keep])
    # the quadratic definition on one head
    o_def, _ = orc.hla_quadratic(qf[1, 5], [kf[1, 5, f] for f in range(3)], f64(V)[1, 5], EPS)
    np.testing.assert_allclose(o_def, Oq[1, 5], rtol=1e-8, atol=1e-12)


def test_tc_bitwise_reproducible():
    s = synth.HlaShape("t", 1, 3, 2000, 128, "bf16", "inv_sqrt_d")
    _, _, V = synth.make_qkv(s)
    qf, kf = synth.make_features(s)
    run = DeviceRun(s, "none", EPS, 4)
    a = run.forward(qf, kf, V)
    b = run.forward(qf, kf, V)
    assert np.array_equal(a, b)


@pytest.mark.parametrize("d,N,B,H,splits", [(128, 1000, 1, 2, 0), (64, 700, 2, 2, 3), (128, 130, 1, 1, 0), (128, 2500, 1, 3, 5)])
def test_core_backward_bf16_features(d, N, B, H, splits):
    """dq, dk^f (fp32 feature gradients) and dV (bf16) of the tensor-core backward against the quadratic-form oracle."""
    s = synth.HlaShape("t", B, H, N, d, "bf16", "inv_sqrt_d")
    _, _, V = synth.make_qkv(s)
    V = synth.bf16_round(V * np.float32(np.sqrt(d)))
    qf, kf = synth.make_features(s)
    dO = synth.make_dO(s)
    run = DeviceRun(s, "none", EPS, splits)
    O = run.forward(qf, kf, V)
    dq, dk, dv = run.backward(dO)
    f64 = lambda a: a.astype(np.float64)
    form = "quadratic" if N <= 1000 else "factored"
    rq, rk, rv = orc.hla_core_backward(f64(qf), f64(kf), f64(V), f64(dO), EPS, form)
    assert relerr(dv, rv) < TOL["bf16"], relerr(dv, rv)
    assert relerr(dq, rq) < TOL["bf16"], relerr(dq, rq)
    assert relerr(dk, rk) < TOL["bf16"], relerr(dk, rk)
    assert run.op.launches() == 3


def test_full_backward_bf16_mlp_stagewise():
    """Training-step shape at reduced size (d=128, ragged N) with the phi maps: every stage against the oracle
    run on that stage's actual inputs, then end to end."""
    s = synth.HlaShape("t", 2, 3, 1500, 128, "bf16", "rms_qk", backward=True)
    Q, K, V = synth.make_qkv(s)
    dO = synth.make_dO(s)
    pq, pk = synth.make_phi_weights(s.d, s.d_phi, s.F, s.dtype)
    run = DeviceRun(s, "mlp", EPS)
    run.set_weights(pq, pk)
    O = run.forward(Q, K, V)
    dQ, dK, dV = run.backward(dO)
    f64 = lambda a: a.astype(np.float64)
    gq, gk = run.features()
    nq = s.B * s.H * s.N * s.d_phi
    dqf = run.region("dqf", nq, (s.B, s.H, s.N, s.d_phi))
    dkf = run.region("dkf", nq * s.F, (s.B, s.H, s.F, s.N, s.d_phi))
    # core gradients at the features the GPU used
    rq, rk, rv = orc.hla_core_backward(gq, gk, f64(V), f64(dO), EPS, "factored")
    assert relerr(dV, rv) < TOL["bf16"]
    assert relerr(dqf, rq) < TOL["bf16"]
    assert relerr(dkf, rk) < TOL["bf16"]
    # phi backward at the feature gradients the GPU produced
    d = s.d
    rQ = orc.phi_mlp_backward(f64(Q).reshape(-1, d), *pq, dqf.reshape(-1, s.d_phi)).reshape(Q.shape)
    rK = sum(orc.phi_mlp_backward(f64(K).reshape(-1, d), *pk[f], dkf[:, :, f].reshape(-1, s.d_phi)).reshape(K.shape) for f in range(s.F))
    # The library takes the ReLU mask from the features its forward kept.  Where that mask differs from the oracle's
    # (only possible where the pre-activation is within the forward's bf16-level error of zero) the row is a different,
    # equally valid one-sided derivative; those rows are counted and left out of the max-norm.
    pre_q = orc.phi_mlp(f64(Q).reshape(-1, d), *pq, relu=False).reshape(gq.shape)
    pre_k = np.stack([orc.phi_mlp(f64(K).reshape(-1, d), *w, relu=False).reshape(gq.shape) for w in pk], axis=2)
    flip_q, flip_k = (gq > 0) != (pre_q > 0), (gk > 0) != (pre_k > 0)
    assert flip_q.mean() < 5e-3 and flip_k.mean() < 5e-3
    assert np.abs(pre_q[flip_q]).max(initial=0) < 5e-3 * np.abs(pre_q).max()
    assert np.abs(pre_k[flip_k]).max(initial=0) < 5e-3 * np.abs(pre_k).max()
    same_q, same_k = ~flip_q.any(axis=-1), ~flip_k.any(axis=(2, 4))
    assert relerr(dQ[same_q], rQ[same_q]) < TOL["bf16"], relerr(dQ[same_q], rQ[same_q])
    assert relerr(dK[same_k], rK[same_k]) < TOL["bf16"], relerr(dK[same_k], rK[same_k])
    # End to end.  The final ReLU makes dQ, dK discontinuous in the input: a token with a pre-activation within the
    # bf16-level error of zero gets (correctly, for the features the GPU computed) an O(1) different gradient row.
    # Those tokens are graded stage-wise above; end to end the bound is on the tokens whose pre-activations are all
    # at least 0.5 % of the largest one away from zero.  dQ is also ill-conditioned where the query features are
    # small: o_i does not change when q_i is scaled, so dq_i grows like 1/|q_i| and the forward's absolute feature
    # error (bf16 rounding of the hidden layer) becomes a large relative error of exactly the rows with the largest
    # gradients; the bound is therefore taken over the queries with |phi_q(q_i)| >= half the median.
    eQ, eK, eV, _, _ = orc.hla_backward(f64(Q), f64(K), f64(V), f64(dO), pq, pk, EPS, "factored")
    assert relerr(dV, eV) < TOL["bf16"], relerr(dV, eV)
    qn = np.linalg.norm(np.maximum(pre_q, 0.0), axis=-1)
    keep_q = (np.abs(pre_q).min(axis=-1) > 5e-3 * np.abs(pre_q).max()) & (qn >= 0.5 * np.median(qn))
    keep_k = np.abs(pre_k).min(axis=(2, 4)) > 5e-3 * np.abs(pre_k).max()
    report("reduced training step end to end", kept_q=keep_q.mean(), kept_k=keep_k.mean(), dV_maxnorm=relerr(dV, eV),
           dQ_l2_kept=l2err(dQ[keep_q], eQ[keep_q]), dK_l2_kept=l2err(dK[keep_k], eK[keep_k]),
           dQ_maxnorm_kept=relerr(dQ[keep_q], eQ[keep_q]), dK_maxnorm_kept=relerr(dK[keep_k], eK[keep_k]),
           flipped_q=flip_q.mean(), flipped_k=flip_k.mean())
    assert keep_q.mean() > 0.7 and keep_k.mean() > 0.5
    assert l2err(dQ[keep_q], eQ[keep_q]) < TOL["bf16"], l2err(dQ[keep_q], eQ[keep_q])
    assert l2err(dK[keep_k], eK[keep_k]) < TOL["bf16"], l2err(dK[keep_k], eK[keep_k])
    assert run.op.launches() == 5


@pytest.mark.parametrize("d,N,B,H", [(128, 1500, 2, 2), (64, 700, 1, 3), (128, 100, 1, 1)])
def test_two_factor_variant_with_the_phi_maps_stagewise(d, N, B, H):
    """The paper's 2-factor variant (two key maps, d_phi = 12) on the tensor-core kernels with the phi maps: every stage of
    the forward, the backward and the weight gradients against the oracle run on that stage's actual inputs."""
    s = synth.HlaShape("t", B, H, N, d, "bf16", "rms_qk", True, 2, 12)
    Q, K, V = synth.make_qkv(s)
    dO = synth.make_dO(s)
    pq, pk = synth.make_phi_weights(s.d, s.d_phi, s.F, s.dtype)
    assert len(pk) == 2 and pq[2].shape == (d, 12)
    run = DeviceRun(s, "mlp", EPS)
    assert run.op.layout.tensor_core == 1 and run.op.layout.state_rows == 78
    run.set_weights(pq, pk)
    O = run.forward(Q, K, V)
    assert run.op.launches() == 3
    f64 = lambda a: a.astype(np.float64)
    gq, gk = run.features()
    _, _, qf, kf = orc.hla_forward(f64(Q), f64(K), f64(V), pq, pk, EPS, "factored")
    assert relerr(gq, qf) < TOL["bf16"] and relerr(gk, kf) < TOL["bf16"]
    Oc, eta = orc.hla_core_forward(gq, gk, f64(V), EPS, "quadratic" if N <= 1500 else "factored")
    assert relerr(O, Oc) < TOL["bf16"], relerr(O, Oc)
    assert relerr(run.eta(), eta) < TOL["bf16"] / 4
    dQ, dK, dV = run.backward(dO)
    assert run.op.launches() == 5
    nq = s.B * s.H * s.N * s.d_phi
    dqf = run.region("dqf", nq, (s.B, s.H, s.N, s.d_phi))
    dkf = run.region("dkf", nq * s.F, (s.B, s.H, s.F, s.N, s.d_phi))
    rq, rk, rv = orc.hla_core_backward(gq, gk, f64(V), f64(dO), EPS, "factored")
    assert relerr(dV, rv) < TOL["bf16"] and relerr(dqf, rq) < TOL["bf16"] and relerr(dkf, rk) < TOL["bf16"]
    rQ = orc.phi_mlp_backward(f64(Q).reshape(-1, d), *pq, dqf.reshape(-1, s.d_phi)).reshape(Q.shape)
    rK = sum(orc.phi_mlp_backward(f64(K).reshape(-1, d), *pk[f], dkf[:, :, f].reshape(-1, s.d_phi)).reshape(K.shape) for f in range(s.F))
    pre_q = orc.phi_mlp(f64(Q).reshape(-1, d), *pq, relu=False).reshape(gq.shape)
    pre_k = np.stack([orc.phi_mlp(f64(K).reshape(-1, d), *w, relu=False).reshape(gq.shape) for w in pk], axis=2)
    flip_q, flip_k = (gq > 0) != (pre_q > 0), (gk > 0) != (pre_k > 0)
    assert flip_q.mean() < 5e-3 and flip_k.mean() < 5e-3
    same_q, same_k = ~flip_q.any(axis=-1), ~flip_k.any(axis=(2, 4))
    assert relerr(dQ[same_q], rQ[same_q]) < TOL["bf16"], relerr(dQ[same_q], rQ[same_q])
    assert relerr(dK[same_k], rK[same_k]) < TOL["bf16"], relerr(dK[same_k], rK[same_k])
    # weight gradients of the three maps at the masked feature gradients the GPU used
    wq, wk = run.op.backward_weights(run.Q, run.K)
    torch.cuda.synchronize()
    assert run.op.device_status() == binding.HLA_OK
    sides = [(Q, pq, gq, dqf, wq)] + [(K, pk[f], gk[:, :, f], dkf[:, :, f], wk[f]) for f in range(s.F)]
    for X, w, feat, dfeat, got in sides:
        acc = None
        for b in range(B):
            for h in range(H):
                g = orc.phi_mlp_backward_weights(f64(X[b, h]), *w, f64(dfeat[b, h]) * (feat[b, h] > 0), relu=False)
                acc = g if acc is None else tuple(a + c for a, c in zip(acc, g))
        for t, ref in zip(got, acc):
            assert relerr(t.float().cpu().numpy(), ref) < TOL["bf16"]


def test_bounded_wait_reports_timeout_and_context_stays_usable():
    """Failure detection without a fault: a wait that nothing satisfies runs out after its limit, the kernel returns,
    the host reads HLA_ERR_DEVICE_TIMEOUT, and the same context computes a correct forward afterwards."""
    s = synth.HlaShape("t", 1, 2, 300, 128, "bf16", "inv_sqrt_d")
    _, _, V = synth.make_qkv(s)
    qf, kf = synth.make_features(s)
    run = DeviceRun(s, "none", EPS)
    binding.hla_selftest_bounded_wait(run.op.ctx, run.op.workspace)
    assert run.op.device_status() == binding.HLA_ERR_DEVICE_TIMEOUT
    O = run.forward(qf, kf, V)                                    # clears the status words; asserts HLA_OK inside
    Oq, _ = orc.hla_core_forward(qf.astype(np.float64), kf.astype(np.float64), V.astype(np.float64), EPS, "quadratic")
    assert relerr(O, Oq) < TOL["bf16"]


def test_forward_backward_replay_in_a_cuda_graph():
    """The library only enqueues work on the caller's stream, so a whole training step can be captured once in a CUDA
    graph and replayed; the replays must reproduce the eager results bit for bit."""
    s = synth.HlaShape("t", 1, 3, 1500, 128, "bf16", "rms_qk", backward=True)
    Q, K, V = synth.make_qkv(s)
    dO = synth.make_dO(s)
    pq, pk = synth.make_phi_weights(s.d, s.d_phi, s.F, s.dtype)
    run = DeviceRun(s, "mlp", EPS)
    run.set_weights(pq, pk)
    O_ref = run.forward(Q, K, V)
    ref = run.backward(dO)
    op = run.op
    O, dQ, dK, dV = (torch.empty_like(run.V) for _ in range(4))
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            binding.hla_forward(op.ctx, run.Q, run.K, run.V, O, op.workspace, side)
            binding.hla_backward(op.ctx, run.Q, run.K, run.V, O, run.dO, dQ, dK, dV, op.workspace, side)
    for _ in range(2):
        for t in (O, dQ, dK, dV):
            t.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert op.device_status() == binding.HLA_OK
        assert np.array_equal(O.float().cpu().numpy(), O_ref.astype(np.float32))
        for got, want in zip((dQ, dK, dV), ref):
            assert np.array_equal(got.float().cpu().numpy(), want.astype(np.float32))
