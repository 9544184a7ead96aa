"""GPU parity of the fp32 SIMT path (and of bf16 shapes outside the tensor-core
set) against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import hla_oracle as orc
from paper_2602_12128_b200 import binding, synth
from hla_testlib import DeviceRun, TOL, oracle_state, relerr

pytestmark = pytest.mark.gpu
EPS = 1e-6


def test_config1_tiny_f32_forward_mlp():
    """B=1,H=2,N=256,d=16 fp32, Q,K,V ~ N(0,1)/sqrt(d): full output against the quadratic definition."""
    s = synth.CONFIGS["tiny_f32"]
    Q, K, V = synth.make_qkv(s)
    pq, pk = synth.make_phi_weights(s.d, s.d_phi, s.F, s.dtype)
    run = DeviceRun(s, "mlp", EPS)
    run.set_weights(pq, pk)
    O = run.forward(Q, K, V)
    Oq, eta, qf, kf = orc.hla_forward(Q, K, V, pq, pk, EPS, "quadratic")
    gq, gk = run.features()
    assert relerr(gq, qf) < TOL["f32"] and relerr(gk, kf) < TOL["f32"]
    assert relerr(run.eta(), eta) < TOL["f32"]
    assert O.shape == (1, 2, 256, 16)
    assert relerr(O, Oq) < TOL["f32"]
    assert run.op.launches() == 5


@pytest.mark.parametrize("F,dphi,d,N,splits", [(3, 6, 16, 256, 0), (2, 12, 32, 333, 3), (1, 8, 8, 50, 1), (4, 4, 128, 97, 0),
                                                (3, 6, 128, 1000, 7), (3, 3, 4, 5, 0)])
def test_core_forward_f32_features(F, dphi, d, N, splits):
    s = synth.HlaShape("t", 2, 3, N, d, "f32", "inv_sqrt_d", F=F, d_phi=dphi)
    _, _, V = synth.make_qkv(s)
    qf, kf = synth.make_features(s)
    run = DeviceRun(s, "none", EPS, splits)
    O = run.forward(qf, kf, V)
    Oq, eta = orc.hla_core_forward(qf.astype(np.float64), kf.astype(np.float64), V.astype(np.float64), EPS, "quadratic")
    assert relerr(O, Oq) < TOL["f32"]
    assert relerr(run.eta(), eta) < TOL["f32"]
    C, z = run.state()
    Co, zo = oracle_state(kf.astype(np.float64), V.astype(np.float64))
    assert relerr(C, Co) < TOL["f32"] and relerr(z, zo) < TOL["f32"]


@pytest.mark.parametrize("F,dphi,d,N", [(3, 6, 16, 200), (2, 12, 64, 77), (1, 8, 8, 40), (3, 4, 128, 130)])
def test_core_backward_f32_features(F, dphi, d, N):
    s = synth.HlaShape("t", 1, 2, N, d, "f32", "inv_sqrt_d", F=F, d_phi=dphi)
    _, _, V = synth.make_qkv(s)
    qf, kf = synth.make_features(s)
    dO = synth.make_dO(s)
    run = DeviceRun(s, "none", EPS)
    run.forward(qf, kf, V)
    dq, dk, dv = run.backward(dO)
    rq, rk, rv = orc.hla_core_backward(qf.astype(np.float64), kf.astype(np.float64), V.astype(np.float64), dO.astype(np.float64), EPS, "quadratic")
    assert relerr(dv, rv) < TOL["f32"]
    assert relerr(dq, rq) < TOL["f32"]
    assert relerr(dk, rk) < TOL["f32"]
    dC, dz = run.state("dstate")
    assert np.all(np.isfinite(dC)) and np.all(np.isfinite(dz))


def test_full_backward_f32_mlp():
    s = synth.HlaShape("t", 1, 2, 150, 16, "f32", "rms_qk")
    Q, K, V = synth.make_qkv(s)
    dO = synth.make_dO(s)
    pq, pk = synth.make_phi_weights(s.d, s.d_phi, s.F, s.dtype)
    run = DeviceRun(s, "mlp", EPS)
    run.set_weights(pq, pk)
    O = run.forward(Q, K, V)
    dQ, dK, dV = run.backward(dO)
    rQ, rK, rV, _, _ = orc.hla_backward(*(a.astype(np.float64) for a in (Q, K, V, dO)), pq, pk, EPS, "quadratic")
    assert relerr(O, orc.hla_forward(Q, K, V, pq, pk, EPS, "quadratic")[0]) < TOL["f32"]
    assert relerr(dV, rV) < TOL["f32"]
    assert relerr(dQ, rQ) < 2 * TOL["f32"]
    assert relerr(dK, rK) < 2 * TOL["f32"]
    assert run.op.launches() == 7


def test_bf16_shape_outside_tensor_core_set_runs_simt():
    s = synth.HlaShape("t", 1, 2, 300, 32, "bf16", "rms_qk")
    Q, K, V = synth.make_qkv(s)
    pq, pk = synth.make_phi_weights(s.d, s.d_phi, s.F, s.dtype)
    run = DeviceRun(s, "mlp", EPS)
    assert run.op.layout.tensor_core == 0
    run.set_weights(pq, pk)
    O = run.forward(Q, K, V)
    gq, gk = run.features()
    Oc, _ = orc.hla_core_forward(gq, gk, V.astype(np.float64), EPS)
    assert relerr(O, Oc) < TOL["bf16"]
    _, _, qf, kf = orc.hla_forward(Q, K, V, pq, pk, EPS)
    assert relerr(gq, qf) < 1e-4 and relerr(gk, kf) < 1e-4


def test_bitwise_reproducible():
    s = synth.HlaShape("t", 1, 2, 500, 16, "f32", "inv_sqrt_d")
    _, _, V = synth.make_qkv(s)
    qf, kf = synth.make_features(s)
    run = DeviceRun(s, "none", EPS, 5)
    a = run.forward(qf, kf, V)
    b = run.forward(qf, kf, V)
    assert np.array_equal(a, b)
