"""GPU parity of the value modulation  Out = T + phi_v1(T) (.) phi_v2(V)  (Section 4.5) and of its input gradients against
the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import hla_oracle as orc
from paper_2602_12128_b200 import binding, synth
from hla_testlib import TOL, relerr, report, to_dev, to_np

pytestmark = pytest.mark.gpu
f64 = lambda a: np.asarray(a, np.float64)


def make_vmlp(d, seed):
    """ln_g ~ 1 + 0.2 N, ln_b ~ 0.1 N, W1, W2 ~ N(0, 1/d), biases 0.1 N; bf16-exact float32 arrays."""
    rng = np.random.default_rng(seed)
    r = lambda *s: rng.standard_normal(s, dtype=np.float32)
    w = (1.0 + 0.2 * r(d), 0.1 * r(d), r(d, d) / np.sqrt(d), 0.1 * r(d), r(d, d) / np.sqrt(d), 0.1 * r(d))
    return tuple(synth.bf16_round(np.asarray(a, np.float32)) for a in w)


def setup(d, N, B, H, seed=0):
    s = synth.HlaShape("t", B, H, N, d, "bf16", "inv_sqrt_d")
    rng = np.random.default_rng(seed)
    T = synth.bf16_round(rng.standard_normal((B, H, N, d), dtype=np.float32) * 0.7 + 0.2)      # attention results: O(1), not centred
    V = synth.bf16_round(rng.standard_normal((B, H, N, d), dtype=np.float32))
    dOut = synth.bf16_round(rng.standard_normal((B, H, N, d), dtype=np.float32))
    v1, v2 = make_vmlp(d, 7), make_vmlp(d, 8)
    op = binding.Hla(B, H, N, d, dtype="bf16", phi="none", eps=1e-6, value_mod=True)
    op.set_phi_v(tuple(to_dev(a, "bf16") for a in v1), tuple(to_dev(a, "bf16") for a in v2))
    return s, op, (T, V, dOut), (v1, v2)


def oracle_forward(T, V, v1, v2):
    B, H = T.shape[:2]
    out = np.empty(T.shape)
    for b in range(B):
        for h in range(H):
            out[b, h] = orc.value_modulation(f64(T[b, h]), f64(V[b, h]), v1, v2)
    return out


@pytest.mark.parametrize("d,N,B,H", [(128, 1000, 1, 2), (64, 777, 2, 2), (128, 77, 1, 1), (128, 4096 + 5, 1, 3)])
def test_value_modulation_forward(d, N, B, H):
    s, op, (T, V, _), (v1, v2) = setup(d, N, B, H)
    Td, Vd = to_dev(T, "bf16"), to_dev(V, "bf16")
    out = op.value_mod_forward(Td, Vd)
    torch.cuda.synchronize()
    assert op.device_status() == binding.HLA_OK
    assert op.launches() == 3                     # weight folding, phi_v2(V), T + phi_v1(T) (.) Y2
    ref = oracle_forward(T, V, v1, v2)
    got = to_np(out)
    # the update alone (Out - T) against the oracle's, so that the residual does not hide an error of the product
    upd, upd_ref = got - f64(T), ref - f64(T)
    report(f"value modulation forward d={d} N={N}", out=relerr(got, ref), update=relerr(upd, upd_ref))
    assert relerr(got, ref) < TOL["bf16"]
    assert relerr(upd, upd_ref) < TOL["bf16"]
    again = to_np(op.value_mod_forward(Td, Vd))
    assert np.array_equal(got, again)


@pytest.mark.parametrize("d,N,B,H", [(128, 900, 1, 2), (64, 300, 1, 2), (128, 130, 1, 1)])
def test_value_modulation_backward(d, N, B, H):
    s, op, (T, V, dOut), (v1, v2) = setup(d, N, B, H, seed=3)
    Td, Vd, dOd = to_dev(T, "bf16"), to_dev(V, "bf16"), to_dev(dOut, "bf16")
    op.value_mod_forward(Td, Vd)                  # the step's forward (it also starts the record of device-side time-outs)
    dT, dV = op.value_mod_backward(Td, Vd, dOd)
    torch.cuda.synchronize()
    assert op.device_status() == binding.HLA_OK
    assert op.launches() == 5                     # folding, both maps forward, the two backward passes
    rT, rV = np.empty(T.shape), np.empty(V.shape)
    for b in range(B):
        for h in range(H):
            rT[b, h], rV[b, h] = orc.value_modulation_backward(f64(T[b, h]), f64(V[b, h]), f64(dOut[b, h]), v1, v2)
    gT, gV = to_np(dT), to_np(dV)
    report(f"value modulation backward d={d} N={N}", dT=relerr(gT, rT), dV=relerr(gV, rV), dT_without_residual=relerr(gT - f64(dOut), rT - f64(dOut)))
    assert relerr(gT, rT) < TOL["bf16"] and relerr(gV, rV) < TOL["bf16"]
    assert relerr(gT - f64(dOut), rT - f64(dOut)) < TOL["bf16"]
    # accumulate_dV adds the V-side gradient to what dV holds
    base = synth.bf16_round(np.random.default_rng(5).standard_normal(V.shape, dtype=np.float32))
    dV2 = to_dev(base, "bf16")
    op.value_mod_backward(Td, Vd, dOd, dT, dV2, accumulate_dV=True)
    torch.cuda.synchronize()
    assert relerr(to_np(dV2), f64(base) + rV) < TOL["bf16"]
    assert op.device_status() == binding.HLA_OK


def test_value_modulation_after_the_operator():
    """The whole block tail on one context: hla_forward, then the value modulation of its output; backward through both,
    with the V gradients of the two stages accumulated by the library."""
    s = synth.HlaShape("t", 1, 2, 1100, 128, "bf16", "rms_qk", backward=True)
    Q, K, V = synth.make_qkv(s)
    dOut = synth.make_dO(s)
    pq, pk = synth.make_phi_weights(s.d, s.d_phi, s.F, s.dtype)
    v1, v2 = make_vmlp(s.d, 7), make_vmlp(s.d, 8)
    op = binding.Hla(s.B, s.H, s.N, s.d, dtype="bf16", phi="mlp", eps=1e-6, value_mod=True)
    op.set_phi(tuple(to_dev(a, "bf16") for a in pq), [tuple(to_dev(a, "bf16") for a in w) for w in pk])
    op.set_phi_v(tuple(to_dev(a, "bf16") for a in v1), tuple(to_dev(a, "bf16") for a in v2))
    Qd, Kd, Vd, dOd = (to_dev(a, "bf16") for a in (Q, K, V, dOut))
    O = op.forward(Qd, Kd, Vd)
    out = op.value_mod_forward(O, Vd)
    # backward: through the modulation first (dT is the upstream gradient of the operator), then the operator, then the
    # V-side gradient of the modulation is added to the dV the operator wrote
    dT, _ = op.value_mod_backward(O, Vd, dOd)
    dQ, dK, dV = op.backward(Qd, Kd, Vd, O, dT)
    op.value_mod_backward(O, Vd, dOd, torch.empty_like(dT), dV, accumulate_dV=True)
    torch.cuda.synchronize()
    assert op.device_status() == binding.HLA_OK
    # stage-wise references: the modulation at the attention output the GPU produced, the operator's dV at the dT the GPU produced
    Og, dTg = to_np(O), to_np(dT)
    ref_out = oracle_forward(Og, V, v1, v2)
    assert relerr(to_np(out), ref_out) < TOL["bf16"]
    nq = s.B * s.H * s.N * s.d_phi
    gq = to_np(op.region("qf")[:nq]).reshape(s.B, s.H, s.N, s.d_phi)
    gk = to_np(op.region("kf")[: nq * s.F]).reshape(s.B, s.H, s.F, s.N, s.d_phi)
    _, _, dV_core = orc.hla_core_backward(gq, gk, f64(V), dTg, 1e-6, "factored")
    dV_mod = np.empty(V.shape)
    for b in range(s.B):
        for h in range(s.H):
            rT, dV_mod[b, h] = orc.value_modulation_backward(Og[b, h], f64(V[b, h]), f64(dOut[b, h]), v1, v2)
            assert relerr(dTg[b, h], rT) < TOL["bf16"]
    assert relerr(to_np(dV), dV_core + dV_mod) < TOL["bf16"]


@pytest.mark.parametrize("name", ["dit_bf16", "train_bf16"])
def test_value_modulation_at_the_benchmark_shapes(name):
    """Full-size shapes (video-DiT forward, training step): forward and input gradients on sampled token rows of every
    head against the oracle (every token is independent of the others in this stage), plus finiteness of everything."""
    c = synth.CONFIGS[name]
    rng = np.random.default_rng(17)
    dims = (c.B, c.H, c.N, c.d)
    g = torch.Generator(device="cuda")
    g.manual_seed(5)
    Td = (torch.randn(dims, generator=g, device="cuda") * 0.7 + 0.2).to(torch.bfloat16)
    Vd = torch.randn(dims, generator=g, device="cuda").to(torch.bfloat16)
    dOd = torch.randn(dims, generator=g, device="cuda").to(torch.bfloat16)
    v1, v2 = make_vmlp(c.d, 7), make_vmlp(c.d, 8)
    op = binding.Hla(c.B, c.H, c.N, c.d, dtype="bf16", phi="none", eps=1e-6, value_mod=True)
    op.set_phi_v(tuple(to_dev(a, "bf16") for a in v1), tuple(to_dev(a, "bf16") for a in v2))
    out = op.value_mod_forward(Td, Vd)
    dT, dV = op.value_mod_backward(Td, Vd, dOd)
    torch.cuda.synchronize()
    assert op.device_status() == binding.HLA_OK
    for t in (out, dT, dV):
        assert bool(torch.isfinite(t).all())
    worst = {"out": 0.0, "dT": 0.0, "dV": 0.0}
    for b in range(c.B):
        for h in range(c.H):
            rows = np.sort(rng.choice(c.N, 64, replace=False))
            rows[-1] = c.N - 1                                   # the ragged tail of the head
            idx = torch.from_numpy(rows).cuda()
            Ts, Vs, dOs = (to_np(x[b, h].index_select(0, idx)) for x in (Td, Vd, dOd))
            ref = orc.value_modulation(Ts, Vs, v1, v2)
            rT, rV = orc.value_modulation_backward(Ts, Vs, dOs, v1, v2)
            worst["out"] = max(worst["out"], relerr(to_np(out[b, h].index_select(0, idx)), ref))
            worst["dT"] = max(worst["dT"], relerr(to_np(dT[b, h].index_select(0, idx)), rT))
            worst["dV"] = max(worst["dV"], relerr(to_np(dV[b, h].index_select(0, idx)), rV))
    report(f"value modulation at {name}", **worst)
    assert max(worst.values()) < TOL["bf16"], worst
