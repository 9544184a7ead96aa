"""The half-pass entry points (hla_forward_keys / _queries, hla_backward_queries / _keys) on one GPU: with one shard they
reproduce the whole calls bit for bit; with a sequence cut into two shards that run one after the other, and the states
added in between (what an all-reduce over two devices would do), every shard gets its slice of the unsharded result."""
import numpy as np
import pytest
import torch

from oracle import hla_oracle as orc
from paper_2602_12128_b200 import binding, multi, synth
from hla_testlib import DeviceRun, TOL, relerr, to_dev, to_np, dev_weights

pytestmark = pytest.mark.gpu
EPS = 1e-6
f64 = lambda a: a.astype(np.float64)


def make(phi, N, d=128, H=2):
    s = synth.HlaShape("t", 1, H, N, d, "bf16", "inv_sqrt_d")
    Q, K, V = synth.make_qkv(s)
    dO = synth.make_dO(s)
    if phi == "none":
        V = synth.bf16_round(V * np.float32(np.sqrt(d)))
        Q, K = synth.make_features(s)
    return s, Q, K, V, dO


@pytest.mark.parametrize("phi", ["none", "mlp"])
def test_one_shard_halves_equal_the_whole_calls(phi):
    s, Q, K, V, dO = make(phi, 1000)
    pq, pk = synth.make_phi_weights(s.d, s.d_phi, s.F, s.dtype)
    run = DeviceRun(s, phi, EPS)
    if phi == "mlp":
        run.set_weights(pq, pk)
    O = run.forward(Q, K, V)
    dq, dk, dv = run.backward(dO)
    op = run.op
    O2 = torch.empty_like(run.O)
    multi.sharded_forward(op, run.Q, run.K, run.V, O2)
    dQ2, dK2, dV2 = torch.empty_like(run.Q), torch.empty_like(run.K), torch.empty_like(run.V)
    multi.sharded_backward(op, run.Q, run.K, run.V, O2, run.dO, dQ2, dK2, dV2)
    torch.cuda.synchronize()
    assert op.device_status() == binding.HLA_OK
    assert np.array_equal(to_np(O2), O)
    assert np.array_equal(to_np(dQ2), dq) and np.array_equal(to_np(dK2), dk) and np.array_equal(to_np(dV2), dv)


@pytest.mark.parametrize("phi,N,cut", [("none", 1000, 437), ("mlp", 1500, 640), ("none", 300, 128)])
def test_two_shards_one_after_the_other(phi, N, cut):
    s, Q, K, V, dO = make(phi, N)
    pq, pk = synth.make_phi_weights(s.d, s.d_phi, s.F, s.dtype)
    whole = DeviceRun(s, phi, EPS)
    if phi == "mlp":
        whole.set_weights(pq, pk)
    O = whole.forward(Q, K, V)
    dq, dk, dv = whole.backward(dO)
    tok = 2 if phi == "mlp" else None          # token axis of Q, K in this mode (features: K is [B,H,F,N,dphi])
    shards = []
    for lo, hi in ((0, cut), (cut, N)):
        sc = synth.HlaShape("t", 1, s.H, hi - lo, s.d, "bf16", "inv_sqrt_d")
        op = binding.Hla(1, s.H, hi - lo, s.d, dtype="bf16", phi=phi, eps=EPS)
        if phi == "mlp":
            op.set_phi(*dev_weights(pq, pk, "bf16"))
        io = "bf16" if phi == "mlp" else "f32"
        q = to_dev(np.ascontiguousarray(Q[:, :, lo:hi]), io)
        k = to_dev(np.ascontiguousarray(K[:, :, lo:hi] if phi == "mlp" else K[:, :, :, lo:hi]), io)
        v = to_dev(np.ascontiguousarray(V[:, :, lo:hi]), "bf16")
        g = to_dev(np.ascontiguousarray(dO[:, :, lo:hi]), "bf16")
        shards.append(dict(op=op, q=q, k=k, v=v, g=g, o=torch.empty_like(v), dq=torch.empty_like(q), dk=torch.empty_like(k), dv=torch.empty_like(v)))
    # forward: key halves, sum of the states, query halves
    for sh in shards:
        binding.hla_forward_keys(sh["op"].ctx, sh["k"], sh["v"], sh["op"].workspace)
    total = shards[0]["op"].state_region() + shards[1]["op"].state_region()
    for sh in shards:
        sh["op"].state_region().copy_(total)
        binding.hla_forward_queries(sh["op"].ctx, sh["q"], sh["o"], sh["op"].workspace)
    # backward: query halves, sum of the gradient states, key halves
    for sh in shards:
        binding.hla_backward_queries(sh["op"].ctx, sh["q"], sh["k"], sh["v"], sh["o"], sh["g"], sh["dq"], sh["dk"], sh["dv"], sh["op"].workspace)
    dtotal = shards[0]["op"].state_region(True) + shards[1]["op"].state_region(True)
    for sh in shards:
        sh["op"].state_region(True).copy_(dtotal)
        binding.hla_backward_keys(sh["op"].ctx, sh["q"], sh["k"], sh["v"], sh["o"], sh["g"], sh["dq"], sh["dk"], sh["dv"], sh["op"].workspace)
    torch.cuda.synchronize()
    for sh in shards:
        assert sh["op"].device_status() == binding.HLA_OK
    cat = lambda key, axis=2: np.concatenate([to_np(sh[key]) for sh in shards], axis=axis)
    O2, dv2, dq2 = cat("o"), cat("dv"), cat("dq")
    dk2 = cat("dk", 2 if phi == "mlp" else 3)
    # the same arithmetic in a different summation order: compare with the unsharded run, tightly
    assert relerr(O2, O) < 5e-3 and relerr(dv2, dv) < 5e-3, (relerr(O2, O), relerr(dv2, dv))
    if phi == "none":
        assert relerr(dq2, dq) < 5e-3 and relerr(dk2, dk) < 5e-3
        rO, _ = orc.hla_core_forward(f64(Q), f64(K), f64(V), EPS, "factored")
        rq, rk, rv = orc.hla_core_backward(f64(Q), f64(K), f64(V), f64(dO), EPS, "factored")
        assert relerr(O2, rO) < TOL["bf16"] and relerr(dv2, rv) < TOL["bf16"] and relerr(dq2, rq) < TOL["bf16"] and relerr(dk2, rk) < TOL["bf16"]
    else:
        # dQ, dK go through ReLU masks taken from features that differ in the last bf16 bit between the two runs: relative L2
        l2 = lambda a, b: float(np.linalg.norm(a - b) / np.linalg.norm(b))
        assert l2(dq2, dq) < 1e-2 and l2(dk2, dk) < 1e-2, (l2(dq2, dq), l2(dk2, dk))


class _TwoRanks:
    """Stands in for torch.distributed with two ranks on one device: `states` holds what each rank's all_gather would
    deliver (the shards run one after the other, so both states exist before the helper is called)."""

    def __init__(self, rank, states):
        self.rank, self.states = rank, states

    def is_initialized(self):
        return True

    def get_world_size(self):
        return len(self.states)

    def get_rank(self):
        return self.rank

    def all_gather(self, parts, local):
        assert torch.equal(local, self.states[self.rank])
        for dst, src in zip(parts, self.states):
            dst.copy_(src)


@pytest.mark.parametrize("phi,N,cut", [("none", 1000, 437), ("mlp", 1500, 640), ("none", 300, 128)])
def test_causal_two_shards_one_after_the_other(phi, N, cut):
    """Causal forward of a sequence cut into two shards: each shard's pass starts from the state of the tokens before
    it (multi.sharded_causal_forward with the exclusive prefix over the ranks) and gives its slice of the unsharded
    causal result."""
    s, Q, K, V, _ = make(phi, N)
    pq, pk = synth.make_phi_weights(s.d, s.d_phi, s.F, s.dtype)
    whole = DeviceRun(s, phi, EPS, causal=True)
    if phi == "mlp":
        whole.set_weights(pq, pk)
    O = whole.forward(Q, K, V)
    io = "bf16" if phi == "mlp" else "f32"
    shards = []
    for lo, hi in ((0, cut), (cut, N)):
        ops = [binding.Hla(1, s.H, hi - lo, s.d, dtype="bf16", phi=phi, eps=EPS, causal=c) for c in (False, True)]
        if phi == "mlp":
            for op in ops:
                op.set_phi(*dev_weights(pq, pk, "bf16"))
        q = to_dev(np.ascontiguousarray(Q[:, :, lo:hi]), io)
        k = to_dev(np.ascontiguousarray(K[:, :, lo:hi] if phi == "mlp" else K[:, :, :, lo:hi]), io)
        v = to_dev(np.ascontiguousarray(V[:, :, lo:hi]), "bf16")
        shards.append(dict(plain=ops[0], causal=ops[1], q=q, k=k, v=v, o=torch.empty_like(v)))
    states = []
    for sh in shards:      # what every rank holds before the all_gather
        binding.hla_forward_keys(sh["plain"].ctx, sh["k"], sh["v"], sh["plain"].workspace)
        states.append(sh["plain"].state_region().clone())
    for r, sh in enumerate(shards):
        multi.sharded_causal_forward(sh["causal"], sh["plain"], sh["q"], sh["k"], sh["v"], sh["o"], dist=_TwoRanks(r, states))
    torch.cuda.synchronize()
    for sh in shards:
        assert sh["causal"].device_status() == binding.HLA_OK and sh["plain"].device_status() == binding.HLA_OK
    O2 = np.concatenate([to_np(sh["o"]) for sh in shards], axis=2)
    assert relerr(O2, O) < 5e-3, relerr(O2, O)
    if phi == "none":
        rO, _ = orc.hla_core_forward(f64(Q), f64(K), f64(V), EPS, "causal_quadratic")
        assert relerr(O2, rO) < TOL["bf16"], relerr(O2, rO)
    # the first shard starts from nothing: its slice is the causal result of its own tokens, bit for bit
    first = binding.Hla(1, s.H, cut, s.d, dtype="bf16", phi=phi, eps=EPS, causal=True)
    if phi == "mlp":
        first.set_phi(*dev_weights(pq, pk, "bf16"))
    o1 = first.forward(shards[0]["q"], shards[0]["k"], shards[0]["v"])
    torch.cuda.synchronize()
    assert np.array_equal(to_np(o1), to_np(shards[0]["o"]))


def test_halves_are_refused_where_they_do_not_exist():
    s, Q, K, V, dO = make("none", 300)
    run = DeviceRun(s, "none", EPS, causal=True)
    run.forward(Q, K, V)
    with pytest.raises(binding.HlaError) as e:
        binding.hla_forward_keys(run.op.ctx, run.K, run.V, run.op.workspace)
    assert e.value.status == binding.HLA_ERR_UNSUPPORTED
