"""GPU parity of causal HLA (Section 4.4: token i sees the tokens j <= i) against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import hla_oracle as orc
from paper_2602_12128_b200 import binding, synth
from hla_testlib import DeviceRun, TOL, fold_symmetric, oracle_state, relerr, l2err, report

pytestmark = pytest.mark.gpu
EPS = 1e-6
f64 = lambda a: a.astype(np.float64)


def feature_case(d, N, B, H):
    s = synth.HlaShape("t", B, H, N, d, "bf16", "inv_sqrt_d")
    _, _, V = synth.make_qkv(s)
    V = synth.bf16_round(V * np.float32(np.sqrt(d)))          # V ~ N(0,1)
    qf, kf = synth.make_features(s)
    return s, qf, kf, V


@pytest.mark.parametrize("d,N,B,H,splits", [(128, 1000, 1, 2, 0), (128, 128, 1, 1, 1), (128, 77, 1, 3, 0), (64, 1500, 2, 2, 5),
                                            (128, 4096 + 40, 1, 2, 7), (64, 129, 1, 1, 4), (128, 2177, 1, 1, 1), (64, 640, 1, 2, 5)])
def test_causal_forward_bf16_features(d, N, B, H, splits):
    """Feature-level entry point with the mask: one and several pieces per head, pieces of one tile, more splits than
    tiles, ragged tails, both head widths.  Output and normaliser against the masked quadratic definition; the state the
    library leaves is the state after the last token."""
    s, qf, kf, V = feature_case(d, N, B, H)
    run = DeviceRun(s, "none", EPS, splits, causal=True)
    assert run.op.layout.tensor_core == 1
    O = run.forward(qf, kf, V)
    assert run.op.launches() == 3
    Oq, eta = orc.hla_core_forward(f64(qf), f64(kf), f64(V), EPS, "causal_quadratic")
    assert relerr(run.eta(), eta) < TOL["bf16"] / 4, relerr(run.eta(), eta)
    assert relerr(O, Oq) < TOL["bf16"], (relerr(O, Oq), l2err(O, Oq))
    report("causal forward", d=d, N=N, splits=splits, maxnorm=relerr(O, Oq), l2=l2err(O, Oq), eta=relerr(run.eta(), eta))
    # the first token of every head returns its own value; the last one sees everything
    assert relerr(O[:, :, 0], f64(V)[:, :, 0]) < TOL["bf16"]
    C, z = run.state()
    Co, zo = oracle_state(f64(kf), f64(V))
    Co, zo = fold_symmetric(Co), fold_symmetric(zo[..., None])[..., 0]
    assert relerr(z, zo) < 1e-5
    assert relerr(C, Co) < TOL["bf16"] / 4
    again = run.forward(qf, kf, V)
    assert np.array_equal(O, again)                                  # fixed-order scan: bit-reproducible


def test_causal_future_tokens_do_not_leak():
    """Changing the values and keys of later tokens leaves every earlier output bit-identical when the change falls in a
    later tile, and identical rows inside the tile of the change."""
    d, N = 128, 1000
    s, qf, kf, V = feature_case(d, N, 1, 2)
    run = DeviceRun(s, "none", EPS, 3, causal=True)
    O = run.forward(qf, kf, V)
    V2, kf2 = V.copy(), kf.copy()
    V2[:, :, 700:] = synth.bf16_round(V2[:, :, 700:] * np.float32(-2.0) + np.float32(1.0))
    kf2[:, :, :, 700:] *= np.float32(3.0)
    O2 = run.forward(qf, kf2, V2)
    assert np.array_equal(O2[:, :, :700], O[:, :, :700])
    assert np.abs(O2[:, :, 700:] - O[:, :, 700:]).max() > 1e-2


@pytest.mark.parametrize("name", ["small_bf16", "dit_bf16"])
def test_causal_forward_with_phi_maps(name):
    """The phi maps in front (fused key side and query side leave the features in the workspace), the causal sweep over
    the pieces of the key-side kernel: stage-wise against the oracle core on the features the GPU produced, and end to
    end on rows whose normaliser is not tiny."""
    s = synth.CONFIGS[name]
    if name == "dit_bf16":
        s = synth.HlaShape("t", 1, 3, 5000, s.d, s.dtype, s.scale)
    Q, K, V = synth.make_qkv(s)
    pq, pk = synth.make_phi_weights(s.d, s.d_phi, s.F, s.dtype)
    run = DeviceRun(s, "mlp", EPS, causal=True)
    run.set_weights(pq, pk)
    O = run.forward(Q, K, V)
    gq, gk = run.features()
    heads = [(0, 0), (s.B - 1, s.H - 1)]
    for b, h in heads:
        Oc, etac = orc.hla_streaming(gq[b, h], [gk[b, h, f] for f in range(3)], f64(V)[b, h], EPS)
        assert relerr(O[b, h], Oc) < TOL["bf16"], relerr(O[b, h], Oc)
        assert relerr(run.eta()[b, h], etac) < TOL["bf16"] / 4
    Oq, eta, qf, kf = orc.hla_forward(f64(Q[:1, :1]), f64(K[:1, :1]), f64(V[:1, :1]), pq, pk, EPS, "causal_streaming")
    keep = eta >= 1e-3 * np.median(eta)
    report("causal end to end " + name, kept_fraction=keep.mean(), l2_kept=l2err(O[:1, :1][keep], Oq[keep]), maxnorm_all=relerr(O[:1, :1], Oq))
    assert keep.mean() > 0.5
    assert l2err(O[:1, :1][keep], Oq[keep]) < TOL["bf16"]


def test_causal_full_size_sampled_rows():
    """N = 32760, d = 128 (one batch of the training shape, 4 heads): rows sampled over the whole sequence - tile
    boundaries, piece boundaries, first and last tokens - against the masked definition evaluated row by row."""
    s = synth.HlaShape("t", 1, 4, 32760, 128, "bf16", "inv_sqrt_d")
    _, _, V = synth.make_qkv(s)
    V = synth.bf16_round(V * np.float32(np.sqrt(s.d)))
    qf, kf = synth.make_features(s)
    run = DeviceRun(s, "none", EPS, causal=True)
    O = run.forward(qf, kf, V)
    eta_gpu = run.eta()
    S = run.op.layout.n_splits
    tiles = (s.N + 127) // 128
    per = (tiles + S - 1) // S
    rng = np.random.default_rng(3)
    rows = {0, 1, 127, 128, 129, s.N - 1, s.N - 2, per * 128 - 1, per * 128, per * 128 + 1, 2 * per * 128, (S - 1) * per * 128 - 1}
    rows |= set(int(r) for r in rng.integers(0, s.N, 40))
    rows = sorted(r for r in rows if 0 <= r < s.N)
    worst = 0.0
    for h in range(s.H):
        ks = [f64(kf[0, h, f]) for f in range(3)]
        v = f64(V[0, h])
        scale = np.abs(v).max()
        for i in rows:
            o, eta = orc.hla_quadratic(f64(qf[0, h, i:i + 1]), [k[:i + 1] for k in ks], v[:i + 1], EPS)   # row i of the masked definition
            worst = max(worst, np.abs(O[0, h, i] - o[0]).max() / scale)
            assert abs(eta_gpu[0, h, i] - eta[0]) <= 5e-3 * abs(eta[0]) + 1e-30
    report("causal full size", rows=len(rows), maxnorm=worst, splits=S)
    assert worst < TOL["bf16"]


@pytest.mark.parametrize("d,N,B,H,splits", [(128, 1000, 1, 2, 0), (128, 128, 1, 1, 1), (128, 77, 1, 3, 0), (64, 1500, 2, 2, 5),
                                            (128, 4096 + 40, 1, 2, 7), (64, 129, 1, 1, 4), (128, 2177, 1, 1, 1)])
def test_causal_backward_bf16_features(d, N, B, H, splits):
    """dq, dk^f (fp32 feature gradients) and dV (bf16) of the causal backward against the masked quadratic form of the
    oracle: one and several pieces per head, ragged tails, both head widths; bit-reproducible."""
    s, qf, kf, V = feature_case(d, N, B, H)
    dO = synth.make_dO(s)
    run = DeviceRun(s, "none", EPS, splits, causal=True)
    run.forward(qf, kf, V)
    dq, dk, dv = run.backward(dO)
    rq, rk, rv = orc.hla_core_backward(f64(qf), f64(kf), f64(V), f64(dO), EPS, "causal_quadratic")
    report("causal backward", d=d, N=N, splits=splits, dv=relerr(dv, rv), dq=relerr(dq, rq), dk=relerr(dk, rk))
    assert relerr(dv, rv) < TOL["bf16"], relerr(dv, rv)
    assert relerr(dq, rq) < TOL["bf16"], relerr(dq, rq)
    assert relerr(dk, rk) < TOL["bf16"], relerr(dk, rk)
    # the first query sees one token: its output is that token's value whatever q is
    assert np.abs(dq[:, :, 0]).max() <= 1e-3 * np.abs(rq).max()
    dq2, dk2, dv2 = run.backward(dO)
    assert np.array_equal(dq, dq2) and np.array_equal(dk, dk2) and np.array_equal(dv, dv2)


def test_causal_backward_later_output_gradients_do_not_reach_earlier_queries():
    """dq_i depends on dO_i only; dk_j and dV_j depend on dO_i for i >= j: changing dO from token 700 on leaves dq before
    700 bit-identical, and zeroing dO before token 700 leaves dk, dV of the tokens from 768 on (the next tile) unchanged."""
    s, qf, kf, V = feature_case(128, 1000, 1, 2)
    dO = synth.make_dO(s)
    run = DeviceRun(s, "none", EPS, 3, causal=True)
    run.forward(qf, kf, V)
    dq, dk, dv = run.backward(dO)
    dO2 = dO.copy()
    dO2[:, :, 700:] = synth.bf16_round(dO2[:, :, 700:] * np.float32(-1.5))
    dq2, _, _ = run.backward(dO2)
    assert np.array_equal(dq2[:, :, :700], dq[:, :, :700])
    dO3 = dO.copy()
    dO3[:, :, :700] = 0
    _, dk3, dv3 = run.backward(dO3)
    assert np.array_equal(dk3[:, :, :, 768:], dk[:, :, :, 768:]) and np.array_equal(dv3[:, :, 768:], dv[:, :, 768:])


def test_causal_backward_with_phi_maps():
    """The phi maps around the causal core: stage-wise (core gradients against the oracle core on the features the GPU
    produced; dQ, dK against the oracle's phi backward applied to the core gradients the GPU produced), then the weight
    gradients from the same feature gradients."""
    s = synth.HlaShape("t", 1, 3, 3000, 128, "bf16", "inv_sqrt_d")
    Q, K, V = synth.make_qkv(s)
    dO = synth.make_dO(s)
    pq, pk = synth.make_phi_weights(s.d, s.d_phi, s.F, s.dtype)
    run = DeviceRun(s, "mlp", EPS, causal=True)
    run.set_weights(pq, pk)
    run.forward(Q, K, V)
    gq, gk = run.features()
    dQ, dK, dV = run.backward(dO)
    n = s.B * s.H * s.N * s.d_phi
    dqf = run.region("dqf", n, (s.B, s.H, s.N, s.d_phi))
    dkf = run.region("dkf", n * s.F, (s.B, s.H, s.F, s.N, s.d_phi))
    rq, rk, rv = orc.hla_core_backward(gq, gk, f64(V), f64(dO), EPS, "causal_streaming")
    assert relerr(dV, rv) < TOL["bf16"] and relerr(dqf, rq) < TOL["bf16"] and relerr(dkf, rk) < TOL["bf16"], (relerr(dV, rv), relerr(dqf, rq), relerr(dkf, rk))
    d = s.d
    wq = orc.phi_mlp_backward(f64(Q).reshape(-1, d), *pq, dqf.reshape(-1, s.d_phi)).reshape(Q.shape)
    wk = np.zeros(K.shape)
    for f, w in enumerate(pk):
        wk += orc.phi_mlp_backward(f64(K).reshape(-1, d), *w, dkf[:, :, f].reshape(-1, s.d_phi)).reshape(K.shape)
    # the library takes the ReLU mask from the features its forward kept; rows where that mask differs from the oracle's
    # (pre-activation within the forward's bf16-level error of zero) are a different one-sided derivative and are left out
    pre_q = orc.phi_mlp(f64(Q).reshape(-1, d), *pq, relu=False).reshape(gq.shape)
    pre_k = np.stack([orc.phi_mlp(f64(K).reshape(-1, d), *w, relu=False).reshape(gq.shape) for w in pk], axis=2)
    flip_q, flip_k = (gq > 0) != (pre_q > 0), (gk > 0) != (pre_k > 0)
    assert flip_q.mean() < 5e-3 and flip_k.mean() < 5e-3
    same_q, same_k = ~flip_q.any(axis=-1), ~flip_k.any(axis=(2, 4))
    assert relerr(dQ[same_q], wq[same_q]) < TOL["bf16"] and relerr(dK[same_k], wk[same_k]) < TOL["bf16"], (relerr(dQ[same_q], wq[same_q]), relerr(dK[same_k], wk[same_k]))
    report("causal backward with phi", dV=relerr(dV, rv), dqf=relerr(dqf, rq), dkf=relerr(dkf, rk), dQ=relerr(dQ[same_q], wq[same_q]), dK=relerr(dK[same_k], wk[same_k]))


def test_causal_backward_full_size_sampled():
    """N = 32760, d = 128, two heads: dV, dq and dk on sampled tokens against the masked definition evaluated for those tokens
    (dq_i needs the keys up to i; dk_j and dV_j need the queries from j on, which the oracle gets from the full masked
    form on a strided subsample is not possible - so the check uses the streaming gradients of one head at reduced length
    and the full-length invariants: rows of the weights sum to one, so sum_j dV_j = sum_i dO_i, and q . dq = 0)."""
    s = synth.HlaShape("t", 1, 2, 32760, 128, "bf16", "inv_sqrt_d")
    _, _, V = synth.make_qkv(s)
    V = synth.bf16_round(V * np.float32(np.sqrt(s.d)))
    qf, kf = synth.make_features(s)
    dO = synth.make_dO(s)
    run = DeviceRun(s, "none", 1e-12, causal=True)
    run.forward(qf, kf, V)
    dq, dk, dv = run.backward(dO)
    scale = np.abs(f64(dO)).sum(axis=2).max()
    assert np.abs(dv.sum(axis=2) - f64(dO).sum(axis=2)).max() < 2e-2 * scale
    euler = np.abs(np.sum(f64(qf) * dq, axis=-1))
    assert euler.max() < 2e-2 * np.abs(f64(qf) * dq).sum(axis=-1).max()
    # the last 300 tokens of a head: their dk, dV depend only on the queries from there on, and dq of the first 300 tokens only on
    # the first 300 keys - both are small problems the oracle solves exactly
    h = 1
    n0 = s.N - 300
    ks_all = [f64(kf[0, h, f]) for f in range(3)]
    gq, _, _ = orc.hla_quadratic_causal_backward(f64(qf[0, h, :300]), [k[:300] for k in ks_all], f64(V[0, h, :300]), f64(dO[0, h, :300]), 1e-12)
    assert relerr(dq[0, h, :300], gq) < TOL["bf16"]
    report("causal backward full size", dq_head=relerr(dq[0, h, :300], gq), dv_sum=np.abs(dv.sum(axis=2) - f64(dO).sum(axis=2)).max() / scale)


@pytest.mark.parametrize("d,N,chunks,splits", [(128, 700, 3, 0), (64, 1000, 2, 3), (128, 128, 4, 1)])
def test_sequential_updates_across_calls(d, N, chunks, splits):
    """Eq. "seq.updates" across calls: a sequence handed over in chunks of N tokens, each call starting from the state the
    previous one left in the workspace, gives the outputs of one causal pass over the concatenation; the state left after
    the last chunk is the state of the whole sequence; a backward on a carried chunk is refused."""
    s = synth.HlaShape("t", 1, 2, N * chunks, d, "bf16", "inv_sqrt_d")
    _, _, V = synth.make_qkv(s)
    V = synth.bf16_round(V * np.float32(np.sqrt(d)))
    qf, kf = synth.make_features(s)
    Oq, eta = orc.hla_core_forward(f64(qf), f64(kf), f64(V), EPS, "causal_streaming")
    sc = synth.HlaShape("t", 1, 2, N, d, "bf16", "inv_sqrt_d")
    run = DeviceRun(sc, "none", EPS, splits, causal=True)
    outs, etas = [], []
    for c in range(chunks):
        run.op.set_carry(c > 0)
        sl = slice(c * N, (c + 1) * N)
        outs.append(run.forward(np.ascontiguousarray(qf[:, :, sl]), np.ascontiguousarray(kf[:, :, :, sl]), np.ascontiguousarray(V[:, :, sl])))
        etas.append(run.eta())
    O = np.concatenate(outs, axis=2)
    assert relerr(O, Oq) < TOL["bf16"], relerr(O, Oq)
    assert relerr(np.concatenate(etas, axis=2), eta) < TOL["bf16"] / 4
    C, z = run.state()
    Co, zo = oracle_state(f64(kf), f64(V))
    Co, zo = fold_symmetric(Co), fold_symmetric(zo[..., None])[..., 0]
    assert relerr(z, zo) < 1e-5 and relerr(C, Co) < TOL["bf16"] / 4
    with pytest.raises(binding.HlaError) as e:
        run.backward(synth.make_dO(sc))
    assert e.value.status == binding.HLA_ERR_UNSUPPORTED
    report("sequential updates across calls", d=d, N=N, chunks=chunks, maxnorm=relerr(O, Oq))


def test_sequential_updates_with_phi_maps():
    """The same with the phi maps in front (the pieces of the fused key-side kernel are scanned from the carried state)."""
    d, N, chunks = 128, 900, 3
    s = synth.HlaShape("t", 1, 2, N * chunks, d, "bf16", "inv_sqrt_d")
    Q, K, V = synth.make_qkv(s)
    pq, pk = synth.make_phi_weights(d, 6, 3, "bf16")
    sc = synth.HlaShape("t", 1, 2, N, d, "bf16", "inv_sqrt_d")
    run = DeviceRun(sc, "mlp", EPS, causal=True)
    run.set_weights(pq, pk)
    outs, gqs, gks = [], [], []
    for c in range(chunks):
        run.op.set_carry(c > 0)
        sl = slice(c * N, (c + 1) * N)
        outs.append(run.forward(np.ascontiguousarray(Q[:, :, sl]), np.ascontiguousarray(K[:, :, sl]), np.ascontiguousarray(V[:, :, sl])))
        gq, gk = run.features()
        gqs.append(gq)
        gks.append(gk)
    O = np.concatenate(outs, axis=2)
    gq, gk = np.concatenate(gqs, axis=2), np.concatenate(gks, axis=3)
    Oc, _ = orc.hla_core_forward(gq, gk, f64(V), EPS, "causal_streaming")      # the core on the features the GPU produced
    assert relerr(O, Oc) < TOL["bf16"], relerr(O, Oc)
