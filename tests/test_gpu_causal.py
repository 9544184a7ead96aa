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


def test_causal_backward_is_refused():
    s, qf, kf, V = feature_case(128, 300, 1, 1)
    run = DeviceRun(s, "none", EPS, causal=True)
    O = run.forward(qf, kf, V)
    with pytest.raises(binding.HlaError) as e:
        run.backward(synth.make_dO(s))
    assert e.value.status == binding.HLA_ERR_UNSUPPORTED
