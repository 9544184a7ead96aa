"""hla_forward_static: the forward on the scratch array that the library itself carries.

It exists for callers that cannot allocate device memory when they need the operator - code running inside a
host application that owns the allocator, or a loop that must not allocate after start-up - so they cannot
provide the workspace hla_forward asks for.  The test calls it through the C ABI twice in a row (the array is
shared and keeps the previous call's contents, so the second call must not be disturbed by the first) and checks
both results against hla_forward with an ordinary workspace.  The file name sorts last on purpose: a run that
stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

from paper_2602_12128_b200 import binding, synth
from hla_testlib import TOL, relerr, to_dev, to_np

EPS = 1e-6


@pytest.mark.gpu
@pytest.mark.parametrize("dtype,d,N,H", [("bf16", 128, 1000, 2), ("f32", 16, 333, 3)])
def test_static_scratch_forward_matches_workspace_forward(dtype, d, N, H):
    s = synth.HlaShape("t", 1, H, N, d, dtype, "inv_sqrt_d")
    _, _, V = synth.make_qkv(s)
    qf, kf = synth.make_features(s)
    qd, kd, vd = to_dev(qf, "f32"), to_dev(kf, "f32"), to_dev(V, dtype)
    op = binding.Hla(s.B, s.H, s.N, s.d, dtype=dtype, phi="none", eps=EPS)
    assert binding.hla_workspace_bytes(op.ctx) <= binding.HLA_STATIC_WS_BYTES
    ref = to_np(op.forward(qd, kd, vd))
    torch.cuda.synchronize()
    assert op.device_status() == binding.HLA_OK

    out = torch.empty_like(vd)            # allocated up front: the calls below allocate nothing
    results = []
    for call in range(2):
        out.fill_(float("nan"))
        scratch = binding.hla_forward_static(op.ctx, qd, kd, vd, out)
        assert scratch and scratch % 256 == 0
        assert binding.hla_last_device_status(op.ctx, scratch) == binding.HLA_OK      # synchronises the stream
        got = to_np(out)
        assert np.all(np.isfinite(got)), call
        assert relerr(got, ref) < TOL[dtype], (call, relerr(got, ref))
        results.append(got)
    # same kernels in the same order with fixed-order reductions: both calls agree with the workspace path bit for bit
    assert np.array_equal(results[0], ref) and np.array_equal(results[1], ref)


class _RawDeviceBytes:
    """Zero-copy view of `nbytes` of device memory at `ptr` for torch.as_tensor."""

    def __init__(self, ptr, nbytes):
        self.__cuda_array_interface__ = {"shape": (nbytes,), "typestr": "|u1", "data": (ptr, False), "version": 2}


@pytest.mark.gpu
def test_static_scratch_with_phi_maps_after_another_user_and_as_backward_workspace():
    """The array is shared by every context and keeps what the last call left.  Here another context (other shape,
    other mode) uses it first and it is then overwritten with NaN bytes, before a forward with the phi maps runs on it;
    hla_backward then takes the array as its workspace (the forward's features and state live there).  Everything
    must agree bit for bit with the same calls on an ordinary workspace: nothing stale is read."""
    s = synth.HlaShape("t", 1, 2, 1000, 128, "bf16", "rms_qk", backward=True)
    Q, K, V = synth.make_qkv(s)
    dO = synth.make_dO(s)
    pq, pk = synth.make_phi_weights(s.d, s.d_phi, s.F, s.dtype)
    op = binding.Hla(s.B, s.H, s.N, s.d, dtype="bf16", phi="mlp", eps=EPS)
    op.set_phi(tuple(to_dev(a, "bf16") for a in pq), [tuple(to_dev(a, "bf16") for a in w) for w in pk])
    assert binding.hla_workspace_bytes(op.ctx) <= binding.HLA_STATIC_WS_BYTES
    Qd, Kd, Vd, dOd = (to_dev(a, "bf16") for a in (Q, K, V, dO))
    O_ref = op.forward(Qd, Kd, Vd)
    ref = [to_np(t) for t in (O_ref,) + tuple(op.backward(Qd, Kd, Vd, O_ref, dOd))]
    torch.cuda.synchronize()
    assert op.device_status() == binding.HLA_OK

    # another user of the array: a feature-level fp32 context of a different shape
    t = synth.HlaShape("u", 1, 3, 333, 16, "f32", "inv_sqrt_d")
    _, _, Vt = synth.make_qkv(t)
    qf, kf = synth.make_features(t)
    other = binding.Hla(t.B, t.H, t.N, t.d, dtype="f32", phi="none", eps=EPS)
    vt = to_dev(Vt, "f32")
    scratch = binding.hla_forward_static(other.ctx, to_dev(qf, "f32"), to_dev(kf, "f32"), vt, torch.empty_like(vt))
    assert binding.hla_last_device_status(other.ctx, scratch) == binding.HLA_OK
    view = torch.as_tensor(_RawDeviceBytes(scratch, binding.HLA_STATIC_WS_BYTES), device="cuda")
    assert view.data_ptr() == scratch

    out, dQ, dK, dV = (torch.empty_like(Vd) for _ in range(4))
    for call in range(2):
        view.fill_(0xFF)                     # every fp32 / bf16 word of the array is now a NaN
        for x in (out, dQ, dK, dV):
            x.fill_(float("nan"))
        assert binding.hla_forward_static(op.ctx, Qd, Kd, Vd, out) == scratch
        binding.hla_backward(op.ctx, Qd, Kd, Vd, out, dOd, dQ, dK, dV, scratch, workspace_bytes=binding.HLA_STATIC_WS_BYTES)
        assert binding.hla_last_device_status(op.ctx, scratch) == binding.HLA_OK
        for got, want in zip((out, dQ, dK, dV), ref):
            assert np.array_equal(to_np(got), want), call


def test_static_scratch_refuses_shapes_that_need_more():
    big = binding.Hla(2, 24, 32760, 128, dtype="bf16", phi="mlp", eps=EPS, device=None)      # no workspace tensor is created
    assert binding.hla_workspace_bytes(big.ctx) > binding.HLA_STATIC_WS_BYTES
    p = 0x10000                                                                               # never dereferenced
    st = binding.load_library().hla_forward_static(big.ctx, p, p, p, p, None, None)
    assert st == binding.HLA_ERR_WORKSPACE
    assert binding.load_library().hla_forward_static(None, p, p, p, p, None, None) == binding.HLA_ERR_INVALID_ARG
