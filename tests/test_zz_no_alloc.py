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


def test_static_scratch_refuses_shapes_that_need_more():
    big = binding.Hla(2, 24, 32760, 128, dtype="bf16", phi="mlp", eps=EPS, device=None)      # no workspace tensor is created
    assert binding.hla_workspace_bytes(big.ctx) > binding.HLA_STATIC_WS_BYTES
    p = 0x10000                                                                               # never dereferenced
    st = binding.load_library().hla_forward_static(big.ctx, p, p, p, p, None, None)
    assert st == binding.HLA_ERR_WORKSPACE
    assert binding.load_library().hla_forward_static(None, p, p, p, p, None, None) == binding.HLA_ERR_INVALID_ARG
