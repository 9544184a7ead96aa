"""Helpers shared by the GPU parity tests: numpy <-> torch marshalling, the
error metric, and running the library / the oracle on the same seeded inputs."""
from __future__ import annotations

import numpy as np
import torch

from oracle import hla_oracle as orc
from paper_2602_12128_b200 import binding, synth

TOL = {"f32": 1e-4, "bf16": 2e-2}   # max |y - ref| / max |ref|, per tensor


def relerr(y, ref) -> float:
    y = np.asarray(y, np.float64)
    ref = np.asarray(ref, np.float64)
    den = np.max(np.abs(ref))
    return float(np.max(np.abs(y - ref)) / (den if den > 0 else 1.0))


def l2err(y, ref) -> float:
    y = np.asarray(y, np.float64)
    ref = np.asarray(ref, np.float64)
    return float(np.linalg.norm(y - ref) / max(np.linalg.norm(ref), 1e-300))


def report(name: str, **values) -> None:
    """Prints measured parity figures (errors, kept fractions) so that a test log shows how far inside its bound a
    comparison is; with HLA_PARITY_REPORT set to a file path the same record is appended there as a JSON line."""
    import json
    import os
    rec = {"check": name, **{k: (float(v) if np.isscalar(v) else v) for k, v in values.items()}}
    print("parity:", json.dumps(rec))
    path = os.environ.get("HLA_PARITY_REPORT")
    if path:
        with open(path, "a") as f:
            f.write(json.dumps(rec) + "\n")


def to_dev(x: np.ndarray, dtype: str):
    t = torch.from_numpy(np.ascontiguousarray(x))
    if dtype == "bf16":
        t = t.to(torch.bfloat16)
    return t.cuda()


def to_np(t) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def dev_weights(phi_q, phi_k, dtype):
    return tuple(to_dev(a, dtype) for a in phi_q), [tuple(to_dev(a, dtype) for a in w) for w in phi_k]


class DeviceRun:
    """One library context fed from numpy inputs; keeps device tensors for reuse."""

    def __init__(self, shape: synth.HlaShape, phi="mlp", eps=0.0, n_splits=0, causal=False):
        self.shape = shape
        self.phi = phi
        self.op = binding.Hla(shape.B, shape.H, shape.N, shape.d, dtype=shape.dtype, phi=phi, F=shape.F, d_phi=shape.d_phi,
                              eps=eps, n_splits=n_splits, causal=causal)

    def set_weights(self, phi_q, phi_k):
        self.op.set_phi(*dev_weights(phi_q, phi_k, self.shape.dtype))

    def forward(self, Q, K, V):
        s = self.shape
        io = s.dtype
        self.Q = to_dev(Q, io if self.phi == "mlp" else "f32")
        self.K = to_dev(K, io if self.phi == "mlp" else "f32")
        self.V = to_dev(V, io)
        self.O = self.op.forward(self.Q, self.K, self.V)
        torch.cuda.synchronize()
        assert self.op.device_status() == binding.HLA_OK
        return to_np(self.O)

    def backward(self, dO):
        self.dO = to_dev(dO, self.shape.dtype)
        dQ, dK, dV = self.op.backward(self.Q, self.K, self.V, self.O, self.dO)
        torch.cuda.synchronize()
        assert self.op.device_status() == binding.HLA_OK
        return to_np(dQ), to_np(dK), to_np(dV)

    def region(self, name, count, shape):
        return to_np(self.op.region(name)[:count]).reshape(shape)

    def features(self):
        s = self.shape
        nq = s.B * s.H * s.N * s.d_phi
        return (self.region("qf", nq, (s.B, s.H, s.N, s.d_phi)),
                self.region("kf", nq * s.F, (s.B, s.H, s.F, s.N, s.d_phi)))

    def state(self, name="state"):
        """(C, z) as the library keeps them: [B,H,state_rows,d] and [B,H,state_rows]."""
        s = self.shape
        R = self.op.layout.state_rows
        ld = self.op.layout.state_ld
        st = self.region(name, s.B * s.H * R * ld, (s.B, s.H, R, ld))
        return st[..., : s.d], st[..., s.d]

    def eta(self):
        s = self.shape
        return self.region("eta", s.B * s.H * s.N, (s.B, s.H, s.N))


def oracle_state(kf, V):
    B, H, F = kf.shape[:3]
    C = np.empty((B, H, kf.shape[-1] ** F, V.shape[-1]))
    z = np.empty((B, H, kf.shape[-1] ** F))
    for b in range(B):
        for h in range(H):
            C[b, h], z[b, h] = orc.context_state([kf[b, h, f] for f in range(F)], V[b, h])
    return C, z


def fold_symmetric(T, dphi=6, F=3):
    """Sum a tensor whose axis -2 (or last axis for a vector field) indexes the P = dphi^F outer-product
    entries over the distinct permutations of each sorted index tuple: [.., P, d] -> [.., n_mono, d].
    This is what the readout of the symmetric query tensor q (x) q (x) q can see of the state."""
    import itertools
    monos = [t for t in itertools.combinations_with_replacement(range(dphi), F)]
    out = np.zeros(T.shape[:-2] + (len(monos), T.shape[-1]))
    for m, t in enumerate(monos):
        for perm in set(itertools.permutations(t)):
            p = 0
            for i in perm:
                p = p * dphi + i
            out[..., m, :] += T[..., p, :]
    return out
