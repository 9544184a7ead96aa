"""ctypes binding of libhla.so: the same entry points as include/hla.h, taking
torch tensors (device memory and streams only - every step of the operator
runs in the library's kernels).  There is no fallback: if the library cannot be
loaded, importing callers get an exception."""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, byref, c_char_p, c_float, c_int32, c_size_t, c_void_p

import torch

from . import build as _build

HLA_OK, HLA_ERR_INVALID_ARG, HLA_ERR_UNSUPPORTED, HLA_ERR_WORKSPACE, HLA_ERR_CUDA, HLA_ERR_DEVICE_TIMEOUT, HLA_ERR_NO_MEMORY = range(7)
HLA_BF16, HLA_F32 = 0, 1
HLA_PHI_MLP, HLA_PHI_NONE = 0, 1

EXPORTS = [
    "hla_create", "hla_set_phi", "hla_workspace_bytes", "hla_workspace_layout", "hla_forward", "hla_backward", "hla_forward_keys", "hla_forward_queries", "hla_backward_queries", "hla_backward_keys", "hla_backward_weights", "hla_set_phi_v", "hla_set_carry", "hla_value_mod_forward", "hla_value_mod_backward", "hla_forward_static",
    "hla_last_device_status", "hla_selftest_bounded_wait", "hla_last_launch_count", "hla_timing_enable", "hla_timing_collect", "hla_timing_get",
    "hla_destroy", "hla_status_string",
]


class HlaConfig(ctypes.Structure):
    _fields_ = [("B", c_int32), ("H", c_int32), ("N", c_int32), ("d", c_int32), ("F", c_int32), ("d_phi", c_int32),
                ("phi", c_int32), ("dtype", c_int32), ("eps", c_float), ("n_splits", c_int32), ("causal", c_int32), ("value_mod", c_int32)]


class HlaMlp(ctypes.Structure):
    _fields_ = [("W1", c_void_p), ("b1", c_void_p), ("W2", c_void_p), ("b2", c_void_p)]


class HlaVmlp(ctypes.Structure):
    _fields_ = [("ln_g", c_void_p), ("ln_b", c_void_p), ("W1", c_void_p), ("b1", c_void_p), ("W2", c_void_p), ("b2", c_void_p)]


class HlaMlpGrad(ctypes.Structure):
    _fields_ = [("dW1", c_void_p), ("db1", c_void_p), ("dW2", c_void_p), ("db2", c_void_p)]


class HlaWsLayout(ctypes.Structure):
    _fields_ = [("status", c_size_t), ("qf", c_size_t), ("kf", c_size_t), ("state", c_size_t), ("eta", c_size_t),
                ("dstate", c_size_t), ("dqf", c_size_t), ("dkf", c_size_t), ("state_ld", c_int32), ("state_rows", c_int32), ("n_splits", c_int32),
                ("tensor_core", c_int32)]


class HlaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (hla_status {status})")


_lib = None


def library_path() -> str:
    return _build.LIB


def load_library(rebuild: bool = False) -> ctypes.CDLL:
    """Loads libhla.so (building it with nvcc first if it is missing or stale)."""
    global _lib
    if _lib is not None and not rebuild:
        return _lib
    path = _build.build(force=rebuild)
    if not os.path.exists(path):
        raise RuntimeError(f"HLA CUDA library missing: {path}")
    lib = ctypes.CDLL(path)
    lib.hla_create.argtypes = [POINTER(HlaConfig), POINTER(c_void_p)]
    lib.hla_create.restype = c_int32
    lib.hla_set_phi.argtypes = [c_void_p, POINTER(HlaMlp), POINTER(HlaMlp)]
    lib.hla_set_phi.restype = c_int32
    lib.hla_workspace_bytes.argtypes = [c_void_p]
    lib.hla_workspace_bytes.restype = c_size_t
    lib.hla_workspace_layout.argtypes = [c_void_p, POINTER(HlaWsLayout)]
    lib.hla_workspace_layout.restype = c_int32
    lib.hla_forward.argtypes = [c_void_p] + [c_void_p] * 4 + [c_void_p, c_size_t, c_void_p]
    lib.hla_forward.restype = c_int32
    lib.hla_backward.argtypes = [c_void_p] + [c_void_p] * 8 + [c_void_p, c_size_t, c_void_p]
    lib.hla_backward.restype = c_int32
    lib.hla_forward_keys.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
    lib.hla_forward_keys.restype = c_int32
    lib.hla_forward_queries.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
    lib.hla_forward_queries.restype = c_int32
    for name in ("hla_backward_queries", "hla_backward_keys"):
        getattr(lib, name).argtypes = [c_void_p] + [c_void_p] * 8 + [c_void_p, c_size_t, c_void_p]
        getattr(lib, name).restype = c_int32
    lib.hla_backward_weights.argtypes = [c_void_p, c_void_p, c_void_p, POINTER(HlaMlpGrad), POINTER(HlaMlpGrad), c_void_p, c_size_t, c_void_p]
    lib.hla_backward_weights.restype = c_int32
    lib.hla_set_carry.argtypes = [c_void_p, c_int32]
    lib.hla_set_carry.restype = c_int32
    lib.hla_set_phi_v.argtypes = [c_void_p, POINTER(HlaVmlp), POINTER(HlaVmlp)]
    lib.hla_set_phi_v.restype = c_int32
    lib.hla_value_mod_forward.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]
    lib.hla_value_mod_forward.restype = c_int32
    lib.hla_value_mod_backward.argtypes = [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int32, c_void_p, c_size_t, c_void_p]
    lib.hla_value_mod_backward.restype = c_int32
    lib.hla_forward_static.argtypes = [c_void_p] + [c_void_p] * 4 + [c_void_p, POINTER(c_void_p)]
    lib.hla_forward_static.restype = c_int32
    lib.hla_last_device_status.argtypes = [c_void_p, c_void_p, c_void_p]
    lib.hla_last_device_status.restype = c_int32
    lib.hla_selftest_bounded_wait.argtypes = [c_void_p, c_void_p, c_size_t, c_void_p]
    lib.hla_selftest_bounded_wait.restype = c_int32
    lib.hla_last_launch_count.argtypes = [c_void_p]
    lib.hla_last_launch_count.restype = c_int32
    lib.hla_timing_enable.argtypes = [c_void_p, c_int32]
    lib.hla_timing_enable.restype = c_int32
    lib.hla_timing_collect.argtypes = [c_void_p]
    lib.hla_timing_collect.restype = c_int32
    lib.hla_timing_get.argtypes = [c_void_p, c_int32, POINTER(c_char_p), POINTER(ctypes.c_double), POINTER(ctypes.c_int64)]
    lib.hla_timing_get.restype = c_int32
    lib.hla_destroy.argtypes = [c_void_p]
    lib.hla_destroy.restype = c_int32
    lib.hla_status_string.argtypes = [c_int32]
    lib.hla_status_string.restype = c_char_p
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().hla_status_string(int(status)).decode()


def _ptr(t) -> int:
    if t is None:
        return 0
    if isinstance(t, int):
        return t
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream if torch.cuda.is_available() else 0
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


# ---- the C entry points, one to one ------------------------------------------
def hla_create(cfg: HlaConfig) -> int:
    out = c_void_p()
    st = load_library().hla_create(byref(cfg), byref(out))
    if st != HLA_OK:
        raise HlaError(st, "hla_create")
    return out.value


def hla_set_phi(ctx: int, phi_q, phi_k) -> None:
    """phi_q = (W1, b1, W2, b2) device tensors; phi_k = list of F such tuples."""
    q = HlaMlp(*[_ptr(t) for t in phi_q])
    ks = (HlaMlp * len(phi_k))(*[HlaMlp(*[_ptr(t) for t in w]) for w in phi_k])
    st = load_library().hla_set_phi(ctx, byref(q), ks)
    if st != HLA_OK:
        raise HlaError(st, "hla_set_phi")


def hla_workspace_bytes(ctx: int) -> int:
    return int(load_library().hla_workspace_bytes(ctx))


def hla_workspace_layout(ctx: int) -> HlaWsLayout:
    out = HlaWsLayout()
    st = load_library().hla_workspace_layout(ctx, byref(out))
    if st != HLA_OK:
        raise HlaError(st, "hla_workspace_layout")
    return out


def hla_forward(ctx: int, Q, K, V, O, workspace, stream=None, workspace_bytes=None) -> None:
    nbytes = workspace.numel() * workspace.element_size() if workspace_bytes is None else workspace_bytes
    st = load_library().hla_forward(ctx, _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(workspace), nbytes, _stream(stream))
    if st != HLA_OK:
        raise HlaError(st, "hla_forward")


def hla_backward(ctx: int, Q, K, V, O, dO, dQ, dK, dV, workspace, stream=None, workspace_bytes=None) -> None:
    nbytes = workspace.numel() * workspace.element_size() if workspace_bytes is None else workspace_bytes
    st = load_library().hla_backward(ctx, _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(dO), _ptr(dQ), _ptr(dK), _ptr(dV),
                                     _ptr(workspace), nbytes, _stream(stream))
    if st != HLA_OK:
        raise HlaError(st, "hla_backward")


def hla_forward_keys(ctx: int, K, V, workspace, stream=None) -> None:
    st = load_library().hla_forward_keys(ctx, _ptr(K), _ptr(V), _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream))
    if st != HLA_OK:
        raise HlaError(st, "hla_forward_keys")


def hla_forward_queries(ctx: int, Q, O, workspace, stream=None) -> None:
    st = load_library().hla_forward_queries(ctx, _ptr(Q), _ptr(O), _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream))
    if st != HLA_OK:
        raise HlaError(st, "hla_forward_queries")


def _backward_half(name, ctx, Q, K, V, O, dO, dQ, dK, dV, workspace, stream):
    st = getattr(load_library(), name)(ctx, _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(dO), _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(workspace),
                                       workspace.numel() * workspace.element_size(), _stream(stream))
    if st != HLA_OK:
        raise HlaError(st, name)


def hla_backward_queries(ctx: int, Q, K, V, O, dO, dQ, dK, dV, workspace, stream=None) -> None:
    _backward_half("hla_backward_queries", ctx, Q, K, V, O, dO, dQ, dK, dV, workspace, stream)


def hla_backward_keys(ctx: int, Q, K, V, O, dO, dQ, dK, dV, workspace, stream=None) -> None:
    _backward_half("hla_backward_keys", ctx, Q, K, V, O, dO, dQ, dK, dV, workspace, stream)


def hla_backward_weights(ctx: int, Q, K, dphi_q, dphi_k, workspace, stream=None, workspace_bytes=None) -> None:
    """dphi_q = (dW1, db1, dW2, db2) fp32 device tensors or None; dphi_k = list of F such tuples or None."""
    nbytes = workspace.numel() * workspace.element_size() if workspace_bytes is None else workspace_bytes
    q = byref(HlaMlpGrad(*[_ptr(t) for t in dphi_q])) if dphi_q is not None else None
    ks = (HlaMlpGrad * len(dphi_k))(*[HlaMlpGrad(*[_ptr(t) for t in w]) for w in dphi_k]) if dphi_k is not None else None
    st = load_library().hla_backward_weights(ctx, _ptr(Q), _ptr(K), q, ks, _ptr(workspace), nbytes, _stream(stream))
    if st != HLA_OK:
        raise HlaError(st, "hla_backward_weights")


def hla_set_carry(ctx: int, carry: bool) -> None:
    st = load_library().hla_set_carry(ctx, 1 if carry else 0)
    if st != HLA_OK:
        raise HlaError(st, "hla_set_carry")


def hla_set_phi_v(ctx: int, v1, v2) -> None:
    """v1, v2 = (ln_g, ln_b, W1, b1, W2, b2) device tensors of the two value-modulation maps."""
    a, b = HlaVmlp(*[_ptr(t) for t in v1]), HlaVmlp(*[_ptr(t) for t in v2])
    st = load_library().hla_set_phi_v(ctx, byref(a), byref(b))
    if st != HLA_OK:
        raise HlaError(st, "hla_set_phi_v")


def hla_value_mod_forward(ctx: int, T, V, Out, workspace, stream=None) -> None:
    st = load_library().hla_value_mod_forward(ctx, _ptr(T), _ptr(V), _ptr(Out), _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream))
    if st != HLA_OK:
        raise HlaError(st, "hla_value_mod_forward")


def hla_value_mod_backward(ctx: int, T, V, dOut, dT, dV, accumulate_dV, workspace, stream=None) -> None:
    st = load_library().hla_value_mod_backward(ctx, _ptr(T), _ptr(V), _ptr(dOut), _ptr(dT), _ptr(dV), 1 if accumulate_dV else 0, _ptr(workspace),
                                               workspace.numel() * workspace.element_size(), _stream(stream))
    if st != HLA_OK:
        raise HlaError(st, "hla_value_mod_backward")


HLA_STATIC_WS_BYTES = 16 * 1024 * 1024


def hla_forward_static(ctx: int, Q, K, V, O, stream=None) -> int:
    """hla_forward on the scratch array the library itself carries (no workspace tensor, nothing allocated).
    Returns that array's device address (an int), usable as `workspace` for hla_last_device_status."""
    scratch = c_void_p()
    st = load_library().hla_forward_static(ctx, _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _stream(stream), byref(scratch))
    if st != HLA_OK:
        raise HlaError(st, "hla_forward_static")
    return scratch.value


def hla_last_device_status(ctx: int, workspace, stream=None) -> int:
    return int(load_library().hla_last_device_status(ctx, _ptr(workspace), _stream(stream)))


def hla_selftest_bounded_wait(ctx: int, workspace, stream=None) -> None:
    nbytes = workspace.numel() * workspace.element_size()
    st = load_library().hla_selftest_bounded_wait(ctx, _ptr(workspace), nbytes, _stream(stream))
    if st != HLA_OK:
        raise HlaError(st, "hla_selftest_bounded_wait")


def hla_last_launch_count(ctx: int) -> int:
    return int(load_library().hla_last_launch_count(ctx))


def hla_timing_enable(ctx: int, on: bool) -> None:
    st = load_library().hla_timing_enable(ctx, 1 if on else 0)
    if st != HLA_OK:
        raise HlaError(st, "hla_timing_enable")


def hla_timing_collect(ctx: int) -> dict:
    """After a stream synchronise: {kernel name: (total_ms, launches)} of the launches recorded since the last collect."""
    lib = load_library()
    n = lib.hla_timing_collect(ctx)
    out = {}
    for i in range(n):
        name = c_char_p()
        ms = ctypes.c_double()
        cnt = ctypes.c_int64()
        st = lib.hla_timing_get(ctx, i, byref(name), byref(ms), byref(cnt))
        if st != HLA_OK:
            raise HlaError(st, "hla_timing_get")
        out[name.value.decode()] = (ms.value, cnt.value)
    return out


def hla_destroy(ctx: int) -> None:
    st = load_library().hla_destroy(ctx)
    if st != HLA_OK:
        raise HlaError(st, "hla_destroy")


# ---- a small convenience holder (context + workspace) -------------------------
class Hla:
    """Owns a context and its workspace tensor.  All compute happens in hla_forward / hla_backward."""

    def __init__(self, B, H, N, d, dtype="bf16", phi="mlp", F=0, d_phi=0, eps=0.0, n_splits=0, device="cuda", value_mod=False, causal=False):
        self.cfg = HlaConfig(B, H, N, d, F, d_phi, HLA_PHI_MLP if phi == "mlp" else HLA_PHI_NONE,
                             HLA_BF16 if dtype == "bf16" else HLA_F32, eps, n_splits, 1 if causal else 0, 1 if value_mod else 0)
        self.torch_dtype = torch.bfloat16 if dtype == "bf16" else torch.float32
        self.ctx = hla_create(self.cfg)
        self.layout = hla_workspace_layout(self.ctx)
        self.device = device
        self.workspace = torch.empty(hla_workspace_bytes(self.ctx), dtype=torch.uint8, device=device) if device else None
        self._weights = None

    def set_phi(self, phi_q, phi_k):
        self._weights = (phi_q, phi_k)      # keep the tensors alive: the library only borrows pointers
        hla_set_phi(self.ctx, phi_q, phi_k)

    def forward(self, Q, K, V, O=None, stream=None):
        if O is None:
            O = torch.empty_like(V)
        hla_forward(self.ctx, Q, K, V, O, self.workspace, stream)
        return O

    def backward(self, Q, K, V, O, dO, dQ=None, dK=None, dV=None, stream=None):
        dQ = torch.empty_like(Q) if dQ is None else dQ
        dK = torch.empty_like(K) if dK is None else dK
        dV = torch.empty_like(V) if dV is None else dV
        hla_backward(self.ctx, Q, K, V, O, dO, dQ, dK, dV, self.workspace, stream)
        return dQ, dK, dV

    def state_region(self, gradient=False):
        """The fp32 state (or gradient state) of the last pass as a flat view of the workspace: what shards of a sequence add."""
        n = self.cfg.B * self.cfg.H * self.layout.state_rows * self.layout.state_ld
        return self.region("dstate" if gradient else "state")[:n]

    def set_carry(self, carry: bool):
        hla_set_carry(self.ctx, carry)

    def set_phi_v(self, v1, v2):
        self._vweights = (v1, v2)           # keep the tensors alive: the library only borrows pointers
        hla_set_phi_v(self.ctx, v1, v2)

    def value_mod_forward(self, T, V, Out=None, stream=None):
        Out = torch.empty_like(T) if Out is None else Out
        hla_value_mod_forward(self.ctx, T, V, Out, self.workspace, stream)
        return Out

    def value_mod_backward(self, T, V, dOut, dT=None, dV=None, accumulate_dV=False, stream=None):
        dT = torch.empty_like(T) if dT is None else dT
        dV = torch.empty_like(V) if dV is None else dV
        hla_value_mod_backward(self.ctx, T, V, dOut, dT, dV, accumulate_dV, self.workspace, stream)
        return dT, dV

    def backward_weights(self, Q, K, stream=None):
        """Weight gradients of phi_q and phi_k1..F (fp32, shapes of the weights), after backward()."""
        F = self.cfg.F or 3
        d, dphi = self.cfg.d, self.cfg.d_phi or (6 if F == 3 else 12)
        mk = lambda: tuple(torch.empty(s, dtype=torch.float32, device=self.device) for s in ((d, d), (d,), (d, dphi), (dphi,)))
        gq, gk = mk(), [mk() for _ in range(F)]
        hla_backward_weights(self.ctx, Q, K, gq, gk, self.workspace, stream)
        return gq, gk

    def region(self, name, dtype=torch.float32):
        """View of a persistent workspace region (see hla_ws_layout) as a flat tensor from its offset to the end."""
        off = getattr(self.layout, name)
        if off == ctypes.c_size_t(-1).value:
            raise KeyError(name)
        return self.workspace[off:].view(dtype)

    def device_status(self, stream=None) -> int:
        return hla_last_device_status(self.ctx, self.workspace, stream)

    def launches(self) -> int:
        return hla_last_launch_count(self.ctx)

    def close(self):
        if self.ctx:
            hla_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
