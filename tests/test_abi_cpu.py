"""Host-side checks of the C ABI that need no GPU: the library builds and loads, exports every
symbol include/hla.h declares, validates configurations and call arguments before any launch,
and sizes its workspace consistently."""
import ctypes
import os
import re

import pytest

from paper_2602_12128_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "hla.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hla_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = binding.load_library()
    names = declared_symbols()
    assert {"hla_create", "hla_forward", "hla_backward", "hla_destroy"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names


def cfg(**kw):
    base = dict(B=1, H=2, N=300, d=128, F=0, d_phi=0, phi=binding.HLA_PHI_MLP, dtype=binding.HLA_BF16, eps=0.0, n_splits=0, causal=0, value_mod=0)
    base.update(kw)
    return binding.HlaConfig(*[base[k] for k, _ in binding.HlaConfig._fields_])


def create(**kw):
    out = ctypes.c_void_p()
    st = binding.load_library().hla_create(ctypes.byref(cfg(**kw)), ctypes.byref(out))
    return st, out.value


def test_create_defaults_and_layout():
    st, ctx = create()
    assert st == binding.HLA_OK and ctx
    L = binding.hla_workspace_layout(ctx)
    assert L.tensor_core == 1 and L.state_rows == 56 and L.state_ld >= 129      # F=3, d_phi=6 folded to 56 monomials
    assert L.n_splits >= 1 and L.n_splits <= 3                                  # never more splits than 128-token tiles
    total = binding.hla_workspace_bytes(ctx)
    none = ctypes.c_size_t(-1).value
    offs = [getattr(L, n) for n in ("status", "qf", "kf", "state", "eta", "dstate", "dqf", "dkf")]
    assert all(o != none and o % 256 == 0 and o < total for o in offs)
    assert offs == sorted(offs)
    binding.hla_destroy(ctx)


def test_feature_level_entry_has_no_feature_regions():
    st, ctx = create(phi=binding.HLA_PHI_NONE, dtype=binding.HLA_F32, d=16, F=2)
    assert st == binding.HLA_OK
    L = binding.hla_workspace_layout(ctx)
    none = ctypes.c_size_t(-1).value
    assert L.qf == none and L.kf == none and L.dqf == none and L.dkf == none
    assert L.tensor_core == 0 and L.state_rows == 144                           # F=2 defaults to d_phi = 12
    binding.hla_destroy(ctx)


@pytest.mark.parametrize("kw,want", [
    (dict(B=0), binding.HLA_ERR_INVALID_ARG),
    (dict(N=-5), binding.HLA_ERR_INVALID_ARG),
    (dict(phi=7), binding.HLA_ERR_INVALID_ARG),
    (dict(dtype=3), binding.HLA_ERR_INVALID_ARG),
    (dict(F=1), binding.HLA_ERR_INVALID_ARG),            # no default d_phi for F = 1
    (dict(causal=2), binding.HLA_ERR_INVALID_ARG),
    (dict(causal=1, F=2), binding.HLA_ERR_UNSUPPORTED),                 # the causal sweep: 3 factors, bf16, d in {64, 128}
    (dict(causal=1, dtype=binding.HLA_F32, d=16), binding.HLA_ERR_UNSUPPORTED),
    (dict(F=3, d_phi=7), binding.HLA_ERR_UNSUPPORTED),   # 343 features > 256
    (dict(F=5, d_phi=2), binding.HLA_ERR_UNSUPPORTED),
    (dict(d=256), binding.HLA_ERR_UNSUPPORTED),
    (dict(d=20), binding.HLA_ERR_UNSUPPORTED),           # bf16 rows must be 16-byte multiples
    (dict(B=300, H=300), binding.HLA_ERR_UNSUPPORTED),
    (dict(value_mod=2), binding.HLA_ERR_INVALID_ARG),
    (dict(value_mod=1, dtype=binding.HLA_F32, d=16), binding.HLA_ERR_UNSUPPORTED),      # value modulation: bf16, d in {64, 128}
])
def test_create_rejects(kw, want):
    st, ctx = create(**kw)
    assert st == want and not ctx


def test_calls_validate_before_launching():
    lib = binding.load_library()
    st, ctx = create(phi=binding.HLA_PHI_NONE)
    assert st == binding.HLA_OK
    need = binding.hla_workspace_bytes(ctx)
    p = 0x10000      # never dereferenced: validation fails first
    assert lib.hla_forward(None, p, p, p, p, p, need, None) == binding.HLA_ERR_INVALID_ARG
    assert lib.hla_forward(ctx, None, p, p, p, p, need, None) == binding.HLA_ERR_INVALID_ARG
    assert lib.hla_forward(ctx, p + 4, p, p, p, p, need, None) == binding.HLA_ERR_INVALID_ARG      # misaligned tensor
    assert lib.hla_forward(ctx, p, p, p, p, p + 16, need, None) == binding.HLA_ERR_INVALID_ARG     # workspace not 256-aligned
    assert lib.hla_forward(ctx, p, p, p, p, p, need - 1, None) == binding.HLA_ERR_WORKSPACE
    assert lib.hla_backward(ctx, p, p, p, p, p, p, p, None, p, need, None) == binding.HLA_ERR_INVALID_ARG
    assert lib.hla_backward(ctx, p, p, p, p, p, p, p, p, p, need - 1, None) == binding.HLA_ERR_WORKSPACE
    binding.hla_destroy(ctx)
    # the phi maps must have been set before a call in HLA_PHI_MLP mode
    st, ctx = create()
    need = binding.hla_workspace_bytes(ctx)
    assert lib.hla_forward(ctx, p, p, p, p, p, need, None) == binding.HLA_ERR_INVALID_ARG
    assert lib.hla_set_phi(ctx, None, None) == binding.HLA_ERR_INVALID_ARG
    # dQ, dK leave the tensor-core phi backward as 32-byte stores: a 16-byte-aligned dK is refused before any launch
    # (the phi weights only have to be set, they are not read by the validation)
    w = binding.HlaMlp(p, p, p, p)
    ws3 = (binding.HlaMlp * 3)(w, w, w)
    assert lib.hla_set_phi(ctx, ctypes.byref(w), ws3) == binding.HLA_OK
    assert lib.hla_backward(ctx, p, p, p, p, p, p, p + 16, p, p, need, None) == binding.HLA_ERR_INVALID_ARG
    assert lib.hla_backward(ctx, p, p, p, p, p, p + 16, p, p, p, need, None) == binding.HLA_ERR_INVALID_ARG
    binding.hla_destroy(ctx)
    assert lib.hla_destroy(None) == binding.HLA_ERR_INVALID_ARG
    assert binding.status_string(binding.HLA_ERR_NO_MEMORY) == "out of host memory"
    # value modulation: refused unless the context was created for it and its weights were given
    st, ctx = create()
    need = binding.hla_workspace_bytes(ctx)
    assert lib.hla_value_mod_forward(ctx, p, p, p + 256, p, need, None) == binding.HLA_ERR_INVALID_ARG
    binding.hla_destroy(ctx)
    st, ctx = create(value_mod=1)
    assert st == binding.HLA_OK and binding.hla_workspace_bytes(ctx) > need
    need = binding.hla_workspace_bytes(ctx)
    assert lib.hla_value_mod_forward(ctx, p, p, p + 256, p, need, None) == binding.HLA_ERR_INVALID_ARG      # weights not set
    v = binding.HlaVmlp(p, p, p, p, p, p)
    assert lib.hla_set_phi_v(ctx, ctypes.byref(v), ctypes.byref(v)) == binding.HLA_OK
    assert lib.hla_value_mod_forward(ctx, p, p, p, p, need, None) == binding.HLA_ERR_INVALID_ARG            # Out aliases T
    assert lib.hla_value_mod_forward(ctx, p, p, p + 16, p, need, None) == binding.HLA_ERR_INVALID_ARG       # Out not 32-byte aligned
    assert lib.hla_value_mod_forward(ctx, p, p, p + 256, p, need - 1, None) == binding.HLA_ERR_WORKSPACE
    assert lib.hla_value_mod_backward(ctx, p, p, p, p + 16, p, 0, p, need, None) == binding.HLA_ERR_INVALID_ARG
    binding.hla_destroy(ctx)
    assert binding.status_string(binding.HLA_ERR_DEVICE_TIMEOUT) == "device-side wait timed out"
    assert binding.hla_workspace_bytes(None) == 0


def test_set_carry_validation():
    """Sequential updates across calls exist for contexts with the mask only; the flag is 0 or 1."""
    lib = binding.load_library()
    st, ctx = create(causal=1)
    assert st == binding.HLA_OK
    assert lib.hla_set_carry(ctx, 1) == binding.HLA_OK
    assert lib.hla_set_carry(ctx, 0) == binding.HLA_OK
    assert lib.hla_set_carry(ctx, 2) == binding.HLA_ERR_INVALID_ARG
    assert lib.hla_set_carry(None, 1) == binding.HLA_ERR_INVALID_ARG
    binding.hla_destroy(ctx)
    st, ctx = create()
    assert st == binding.HLA_OK
    assert lib.hla_set_carry(ctx, 1) == binding.HLA_ERR_INVALID_ARG
    binding.hla_destroy(ctx)
