"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, and rejects bad arguments with the documented status codes before any CUDA call."""
import ctypes as C
import os
import re

import pytest

import paper_2605_02888_b200 as speckv
from paper_2605_02888_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "speckv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(speckv_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    L = speckv.load_library()
    names = _declared()
    assert {"speckv_signals", "speckv_select_gamma", "speckv_verify", "speckv_step",
            "speckv_workspace_size"} <= set(names)
    for n in names:
        assert hasattr(L, n), n


def test_version_and_status_strings():
    assert speckv.version() >= 100
    assert speckv.status_string(0) == "ok"
    assert "workspace" in speckv.status_string(3)


def _cb(**kw):
    b = binding._CBatch()
    b.B, b.gamma_max, b.V, b.dtype = 4, 8, 128256, binding.BF16
    b.draft_logits = 0x1000
    b.draft_stride_b, b.draft_stride_pos = 8 * 128256, 128256
    b.temperature_scalar = 1.0
    for k, v in kw.items():
        setattr(b, k, v)
    return b


def test_workspace_size_and_argument_checks_without_a_gpu():
    L = speckv.load_library()
    n = C.c_size_t(0)
    assert L.speckv_workspace_size(C.byref(_cb()), C.byref(n)) == binding.OK and n.value >= 256
    small = n.value
    assert L.speckv_workspace_size(C.byref(_cb(B=64)), C.byref(n)) == binding.OK and n.value > small
    assert L.speckv_workspace_size(C.byref(_cb(V=0)), C.byref(n)) == binding.ERR_INVALID_ARG
    assert L.speckv_workspace_size(C.byref(_cb(gamma_max=17)), C.byref(n)) == binding.ERR_UNSUPPORTED
    assert L.speckv_workspace_size(C.byref(_cb()), None) == binding.ERR_INVALID_ARG
    # signals: NULL logits, bad dtype, bad strides, missing / misaligned / short workspace
    call = lambda b, ws, nb: L.speckv_signals(C.byref(b), None, None, None, None, ws, nb, None)
    assert call(_cb(draft_logits=None), 0x100, 1 << 30) == binding.ERR_INVALID_ARG
    assert call(_cb(dtype=7), 0x100, 1 << 30) == binding.ERR_UNSUPPORTED
    assert call(_cb(draft_stride_pos=100), 0x100, 1 << 30) == binding.ERR_INVALID_ARG
    assert call(_cb(), None, 1 << 30) == binding.ERR_INVALID_ARG
    assert call(_cb(), 0x101, 1 << 30) == binding.ERR_INVALID_ARG
    assert call(_cb(), 0x100, 16) == binding.ERR_WORKSPACE
    assert call(_cb(B=-1), 0x100, 1 << 30) == binding.ERR_INVALID_ARG
    # flags: the value 2 (no kernel behind it any more) and unknown bits are refused before anything is launched
    assert call(_cb(flags=2), 0x100, 1 << 30) == binding.ERR_INVALID_ARG
    assert call(_cb(flags=8), 0x100, 1 << 30) == binding.ERR_INVALID_ARG
    assert call(_cb(B=0), None, 0) == binding.OK          # empty batch: nothing to do
    # verify needs target, tokens and uniforms
    assert L.speckv_verify(C.byref(_cb()), 0x100, 0x100, None, 0x100, 1 << 30, None) == binding.ERR_INVALID_ARG
    # controller checks
    m = binding._CMlp()
    assert L.speckv_select_gamma(4, 0x100, None, C.byref(m), None, 0x100, None) == binding.ERR_INVALID_ARG
    m.n_in, m.n_hidden, m.n_out = 5, 64, 4
    m.W1 = m.b1 = m.W2 = m.b2 = 0x100
    assert L.speckv_select_gamma(4, 0x100, None, C.byref(m), None, 0x100, None) == binding.ERR_UNSUPPORTED


def test_binding_refuses_cpu_tensors():
    import torch
    with pytest.raises(ValueError, match="CUDA"):
        speckv.speckv_signals(speckv.Batch(draft_logits=torch.zeros(1, 2, 16)))
