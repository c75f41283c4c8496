"""Host-side checks of the C ABI that need no GPU: the library loads, exports every
symbol include/psk.h declares, and rejects bad arguments before touching a device."""
import ctypes
import os
import re
from ctypes import byref, c_void_p

import pytest

import paper_2310_01655_b200 as psk
from paper_2310_01655_b200.binding import Shape

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    from paper_2310_01655_b200 import build
    build.build()
    return psk.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "psk.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(psk_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = declared_symbols()
    assert {"psk_sketch", "psk_causal_attn_fwd", "psk_causal_attn_bwd", "psk_workspace_bytes",
            "psk_check", "psk_status_string", "psk_version"} <= set(names)
    for name in names:
        assert hasattr(L, name), name


def good():
    return Shape(1, 2, 512, 64, 32, 4, 256, 1, 2 * 512 * 64, 512 * 64, 64, 2, 0, 0, 0)


def test_status_strings(L):
    assert psk.status_string(0) == "ok"
    for code in range(-7, 0):
        assert psk.status_string(code) not in ("ok", "unknown status")
    assert psk.status_string(-99) == "unknown status"


def test_workspace_size_formula(L):
    s = good()
    s.path = psk.PATH_CUDA_CORES
    rows = 2 * 512
    states = 2 * 2 * 32 * 32 * 65 * 4
    fwd = psk.workspace_bytes(s, False)
    bwd = psk.workspace_bytes(s, True)
    assert fwd >= 256 + rows * (32 + 32 + 65) * 4 + states
    assert bwd >= fwd + rows * (65 + 32 + 32) * 4 + states
    assert fwd % 256 == 0 and bwd % 256 == 0


@pytest.mark.parametrize("field,value,code", [
    ("p", 2, -2), ("p", 6, -2), ("p", 16, -2), ("h", 128, -2), ("r", 48, -2),      # (p = 2 needs r = h)
    ("b", 100, -3), ("n", 500, -3), ("B", 0, -3), ("g_heads", 3, -3),
    ("dtype", 7, -1), ("path", 9, -1), ("flags", 8, -1), ("stride_n", 66, -4),
    ("flags", 6, -2),                                   # no mask together with exact same-block weights
    ("seq_segments", -1, -1), ("seq_segments", 3, -3),   # runs must divide the n / b = 2 blocks
])
def test_bad_shapes_are_rejected_before_any_launch(L, field, value, code):
    s = good()
    setattr(s, field, value)
    assert psk.workspace_bytes(s, False) == 0
    fake = c_void_p(256)   # never dereferenced: validation fails first
    st = L.psk_causal_attn_fwd(byref(s), fake, fake, fake, fake, fake, fake, None, fake, 1 << 40, None)
    assert st == code, (field, psk.status_string(st))
    st = L.psk_causal_attn_bwd(byref(s), *([fake] * 12), 1 << 40, None)
    assert st == code
    st = L.psk_sketch(byref(s), fake, fake, fake, fake, None, None)
    assert st == code


def test_null_misaligned_and_small_workspace(L):
    s = good()
    fake = c_void_p(256)
    args = [fake] * 6
    assert L.psk_causal_attn_fwd(byref(s), None, fake, fake, fake, fake, fake, None, fake, 1 << 40, None) == -1
    assert L.psk_causal_attn_fwd(byref(s), c_void_p(260), fake, fake, fake, fake, fake, None, fake, 1 << 40, None) == -4
    assert L.psk_causal_attn_fwd(byref(s), *args, None, fake, 16, None) == -5
    assert L.psk_causal_attn_fwd(byref(s), *args, None, None, 1 << 40, None) == -5
    assert L.psk_causal_attn_fwd(byref(s), *args, None, c_void_p(264), 1 << 40, None) == -5
    assert L.psk_causal_attn_bwd(byref(s), *([fake] * 6), None, *([fake] * 5), 1 << 40, None) == -1
    assert L.psk_sketch(None, fake, fake, fake, fake, None, None) == -1


def test_binding_refuses_cpu_tensors(L):
    import torch
    x = torch.zeros(1, 1, 128, 64)
    g = torch.zeros(1, 64, 16)
    with pytest.raises(RuntimeError, match="CUDA"):
        psk.causal_attn_fwd(x, x, x, g, g, 128)
    with pytest.raises(RuntimeError, match="CUDA"):
        psk.sketch(x, g, g)
