"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every
function that include/swila.h declares, sizes states correctly and rejects bad arguments
before touching the device."""
import ctypes
import os
import re

import pytest

from paper_2609_39034_b200 import build as swila_build
from paper_2609_39034_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    swila_build.build()
    from paper_2609_39034_b200 import binding as b

    return b


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "swila.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(swila_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(binding):
    names = _declared_functions()
    assert "swila_forward" in names and "swila_decode_step" in names
    raw = ctypes.CDLL(binding.LIB_PATH)
    for n in names:
        assert hasattr(raw, n), f"{n} declared in swila.h but not exported"
    assert set(binding.EXPORTS) <= set(names)


def test_version_and_strerror(binding):
    assert binding.lib.swila_version() >= 100
    for code in range(0, -8, -1):
        assert binding.lib.swila_strerror(code)
    assert binding.lib.swila_strerror(-99) == b"unknown status"


def test_state_bytes(binding):
    w = wl.CONFIGS[2]
    sh = binding.make_shape(w)
    assert binding.lib.swila_state_w_bytes(ctypes.byref(sh)) == w.B * w.H * w.J * w.Dv * w.Dk * 4
    assert binding.lib.swila_state_r_bytes(ctypes.byref(sh)) == w.B * w.H * w.J * w.Dv * 4
    bad = binding.make_shape(w.with_(Dk=48))
    assert binding.lib.swila_state_w_bytes(ctypes.byref(bad)) == 0


@pytest.mark.parametrize("change,status", [
    (dict(B=0), -2), (dict(Dv=12), -2), (dict(T=-1), -2), (dict(Dk=48), -3), (dict(J=3), -3),
    (dict(flags=wl.FLAG_POST_DECAY), -3), (dict(flags=wl.FLAG_GATED), -3),
    (dict(gate_granularity=wl.GRAN_PER_KEY), -3), (dict(flags=16), -3),
])
def test_forward_rejects_bad_shapes_on_the_host(binding, change, status):
    w = wl.CONFIGS[0].with_(**change)
    sh = binding.make_shape(w)
    g = binding.Gates()
    rc = binding.lib.swila_forward(ctypes.byref(sh), None, None, None, ctypes.byref(g), None, None, None, None, None)
    assert rc == status


def test_forward_rejects_null_misaligned_and_aliased_pointers(binding):
    w = wl.CONFIGS[0]
    sh = binding.make_shape(w)
    g = binding.Gates()
    f = binding.lib.swila_forward
    assert f(ctypes.byref(sh), None, None, None, ctypes.byref(g), None, None, None, None, None) == binding.ERR_NULL
    # fake (never dereferenced) addresses: validation happens before any launch
    a = 0x10000
    g = binding.Gates(a, a, a, None, None, None)
    assert f(ctypes.byref(sh), a, a, a, ctypes.byref(g), None, None, a + 0x100000 + 4, None, None) == binding.ERR_ALIGN
    assert f(ctypes.byref(sh), a, a, a, ctypes.byref(g), None, None, a, None, None) == binding.ERR_ALIAS
    sh_t = binding.make_shape(w.variant(temporal=True))
    assert f(ctypes.byref(sh_t), a, a, a, ctypes.byref(g), None, None, a + 0x100000, None, None) == binding.ERR_NULL
    assert binding.lib.swila_decode_step(ctypes.byref(sh), a, a, a, ctypes.byref(g), None, a, None) == binding.ERR_NULL
