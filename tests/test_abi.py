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


def _declared_functions(header="swila.h"):
    text = open(os.path.join(ROOT, "include", header)).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(swila_[a-z_0-9]+)\s*\(", text)))


# The product's C ABI: the calls of the hot path (prefill, decode, state helpers, status) plus the documented
# extras (host-buffer front ends, statistics, output norm).  Anything else belongs in swila_dev.h.
PRODUCT_ABI = {"swila_version", "swila_strerror", "swila_last_cuda_error", "swila_device_status",
               "swila_state_w_bytes", "swila_state_r_bytes", "swila_state_init", "swila_forward",
               "swila_decode_step", "swila_forward_stats", "swila_output_norm",
               "swila_forward_host", "swila_forward_host_workspace_bytes",
               "swila_forward_host_static", "swila_forward_host_static_capacity"}
DEV_ABI = {"swila_auto_algo", "swila_selftest_wait_timeout", "swila_bench_fma_chain", "swila_selftest_tf32_mma", "swila_selftest_bf16_mma",
           "swila_chunk_plan", "swila_chunk_run_pieces"}


def test_headers_declare_exactly_the_documented_sets():
    assert set(_declared_functions("swila.h")) == PRODUCT_ABI
    assert set(_declared_functions("swila_dev.h")) == DEV_ABI


def test_library_exports_every_declared_symbol_and_nothing_else(binding):
    names = _declared_functions("swila.h") + _declared_functions("swila_dev.h")
    raw = ctypes.CDLL(binding.LIB_PATH)
    for n in names:
        assert hasattr(raw, n), f"{n} declared in a header but not exported"
    assert set(binding.EXPORTS) <= set(names)
    import subprocess
    out = subprocess.run(["nm", "-D", "--defined-only", binding.LIB_PATH], capture_output=True, text=True).stdout
    exported = {line.split()[-1] for line in out.splitlines() if " T " in line and line.split()[-1].startswith("swila_")}
    assert exported == set(names), exported ^ set(names)


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


def test_alias_check_covers_every_written_tensor(binding):
    """o, r_debug and the output state may overlap no streamed input and not each other; state_out == state_in is
    allowed (in place).  Fake addresses: validation happens on the host before any launch."""
    w = wl.CONFIGS[0].variant(temporal=True, gated=True)
    sh = binding.make_shape(w)
    f = binding.lib.swila_forward
    M = 0x1000000  # 16 MB apart: far more than any tensor of this shape
    q, k, v, be, pk, pq, gk, gq, al, o, rdbg, W, r, rho = (0x10000000 + i * M for i in range(14))
    g = binding.Gates(be, pk, pq, gk, gq, al)
    st = binding.State(W, r, rho)
    call = lambda gates=g, out=o, dbg=rdbg, sin=st, sout=st: f(  # noqa: E731
        ctypes.byref(sh), q, k, v, ctypes.byref(gates), ctypes.byref(sin) if sin else None,
        ctypes.byref(sout) if sout else None, out, dbg, None)
    # (every call below must fail validation: a call that passed it would launch on the fake addresses)
    for bad in (dict(out=gk), dict(out=gq), dict(out=al), dict(dbg=q), dict(dbg=o), dict(out=W),
                dict(sout=binding.State(k, r, rho)), dict(sout=binding.State(W, be, rho)),
                dict(sout=binding.State(W, r, r)), dict(sout=binding.State(W + 16, r, rho))):
        assert call(**bad) == binding.ERR_ALIAS, bad


def test_auto_dispatch_rule(binding):
    """What sends an AUTO call to the scan kernel, as the header states it."""
    auto = lambda w, aux=0: binding.lib.swila_auto_algo(ctypes.byref(binding.make_shape(w)), aux)  # noqa: E731
    lm = wl.CONFIGS[2]
    assert auto(lm) == binding.ALGO_CHUNK and auto(lm.variant(temporal=True)) == binding.ALGO_CHUNK
    assert auto(lm, 1) == binding.ALGO_CHUNK and auto(lm.variant(temporal=True), 1) == binding.ALGO_CHUNK
    assert auto(wl.CONFIGS[1].with_(J=16)) == binding.ALGO_CHUNK and auto(wl.CONFIGS[1].with_(J=16), 1) == binding.ALGO_SCAN
    rows = dict(gated=True, granularity=wl.GRAN_PER_OUT)
    assert auto(lm.variant(**rows)) == binding.ALGO_CHUNK and auto(lm.variant(gated=True, granularity=wl.GRAN_SCALAR, post_decay=True)) == binding.ALGO_CHUNK
    assert auto(lm.variant(**rows), 1) == binding.ALGO_SCAN and auto(lm.variant(temporal=True, **rows)) == binding.ALGO_SCAN and auto(wl.CONFIGS[1].variant(temporal=True, **rows)) == binding.ALGO_CHUNK
    assert auto(lm.with_(J=8).variant(**rows)) == binding.ALGO_SCAN and auto(wl.CONFIGS[1].with_(J=8).variant(**rows)) == binding.ALGO_CHUNK
    for w in (lm.with_(T=63), lm.with_(io_dtype="fp32"), lm.variant(gated=True), lm.with_(J=2), lm.with_(J=16),
              lm.variant(gated=True, granularity=wl.GRAN_ELEMENTWISE),
              wl.CONFIGS[0], wl.CONFIGS[3], lm.with_(flags=wl.FLAG_QKV_ACT)):
        assert auto(w) == binding.ALGO_SCAN, w
    assert auto(lm.with_(J=3)) == binding.ERR_UNSUPPORTED
