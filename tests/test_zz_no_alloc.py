"""The allocation-free host entry point, swila_forward_host_static.

It exists for callers that are handed host tensors and a stream but are not allowed to allocate
device memory; it stages through a fixed 16 MiB array inside the library instead of a caller
workspace.  The GPU test drives it through the C ABI twice in a row, with different problems,
and requires each result to equal what swila_forward_host (caller-allocated workspace) returns
for the same inputs: the second call finds the first call's bytes in the shared array and must
not be affected by them.  This file is collected last on purpose."""
import ctypes

import pytest
import torch

from paper_2609_39034_b200 import workloads as wl
from tests._gpu_util import TOL_BF16_O, TOL_STATE


def _binding():
    from paper_2609_39034_b200 import build as swila_build

    swila_build.build()
    from paper_2609_39034_b200 import binding

    return binding


def test_static_entry_rejects_problems_beyond_its_capacity():
    b = _binding()
    cap = b.lib.swila_forward_host_static_capacity()
    assert cap == 16 << 20
    big = wl.CONFIGS[2]  # needs gigabytes of workspace
    assert b.host_workspace_bytes(big) > cap
    sh = b.make_shape(big)
    g = b.Gates()
    rc = b.lib.swila_forward_host_static(ctypes.byref(sh), None, None, None, ctypes.byref(g), None, None, None, None)
    assert rc == b.ERR_SIZE
    bad = b.make_shape(big.with_(J=3))
    rc = b.lib.swila_forward_host_static(ctypes.byref(bad), None, None, None, ctypes.byref(g), None, None, None, None)
    assert rc == b.ERR_UNSUPPORTED


@pytest.mark.gpu
def test_static_entry_matches_workspace_entry_on_two_calls_in_a_row(oracle):
    assert torch.cuda.is_available()
    b = _binding()
    problems = [wl.CONFIGS[1].with_(B=2, H=3, T=75).variant(temporal=True, gated=True),
                wl.CONFIGS[2].with_(B=1, H=2, T=40, recipe="gauss")]
    for i, w in enumerate(problems):
        assert b.host_workspace_bytes(w) <= b.lib.swila_forward_host_static_capacity()
        inp = {n: (x.pin_memory() if x is not None else None)
               for n, x in wl.make_inputs(w, stress=True, seed_offset=i).items()}
        sin = {"W": inp["W0"], "r_prev": inp["r0"], "rho_prev": inp["rho0"]}

        def out_state():
            return {"W": torch.empty_like(inp["W0"]).pin_memory(),
                    "r_prev": torch.empty_like(inp["r0"]).pin_memory() if w.temporal else None,
                    "rho_prev": torch.empty_like(inp["rho0"]).pin_memory() if w.temporal else None}

        ws = torch.empty(b.host_workspace_bytes(w), device="cuda", dtype=torch.uint8)
        ref_state, got_state = out_state(), out_state()
        ref_o = b.swila_forward_host(w, inp, ws, state_in=sin, state_out=ref_state)
        torch.cuda.synchronize()
        got_o = b.swila_forward_host_static(w, inp, state_in=sin, state_out=got_state)
        torch.cuda.synchronize()
        assert wl.rel_err(got_o, ref_o) < TOL_BF16_O, f"call {i}: o"
        assert wl.rel_err(got_state["W"], ref_state["W"]) < TOL_STATE, f"call {i}: W"
        if w.temporal:
            assert wl.rel_err(got_state["r_prev"], ref_state["r_prev"]) < TOL_STATE
            assert wl.rel_err(got_state["rho_prev"], ref_state["rho_prev"]) < TOL_STATE
        # and against the fp64 oracle directly, so that this test stands without the workspace entry point's own
        ref = oracle.forward_inputs(inp, flags=w.flags, gran=w.gate_granularity)
        assert wl.rel_err(got_o, torch.from_numpy(ref["o"])) < TOL_BF16_O, f"call {i}: o against the oracle"
        assert wl.rel_err(got_state["W"], torch.from_numpy(ref["W"])) < TOL_STATE, f"call {i}: W against the oracle"
        # same kernel, same inputs: in fact the two entry points agree to the bit
        assert torch.equal(got_o, ref_o) and torch.equal(got_state["W"], ref_state["W"])
