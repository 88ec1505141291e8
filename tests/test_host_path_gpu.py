"""GPU: the host-buffer entry point (pinned host tensors staged through a caller-owned device
workspace) gives exactly the device-pointer entry point's results, and matches the oracle."""
import pytest
import torch

from paper_2609_39034_b200 import workloads as wl
from tests._gpu_util import assert_close, gpu_forward, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    assert torch.cuda.is_available()
    from paper_2609_39034_b200 import binding as b

    return b


def _pin(inp):
    return {n: (x.pin_memory() if x is not None else None) for n, x in inp.items()}


@pytest.mark.parametrize("var", [dict(), dict(temporal=True), dict(temporal=True, gated=True)],
                         ids=["vanilla", "temporal", "gated_temporal"])
def test_host_entry_equals_device_entry(binding, oracle, var):
    w = wl.CONFIGS[1].with_(B=2, H=3, T=75).variant(**var)
    inp = wl.make_inputs(w, stress=True)
    ref = oracle.forward_inputs(inp, flags=w.flags, gran=w.gate_granularity)
    dev = gpu_forward(binding, w, to_dev(inp))
    host = _pin(inp)
    ws = torch.empty(binding.host_workspace_bytes(w), device="cuda", dtype=torch.uint8)
    sin = {"W": host["W0"], "r_prev": host["r0"], "rho_prev": host["rho0"]}
    sout = {"W": torch.empty_like(inp["W0"]).pin_memory(),
            "r_prev": torch.empty_like(inp["r0"]).pin_memory() if w.temporal else None,
            "rho_prev": torch.empty_like(inp["rho0"]).pin_memory() if w.temporal else None}
    o = binding.swila_forward_host(w, host, ws, state_in=sin, state_out=sout)
    torch.cuda.synchronize()
    assert torch.equal(o, dev["o"]) and torch.equal(sout["W"], dev["W"])
    if w.temporal:
        assert torch.equal(sout["r_prev"], dev["r_prev"]) and torch.equal(sout["rho_prev"], dev["rho_prev"])
    assert_close(w, {"o": o, "W": sout["W"], "r_prev": sout["r_prev"], "rho_prev": sout["rho_prev"]}, ref, "host")


def test_host_entry_rejects_a_small_workspace(binding):
    w = wl.CONFIGS[0]
    host = _pin(wl.make_inputs(w))
    ws = torch.empty(binding.host_workspace_bytes(w) - 256, device="cuda", dtype=torch.uint8)
    with pytest.raises(binding.SwilaError) as e:
        binding.swila_forward_host(w, host, ws)
    assert e.value.status == binding.ERR_SIZE


@pytest.mark.parametrize("var,T", [(dict(), 2304), (dict(temporal=True), 2304), (dict(temporal=True, gated=True), 1400),
                                   (dict(gated=True, granularity=wl.GRAN_PER_OUT), 2048)],
                         ids=["vanilla", "temporal", "gated_temporal", "gated_rows"])
def test_host_entry_in_slabs_equals_device_entry(binding, var, T):
    """Problems of 64 MB and more go through in slabs of (batch, head) pairs over internal copy streams; with 15
    pairs the 8 slabs are uneven.  The results must be those of one call on device tensors."""
    w = wl.CONFIGS[1].with_(B=3, H=5, T=T).variant(**var)
    assert binding.host_workspace_bytes(w) >= 64 << 20
    inp = wl.make_inputs(w, stress=True)
    dev = gpu_forward(binding, w, to_dev(inp))
    host = _pin(inp)
    ws = torch.empty(binding.host_workspace_bytes(w), device="cuda", dtype=torch.uint8)
    sin = {"W": host["W0"], "r_prev": host["r0"], "rho_prev": host["rho0"]}
    sout = {"W": torch.empty_like(inp["W0"]).pin_memory(),
            "r_prev": torch.empty_like(inp["r0"]).pin_memory() if w.temporal else None,
            "rho_prev": torch.empty_like(inp["rho0"]).pin_memory() if w.temporal else None}
    for _ in range(2):  # twice in a row: the second call reuses the streams and events of the first
        o = binding.swila_forward_host(w, host, ws, state_in=sin, state_out=sout)
        torch.cuda.synchronize()
        assert torch.equal(o, dev["o"]) and torch.equal(sout["W"], dev["W"])
        if w.temporal:
            assert torch.equal(sout["r_prev"], dev["r_prev"]) and torch.equal(sout["rho_prev"], dev["rho_prev"])


def test_host_entry_from_two_threads_at_once(binding):
    """Two host threads call the pipelined host path on one device at the same time, each with its own stream,
    workspace and tensors; they share the library's copy streams and events.  Each must get what it gets alone."""
    import threading

    ws_ = [wl.CONFIGS[1].with_(B=3, H=5, T=2304), wl.CONFIGS[1].with_(B=2, H=8, T=2304).variant(temporal=True)]
    jobs = []
    for i, w in enumerate(ws_):
        assert binding.host_workspace_bytes(w) >= 64 << 20
        inp = wl.make_inputs(w, stress=True, seed_offset=i)
        dev = gpu_forward(binding, w, to_dev(inp))
        host = _pin(inp)
        jobs.append(dict(w=w, host=host, dev=dev, stream=torch.cuda.Stream(),
                         ws=torch.empty(binding.host_workspace_bytes(w), device="cuda", dtype=torch.uint8),
                         sin={"W": host["W0"], "r_prev": host["r0"], "rho_prev": host["rho0"]}))
    torch.cuda.synchronize()
    errors = []

    def work(job):
        try:
            for _ in range(6):
                sout = {"W": torch.empty_like(job["host"]["W0"]).pin_memory(),
                        "r_prev": torch.empty_like(job["host"]["r0"]).pin_memory() if job["w"].temporal else None,
                        "rho_prev": torch.empty_like(job["host"]["rho0"]).pin_memory() if job["w"].temporal else None}
                o = binding.swila_forward_host(job["w"], job["host"], job["ws"], state_in=job["sin"], state_out=sout,
                                               stream=job["stream"])
                job["stream"].synchronize()
                if not (torch.equal(o, job["dev"]["o"]) and torch.equal(sout["W"], job["dev"]["W"])):
                    errors.append(job["w"].name + ": result differs from the single-threaded call")
        except Exception as e:  # noqa: BLE001
            errors.append(repr(e))

    threads = [threading.Thread(target=work, args=(j,)) for j in jobs]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    torch.cuda.synchronize()
    assert not errors, errors
