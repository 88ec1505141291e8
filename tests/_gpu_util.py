"""Helpers shared by the GPU parity tests: run the same seeded inputs through the CUDA
library (via its C ABI) and through the fp64 oracle, and compare with the stated bars."""
import torch

from paper_2609_39034_b200 import workloads as wl

# Tolerances (max |x - y| / max(|y|, rms(y)), y = oracle):
#   fp32 inputs: 1e-4 on o and on the state;
#   bf16 inputs with fp32 state: 2e-2 on o (bf16 output rounding alone is 2^-9); the state never
#   passes through bf16 (identical rounded inputs, fp32 arithmetic), so it keeps the 1e-4 bar.
TOL_FP32 = 1e-4
TOL_BF16_O = 2e-2
TOL_STATE = 1e-4


def to_dev(inp, device="cuda"):
    return {n: (x.to(device) if x is not None else None) for n, x in inp.items()}


def gpu_forward(binding, w, inp_dev, *, want_r=False, algo=0, state_in="from_inputs"):
    """Returns dict(o, W, r_prev, rho_prev, r) of CPU tensors."""
    st_out = binding.state_alloc(w, init=False)
    if state_in == "from_inputs":
        sin = {"W": inp_dev["W0"], "r_prev": inp_dev.get("r0"), "rho_prev": inp_dev.get("rho0")}
    else:
        sin = state_in
    T = inp_dev["q"].shape[2]
    r = torch.empty((w.B, w.H, T, w.J, w.Dv), device="cuda", dtype=torch.float32) if want_r else None
    o = binding.swila_forward(w, inp_dev, state_in=sin, state_out=st_out, r_debug=r, algo=algo)
    torch.cuda.synchronize()
    return {"o": o.cpu(), "W": st_out["W"].cpu(),
            "r_prev": st_out["r_prev"].cpu() if w.temporal else None,
            "rho_prev": st_out["rho_prev"].cpu() if w.temporal else None,
            "r": r.cpu() if want_r else None}


def assert_close(w, got, ref, what=""):
    """got: gpu_forward output; ref: oracle output (numpy fp64)."""
    tol_o = TOL_BF16_O if w.io_dtype == "bf16" else TOL_FP32
    e_o = wl.rel_err(got["o"], torch.from_numpy(ref["o"]))
    e_w = wl.rel_err(got["W"], torch.from_numpy(ref["W"]))
    assert e_o < tol_o, f"{what} o: rel err {e_o:.3e} >= {tol_o}"
    assert e_w < TOL_STATE, f"{what} W: rel err {e_w:.3e} >= {TOL_STATE}"
    if w.temporal:
        for n in ("r_prev", "rho_prev"):
            e = wl.rel_err(got[n], torch.from_numpy(ref[n]))
            assert e < TOL_STATE, f"{what} {n}: rel err {e:.3e}"
    if got.get("r") is not None and ref.get("r") is not None:
        e = float((got["r"].double() - torch.from_numpy(ref["r"])).abs().max())
        assert e < 1e-4, f"{what} r: abs err {e:.3e}"
    return e_o, e_w
