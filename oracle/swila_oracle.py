"""ctypes front end of the fp64 C oracle (oracle/swila_ref.c): test infrastructure only.

``forward`` takes torch tensors or numpy arrays of any float dtype, upcasts them to
fp64 and runs the sequential recurrence of Sec. 3.2 (Eqs. 3.3-3.5) with the Temporal
(App. B.3) and Gated (Sec. 3.4, App. B.4) variants.  The arithmetic lives in the C
file; this wrapper only marshals arrays."""
from __future__ import annotations

import ctypes
from typing import Dict, Optional

import numpy as np

from . import build as _build

_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build())
        dp = ctypes.POINTER(ctypes.c_double)
        lib.swila_ref_forward.argtypes = [ctypes.c_int] * 8 + [dp] * 14
        lib.swila_ref_forward.restype = ctypes.c_int
        lib.swila_ref_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def threads() -> int:
    """Number of OpenMP threads the oracle will use."""
    return int(_load().swila_ref_threads())


def _f64(x) -> Optional[np.ndarray]:
    if x is None:
        return None
    if hasattr(x, "detach"):  # torch tensor (possibly bf16, possibly on a GPU)
        x = x.detach().to("cpu").double().numpy()
    return np.ascontiguousarray(np.asarray(x, dtype=np.float64))


def _ptr(a: Optional[np.ndarray]):
    dp = ctypes.POINTER(ctypes.c_double)
    return a.ctypes.data_as(dp) if a is not None else ctypes.cast(None, dp)


def forward(q, k, v, beta_logit, pik_logit, piq_logit, *, gk_logit=None, gq_logit=None,
            alpha=None, W0=None, r0=None, rho0=None, flags: int = 0, gran: int = 0,
            want_r: bool = False) -> Dict[str, np.ndarray]:
    """Run the oracle.  Shapes: q,k [B,H,T,Dk]; v [B,H,T,Dv]; gate logits [B,H,T,J,Dv];
    gk/gq logits [B,H,T,Dv]; alpha by granularity; W0 [B,H,J,Dv,Dk] (zeros if None);
    r0, rho0 [B,H,J,Dv] (uniform 1/J if None and TEMPORAL).

    Returns {"o": [B,H,T,Dv], "W": final state, "r_prev", "rho_prev" (TEMPORAL),
    "r": [B,H,T,J,Dv] if want_r}, all fp64."""
    lib = _load()
    q, k, v = _f64(q), _f64(k), _f64(v)
    bl, pk, pq = _f64(beta_logit), _f64(pik_logit), _f64(piq_logit)
    B, H, T, Dk = q.shape
    Dv = v.shape[-1]
    J = bl.shape[3]
    assert k.shape == q.shape and v.shape == (B, H, T, Dv)
    assert bl.shape == pk.shape == pq.shape == (B, H, T, J, Dv)
    W = np.zeros((B, H, J, Dv, Dk)) if W0 is None else _f64(W0).copy()
    assert W.shape == (B, H, J, Dv, Dk)
    temporal = bool(flags & 1)
    gated = bool(flags & 2)
    gk = gq = rp = rh = al = None
    if temporal:
        gk, gq = _f64(gk_logit), _f64(gq_logit)
        assert gk.shape == gq.shape == (B, H, T, Dv)
        rp = np.full((B, H, J, Dv), 1.0 / J) if r0 is None else _f64(r0).copy()
        rh = np.full((B, H, J, Dv), 1.0 / J) if rho0 is None else _f64(rho0).copy()
    if gated:
        al = _f64(alpha)
        want = {1: (B, H, T, J, Dk), 2: (B, H, T, J, Dv), 3: (B, H, T, J), 4: (B, H, T, J, Dv, Dk)}[gran]
        assert al.shape == want, (al.shape, want)
    o = np.zeros((B, H, T, Dv))
    r = np.zeros((B, H, T, J, Dv)) if want_r else None
    rc = lib.swila_ref_forward(B, H, T, Dk, Dv, J, int(flags), int(gran), _ptr(q), _ptr(k), _ptr(v),
                               _ptr(bl), _ptr(pk), _ptr(pq), _ptr(gk), _ptr(gq), _ptr(al),
                               _ptr(W), _ptr(rp), _ptr(rh), _ptr(o), _ptr(r))
    if rc != 0:
        raise ValueError(f"swila_ref_forward rejected its arguments (rc={rc})")
    out = {"o": o, "W": W}
    if temporal:
        out["r_prev"], out["rho_prev"] = rp, rh
    if want_r:
        out["r"] = r
    return out


def forward_inputs(inp: dict, *, flags: int = 0, gran: int = 0, want_r: bool = False,
                   state: Optional[dict] = None) -> Dict[str, np.ndarray]:
    """``forward`` on a dict laid out like the seeded input generator's; ``state``
    (keys W, r_prev, rho_prev) overrides the dict's initial state when given."""
    W0, r0, rho0 = inp.get("W0"), inp.get("r0"), inp.get("rho0")
    if state is not None:
        W0, r0, rho0 = state["W"], state.get("r_prev"), state.get("rho_prev")
    return forward(inp["q"], inp["k"], inp["v"], inp["beta_logit"], inp["pik_logit"], inp["piq_logit"],
                   gk_logit=inp.get("gk_logit"), gq_logit=inp.get("gq_logit"), alpha=inp.get("alpha"),
                   W0=W0, r0=r0, rho0=rho0, flags=flags, gran=gran, want_r=want_r)
