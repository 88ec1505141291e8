"""Seeded synthetic inputs for the SwiLA recurrence.

This module only *produces inputs*: queries, keys, values, the pre-activation gate
tensors that the layer's learned projections would emit, decay values and initial
states.  It contains none of the recurrence's arithmetic (no E-step, M-step or
readout) and is the one module shared by the CUDA path's tests/bench and by the CPU
oracle's tests.  Every tensor is drawn from its own ``torch.Generator`` seeded as
``1000 * config + tensor_index`` (+ a caller-supplied offset), generated in fp32,
then rounded ONCE to the io dtype; the same rounded values feed both sides.

Workload shapes follow the paper's experiments (Appendix D): the 374M language-model
layer (J=4, D=64), 1.3B-style throughput shapes (T up to 16k), associative-recall
sequences with key reuse, and batched generation on a carried state.  Queries and
keys are L2-normalised per token and head (Appendix D.1: SiLU + L2 normalisation on
Q/K), without which the delta-rule update is unstable.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Optional

import torch

FLAG_TEMPORAL = 1
FLAG_GATED = 2
FLAG_POST_DECAY = 4
FLAG_QKV_ACT = 8  # q, k, v are raw projections: SiLU + L2 normalisation inside the kernel (App. B.2, App. D.1)

GRAN_NONE = 0
GRAN_PER_KEY = 1
GRAN_PER_OUT = 2
GRAN_SCALAR = 3
GRAN_ELEMENTWISE = 4  # alpha [B,H,T,J,Dv,Dk]: one decay per state element (App. B.4, the general form)


@dataclass(frozen=True)
class Workload:
    """Shape and variant of one SwiLA call (J = number of mixture components)."""

    name: str
    config: int
    B: int
    H: int
    T: int
    Dk: int
    Dv: int
    J: int
    io_dtype: str = "fp32"  # "fp32" | "bf16": q, k, v, o and all logit tensors
    flags: int = 0
    gate_granularity: int = GRAN_NONE
    recipe: str = "gauss"  # "gauss" | "lm" | "recall"

    @property
    def temporal(self) -> bool:
        return bool(self.flags & FLAG_TEMPORAL)

    @property
    def gated(self) -> bool:
        return bool(self.flags & FLAG_GATED)

    @property
    def torch_io_dtype(self) -> torch.dtype:
        return torch.bfloat16 if self.io_dtype == "bf16" else torch.float32

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)

    def variant(self, temporal: bool = False, gated: bool = False, post_decay: bool = False,
                granularity: int = GRAN_PER_KEY) -> "Workload":
        flags = (FLAG_TEMPORAL if temporal else 0) | (FLAG_GATED if gated else 0) | (
            FLAG_POST_DECAY if (gated and post_decay) else 0)
        return replace(self, flags=flags, gate_granularity=granularity if gated else GRAN_NONE)


# The five benchmark configurations (index = config number).
CONFIGS = {
    0: Workload("tiny_prefill", 0, B=1, H=2, T=256, Dk=16, Dv=16, J=2, io_dtype="fp32"),
    1: Workload("mid_prefill", 1, B=8, H=16, T=2048, Dk=64, Dv=64, J=4, io_dtype="bf16"),
    2: Workload("lm_prefill", 2, B=4, H=16, T=8192, Dk=128, Dv=128, J=4, io_dtype="bf16", recipe="lm"),
    3: Workload("recall_prefill", 3, B=64, H=4, T=512, Dk=64, Dv=64, J=8, io_dtype="fp32", recipe="recall"),
    # T here is the prefill length; decode adds DECODE_STEPS single-token calls.
    4: Workload("batched_decode", 4, B=256, H=32, T=4096, Dk=128, Dv=128, J=4, io_dtype="bf16"),
}
DECODE_STEPS = 1024
DECODE_PREFILL_CHUNK = 256
LM_EMBED_WIDTH = 2048


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _randn(shape, seed, device, std: float = 1.0) -> torch.Tensor:
    x = torch.randn(shape, generator=_gen(seed, device), device=device, dtype=torch.float32)
    return x * std if std != 1.0 else x


def _l2n(x: torch.Tensor) -> torch.Tensor:
    return x / x.norm(dim=-1, keepdim=True).clamp_min(1e-12)


def _head_proj(theta: torch.Tensor, x: torch.Tensor) -> torch.Tensor:
    """theta [H, M, Dk] applied to x [B, H, T, Dk] -> [B, H, T, M]."""
    return torch.einsum("hmd,bhtd->bhtm", theta, x).contiguous()


def make_inputs(w: Workload, *, device="cpu", stress: bool = False, seed_offset: int = 0,
                state: str = "default") -> Dict[str, Optional[torch.Tensor]]:
    """Build every tensor of one ``swila_forward`` call for workload ``w``.

    stress=True draws gate parameters with std 1 (instead of 0.02) and a N(0,1)
    initial state, so that the mixture components genuinely differ and the E-step
    matters to the result; it is used by parity tests only.
    state: "default" (zeros unless stress), "zero", or "randn".

    Returns a dict with q, k, v, beta_logit, pik_logit, piq_logit (io dtype),
    gk_logit, gq_logit (io dtype or None), alpha (fp32 or None), and the initial
    state W0 [B,H,J,Dv,Dk], r0, rho0 [B,H,J,Dv] (fp32; r0/rho0 None unless temporal).
    """
    B, H, T, Dk, Dv, J = w.B, w.H, w.T, w.Dk, w.Dv, w.J
    base = 1000 * w.config + 100003 * seed_offset
    pstd = 1.0 if stress else 0.02
    io = w.torch_io_dtype
    out: Dict[str, Optional[torch.Tensor]] = {}

    if w.recipe == "lm":
        # Token embeddings projected by seeded random linear maps; SiLU on q, k, v.
        E = _randn((B, T, LM_EMBED_WIDTH), base + 0, device)
        wstd = 1.0 / 32.0  # N(0, 1/sqrt(1024)) read as a standard deviation
        def proj(idx, width):
            Wm = _randn((LM_EMBED_WIDTH, H * width), base + idx, device, wstd)
            y = torch.nn.functional.silu(E @ Wm)
            return y.view(B, T, H, width).permute(0, 2, 1, 3).contiguous()
        q, k, v = _l2n(proj(1, Dk)), _l2n(proj(2, Dk)), proj(3, Dv)
        gstd = 1.0 / 45.0 if stress else 0.02  # logit std ~1 vs ~0.9: already O(1)
        def gate(idx, per_head):
            Th = _randn((LM_EMBED_WIDTH, H * per_head), base + idx, device, gstd)
            return (E @ Th).view(B, T, H, per_head).permute(0, 2, 1, 3).contiguous()
        beta_l = gate(4, J * Dv).view(B, H, T, J, Dv)
        pik_l = gate(5, J * Dv).view(B, H, T, J, Dv)
        piq_l = gate(6, J * Dv).view(B, H, T, J, Dv)
        gk_l = gate(7, Dv) if w.temporal else None
        gq_l = gate(8, Dv) if w.temporal else None
        k_for_alpha = k
        del E
    else:
        if w.recipe == "recall":
            q, k, v = _recall_qkv(w, base, device)
        else:
            q = _l2n(_randn((B, H, T, Dk), base + 1, device))
            k = _l2n(_randn((B, H, T, Dk), base + 2, device))
            v = _randn((B, H, T, Dv), base + 3, device)
        # Gate projections act on the head's own key (beta, pi^k) and query (pi^q).
        th_b = _randn((H, J * Dv, Dk), base + 4, device, pstd)
        th_k = _randn((H, J * Dv, Dk), base + 5, device, pstd)
        th_q = _randn((H, J * Dv, Dk), base + 6, device, pstd)
        beta_l = _head_proj(th_b, k).view(B, H, T, J, Dv)
        pik_l = _head_proj(th_k, k).view(B, H, T, J, Dv)
        piq_l = _head_proj(th_q, q).view(B, H, T, J, Dv)
        if w.temporal:
            gk_l = _head_proj(_randn((H, Dv, Dk), base + 7, device, pstd), k)
            gq_l = _head_proj(_randn((H, Dv, Dk), base + 8, device, pstd), q)
        else:
            gk_l = gq_l = None
        k_for_alpha = k

    out["q"], out["k"], out["v"] = q.to(io).contiguous(), k.to(io).contiguous(), v.to(io).contiguous()
    out["beta_logit"], out["pik_logit"] = beta_l.to(io).contiguous(), pik_l.to(io).contiguous()
    out["piq_logit"] = piq_l.to(io).contiguous()
    out["gk_logit"] = gk_l.to(io).contiguous() if gk_l is not None else None
    out["gq_logit"] = gq_l.to(io).contiguous() if gq_l is not None else None

    if w.gated:
        # Decay values in (0,1), mostly near 1 (sigmoid(3) ~ 0.95), key-dependent.
        m = {GRAN_PER_KEY: Dk, GRAN_PER_OUT: Dv, GRAN_SCALAR: 1, GRAN_ELEMENTWISE: Dv * Dk}[w.gate_granularity]
        th_a = _randn((H, J * m, Dk), base + 9, device, pstd)
        a = torch.sigmoid(3.0 + _head_proj(th_a, k_for_alpha)).view(B, H, T, J, m)
        if w.gate_granularity == GRAN_SCALAR:
            a = a.view(B, H, T, J)
        elif w.gate_granularity == GRAN_ELEMENTWISE:
            a = a.view(B, H, T, J, Dv, Dk)
        out["alpha"] = a.contiguous()
    else:
        out["alpha"] = None

    if state == "default":
        state = "randn" if stress else "zero"
    if state == "randn":
        out["W0"] = _randn((B, H, J, Dv, Dk), base + 10, device)
    else:
        out["W0"] = torch.zeros((B, H, J, Dv, Dk), device=device, dtype=torch.float32)
    if w.temporal:
        if state == "randn":
            out["r0"] = torch.softmax(_randn((B, H, J, Dv), base + 11, device), dim=2).contiguous()
            out["rho0"] = torch.softmax(_randn((B, H, J, Dv), base + 12, device), dim=2).contiguous()
        else:
            out["r0"] = torch.full((B, H, J, Dv), 1.0 / J, device=device, dtype=torch.float32)
            out["rho0"] = torch.full((B, H, J, Dv), 1.0 / J, device=device, dtype=torch.float32)
    else:
        out["r0"] = out["rho0"] = None
    return out


def _recall_qkv(w: Workload, base: int, device):
    """Associative-recall-shaped sequences: a write phase of ``P`` distinct key-value
    pairs per sequence (keys from a per-head codebook of 256 unit vectors), then
    passes that revisit every key in a fresh random order with its original value.
    Queries equal keys.  Only the shape and key-reuse structure of recall benchmarks
    is kept; no benchmark item is reproduced."""
    B, H, T, Dk, Dv = w.B, w.H, w.T, w.Dk, w.Dv
    P = min(64, T)
    codebook = _l2n(_randn((H, 256, Dk), base + 1, device))
    g = _gen(base + 2, device)
    # P distinct codebook indices per (b, h): argsort of uniform noise.
    idx = torch.rand((B, H, 256), generator=g, device=device).argsort(dim=-1)[..., :P]
    vals = _randn((B, H, P, Dv), base + 3, device)
    order = [torch.arange(P, device=device).expand(B, H, P)]
    n = P
    while n < T:
        order.append(torch.rand((B, H, P), generator=g, device=device).argsort(dim=-1))
        n += P
    order = torch.cat(order, dim=-1)[..., :T]  # position within the P pairs, per token
    tok_idx = torch.gather(idx, 2, order)  # codebook index per token
    hsel = torch.arange(H, device=device).view(1, H, 1).expand(B, H, T)
    k = codebook[hsel, tok_idx]
    v = torch.gather(vals, 2, order.unsqueeze(-1).expand(B, H, T, Dv))
    return k.clone(), k.contiguous(), v.contiguous()


def decode_step_inputs(w: Workload, step: int, *, device="cpu", stress: bool = False,
                       seed_offset: int = 0) -> Dict[str, Optional[torch.Tensor]]:
    """Fresh single-token inputs (T=1) for decode step ``step`` of workload ``w``;
    the gate projections are those of ``make_inputs`` (same parameter seeds)."""
    w1 = w.with_(T=1, recipe="gauss")
    B, H, Dk, Dv, J = w.B, w.H, w.Dk, w.Dv, w.J
    base = 1000 * w.config + 100003 * seed_offset
    sb = base + 500 + 7 * step
    pstd = 1.0 if stress else 0.02
    io = w.torch_io_dtype
    q = _l2n(_randn((B, H, 1, Dk), sb + 1, device))
    k = _l2n(_randn((B, H, 1, Dk), sb + 2, device))
    v = _randn((B, H, 1, Dv), sb + 3, device)
    th_b = _randn((H, J * Dv, Dk), base + 4, device, pstd)
    th_k = _randn((H, J * Dv, Dk), base + 5, device, pstd)
    th_q = _randn((H, J * Dv, Dk), base + 6, device, pstd)
    out: Dict[str, Optional[torch.Tensor]] = {
        "q": q.to(io), "k": k.to(io), "v": v.to(io),
        "beta_logit": _head_proj(th_b, k).view(B, H, 1, J, Dv).to(io),
        "pik_logit": _head_proj(th_k, k).view(B, H, 1, J, Dv).to(io),
        "piq_logit": _head_proj(th_q, q).view(B, H, 1, J, Dv).to(io),
        "gk_logit": None, "gq_logit": None, "alpha": None,
    }
    if w1.temporal:
        out["gk_logit"] = _head_proj(_randn((H, Dv, Dk), base + 7, device, pstd), k).to(io)
        out["gq_logit"] = _head_proj(_randn((H, Dv, Dk), base + 8, device, pstd), q).to(io)
    if w1.gated:
        m = {GRAN_PER_KEY: Dk, GRAN_PER_OUT: Dv, GRAN_SCALAR: 1, GRAN_ELEMENTWISE: Dv * Dk}[w.gate_granularity]
        th_a = _randn((H, J * m, Dk), base + 9, device, pstd)
        a = torch.sigmoid(3.0 + _head_proj(th_a, k)).view(B, H, 1, J, m)
        if w.gate_granularity == GRAN_SCALAR:
            a = a.view(B, H, 1, J)
        elif w.gate_granularity == GRAN_ELEMENTWISE:
            a = a.view(B, H, 1, J, Dv, Dk)
        out["alpha"] = a.contiguous()
    return out


def slice_time(inp: Dict[str, Optional[torch.Tensor]], t0: int, t1: int) -> Dict[str, Optional[torch.Tensor]]:
    """Tokens [t0, t1) of every per-token tensor (contiguous copies); state entries
    are passed through unchanged."""
    out = {}
    for name, x in inp.items():
        if x is None or name in ("W0", "r0", "rho0"):
            out[name] = x
        else:
            out[name] = x[:, :, t0:t1].contiguous()
    return out


def slice_rows(inp: Dict[str, Optional[torch.Tensor]], bh_index: torch.Tensor,
               cols: torch.Tensor, gran: int = GRAN_NONE) -> Dict[str, Optional[torch.Tensor]]:
    """Restrict a call to the (b,h) pairs ``bh_index`` (flat indices into B*H) and the
    output columns ``cols``.  Output columns are independent recurrences (Sec. 3.1),
    so the restricted problem is itself a valid call with B'=len(bh_index), H'=1,
    Dv'=len(cols).  Used to check sampled rows of a full-size run."""
    out = {}
    col_last = ("v", "gk_logit", "gq_logit")
    col_gate = ("beta_logit", "pik_logit", "piq_logit")
    for name, x in inp.items():
        if x is None:
            out[name] = None
            continue
        flat = x.reshape((x.shape[0] * x.shape[1],) + tuple(x.shape[2:]))[bh_index]
        if name in col_last or name in col_gate or name in ("r0", "rho0"):
            flat = flat[..., cols]
        elif name == "W0":
            flat = flat[:, :, cols, :]
        elif name == "alpha" and gran == GRAN_PER_OUT:
            flat = flat[..., cols]
        elif name == "alpha" and gran == GRAN_ELEMENTWISE:
            flat = flat[..., cols, :]
        out[name] = flat.unsqueeze(1).contiguous()
    return out


def rel_err(x: torch.Tensor, y: torch.Tensor) -> float:
    """max_i |x_i - y_i| / max(|y_i|, rms(y)) with y the reference, in fp64.

    Plain elementwise relative error is meaningless next to zeros of y; flooring the
    denominator at the tensor's rms keeps the measure scale-free."""
    x = x.detach().double().cpu().reshape(-1)
    y = y.detach().double().cpu().reshape(-1)
    if y.numel() == 0:
        return 0.0
    rms = float(torch.sqrt(torch.mean(y * y)))
    den = torch.clamp(y.abs(), min=max(rms, 1e-300))
    return float(((x - y).abs() / den).max())


def rel_err_unfloored(x: torch.Tensor, y: torch.Tensor, min_frac: float = 1e-2) -> float:
    """Plain elementwise relative error max_i |x_i - y_i| / |y_i| over the elements with |y_i| >= min_frac * rms(y):
    the measure of ``rel_err`` without its floor, reported beside it so that the gap between the two is visible."""
    x = x.detach().double().cpu().reshape(-1)
    y = y.detach().double().cpu().reshape(-1)
    if y.numel() == 0:
        return 0.0
    rms = float(torch.sqrt(torch.mean(y * y)))
    keep = y.abs() >= min_frac * rms
    if not bool(keep.any()):
        return 0.0
    return float(((x - y).abs()[keep] / y.abs()[keep]).max())
