"""Thin ctypes binding of libswila.so: argument marshalling only.

Every step of the recurrence runs inside the CUDA library; this module turns torch
tensors into raw device pointers and mirrors the C structs of include/swila.h.  There
is no CPU fallback: importing this module raises if the library has not been built."""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from .workloads import Workload

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libswila.so")

SWILA_OK = 0
ERR_NULL, ERR_SHAPE, ERR_UNSUPPORTED, ERR_ALIGN, ERR_ALIAS, ERR_CUDA, ERR_SIZE = -1, -2, -3, -4, -5, -6, -7
IO_FP32, IO_BF16 = 0, 1
ALGO_AUTO, ALGO_SCAN, ALGO_SCAN_WIDE, ALGO_SCAN_NARROW, ALGO_CHUNK = 0, 1, 2, 3, 4

EXPORTS = ("swila_version", "swila_strerror", "swila_last_cuda_error", "swila_state_w_bytes",
           "swila_state_r_bytes", "swila_state_init", "swila_forward", "swila_decode_step",
           "swila_bench_fma_chain", "swila_forward_host", "swila_forward_host_workspace_bytes",
           "swila_forward_host_static", "swila_forward_host_static_capacity", "swila_selftest_tf32_mma", "swila_selftest_bf16_mma", "swila_device_status", "swila_chunk_plan", "swila_chunk_run_pieces",
           "swila_forward_stats", "swila_output_norm", "swila_auto_algo", "swila_selftest_wait_timeout")


class Shape(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("B", "H", "T", "Dk", "Dv", "J", "io_dtype", "flags", "gate_granularity", "algo")]


class Gates(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in
                ("beta_logit", "pik_logit", "piq_logit", "gk_logit", "gq_logit", "alpha")]


class State(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("W", "r_prev", "rho_prev")]


class Stats(ctypes.Structure):
    _fields_ = [("r_sum", ctypes.c_void_p), ("r_ent", ctypes.c_void_p), ("rho_sum", ctypes.c_void_p),
                ("rho_ent", ctypes.c_void_p)]


class SwilaError(RuntimeError):
    def __init__(self, status: int):
        self.status = status
        msg = lib.swila_strerror(status).decode()
        if status == ERR_CUDA:
            msg += ": " + lib.swila_last_cuda_error().decode()
        super().__init__(f"swila status {status}: {msg}")


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2609_39034_b200.build` "
            "(there is no fallback implementation)")
    L = ctypes.CDLL(LIB_PATH)
    L.swila_version.restype = ctypes.c_int
    L.swila_strerror.restype = ctypes.c_char_p
    L.swila_strerror.argtypes = [ctypes.c_int]
    L.swila_last_cuda_error.restype = ctypes.c_char_p
    for f in (L.swila_state_w_bytes, L.swila_state_r_bytes):
        f.restype = ctypes.c_size_t
        f.argtypes = [ctypes.POINTER(Shape)]
    L.swila_state_init.restype = ctypes.c_int
    L.swila_state_init.argtypes = [ctypes.POINTER(Shape), ctypes.POINTER(State), ctypes.c_void_p]
    L.swila_forward.restype = ctypes.c_int
    L.swila_forward.argtypes = [ctypes.POINTER(Shape), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                ctypes.POINTER(Gates), ctypes.POINTER(State), ctypes.POINTER(State),
                                ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
    L.swila_forward_stats.restype = ctypes.c_int
    L.swila_forward_stats.argtypes = [ctypes.POINTER(Shape), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                      ctypes.POINTER(Gates), ctypes.POINTER(State), ctypes.POINTER(State),
                                      ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(Stats), ctypes.c_void_p]
    L.swila_output_norm.restype = ctypes.c_int
    L.swila_output_norm.argtypes = [ctypes.POINTER(Shape), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_float,
                                    ctypes.c_void_p]
    L.swila_decode_step.restype = ctypes.c_int
    L.swila_decode_step.argtypes = [ctypes.POINTER(Shape), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                    ctypes.POINTER(Gates), ctypes.POINTER(State), ctypes.c_void_p, ctypes.c_void_p]
    L.swila_forward_host_workspace_bytes.restype = ctypes.c_size_t
    L.swila_forward_host_workspace_bytes.argtypes = [ctypes.POINTER(Shape)]
    L.swila_forward_host.restype = ctypes.c_int
    L.swila_forward_host.argtypes = [ctypes.POINTER(Shape), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                     ctypes.POINTER(Gates), ctypes.POINTER(State), ctypes.POINTER(State),
                                     ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
    L.swila_forward_host_static_capacity.restype = ctypes.c_size_t
    L.swila_forward_host_static.restype = ctypes.c_int
    L.swila_forward_host_static.argtypes = [ctypes.POINTER(Shape), ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                            ctypes.POINTER(Gates), ctypes.POINTER(State), ctypes.POINTER(State),
                                            ctypes.c_void_p, ctypes.c_void_p]
    L.swila_selftest_bf16_mma.restype = ctypes.c_int
    L.swila_selftest_bf16_mma.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int,
                                          ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p]
    L.swila_selftest_tf32_mma.restype = ctypes.c_int
    L.swila_selftest_tf32_mma.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int,
                                          ctypes.c_void_p, ctypes.c_void_p]
    L.swila_chunk_plan.restype = ctypes.c_int
    L.swila_chunk_plan.argtypes = [ctypes.c_int] * 7 + [ctypes.POINTER(ctypes.c_longlong)]
    L.swila_chunk_run_pieces.restype = ctypes.c_int
    L.swila_chunk_run_pieces.argtypes = [ctypes.c_longlong, ctypes.c_int, ctypes.c_int, ctypes.c_longlong,
                                         ctypes.POINTER(ctypes.c_int), ctypes.c_int]
    L.swila_device_status.restype = ctypes.c_int
    L.swila_selftest_wait_timeout.restype = ctypes.c_int
    L.swila_selftest_wait_timeout.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
    L.swila_auto_algo.restype = ctypes.c_int
    L.swila_auto_algo.argtypes = [ctypes.POINTER(Shape), ctypes.c_int]
    L.swila_bench_fma_chain.restype = ctypes.c_int
    L.swila_bench_fma_chain.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p,
                                        ctypes.POINTER(ctypes.c_double), ctypes.c_void_p]
    return L


lib = _load()


def make_shape(w: Workload, T: Optional[int] = None, algo: int = ALGO_AUTO) -> Shape:
    return Shape(w.B, w.H, w.T if T is None else T, w.Dk, w.Dv, w.J,
                 IO_BF16 if w.io_dtype == "bf16" else IO_FP32, w.flags, w.gate_granularity, algo)


def _p(t: Optional[torch.Tensor], host: bool = False):
    if t is None:
        return None
    assert t.is_contiguous() and t.is_cuda != host, "contiguous tensors on the side the entry point expects"
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _gates(inp: dict, host: bool = False) -> Gates:
    return Gates(*[(_p(inp.get(n), host) or ctypes.c_void_p(None)).value for n in
                   ("beta_logit", "pik_logit", "piq_logit", "gk_logit", "gq_logit", "alpha")])


def _state(W, r, rho) -> State:
    return State(W.data_ptr(), r.data_ptr() if r is not None else None, rho.data_ptr() if rho is not None else None)


def check(status: int) -> None:
    if status != SWILA_OK:
        raise SwilaError(status)


def state_alloc(w: Workload, device="cuda", init: bool = True, stream=None) -> dict:
    """Allocate (torch) and optionally initialise (library) a carried state."""
    st = {"W": torch.empty((w.B, w.H, w.J, w.Dv, w.Dk), device=device, dtype=torch.float32),
          "r_prev": None, "rho_prev": None}
    if w.temporal:
        st["r_prev"] = torch.empty((w.B, w.H, w.J, w.Dv), device=device, dtype=torch.float32)
        st["rho_prev"] = torch.empty((w.B, w.H, w.J, w.Dv), device=device, dtype=torch.float32)
    if init:
        sh = make_shape(w)
        s = _state(st["W"], st["r_prev"], st["rho_prev"])
        check(lib.swila_state_init(ctypes.byref(sh), ctypes.byref(s), _stream(stream)))
    return st


def swila_forward(w: Workload, inp: dict, *, state_in: Optional[dict] = None, state_out: Optional[dict] = None,
                  o: Optional[torch.Tensor] = None, r_debug: Optional[torch.Tensor] = None,
                  algo: int = ALGO_AUTO, stream=None, T: Optional[int] = None) -> torch.Tensor:
    """Prefill over inp's q,k,v and gate tensors (device tensors laid out as in
    include/swila.h).  state_in / state_out: dicts with W (and r_prev, rho_prev when
    TEMPORAL), or None (initial state / discard).  Returns o."""
    T = inp["q"].shape[2] if T is None else T
    sh = make_shape(w, T=T, algo=algo)
    if o is None:
        o = torch.empty((w.B, w.H, T, w.Dv), device=inp["q"].device, dtype=w.torch_io_dtype)
    g = _gates(inp)
    sin = _state(state_in["W"], state_in.get("r_prev"), state_in.get("rho_prev")) if state_in else None
    sout = _state(state_out["W"], state_out.get("r_prev"), state_out.get("rho_prev")) if state_out else None
    check(lib.swila_forward(ctypes.byref(sh), _p(inp["q"]), _p(inp["k"]), _p(inp["v"]), ctypes.byref(g),
                            ctypes.byref(sin) if sin else None, ctypes.byref(sout) if sout else None,
                            _p(o), _p(r_debug), _stream(stream)))
    return o


def stats_alloc(w: Workload, device="cuda") -> dict:
    """Zeroed buffers for swila_forward_stats: r_sum, rho_sum [B,H,J,Dv]; r_ent, rho_ent [B,H,Dv]."""
    z = lambda *shape: torch.zeros(shape, device=device, dtype=torch.float32)  # noqa: E731
    return {"r_sum": z(w.B, w.H, w.J, w.Dv), "r_ent": z(w.B, w.H, w.Dv),
            "rho_sum": z(w.B, w.H, w.J, w.Dv), "rho_ent": z(w.B, w.H, w.Dv)}


def swila_forward_stats(w: Workload, inp: dict, stats: dict, *, state_in: Optional[dict] = None,
                        state_out: Optional[dict] = None, o: Optional[torch.Tensor] = None,
                        r_debug: Optional[torch.Tensor] = None, algo: int = ALGO_AUTO, stream=None,
                        T: Optional[int] = None) -> torch.Tensor:
    """swila_forward that also ADDS the sums over time of the mixture weights (Sec. 3.5) to the
    buffers in ``stats`` (keys r_sum, r_ent, rho_sum, rho_ent; a missing key or None skips that sum)."""
    T = inp["q"].shape[2] if T is None else T
    sh = make_shape(w, T=T, algo=algo)
    if o is None:
        o = torch.empty((w.B, w.H, T, w.Dv), device=inp["q"].device, dtype=w.torch_io_dtype)
    g = _gates(inp)
    sin = _state(state_in["W"], state_in.get("r_prev"), state_in.get("rho_prev")) if state_in else None
    sout = _state(state_out["W"], state_out.get("r_prev"), state_out.get("rho_prev")) if state_out else None
    st = Stats(*[(_p(stats.get(n)) or ctypes.c_void_p(None)).value for n in ("r_sum", "r_ent", "rho_sum", "rho_ent")])
    check(lib.swila_forward_stats(ctypes.byref(sh), _p(inp["q"]), _p(inp["k"]), _p(inp["v"]), ctypes.byref(g),
                                  ctypes.byref(sin) if sin else None, ctypes.byref(sout) if sout else None,
                                  _p(o), _p(r_debug), ctypes.byref(st), _stream(stream)))
    return o


def swila_output_norm(w: Workload, o: torch.Tensor, weight: Optional[torch.Tensor] = None, eps: float = 1e-6,
                      stream=None) -> torch.Tensor:
    """RMSNorm of o [B,H,T,Dv] over its last axis, in place (App. D.1); weight fp32 [Dv] or None."""
    sh = make_shape(w, T=o.shape[2])
    check(lib.swila_output_norm(ctypes.byref(sh), _p(o), _p(weight), ctypes.c_float(eps), _stream(stream)))
    return o


def swila_decode_step(w: Workload, inp: dict, state: dict, *, o: Optional[torch.Tensor] = None,
                      algo: int = ALGO_AUTO, stream=None) -> torch.Tensor:
    """One token on a carried state (updated in place).  Returns o [B,H,1,Dv]."""
    sh = make_shape(w, T=1, algo=algo)
    if o is None:
        o = torch.empty((w.B, w.H, 1, w.Dv), device=inp["q"].device, dtype=w.torch_io_dtype)
    g = _gates(inp)
    st = _state(state["W"], state.get("r_prev"), state.get("rho_prev"))
    check(lib.swila_decode_step(ctypes.byref(sh), _p(inp["q"]), _p(inp["k"]), _p(inp["v"]), ctypes.byref(g),
                                ctypes.byref(st), _p(o), _stream(stream)))
    return o


def bench_fma_chain(packed: bool, chains: int, blocks: int, iters: int, scratch: torch.Tensor, stream=None) -> float:
    """Launch the FMA-chain microbenchmark once; returns the FMAs it performs."""
    n = ctypes.c_double(0.0)
    check(lib.swila_bench_fma_chain(int(packed), chains, blocks, iters, _p(scratch), ctypes.byref(n), _stream(stream)))
    return n.value


def host_workspace_bytes(w: Workload, T: Optional[int] = None) -> int:
    sh = make_shape(w, T=T)
    return int(lib.swila_forward_host_workspace_bytes(ctypes.byref(sh)))


def swila_forward_host(w: Workload, inp: dict, workspace: torch.Tensor, *, state_in: Optional[dict] = None,
                       state_out: Optional[dict] = None, o: Optional[torch.Tensor] = None, algo: int = ALGO_AUTO,
                       stream=None) -> torch.Tensor:
    """Prefill on HOST tensors (pinned for asynchronous copies) staged through the caller's
    device ``workspace`` (a uint8 CUDA tensor).  Returns the host tensor o; synchronise the
    stream before reading it."""
    T = inp["q"].shape[2]
    sh = make_shape(w, T=T, algo=algo)
    if o is None:
        o = torch.empty((w.B, w.H, T, w.Dv), dtype=w.torch_io_dtype).pin_memory()
    g = _gates(inp, host=True)
    sin = _state(state_in["W"], state_in.get("r_prev"), state_in.get("rho_prev")) if state_in else None
    sout = _state(state_out["W"], state_out.get("r_prev"), state_out.get("rho_prev")) if state_out else None
    check(lib.swila_forward_host(ctypes.byref(sh), _p(inp["q"], True), _p(inp["k"], True), _p(inp["v"], True),
                                 ctypes.byref(g), ctypes.byref(sin) if sin else None,
                                 ctypes.byref(sout) if sout else None, _p(o, True), _p(workspace),
                                 workspace.numel() * workspace.element_size(), _stream(stream)))
    return o


def swila_forward_host_static(w: Workload, inp: dict, *, state_in: Optional[dict] = None,
                              state_out: Optional[dict] = None, o: Optional[torch.Tensor] = None,
                              algo: int = ALGO_AUTO, stream=None) -> torch.Tensor:
    """swila_forward_host without a caller workspace: the library stages through its own fixed
    16 MiB device array, for callers that may not allocate device memory.  The output tensor
    must be supplied (or is created here in pinned host memory, which is a host allocation).
    Calls that overlap on the GPU race on the shared array; keep them on one stream."""
    T = inp["q"].shape[2]
    sh = make_shape(w, T=T, algo=algo)
    if o is None:
        o = torch.empty((w.B, w.H, T, w.Dv), dtype=w.torch_io_dtype).pin_memory()
    g = _gates(inp, host=True)
    sin = _state(state_in["W"], state_in.get("r_prev"), state_in.get("rho_prev")) if state_in else None
    sout = _state(state_out["W"], state_out.get("r_prev"), state_out.get("rho_prev")) if state_out else None
    check(lib.swila_forward_host_static(ctypes.byref(sh), _p(inp["q"], True), _p(inp["k"], True), _p(inp["v"], True),
                                        ctypes.byref(g), ctypes.byref(sin) if sin else None,
                                        ctypes.byref(sout) if sout else None, _p(o, True), _stream(stream)))
    return o


def selftest_tf32_mma(A: torch.Tensor, B: torch.Tensor) -> torch.Tensor:
    """D = A @ B.T on the tcgen05 path (A [128,K], B [N,K], fp32 on the device)."""
    N, K = B.shape
    D = torch.zeros((128, N), device=A.device, dtype=torch.float32)
    status = torch.zeros(1, device=A.device, dtype=torch.int32)
    check(lib.swila_selftest_tf32_mma(_p(A), _p(B), _p(D), N, K, _p(status), _stream(None)))
    torch.cuda.synchronize()
    if int(status.item()) != 0:
        raise RuntimeError("tcgen05 self-test: the MMA did not signal completion")
    return D


def selftest_bf16_mma(A: torch.Tensor, B: torch.Tensor, a_in_smem: int = 0) -> torch.Tensor:
    """D = bf16(A) @ bf16(B).T on the tcgen05 path (A [128,K], B [N,K], fp32 on the device).
    a_in_smem: 0 = A through tensor memory, 1 = A through shared memory, 2 = both operands in
    the 128-byte-swizzle shared-memory layout, 3 = A through tensor memory and B MN-major with that swizzle."""
    N, K = B.shape
    D = torch.zeros((128, N), device=A.device, dtype=torch.float32)
    status = torch.zeros(1, device=A.device, dtype=torch.int32)
    check(lib.swila_selftest_bf16_mma(_p(A), _p(B), _p(D), N, K, int(a_in_smem), _p(status), _stream(None)))
    torch.cuda.synchronize()
    if int(status.item()) != 0:
        raise RuntimeError("tcgen05 self-test: the MMA did not signal completion")
    return D


def chunk_plan(B: int, H: int, T: int, Dv: int, J: int, sm_count: int, has_state_out: bool = True) -> dict:
    """Work layout SWILA_ALGO_CHUNK would choose (host arithmetic only)."""
    out = (ctypes.c_longlong * 6)()
    check(lib.swila_chunk_plan(B, H, T, Dv, J, sm_count, int(has_state_out), out))
    return dict(zip(("split", "gang", "nch", "per", "units", "grid"), (int(x) for x in out)))


def chunk_run_pieces(units: int, nch: int, per: int, run: int) -> list:
    """Pieces (unit, first chunk, end chunk) of one run, in processing order (host arithmetic only)."""
    cap = 16 + per // max(nch, 1)
    buf = (ctypes.c_int * (3 * cap))()
    n = lib.swila_chunk_run_pieces(units, nch, per, run, buf, cap)
    if n < 0:
        check(n)
    return [(buf[3 * i], buf[3 * i + 1], buf[3 * i + 2]) for i in range(n)]


def auto_algo(w: Workload, aux_outputs: bool = False) -> int:
    """The kernel ALGO_AUTO resolves to for this workload (ALGO_CHUNK or ALGO_SCAN)."""
    sh = make_shape(w)
    rc = int(lib.swila_auto_algo(ctypes.byref(sh), int(aux_outputs)))
    if rc < 0:
        check(rc)
    return rc


def device_status() -> None:
    """Synchronise and raise if a kernel of the library recorded a device-side failure."""
    check(lib.swila_device_status())
