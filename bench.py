#!/usr/bin/env python
"""Benchmark of the SwiLA recurrence on B200.

A step is one pass of the whole hot path -- one ``swila_forward`` over the language-model
shaped prefill workload (B=4, H=16, T=8192, Dk=Dv=128, J=4, bf16 inputs, fp32 state) with
inputs resident in HBM (the library picks the chunked tensor-core kernel).  Reported beside it: the same call end to end from pinned host
buffers (``e2e``), the batched decode leg (B=256 streams, H=32, 1024 single-token steps),
the roofline of the scan kernel, and the fp64 CPU oracle timed on the host cores.

    python bench.py --gpus 1 --steps 10 --warmup 3
    python -m torch.distributed.run --nproc-per-node N ... bench.py --gpus N ...   (independent replicas)
    python bench.py --impl reference      (the CPU oracle alone, same metric and workload)
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2609_39034_b200 import workloads as wl  # noqa: E402

METRIC = "swila_fwd_tokens_per_s"
UNIT = "tokens/s"
HEADLINE = 2  # config index of the workload the metric is quoted on
VARIANTS = {"vanilla": {}, "temporal": dict(temporal=True), "gated_pre_per_key": dict(gated=True),
            "gated_post_per_key": dict(gated=True, post_decay=True),
            "gated_pre_per_out": dict(gated=True, granularity=wl.GRAN_PER_OUT),
            "gated_pre_scalar": dict(gated=True, granularity=wl.GRAN_SCALAR),
            "gated_temporal": dict(temporal=True, gated=True)}

# DRAM traffic per launch comes from profiles/traffic.json (ncu: dram__bytes_read.sum + dram__bytes_write.sum of one
# captured launch), keyed by kernel and workload; an entry counts only while the kernel source it was captured from
# is unchanged (sha256 of the file), else the bench line reports null.
def ncu_traffic(kernel: str, workload: str):
    import hashlib

    path = os.path.join(ROOT, "profiles", "traffic.json")
    if not os.path.exists(path):
        return None
    for e in json.load(open(path)).get("entries", []):
        if e.get("kernel") == kernel and e.get("workload") == workload:
            src = os.path.join(ROOT, e.get("source", ""))
            if os.path.exists(src) and hashlib.sha256(open(src, "rb").read()).hexdigest()[:16] == e.get("source_sha16"):
                return e.get("dram_bytes_per_launch")
    return None


# ----------------------------------------------------------------------------------------------
def algorithmic_bytes(w: wl.Workload) -> float:
    """HBM bytes one prefill must move: q, k, v, o, three gate tensors, plus the state once
    each way."""
    es = 2 if w.io_dtype == "bf16" else 4
    per_tok_head = (2 * w.Dk + 2 * w.Dv + 3 * w.J * w.Dv) * es
    if w.temporal:
        per_tok_head += 2 * w.Dv * es
    if w.gated:
        per = {wl.GRAN_PER_KEY: w.Dk, wl.GRAN_PER_OUT: w.Dv, wl.GRAN_SCALAR: 1,
               wl.GRAN_ELEMENTWISE: w.Dk * w.Dv}[w.gate_granularity]
        per_tok_head += w.J * per * 4
    state = 2 * w.J * w.Dk * w.Dv * 4
    return float(w.B * w.H * (w.T * per_tok_head + state))


def algorithmic_flops(w: wl.Workload, T=None) -> float:
    """FP32 flops of the recurrence: prediction, update and readout are J*Dk*Dv FMAs each."""
    T = w.T if T is None else T
    return 6.0 * w.J * w.Dk * w.Dv * w.B * w.H * T


class ClockSampler:
    """nvidia-smi samples (SM clock, throttle reasons) taken DURING a timed region."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.path = index, None, None

    def start(self):
        fd, self.path = tempfile.mkstemp(suffix=".csv")
        os.close(fd)
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        clocks, reasons, mx, power = [], set(), None, []
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for ln in open(self.path):
            parts = [x.strip() for x in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                clocks.append(float(parts[0]))
                mx = float(parts[1])
                power.append(float(parts[2]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        os.unlink(self.path)
        if clocks:
            out.update(sm_mhz=statistics.median(clocks), sm_max_mhz=mx, reasons=sorted(reasons),
                       samples=len(clocks), power_w_max=max(power))
        return out


def max_over_ranks(ms: float, world: int, device="cpu") -> float:
    """The slowest rank's time: every multi-GPU number is the maximum over ranks (all-reduce MAX on
    whatever process group is initialised; identity for a single process)."""
    if world <= 1:
        return float(ms)
    import torch.distributed as dist

    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(world: int, B: int, T: int, ms_per_step: float) -> float:
    """Independent replicas (weak scaling): every rank processes its own B x T tokens per step."""
    return world * B * T / (ms_per_step * 1e-3)


def time_blocks(fn, steps: int, stream, min_seconds: float = 2.0, max_blocks: int = 400):
    """Blocks of `steps` back-to-back calls, each block timed with its own CUDA event pair, repeated until
    `min_seconds` of device time have been covered: the per-step times of the blocks (ms)."""
    out, total = [], 0.0
    while not out or (total < min_seconds * 1e3 and len(out) < max_blocks):
        ms = time_steps(fn, steps, stream)
        out.append(ms / steps)
        total += ms
    return out


def time_steps(fn, steps: int, stream) -> float:
    """Milliseconds for `steps` back-to-back calls of fn, CUDA events on `stream`."""
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(steps):
        fn()
    b.record(stream)
    b.synchronize()
    return a.elapsed_time(b)


# ----------------------------------------------------------------------------------------------
def cpu_baseline(w: wl.Workload, n_bh: int, repeats: int = 1, warmup: int = 0):
    """The fp64 oracle, as it stands, on the first n_bh (batch, head) pairs of workload w
    (all T tokens, all Dv columns).  Returns (tokens/s, seconds per pass, threads)."""
    from oracle import swila_oracle

    small = w.with_(B=1, H=n_bh)
    inp = wl.make_inputs(small)  # CPU tensors; same shapes and dtypes as the workload's rows
    cores = swila_oracle.threads()
    for _ in range(warmup):
        swila_oracle.forward_inputs(inp)
    ts = []
    for _ in range(repeats):
        t0 = time.perf_counter()
        swila_oracle.forward_inputs(inp)
        ts.append(time.perf_counter() - t0)
    sec = sum(ts) / len(ts)
    # a token counts once for all H heads of the workload
    tokens = n_bh * w.T / w.H
    return tokens / sec, sec, cores


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = wl.CONFIGS[HEADLINE]
    n_bh = 2
    val, sec, cores = cpu_baseline(w, n_bh, repeats=max(1, args.steps), warmup=args.warmup)
    sample = f"{n_bh} of {w.B * w.H} (batch, head) rows of {w.name}, all {w.T} tokens and {w.Dv} columns, per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "H": w.H, "T": w.T, "Dk": w.Dk, "Dv": w.Dv, "J": w.J,
                   "note": "fp64 CPU oracle on a bounded sample; tokens/s scaled by sampled rows / H"},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------
def measure_fma_peak(binding, stream) -> float:
    """FP32 FMA-chain microbenchmark (scalar FMAs, 16 chains/thread, 8 blocks/SM): TFLOP/s."""
    scratch = torch.zeros(4, device="cuda")
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    best = 0.0
    for _ in range(3):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        n = binding.bench_fma_chain(False, 16, sms * 8, 20000, scratch)
        b.record(stream)
        b.synchronize()
        best = max(best, 2.0 * n / (a.elapsed_time(b) * 1e-3) / 1e12)
    return best


def decode_leg(binding, args, stream, dev_index):
    """Config 4: B=256 streams, H=32; states from a seeded 4096-token prefill fed in chunks of
    256 tokens, then `decode_steps` single-token calls with fresh inputs, timed back to back."""
    w = wl.CONFIGS[4]
    if args.decode_batch:
        w = w.with_(B=args.decode_batch)
    st = binding.state_alloc(w)
    chunk = wl.DECODE_PREFILL_CHUNK
    for c in range(args.decode_prefill // chunk):
        inp = wl.make_inputs(w.with_(T=chunk), device="cuda", seed_offset=1 + c)
        binding.swila_forward(w, inp, state_in=st, state_out=st)
        torch.cuda.synchronize()
        del inp
    steps = args.decode_steps
    ins = [wl.decode_step_inputs(w, s, device="cuda") for s in range(steps)]
    o = torch.empty((w.B, w.H, 1, w.Dv), device="cuda", dtype=w.torch_io_dtype)
    # warm-up on a scratch copy of the state
    warm = {k: (v.clone() if v is not None else None) for k, v in st.items()}
    for s in range(min(8, steps)):
        binding.swila_decode_step(w, ins[s], warm, o=o)
    torch.cuda.synchronize()
    del warm
    sampler = ClockSampler(dev_index)
    sampler.start()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for s in range(steps):
        binding.swila_decode_step(w, ins[s], st, o=o)
    b.record(stream)
    b.synchronize()
    clocks = sampler.stop()
    ms = a.elapsed_time(b)
    es = 2
    per_bh_inputs = (2 * w.Dk + 2 * w.Dv + 3 * w.J * w.Dv) * es
    bytes_step = w.B * w.H * (per_bh_inputs + 2 * w.J * w.Dk * w.Dv * 4)
    peaks = _peaks()
    ach = bytes_step * steps / (ms * 1e-3) / 1e9
    return {
        "workload": w.name, "B": w.B, "H": w.H, "Dk": w.Dk, "Dv": w.Dv, "J": w.J, "prefill_tokens": args.decode_prefill,
        "steps": steps, "steps_per_s": steps / (ms * 1e-3), "tokens_per_s": w.B * steps / (ms * 1e-3),
        "ms_per_step": ms / steps, "gpu_launches": steps,
        "roofline": {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": ach / peaks["hbm_gbs"], "peak_source": peaks["source"], "traffic": None,
                     "algorithmic_bytes_per_launch": bytes_step},
        "clocks": clocks,
    }


def paper_shapes_leg(binding, stream):
    """Shapes the paper quotes (not the headline): the 374M LM layer (H=8, J=4, D=64) at B=16, T=4096
    (App. C), and the generation protocol of App. D.4 (2048-token prompt + 128 decoded tokens) at several
    batch sizes; generation time includes prefill and decode, as in the paper."""
    out = {}
    lm = wl.CONFIGS[1].with_(name="lm374m_layer", B=16, H=8, T=4096)
    inp = wl.make_inputs(lm, device="cuda")
    st = binding.state_alloc(lm, init=False)
    o = torch.empty((lm.B, lm.H, lm.T, lm.Dv), device="cuda", dtype=lm.torch_io_dtype)
    f = lambda: binding.swila_forward(lm, inp, state_in=None, state_out=st, o=o)
    for _ in range(3):
        f()
    torch.cuda.synchronize()
    ms = time_steps(f, 10, stream) / 10
    out["lm374m_layer_prefill"] = {"B": lm.B, "H": lm.H, "T": lm.T, "D": lm.Dk, "J": lm.J, "ms": ms,
                                   "tokens_per_s": lm.B * lm.T / (ms * 1e-3)}
    del inp, o, st
    # the component-count ablation of Sec. 5: the same layer with J = 16 (scan kernel)
    lm16 = lm.with_(name="lm374m_layer_j16", J=16)
    inp = wl.make_inputs(lm16, device="cuda")
    st = binding.state_alloc(lm16, init=False)
    o = torch.empty((lm16.B, lm16.H, lm16.T, lm16.Dv), device="cuda", dtype=lm16.torch_io_dtype)
    f16 = lambda: binding.swila_forward(lm16, inp, state_in=None, state_out=st, o=o)
    for _ in range(3):
        f16()
    torch.cuda.synchronize()
    ms = time_steps(f16, 10, stream) / 10
    out["lm374m_layer_prefill_j16"] = {"B": lm16.B, "H": lm16.H, "T": lm16.T, "D": lm16.Dk, "J": lm16.J, "ms": ms,
                                       "tokens_per_s": lm16.B * lm16.T / (ms * 1e-3)}
    del inp, o, st
    gen_out = []
    for B in (1, 2, 4, 8, 16, 32, 64, 128):
        g = wl.CONFIGS[1].with_(name="generation", B=B, H=8, T=2048)
        prompt = wl.make_inputs(g, device="cuda")
        steps = [wl.decode_step_inputs(g, s, device="cuda") for s in range(128)]
        st = binding.state_alloc(g)
        o = torch.empty((g.B, g.H, g.T, g.Dv), device="cuda", dtype=g.torch_io_dtype)
        o1 = torch.empty((g.B, g.H, 1, g.Dv), device="cuda", dtype=g.torch_io_dtype)

        def generate():
            binding.swila_forward(g, prompt, state_in=None, state_out=st, o=o)
            for s in range(128):
                binding.swila_decode_step(g, steps[s], st, o=o1)

        generate()
        torch.cuda.synchronize()
        ms = time_steps(generate, 3, stream) / 3
        gen_out.append({"batch": B, "ms_per_call": ms, "tokens_per_s": B * (2048 + 128) / (ms * 1e-3)})
    out["generation_2048_plus_128"] = {"H": 8, "D": 64, "J": 4, "runs": gen_out,
                                       "note": "one layer's recurrence only; 1 warm-up + 3 timed calls"}
    return out


def variants_leg(binding, stream, fma_peak_tflops: float):
    """The Temporal and Gated variants (App. B.3, Eqs. 3.7-3.8, App. B.4) on all five configurations: prefill time per
    variant for configs 0-3, decode time per step for config 4 (after a 256-token prefill).  Every line is ALGO_AUTO;
    `kernel` says which kernel that resolved to, and `roofline` is taken against the slower bound of that kernel's
    pipes: the FP32 ALUs (3 FMAs per state element and token, one more multiply when gated) or HBM for the scan, HBM
    or the bf16 tensor peak for the chunked kernel."""
    names = list(VARIANTS.items())
    peaks = _peaks()

    def roofline(w, ms, chunk):
        sec = ms * 1e-3
        t_hbm = algorithmic_bytes(w) / (peaks["hbm_gbs"] * 1e9)
        if chunk:
            t_pipe, pipe = algorithmic_flops(w) / (peaks["bf16_tflops"] * 1e12), "tensor"
        else:  # FP32 instruction slots: 3 FMAs (+ 1 multiply when gated) per state element and token, 2 flop each slot
            slots = (4.0 if w.gated else 3.0) / 3.0 * algorithmic_flops(w)
            t_pipe, pipe = slots / (fma_peak_tflops * 1e12), "alu"
        bound = "hbm" if t_hbm >= t_pipe else pipe
        return {"bound": bound, "frac": max(t_hbm, t_pipe) / sec, "t_hbm_ms": t_hbm * 1e3, "t_pipe_ms": t_pipe * 1e3}

    out = {}
    for cfg in (0, 1, 2, 3):
        rows = {}
        for name, kw in names:
            w = wl.CONFIGS[cfg].variant(**kw)
            inp = wl.make_inputs(w, device="cuda")
            st = binding.state_alloc(w)
            o = torch.empty((w.B, w.H, w.T, w.Dv), device="cuda", dtype=w.torch_io_dtype)
            f = lambda: binding.swila_forward(w, inp, state_in=None, state_out=st, o=o)
            for _ in range(3):
                f()
            torch.cuda.synchronize()
            ms = time_steps(f, 10, stream) / 10
            chunk = binding.auto_algo(w) == binding.ALGO_CHUNK
            rows[name] = {"ms": ms, "tokens_per_s": w.B * w.T / (ms * 1e-3), "kernel": "chunk" if chunk else "scan",
                          "roofline": roofline(w, ms, chunk)}
            del inp, st, o
        out[wl.CONFIGS[cfg].name] = rows
    rows = {}
    for name, kw in names:
        w = wl.CONFIGS[4].variant(**kw).with_(T=256)
        st = binding.state_alloc(w)
        pre = wl.make_inputs(w, device="cuda", seed_offset=1)
        binding.swila_forward(w, pre, state_in=st, state_out=st)
        del pre
        steps = [wl.decode_step_inputs(w, s, device="cuda") for s in range(8)]
        o1 = torch.empty((w.B, w.H, 1, w.Dv), device="cuda", dtype=w.torch_io_dtype)
        k = [0]

        def step():
            binding.swila_decode_step(w, steps[k[0] % 8], st, o=o1)
            k[0] += 1

        for _ in range(8):
            step()
        torch.cuda.synchronize()
        ms = time_steps(step, 64, stream) / 64
        rows[name] = {"ms_per_step": ms, "steps_per_s": 1e3 / ms, "kernel": "scan",
                      "roofline": {"bound": "hbm",
                                   "frac": algorithmic_bytes(w.with_(T=1)) / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}}
        del st, steps, o1
    out[wl.CONFIGS[4].name + "_decode"] = rows
    return out


def fusions_leg(binding, stream):
    """The steps either side of the recurrence (App. B.2, App. D.1, Sec. 3.5) on the LM-shaped prefill: what the
    in-kernel q/k/v activation and the sums over time cost the scan kernel, and the output RMSNorm pass against
    the copy bandwidth (it reads and writes o once)."""
    peaks = _peaks()
    w = wl.CONFIGS[HEADLINE]
    inp = wl.make_inputs(w, device="cuda")
    st = binding.state_alloc(w)
    o = torch.empty((w.B, w.H, w.T, w.Dv), device="cuda", dtype=w.torch_io_dtype)
    stats = binding.stats_alloc(w)
    wa = w.with_(flags=w.flags | wl.FLAG_QKV_ACT)
    wgt = torch.ones(w.Dv, device="cuda")
    w4 = w.with_(B=4 * w.B)  # 537 MB of outputs: four times the L2, so the pass runs from HBM
    o4 = torch.randn((w4.B, w4.H, w4.T, w4.Dv), device="cuda").to(w.torch_io_dtype)
    calls = {
        "scan_plain": lambda: binding.swila_forward(w, inp, state_in=None, state_out=st, o=o, algo=binding.ALGO_SCAN),
        "scan_qkv_act": lambda: binding.swila_forward(wa, inp, state_in=None, state_out=st, o=o, algo=binding.ALGO_SCAN),
        "scan_stats": lambda: binding.swila_forward_stats(w, inp, stats, state_in=None, state_out=st, o=o,
                                                          algo=binding.ALGO_SCAN),
        "chunk_plain": lambda: binding.swila_forward(w, inp, state_in=None, state_out=st, o=o, algo=binding.ALGO_CHUNK),
        "chunk_stats": lambda: binding.swila_forward_stats(w, inp, stats, state_in=None, state_out=st, o=o,
                                                           algo=binding.ALGO_CHUNK),
        "output_norm": lambda: binding.swila_output_norm(w4, o4, wgt),
    }
    out = {}
    for name, f in calls.items():
        for _ in range(3):
            f()
        torch.cuda.synchronize()
        out[name] = {"ms": time_steps(f, 10, stream) / 10}
    norm_bytes = 2 * o4.numel() * o4.element_size()
    out["output_norm"].update({"bytes": norm_bytes, "gbs": norm_bytes / (out["output_norm"]["ms"] * 1e-3) / 1e9,
                               "hbm_frac": norm_bytes / (out["output_norm"]["ms"] * 1e-3) / 1e9 / peaks["hbm_gbs"],
                               "note": "o of four LM-shaped prefills (537 MB, larger than L2), read and written once"})
    return out


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "source": "measured (MEASURED_PEAKS.json)"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "source": "fallback"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--algo", type=int, default=0, help="SWILA_ALGO_* kernel choice (0 = auto)")
    ap.add_argument("--no-decode", action="store_true", help="skip the batched decode leg")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle baseline")
    ap.add_argument("--no-scan", action="store_true", help="skip the scan-kernel comparison leg")
    ap.add_argument("--no-paper-shapes", action="store_true", help="skip the shapes the paper itself quotes")
    ap.add_argument("--no-variants", action="store_true", help="skip the Temporal / Gated variants on all five configs")
    ap.add_argument("--no-fusions", action="store_true", help="skip the q/k/v activation, the statistics and the output norm")
    ap.add_argument("--only-headline", action="store_true", help="time the headline step only (profiling runs)")
    ap.add_argument("--min-seconds", type=float, default=2.0, help="repeat the block of --steps until this much is timed")
    # accepted for older command lines; these legs now run by default
    ap.add_argument("--paper-shapes", action="store_true", help=argparse.SUPPRESS)
    ap.add_argument("--variants", action="store_true", help=argparse.SUPPRESS)
    ap.add_argument("--fusions", action="store_true", help=argparse.SUPPRESS)
    ap.add_argument("--decode-steps", type=int, default=wl.DECODE_STEPS)
    ap.add_argument("--decode-prefill", type=int, default=4096)
    ap.add_argument("--decode-batch", type=int, default=0, help="override B of the decode leg (0 = 256)")
    ap.add_argument("--batch", type=int, default=0, help="override B of the prefill workload (profiling only)")
    ap.add_argument("--variant", default="vanilla", choices=sorted(VARIANTS), help="variant of the timed step (profiling only; the metric is quoted on vanilla)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.only_headline:
        args.no_decode = args.no_e2e = args.no_cpu = args.no_scan = True
        args.no_paper_shapes = args.no_variants = args.no_fusions = True

    if args.impl == "reference":
        run_reference(args)
        return

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device; there is no CPU fallback"
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    from paper_2609_39034_b200 import build as swila_build

    if rank == 0 or world == 1:
        swila_build.build()
    if world > 1:
        dist.barrier()
    from paper_2609_39034_b200 import binding

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    w = wl.CONFIGS[HEADLINE].variant(**VARIANTS[args.variant])
    if args.variant != "vanilla":
        w = w.with_(name=w.name + "+" + args.variant)
    if args.batch:
        w = w.with_(B=args.batch)
    stream = torch.cuda.current_stream()
    inp = wl.make_inputs(w, device="cuda")
    st_out = binding.state_alloc(w, init=False)
    o = torch.empty((w.B, w.H, w.T, w.Dv), device="cuda", dtype=w.torch_io_dtype)

    def step():
        binding.swila_forward(w, inp, state_in=None, state_out=st_out, o=o, algo=args.algo)

    for _ in range(args.warmup):
        step()
    barrier()
    # Timed region: blocks of exactly --steps launches, each with its own event pair, repeated until --min-seconds
    # have been covered, so that the clock samples below see the load.  ms_per_step is the median block; the minimum
    # and the block count are reported beside it.
    sampler = ClockSampler(local)
    sampler.start()
    blocks = time_blocks(step, args.steps, stream, args.min_seconds)
    barrier()
    clocks = sampler.stop()
    ms_per_step = max_over_ranks(statistics.median(blocks), world, "cuda")
    ms_min = max_over_ranks(min(blocks), world, "cuda")
    value = whole_job_tokens_per_s(world, w.B, w.T, ms_per_step)
    timing = {"blocks": len(blocks), "steps_per_block": args.steps, "ms_per_step_median": ms_per_step,
              "ms_per_step_min": ms_min, "timed_seconds": sum(blocks) * args.steps * 1e-3,
              "ms_x_sm_mhz": ms_per_step * clocks["sm_mhz"] if clocks.get("sm_mhz") else None}

    # ---- roofline of the kernel the step launches (one launch per step) ----
    props = torch.cuda.get_device_properties(local)
    peaks = _peaks()
    fma_peak_nominal = props.multi_processor_count * 128 * 2 * 1.965e9 / 1e12  # TFLOP/s at the max SM clock
    fma_peak_measured = measure_fma_peak(binding, stream)
    flops = algorithmic_flops(w)
    abytes = algorithmic_bytes(w)
    sec = ms_per_step * 1e-3
    chunked = args.algo == binding.ALGO_CHUNK or (args.algo == 0 and binding.auto_algo(w) == binding.ALGO_CHUNK)
    if chunked:
        # The chunked kernel runs the state contractions on the tensor cores (bf16 operands, fp32
        # accumulation), so of the two bounds -- HBM bytes at the measured copy bandwidth, flops at the
        # measured bf16 tensor peak -- HBM is by far the slower one (0.33 ms vs 0.13 ms on this workload)
        # and is the roofline reported.
        bf16_peak = peaks["bf16_tflops"]
        roofline = {
            "bound": "hbm", "achieved": abytes / sec / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": abytes / sec / 1e9 / peaks["hbm_gbs"], "peak_source": peaks["source"],
            "traffic": ncu_traffic("swila_chunk_kernel", w.name) if not args.batch else None,
            "algorithmic_bytes_per_launch": abytes, "algorithmic_flops_per_launch": flops,
            "kernel": "swila_chunk_kernel",
            "tensor_bound": {"achieved_tflops": flops / sec / 1e12, "peak_tflops": bf16_peak,
                             "frac": flops / sec / 1e12 / bf16_peak,
                             "peak_source": "measured bf16 peak (the kernel's MMAs take bf16 operands)"},
            "note": "latency-bound: the T tokens of a row are a serial dependency chain "
                    "(~180 cycles per token for a row warp running alone, ~210 beside the helper warps)",
        }
    else:
        ach_tflops = flops / sec / 1e12
        roofline = {
            "bound": "alu", "achieved": ach_tflops, "peak": fma_peak_nominal, "unit": "TFLOP/s",
            "frac": ach_tflops / fma_peak_nominal, "peak_source": "derived: SMs x 128 FP32 lanes x 2 x 1.965 GHz",
            "peak_measured_fma_chain": fma_peak_measured, "frac_of_measured_fma_chain": ach_tflops / fma_peak_measured,
            "traffic": ncu_traffic("swila_scan_kernel", w.name) if not args.batch else None,
            "algorithmic_bytes_per_launch": abytes, "algorithmic_flops_per_launch": flops,
            "hbm_achieved_gbs": abytes / sec / 1e9, "hbm_peak_gbs": peaks["hbm_gbs"], "kernel": "swila_scan_kernel",
        }

    # ---- the register-resident scan kernel on the same workload (the path of fp32 io, the TEMPORAL /
    #      GATED variants and decode), with its FP32-ALU roofline ----
    scan = None
    if chunked and not args.no_scan:
        def step_scan():
            binding.swila_forward(w, inp, state_in=None, state_out=st_out, o=o, algo=binding.ALGO_SCAN)
        for _ in range(3):
            step_scan()
        barrier()
        n_scan = max(3, min(args.steps, 10))
        ms_s = time_steps(step_scan, n_scan, stream) / n_scan
        barrier()
        ach = flops / (ms_s * 1e-3) / 1e12
        scan = {"ms_per_step": ms_s, "tokens_per_s": world * w.B * w.T / (ms_s * 1e-3), "steps": n_scan,
                "roofline": {"bound": "alu", "achieved": ach, "peak": fma_peak_nominal, "unit": "TFLOP/s",
                             "frac": ach / fma_peak_nominal,
                             "peak_source": "derived: SMs x 128 FP32 lanes x 2 x 1.965 GHz",
                             "peak_measured_fma_chain": fma_peak_measured,
                             "frac_of_measured_fma_chain": ach / fma_peak_measured, "kernel": "swila_scan_kernel"}}

    # ---- end to end from pinned host buffers through the C ABI ----
    e2e = None
    if not args.no_e2e:
        names = tuple(n for n in ("q", "k", "v", "beta_logit", "pik_logit", "piq_logit", "gk_logit", "gq_logit", "alpha")
                      if inp.get(n) is not None)
        host = {n: None for n in ("gk_logit", "gq_logit", "alpha")}
        host.update({n: inp[n].cpu().pin_memory() for n in names})
        o_host = torch.empty(o.shape, dtype=o.dtype).pin_memory()
        ws = torch.empty(binding.host_workspace_bytes(w), device="cuda", dtype=torch.uint8)

        def step_host():
            binding.swila_forward_host(w, host, ws, state_in=None, state_out=None, o=o_host, algo=args.algo)

        n_e2e = max(2, min(args.steps, 5))
        step_host()
        barrier()
        ms_e = time_steps(step_host, n_e2e, stream)
        barrier()
        ms_e = max_over_ranks(ms_e, world, "cuda")
        h2d = sum(host[n].numel() * host[n].element_size() for n in names)
        d2h = o_host.numel() * o_host.element_size()
        e2e = {"value": whole_job_tokens_per_s(world, w.B, w.T, ms_e / n_e2e), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": ms_e / n_e2e, "steps": n_e2e,
               "note": "swila_forward_host: pinned host inputs -> device workspace -> kernel -> o to pinned host"}
        del host, o_host, ws
    del inp, o, st_out
    torch.cuda.empty_cache()

    decode = None
    if not args.no_decode:
        decode = decode_leg(binding, args, stream, local)
        torch.cuda.empty_cache()

    extras = world == 1  # the further legs describe one GPU; a scaling run times the headline step only
    paper = paper_shapes_leg(binding, stream) if extras and not args.no_paper_shapes else None
    variants = variants_leg(binding, stream, fma_peak_nominal) if extras and not args.no_variants else None
    fusions = fusions_leg(binding, stream) if extras and not args.no_fusions else None

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        n_bh = wl.CONFIGS[HEADLINE].B * wl.CONFIGS[HEADLINE].H  # the whole workload: a few seconds on 16 cores
        val, sec, cores = cpu_baseline(wl.CONFIGS[HEADLINE], n_bh)
        cpu = {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "seconds": sec,
               "sample": f"{n_bh} of {wl.CONFIGS[HEADLINE].B * wl.CONFIGS[HEADLINE].H} (batch, head) rows, all tokens "
                         f"and columns, one pass; tokens/s = rows*T/H / s"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "B": w.B, "H": w.H, "T": w.T, "Dk": w.Dk, "Dv": w.Dv, "J": w.J,
                       "io_dtype": w.io_dtype, "state_dtype": "fp32", "algo": args.algo,
                       "arithmetic": "E-step, corrections inside a chunk and every accumulation in fp32",
                       "mma_operands": ("bf16 hi+lo (16 bit) for the state and Gram operands, update coefficients 24 bit, "
                                        "k and q exact bf16, fp32 accumulate") if chunked else None,
                       "error_measure": "max |x - y| / max(|y|, rms(y)) per tensor against the fp64 oracle",
                       "l2": "inputs (2.1 GB) larger than L2; no flush needed",
                       "multi_gpu": "independent replicas, no collective"},
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": args.steps * len(blocks),
            "timing": timing, "clocks": clocks, "decode": decode, "scan": scan, "paper_shapes": paper, "variants": variants, "fusions": fusions,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
