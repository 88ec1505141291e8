"""Time `swila_forward` on one of the named workloads with CUDA events (inputs resident on the device).

    python -m paper_2609_39034_b200.timing 2 1 --algo chunk

prints, per configuration index, the minimum and median time of a few launches and the tokens per
second they correspond to.  It is the small fixed loop the profiler captures under `profiles/` wrap:
three warm-up launches, then the timed ones, nothing else on the stream.

    python -m paper_2609_39034_b200.timing 2 --norm

times `swila_output_norm` instead, in place on four outputs of the configuration (larger than L2).
"""
import argparse

import torch

from . import binding
from . import workloads as wl

ALGOS = {"auto": binding.ALGO_AUTO, "scan": binding.ALGO_SCAN, "chunk": binding.ALGO_CHUNK}


def time_config(index: int, algo: int, launches: int = 7, warmup: int = 3, temporal: bool = False):
    w = wl.CONFIGS[index].variant(temporal=temporal)
    inp = wl.make_inputs(w, device="cuda")
    state = binding.state_alloc(w)
    o = torch.empty((w.B, w.H, w.T, w.Dv), device="cuda", dtype=w.torch_io_dtype)

    def launch():
        binding.swila_forward(w, inp, state_in=None, state_out=state, o=o, algo=algo)

    for _ in range(warmup):
        launch()
    torch.cuda.synchronize()
    times = []
    for _ in range(launches):
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record()
        launch()
        stop.record()
        torch.cuda.synchronize()
        times.append(start.elapsed_time(stop))
    binding.device_status()
    times.sort()
    return w, times[0], times[len(times) // 2]


def time_norm(index: int, launches: int = 7, warmup: int = 3):
    w = wl.CONFIGS[index]
    w4 = w.with_(B=4 * w.B)
    o = torch.randn((w4.B, w4.H, w4.T, w4.Dv), device="cuda").to(w.torch_io_dtype)
    weight = torch.ones(w.Dv, device="cuda")
    for _ in range(warmup):
        binding.swila_output_norm(w4, o, weight)
    torch.cuda.synchronize()
    times = []
    for _ in range(launches):
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record()
        binding.swila_output_norm(w4, o, weight)
        stop.record()
        torch.cuda.synchronize()
        times.append(start.elapsed_time(stop))
    times.sort()
    return w4, 2 * o.numel() * o.element_size(), times[0], times[len(times) // 2]


def main():
    ap = argparse.ArgumentParser(description=__doc__)
    ap.add_argument("configs", nargs="*", type=int, default=[2, 1])
    ap.add_argument("--algo", choices=sorted(ALGOS), default="auto")
    ap.add_argument("--launches", type=int, default=7)
    ap.add_argument("--norm", action="store_true", help="time swila_output_norm instead of swila_forward")
    ap.add_argument("--temporal", action="store_true", help="the Temporal variant (App. B.3) of the configurations")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("a CUDA device is required")
    for index in args.configs if args.norm else []:
        w, nbytes, t_min, t_med = time_norm(index, args.launches)
        print(f"config {index} x4 ({w.B}x{w.H}x{w.T}x{w.Dv} {w.io_dtype}) output norm: min {t_min:.4f} ms, median "
              f"{t_med:.4f} ms, {nbytes / t_min * 1e3 / 1e9:.0f} GB/s (read + write)", flush=True)
    for index in [] if args.norm else args.configs:
        w, t_min, t_med = time_config(index, ALGOS[args.algo], args.launches, temporal=args.temporal)
        print(f"config {index} ({w.name}{' temporal' if args.temporal else ''}) {args.algo}: min {t_min:.3f} ms, median {t_med:.3f} ms, "
              f"{w.B * w.T / t_min * 1e3 / 1e6:.2f} M tokens/s", flush=True)


if __name__ == "__main__":
    main()
