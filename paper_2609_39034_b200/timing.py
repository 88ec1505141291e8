"""Time `swila_forward` on one of the named workloads with CUDA events (inputs resident on the device).

    python -m paper_2609_39034_b200.timing 2 1 --algo chunk

prints, per configuration index, the minimum and median time of a few launches and the tokens per
second they correspond to.  It is the small fixed loop the profiler captures under `profiles/` wrap:
three warm-up launches, then the timed ones, nothing else on the stream.
"""
import argparse

import torch

from . import binding
from . import workloads as wl

ALGOS = {"auto": binding.ALGO_AUTO, "scan": binding.ALGO_SCAN, "chunk": binding.ALGO_CHUNK}


def time_config(index: int, algo: int, launches: int = 7, warmup: int = 3):
    w = wl.CONFIGS[index]
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


def main():
    ap = argparse.ArgumentParser(description=__doc__)
    ap.add_argument("configs", nargs="*", type=int, default=[2, 1])
    ap.add_argument("--algo", choices=sorted(ALGOS), default="auto")
    ap.add_argument("--launches", type=int, default=7)
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("a CUDA device is required")
    for index in args.configs:
        w, t_min, t_med = time_config(index, ALGOS[args.algo], args.launches)
        print(f"config {index} ({w.name}) {args.algo}: min {t_min:.3f} ms, median {t_med:.3f} ms, "
              f"{w.B * w.T / t_min * 1e3 / 1e6:.2f} M tokens/s", flush=True)


if __name__ == "__main__":
    main()
