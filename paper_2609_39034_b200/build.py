"""Build libswila.so (the C-ABI CUDA library) in-tree for sm_100a with nvcc.

The scan kernel is instantiated for every supported (Dk, J, io dtype, decay mode); each
(Dk, decay mode) pair is its own translation unit so the units compile in parallel.
nvcc cross-compiles without a GPU."""
from __future__ import annotations

import concurrent.futures as cf
import hashlib
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INC = os.path.join(os.path.dirname(HERE), "include")
OBJ = os.path.join(HERE, "build")
LIB = os.path.join(HERE, "libswila.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr"]
DKS = (16, 64, 128)
GATE_MODES = ((0, 0), (1, 0), (1, 1), (2, 0), (2, 1), (3, 0), (3, 1))  # (decay mode, post-decay)


def _deps(path, seen=None):
    """The file and every file it includes with #include "..." (recursively), as absolute paths."""
    seen = set() if seen is None else seen
    path = os.path.normpath(path)
    if path in seen or not os.path.exists(path):
        return seen
    seen.add(path)
    for line in open(path, errors="replace"):
        line = line.strip()
        if line.startswith("#include \""):
            _deps(os.path.join(os.path.dirname(path), line.split('"')[1]), seen)
    return seen


def _unit_stamp(unit) -> str:
    name, src, defs = unit
    h = hashlib.sha256()
    for f in sorted(_deps(src)):
        h.update(f.encode())
        h.update(open(f, "rb").read())
    h.update(" ".join(NVCC_FLAGS + defs).encode())
    return h.hexdigest()


def _units():
    units = [("swila_api.o", os.path.join(CSRC, "swila_api.cu"), [])]
    for dk in DKS:
        for gate, post in GATE_MODES:
            units.append((f"scan_dk{dk}_g{gate}_p{post}.o", os.path.join(CSRC, "swila_scan_inst.cu"),
                          [f"-DSWILA_DK={dk}", f"-DSWILA_GATE={gate}", f"-DSWILA_POST={post}"]))
    for f in sorted(os.listdir(CSRC)):  # any further stand-alone translation units
        if f.endswith(".cu") and f not in ("swila_api.cu", "swila_scan_inst.cu"):
            units.append((f[:-3] + ".o", os.path.join(CSRC, f), []))
    return units


def _compile(unit, verbose):
    name, src, defs = unit
    out = os.path.join(OBJ, name)
    cmd = ["nvcc", *NVCC_FLAGS, *defs, "-I", INC, "-c", src, "-o", out]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"nvcc failed for {name}:\n{r.stdout}\n{r.stderr}")
    return out, r.stderr


def build(force: bool = False, verbose: bool = False, jobs: int | None = None) -> str:
    """Compile what changed (an object is rebuilt when its source, a file it includes or the flags change) and link."""
    os.makedirs(OBJ, exist_ok=True)
    units = _units()
    stamps = {u[0]: _unit_stamp(u) for u in units}
    stale = []
    for u in units:
        sf = os.path.join(OBJ, u[0] + ".stamp")
        if force or not os.path.exists(os.path.join(OBJ, u[0])) or not os.path.exists(sf) or open(sf).read() != stamps[u[0]]:
            stale.append(u)
    link_stamp = hashlib.sha256("".join(sorted(stamps.values())).encode()).hexdigest()
    link_file = os.path.join(OBJ, "stamp")
    if not stale and os.path.exists(LIB) and os.path.exists(link_file) and open(link_file).read() == link_stamp:
        return LIB
    logs = []
    if stale:
        jobs = jobs or min(len(stale), os.cpu_count() or 4)
        with cf.ThreadPoolExecutor(max_workers=jobs) as ex:
            for (name, _, _), (out, log) in zip(stale, ex.map(lambda u: _compile(u, verbose), stale)):
                logs.append(log)
                with open(os.path.join(OBJ, name + ".stamp"), "w") as f:
                    f.write(stamps[name])
    objs = [os.path.join(OBJ, u[0]) for u in units]
    tmp = LIB + f".tmp{os.getpid()}"
    r = subprocess.run(["nvcc", "-shared", "-o", tmp, *objs, "-lcudart"], capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"link failed:\n{r.stdout}\n{r.stderr}")
    os.replace(tmp, LIB)
    with open(link_file, "w") as f:
        f.write(link_stamp)
    if verbose:
        sys.stderr.write("\n".join(logs))
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
