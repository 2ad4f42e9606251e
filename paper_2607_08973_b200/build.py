"""Builds the two CUDA libraries (sm_100a) in-tree with nvcc.

``libsifar.so``        the all-reduce itself: context, producer-side store path,
                       reducer kernels, the allocation-free entry point
                       (``include/sifar.h``).
``libsifar_bench.so``  the synthetic decode-step chains, generator probes and
                       measurement helpers (``include/sifar_workload.h``); it
                       links against ``libsifar.so`` and is found next to it.

``libsifar_s8x2.so``   ``libsifar.so`` once more with the fallback slot format (two self-validating
                       8-byte halves per slot, ``-DSIFAR_SLOT_S8X2``): kept building and tested so that
                       it is there should 16-byte accesses ever be seen torn.

``python -m paper_2607_08973_b200.build`` or ``build()``; nvcc cross-compiles
without a GPU.  Every ``.cu`` file is compiled to an object of its own (in
parallel, only if stale), then the two libraries are linked.  Both link the CUDA
runtime statically, so loading them next to torch needs nothing else.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
OBJ = os.path.join(PKG, "build")
LIB = os.path.join(PKG, "libsifar.so")
LIB_BENCH = os.path.join(PKG, "libsifar_bench.so")
LIB_S8X2 = os.path.join(PKG, "libsifar_s8x2.so")

# which translation units go into which library
CORE_UNITS = ("sifar_core", "sifar_noalloc")
BENCH_UNITS = ("sifar_workload", "sifar_symmetric")

NVCC_FLAGS = [
    "-std=c++17", "-O3", "-lineinfo",
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-Xcompiler", "-fPIC",
    "-I" + os.path.join(ROOT, "include"), "-I" + CSRC,
]


def sources() -> list[str]:
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _headers() -> list[str]:
    return glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(ROOT, "include", "*"))


def _newer(deps, target) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def _nvcc() -> str:
    return os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")


def _compile(unit: str, force: bool, verbose: bool, variant: str = "") -> str:
    src = os.path.join(CSRC, unit + ".cu")
    obj = os.path.join(OBJ, unit + (("." + variant) if variant else "") + ".o")
    if force or _newer([src] + _headers(), obj):
        tmp = obj + f".tmp{os.getpid()}"
        defs = ["-DSIFAR_SLOT_S8X2"] if variant == "s8x2" else []
        cmd = [_nvcc()] + NVCC_FLAGS + defs + (["-Xptxas", "-v"] if verbose else []) + ["-c", "-o", tmp, src]
        subprocess.check_call(cmd)
        os.replace(tmp, obj)
    return obj


def _link(lib: str, objs: list[str], extra: list[str]) -> None:
    if not _newer(objs, lib):
        return
    tmp = lib + f".tmp{os.getpid()}"
    cmd = [_nvcc(), "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp] + objs + extra
    subprocess.check_call(cmd)
    os.replace(tmp, lib)


def build(force: bool = False, verbose: bool = False) -> str:
    units = [os.path.splitext(os.path.basename(s))[0] for s in sources()]
    unknown = [u for u in units if u not in CORE_UNITS + BENCH_UNITS]
    if unknown:
        raise RuntimeError(f"csrc/{unknown[0]}.cu is assigned to neither library (see build.py)")
    os.makedirs(OBJ, exist_ok=True)
    jobs = [(u, "") for u in units] + [(u, "s8x2") for u in CORE_UNITS]
    with ThreadPoolExecutor(max_workers=min(len(jobs), os.cpu_count() or 1)) as pool:
        objs = dict(zip(jobs, pool.map(lambda j: _compile(j[0], force, verbose, j[1]), jobs)))
    fallback = [objs[(u, "s8x2")] for u in CORE_UNITS]
    objs = {u: objs[(u, "")] for u in units}
    _link(LIB_S8X2, fallback, ["-Xlinker", "-soname=libsifar_s8x2.so"])
    _link(LIB, [objs[u] for u in CORE_UNITS], ["-Xlinker", "-soname=libsifar.so"])
    _link(LIB_BENCH, [objs[u] for u in BENCH_UNITS],
          ["-Xlinker", "-soname=libsifar_bench.so", "-Xlinker", "-rpath=$ORIGIN", "-L" + PKG, "-lsifar"])
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
