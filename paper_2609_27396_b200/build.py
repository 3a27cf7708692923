"""Builds libdpara.so in-tree with nvcc for sm_100a (cross-compiles without a GPU).

Each csrc/*.cu is compiled to an object file of its own (in parallel, only when it or a header changed),
then linked into one shared library.  No translation unit uses another's device symbols, so no relocatable
device code is needed."""
from __future__ import annotations

import glob
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "build")
LIB = os.path.join(HERE, "libdpara.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
    "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr", "-Xptxas", "-v",
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _headers():
    return glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(HERE, "..", "include", "*.h"))


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(d) > t for d in sources() + _headers())


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not needs_build():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    os.makedirs(OBJ, exist_ok=True)
    hdr_time = max(os.path.getmtime(h) for h in _headers())
    log_path = os.path.join(HERE, "build.log")
    logs = []

    def compile_one(src: str):
        obj = os.path.join(OBJ, os.path.basename(src)[:-3] + ".o")
        if not force and os.path.exists(obj) and os.path.getmtime(obj) > max(os.path.getmtime(src), hdr_time):
            return obj, 0, ""
        cmd = [nvcc] + NVCC_FLAGS + ["-c", "-o", obj, src]
        r = subprocess.run(cmd, capture_output=True, text=True)
        return obj, r.returncode, " ".join(cmd) + "\n" + r.stdout + r.stderr

    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as ex:
        results = list(ex.map(compile_one, sources()))
    failed = False
    for obj, rc, text in results:
        logs.append(text)
        failed |= rc != 0
    if not failed:
        cmd = [nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", LIB] + [o for o, _, _ in results]
        r = subprocess.run(cmd, capture_output=True, text=True)
        logs.append(" ".join(cmd) + "\n" + r.stdout + r.stderr)
        failed |= r.returncode != 0
    with open(log_path, "w") as f:
        f.write("\n".join(logs))
    if verbose or failed:
        sys.stderr.write("\n".join(logs))
    if failed:
        raise RuntimeError(f"nvcc failed (see {log_path})")
    return LIB


if __name__ == "__main__":
    build(force="--incremental" not in sys.argv, verbose=True)
    print(LIB)
