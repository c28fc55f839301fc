"""Builds ``libgleam_dc.so`` (the CUDA library behind include/gleam.h) with nvcc for sm_100a.

The kernels are instantiated per group of transform lengths in separate translation units that are
compiled in parallel and linked into one shared object next to this file.  Nothing here needs a
GPU: nvcc cross-compiles.
"""
from __future__ import annotations

import concurrent.futures
import hashlib
import os
import re
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
BUILD = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libgleam_dc.so")

NVCC_FLAGS = ["-std=c++17", "--expt-relaxed-constexpr", "-gencode", "arch=compute_100a,code=sm_100a",
              "-lineinfo", "-O3", "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden"]


def _groups():
    text = open(os.path.join(CSRC, "sizes.def")).read()
    return sorted({int(g) for g in re.findall(r"GLEAM_GROUP == (\d+)", text)})


def _sources_digest():
    h = hashlib.sha256()
    for name in sorted(os.listdir(CSRC)):
        h.update(name.encode())
        h.update(open(os.path.join(CSRC, name), "rb").read())
    h.update(open(os.path.join(HERE, "..", "include", "gleam.h"), "rb").read())
    h.update(" ".join(NVCC_FLAGS).encode())
    return h.hexdigest()


def _run(cmd):
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError("command failed: %s\n%s\n%s" % (" ".join(cmd), r.stdout, r.stderr))
    return r.stdout + r.stderr


def build(force: bool = False, verbose: bool = False) -> str:
    os.makedirs(BUILD, exist_ok=True)
    stamp = os.path.join(BUILD, "digest.txt")
    digest = _sources_digest()
    if not force and os.path.exists(LIB) and os.path.exists(stamp) and open(stamp).read() == digest:
        return LIB
    jobs = []
    for g in _groups():
        obj = os.path.join(BUILD, "kernels_group%d.o" % g)
        jobs.append((["nvcc"] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) +
                     ["-DGLEAM_GROUP=%d" % g, "-c", os.path.join(CSRC, "kernels_group.cu"), "-o", obj], obj))
    npair = len(set(re.findall(r"GLEAM_PAIR_GROUP == (\d+)", open(os.path.join(CSRC, "pairs.def")).read())))
    for g in range(npair):
        obj = os.path.join(BUILD, "kernels_pairs%d.o" % g)
        jobs.append((["nvcc"] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) +
                     ["-DGLEAM_PAIR_GROUP=%d" % g, "-c", os.path.join(CSRC, "kernels_pairs.cu"), "-o", obj], obj))
    for name in ("gleam_dc", "kernels_fused", "modl_cg"):
        obj = os.path.join(BUILD, name + ".o")
        jobs.append((["nvcc"] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) +
                     ["-c", os.path.join(CSRC, name + ".cu"), "-o", obj], obj))
    with concurrent.futures.ThreadPoolExecutor(max_workers=min(len(jobs), os.cpu_count() or 4)) as ex:
        outs = list(ex.map(lambda j: _run(j[0]), jobs))
    if verbose:
        print("\n".join(outs))
    _run(["nvcc", "-shared", "-o", LIB] + [j[1] for j in jobs] + ["-gencode", "arch=compute_100a,code=sm_100a"])
    with open(stamp, "w") as fh:
        fh.write(digest)
    return LIB


if __name__ == "__main__":
    import sys
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
