"""Build the C-ABI library ``libdynamo.so`` in-tree with nvcc for sm_100a (no GPU needed to compile).

Every ``.cu`` file is compiled to its own object (in parallel; only the stale ones) and the objects are linked
into the shared library.  No file uses relocatable device code, so plain ``-c`` objects link.
"""
from __future__ import annotations

import hashlib
import json
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "build")
LIB = os.path.join(HERE, "libdynamo.so")
SOURCES = ["api.cu", "pack.cu", "route.cu", "switch.cu", "stats.cu", "ffn_stream.cu", "ffn_tc2.cu",
           "noalloc.cu", "assign.cu", "downside.cu", "debug.cu"]
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]
CFLAGS = ARCH + ["-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC"]
LFLAGS = ARCH + ["-shared", "-Xcompiler", "-fPIC", "-cudart", "static"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def _headers():
    hs = [os.path.join(CSRC, f) for f in sorted(os.listdir(CSRC)) if f.endswith((".cuh", ".h"))]
    hs.append(os.path.join(os.path.dirname(HERE), "include", "dynamo.h"))
    return hs


def _digest(paths) -> str:
    h = hashlib.sha1()
    for p in paths:
        with open(p, "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def _compile(src: str, verbose: bool) -> None:
    obj = os.path.join(OBJ, os.path.splitext(src)[0] + ".o")
    cmd = [_nvcc()] + CFLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-c", "-o", obj, os.path.join(CSRC, src)]
    subprocess.check_call(cmd)


def build_library(force: bool = False, verbose: bool = False) -> str:
    """Staleness goes by content (a digest of every source with all headers, kept beside the objects), not by
    modification times, which a copy of the tree does not preserve."""
    os.makedirs(OBJ, exist_ok=True)
    manifest_path = os.path.join(OBJ, "manifest.json")
    try:
        with open(manifest_path) as f:
            manifest = json.load(f)
    except (OSError, ValueError):
        manifest = {}
    hdr = _digest(_headers())
    want = {s: _digest([os.path.join(CSRC, s)]) + hdr for s in SOURCES}
    stale = [s for s in SOURCES
             if force or manifest.get(s) != want[s] or not os.path.exists(os.path.join(OBJ, os.path.splitext(s)[0] + ".o"))]
    if stale:
        with ThreadPoolExecutor(max_workers=min(len(stale), os.cpu_count() or 4)) as pool:
            list(pool.map(lambda s: _compile(s, verbose), stale))
    objs = [os.path.join(OBJ, os.path.splitext(s)[0] + ".o") for s in SOURCES]
    if stale or not os.path.exists(LIB) or manifest.get("__sources__") != SOURCES:
        subprocess.check_call([_nvcc()] + LFLAGS + ["-o", LIB] + objs)
        want["__sources__"] = SOURCES
        with open(manifest_path, "w") as f:
            json.dump(want, f)
    return LIB


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv))
