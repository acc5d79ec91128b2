"""In-tree build of the CUDA libraries for sm_100a with nvcc (cross-compiles without a GPU).

  liboda_b200.so    -- the C-ABI library declared in include/oda.h
  libsynth_fill.so  -- the device half of the seeded input generator (synth.py)
"""
from __future__ import annotations

import concurrent.futures
import hashlib
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "build")
LIB_ODA = os.path.join(HERE, "liboda_b200.so")
LIB_SYNTH = os.path.join(HERE, "libsynth_fill.so")

NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]
CFLAGS = ["-O3", "-std=c++17", "-lineinfo", "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr"]

ODA_SOURCES = ["oda_api.cu", "splitkv_simt.cu", "splitkv_tma.cu", "recall_head.cu", "recall_exchange.cu", "recall_head_full.cu", "recall_head_fused.cu", "commit.cu", "oda_static.cu"]
SYNTH_SOURCES = ["synth_fill.cu"]


def _deps_digest(src: str) -> str:
    h = hashlib.sha1()
    for name in sorted(os.listdir(CSRC)) + ["../../include/oda.h"]:
        path = os.path.join(CSRC, name)
        if name.endswith((".cuh", ".h")) or os.path.basename(path) == os.path.basename(src):
            with open(path, "rb") as f:
                h.update(f.read())
    h.update(" ".join(ARCH + CFLAGS).encode())
    return h.hexdigest()


def _compile(src: str, verbose: bool) -> str:
    os.makedirs(OBJ, exist_ok=True)
    obj = os.path.join(OBJ, os.path.splitext(src)[0] + ".o")
    stamp = obj + ".sha1"
    digest = _deps_digest(src)
    if os.path.exists(obj) and os.path.exists(stamp) and open(stamp).read() == digest:
        return obj
    cmd = [NVCC, *ARCH, *CFLAGS, "-c", os.path.join(CSRC, src), "-o", obj]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    r = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or r.returncode:
        sys.stderr.write(r.stdout + r.stderr)
    if r.returncode:
        raise RuntimeError(f"nvcc failed on {src}")
    with open(stamp, "w") as f:
        f.write(digest)
    return obj


def _link(objs, out):
    tmp = out + f".tmp{os.getpid()}"
    subprocess.check_call([NVCC, *ARCH, "-shared", "-o", tmp, *objs, "-cudart", "static"])
    os.replace(tmp, out)


def build_all(verbose: bool = False) -> None:
    with concurrent.futures.ThreadPoolExecutor(max_workers=8) as ex:
        oda_objs = list(ex.map(lambda s: _compile(s, verbose), ODA_SOURCES))
        syn_objs = list(ex.map(lambda s: _compile(s, verbose), SYNTH_SOURCES))
    for objs, out in ((oda_objs, LIB_ODA), (syn_objs, LIB_SYNTH)):
        if not os.path.exists(out) or any(os.path.getmtime(o) > os.path.getmtime(out) for o in objs):
            _link(objs, out)


if __name__ == "__main__":
    build_all(verbose="-v" in sys.argv)
    print(LIB_ODA)
    print(LIB_SYNTH)
