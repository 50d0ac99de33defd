"""Builds libresq.so (sm_100a) in-tree with nvcc.  `python paper_2412_14363_b200/build.py [--force] [-v]` (or `python __graft_entry__.py`)."""
from __future__ import annotations

import hashlib
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libresq.so")
SOURCES = ["api.cu", "quantize.cu", "quantize_asym.cu", "mixed_gemm.cu", "decode_stream.cu", "project.cu", "static_scratch.cu",
           "kv_cache.cu", "kv_attention.cu", "kv_prefill.cu", "kv_d64.cu", "gptq.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr"]


def _digest(paths, extra=()) -> str:
    h = hashlib.sha256()
    for x in extra:
        h.update(x.encode())
        h.update(b"\0")
    for path in paths:
        h.update(os.path.basename(path).encode())
        with open(path, "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def _headers():
    inc = os.path.join(HERE, "..", "include")
    out = [os.path.join(inc, f) for f in sorted(os.listdir(inc)) if f.endswith(".h")]
    out += [os.path.join(CSRC, f) for f in sorted(os.listdir(CSRC)) if f.endswith((".h", ".cuh"))]
    return out


def _read(path: str) -> str:
    try:
        with open(path) as f:
            return f.read().strip()
    except OSError:
        return ""


def build(force: bool = False, verbose: bool = False) -> str:
    """An object is rebuilt when the digest of its source, of every header and of the flags differs from the one
    stored beside it; the library when the digest over all of those differs from the one stored beside the library
    (time stamps play no part: a copied tree with fresh mtimes but stale contents is rebuilt)."""
    os.makedirs(OBJ, exist_ok=True)
    hdrs = _headers()
    jobs = []
    objs = []
    stamps = []
    for src in SOURCES:
        s = os.path.join(CSRC, src)
        o = os.path.join(OBJ, src.replace(".cu", ".o"))
        want = _digest([s, *hdrs], NVCC_FLAGS)
        objs.append(o)
        stamps.append(want)
        if force or not os.path.exists(o) or _read(o + ".hash") != want:
            cmd = ["nvcc", *NVCC_FLAGS, *( ["-Xptxas", "-v"] if verbose else []), "-c", s, "-o", o]
            jobs.append((cmd, o + ".hash", want))

    def run(cmd):
        r = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or r.returncode:
            sys.stderr.write(r.stdout + r.stderr)
        if r.returncode:
            raise RuntimeError("nvcc failed: " + " ".join(cmd))

    def compile_one(job):
        cmd, stamp_path, want = job
        if os.path.exists(stamp_path):
            os.remove(stamp_path)
        run(cmd)
        with open(stamp_path, "w") as f:
            f.write(want)

    with ThreadPoolExecutor(max_workers=4) as ex:
        list(ex.map(compile_one, jobs))
    lib_want = hashlib.sha256("".join(stamps).encode()).hexdigest()
    if jobs or not os.path.exists(LIB) or _read(LIB + ".hash") != lib_want:
        tmp = LIB + f".tmp{os.getpid()}"
        run(["nvcc", "-shared", "-o", tmp, *objs, "-gencode", "arch=compute_100a,code=sm_100a"])
        os.replace(tmp, LIB)
        with open(LIB + ".hash", "w") as f:
            f.write(lib_want)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
