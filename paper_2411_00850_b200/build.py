"""Builds the C-ABI shared library (libgwq.so) in-tree with nvcc for sm_100a.

Every source is compiled to an object of its own (in parallel, rebuilt only when it or a header
is newer), then the objects are linked into the shared library."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libgwq.so")
AID_SRC = os.path.join(HERE, "bench_aid", "read_probe.cu")    # the benchmark's read-only launch, a library of its own
AID_LIB = os.path.join(HERE, "bench_aid", "libbench_read_probe.so")
SOURCES = ("decode_w4_f16.cu", "decode_w4_bf16.cu", "decode_w3_f16.cu", "decode_w3_bf16.cu", "decode_w8_f16.cu",
           "decode_w8_bf16.cu", "decode_w2_f16.cu", "decode_w2_bf16.cu", "select.cu",
           "select_static.cu", "pack.cu", "linear_simt.cu", "linear_decode.cu", "linear_skinny.cu", "linear_prefill.cu",
           "quality.cu", "gradmean.cu", "api.cu")
NVCC_FLAGS = (
    "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
    "-Xcompiler", "-fPIC",
)


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    raise RuntimeError("nvcc not found")


def _headers():
    hs = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    hs.append(os.path.join(os.path.dirname(HERE), "include", "gwq.h"))
    return hs


def _stale(target: str, deps) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def needs_build() -> bool:
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + _headers()
    return _stale(LIB, deps) or _stale(AID_LIB, [AID_SRC])


def _build_aid(force: bool) -> None:
    if not force and not _stale(AID_LIB, [AID_SRC]):
        return
    res = subprocess.run([_nvcc(), *NVCC_FLAGS, "-shared", AID_SRC, "-o", AID_LIB, "-lcudart"],
                         capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed on read_probe.cu:\n" + res.stdout + res.stderr)


def _compile(src: str, force: bool, verbose: bool) -> str:
    path = os.path.join(CSRC, src)
    obj = os.path.join(OBJ, src[:-3] + ".o")
    if not force and not _stale(obj, [path] + _headers()):
        return ""
    cmd = [_nvcc(), *NVCC_FLAGS, "-c", path, "-o", obj]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError(f"nvcc failed on {src}:\n" + res.stdout + res.stderr)
    return res.stderr


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every CUDA source and link libgwq.so; returns the library path."""
    if not force and not needs_build():
        return LIB
    os.makedirs(OBJ, exist_ok=True)
    _build_aid(force)
    with ThreadPoolExecutor(max_workers=min(len(SOURCES), os.cpu_count() or 4)) as pool:
        logs = list(pool.map(lambda s: _compile(s, force, verbose), SOURCES))
    if verbose:
        sys.stderr.write("".join(logs))
    objs = [os.path.join(OBJ, s[:-3] + ".o") for s in SOURCES]
    res = subprocess.run([_nvcc(), "-shared", "-o", LIB, *objs, "-lcudart"], capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("link failed:\n" + res.stdout + res.stderr)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
