"""Builds libkvq.so in-tree with nvcc for sm_100a (no JIT cache, no torch extension)."""
from __future__ import annotations

import concurrent.futures
import fcntl
import hashlib
import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libkvq.so")
SOURCES = ["kvq_api.cu", "quantize_append.cu", "rotate_rows.cu", "attn_mma_sync.cu", "attn_jsd.cu", "attn_sm100.cu"]
HEADERS = [os.path.join(CSRC, "kvq_common.cuh"), os.path.join(ROOT, "include", "kvq.h")]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-Xptxas", "-v", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
]


def _nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def _digest(paths: list[str], extra: str = "") -> str:
    h = hashlib.sha256(extra.encode())
    for p in paths:
        with open(p, "rb") as f:
            h.update(os.path.relpath(p, ROOT).encode() + b"\0" + f.read())
    return h.hexdigest()


def _current(target: str, digest: str) -> bool:
    """True if `target` exists and was built from exactly these inputs (file times are not trusted: a copy of the
    tree may have shuffled them)."""
    try:
        with open(target + ".stamp") as f:
            return os.path.exists(target) and f.read().strip() == digest
    except OSError:
        return False


def _stamp(target: str, digest: str) -> None:
    with open(target + ".stamp", "w") as f:
        f.write(digest + "\n")


def build_library(force: bool = False, verbose: bool = False) -> str:
    """Compile every CUDA source and link libkvq.so next to this file; returns its path.  Several processes
    (one per GPU) may call this at once: a file lock lets one of them build and the others find the result."""
    with open(os.path.join(PKG, ".build.lock"), "w") as lock:
        fcntl.flock(lock, fcntl.LOCK_EX)
        try:
            return _build_locked(force, verbose)
        finally:
            fcntl.flock(lock, fcntl.LOCK_UN)


def _build_locked(force: bool, verbose: bool) -> str:
    headers = sorted(set(HEADERS + [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]))

    def compile_one(src: str):
        s = os.path.join(CSRC, src)
        o = os.path.join(CSRC, src[:-3] + ".o")
        d = _digest([s] + headers, " ".join(NVCC_FLAGS[:-4]))     # the flags without the include paths
        if force or not _current(o, d):
            cmd = [_nvcc()] + NVCC_FLAGS + ["-c", s, "-o", o]
            r = subprocess.run(cmd, capture_output=True, text=True)
            log = r.stdout + r.stderr
            with open(o + ".log", "w") as f:
                f.write(" ".join(cmd) + "\n" + log)
            if verbose or r.returncode != 0:
                sys.stderr.write(log)
            if r.returncode != 0:
                raise RuntimeError(f"nvcc failed for {src}")
            _stamp(o, d)
        return o, d

    with concurrent.futures.ThreadPoolExecutor(max_workers=len(SOURCES)) as pool:     # nvcc runs as child processes
        results = list(pool.map(compile_one, SOURCES))
    objs = [o for o, _ in results]
    digests = [d for _, d in results]
    lib_digest = hashlib.sha256("".join(digests).encode()).hexdigest()
    if force or not _current(LIB, lib_digest):
        cmd = [_nvcc(), "-shared", "-o", LIB] + objs + ["-gencode", "arch=compute_100a,code=sm_100a"]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            sys.stderr.write(r.stdout + r.stderr)
            raise RuntimeError("link failed")
        _stamp(LIB, lib_digest)
    return LIB


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose=True))
