"""Builds libhydra_attn.so in-tree with nvcc for sm_100a (cross-compiles without a GPU).

    python -m paper_2609_34318_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG, "csrc")
OUT = os.path.join(PKG, "libhydra_attn.so")
OBJ_DIR = os.path.join(PKG, "build")
SOURCES = ["api.cu", "fwd_kernel.cu", "fwd_short_kernel.cu", "bwd_kernels.cu", "aux_kernels.cu", "mla_ops.cu", "sched.cu"]
# the tensor-core kernel files are compiled a second time for q / k heads of 128 (own symbol names)
VARIANTS = [("fwd_kernel.cu", "d128", ["-DHYDRA_KERNEL_DQK=128"]), ("fwd_short_kernel.cu", "d128", ["-DHYDRA_KERNEL_DQK=128"]),
            ("bwd_kernels.cu", "d128", ["-DHYDRA_KERNEL_DQK=128"])]
HEADERS = ["hydra_internal.h", "sm100_ptx.cuh", os.path.join("..", "..", "include", "hydra_attn.h"),
           os.path.join("..", "..", "include", "hydra_sched.h")]
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
         "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "-Xptxas", "-v"]


def _source_hash() -> str:
    """Content hash of everything the library is built from (file times do not survive a copy)."""
    import hashlib
    h = hashlib.sha1((" ".join(FLAGS) + repr(VARIANTS)).encode())
    for name in SOURCES + HEADERS:
        with open(os.path.join(CSRC, name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def _stale() -> bool:
    if not os.path.exists(OUT) or not os.path.exists(OUT + ".srchash"):
        return True
    with open(OUT + ".srchash") as f:
        return f.read().strip() != _source_hash()


def _compile(job) -> str:
    src, tag, defines = job
    obj = os.path.join(OBJ_DIR, src.replace(".cu", (("_" + tag) if tag else "") + ".o"))
    cmd = [NVCC] + FLAGS + list(defines) + ["-c", os.path.join(CSRC, src), "-o", obj]
    r = subprocess.run(cmd, capture_output=True, text=True)
    with open(obj + ".log", "w") as f:
        f.write(" ".join(cmd) + "\n" + r.stdout + r.stderr)
    if r.returncode != 0:
        raise RuntimeError(f"nvcc failed on {src}:\n{r.stdout}\n{r.stderr}")
    return obj


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return OUT
    os.makedirs(OBJ_DIR, exist_ok=True)
    jobs = [(src, "", []) for src in SOURCES] + VARIANTS
    with ThreadPoolExecutor(max_workers=len(jobs)) as pool:
        objs = list(pool.map(_compile, jobs))
    tmp = OUT + f".tmp{os.getpid()}"
    cmd = [NVCC, "-shared", "-o", tmp] + objs + ["-Xcompiler", "-fPIC"]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"link failed:\n{r.stdout}\n{r.stderr}")
    os.replace(tmp, OUT)
    with open(OUT + ".srchash", "w") as f:
        f.write(_source_hash())
    if verbose:
        for o in objs:
            with open(o + ".log") as f:
                sys.stdout.write(f.read())
    return OUT


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
