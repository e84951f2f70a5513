"""Builds libmpq.so (CUDA, sm_100a) in-tree with nvcc.  ``python -m paper_1905_13389_b200.build``."""
from __future__ import annotations

import concurrent.futures
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
OBJ_DIR = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libmpq.so")
# context only, never linked into libmpq.so: the decoded-integer tensor-core comparison kernel
CONTEXT_SRC = os.path.join(CSRC, "context_i8_gemm.cu")
CONTEXT_LIB = os.path.join(HERE, "libmpq_context.so")

NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]
FLAGS = ["-O3", "-std=c++17", "-lineinfo", "-Xcompiler", "-fPIC", "-I", INCLUDE, "-I", CSRC]
# IEEE arithmetic is part of the contract (bit-exact codes): never --use_fast_math / -ftz.

PLAIN = ["mpq_api.cu", "mpq_encode.cu", "mpq_encode_trig.cu", "mpq_gemm.cu", "mpq_glue.cu", "mpq_probe.cu"]
HEADERS = ["mpq_common.cuh", "mpq_branch_kernel.cuh", "mpq_branch_launch.cuh", "mpq_pointwise_kernel.cuh", os.path.join(INCLUDE, "mpq.h")]


def _jobs():
    jobs = [(os.path.join(CSRC, f), os.path.join(OBJ_DIR, f[:-3] + ".o"), []) for f in PLAIN]
    for hb in range(1, 9):
        jobs.append((os.path.join(CSRC, "mpq_branch_inst.cu"), os.path.join(OBJ_DIR, "mpq_branch_hb%d.o" % hb),
                     ["-DMPQ_HB=%d" % hb]))
    return jobs


def _newest_header():
    paths = [h if os.path.isabs(h) else os.path.join(CSRC, h) for h in HEADERS]
    return max(os.path.getmtime(p) for p in paths)


def _compile(job, verbose):
    src, obj, defs = job
    cmd = [NVCC] + ARCH + FLAGS + defs + (["-Xptxas", "-v"] if verbose else []) + ["-c", src, "-o", obj]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError("nvcc failed for %s:\n%s\n%s" % (src, r.stdout, r.stderr))
    return r.stderr


def build(force: bool = False, verbose: bool = False) -> str:
    os.makedirs(OBJ_DIR, exist_ok=True)
    hdr = _newest_header()
    todo = []
    for job in _jobs():
        src, obj, _ = job
        if force or not os.path.exists(obj) or os.path.getmtime(obj) < max(os.path.getmtime(src), hdr):
            todo.append(job)
    if todo:
        with concurrent.futures.ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as ex:
            for log in ex.map(lambda j: _compile(j, verbose), todo):
                if verbose:
                    sys.stderr.write(log)
    objs = [j[1] for j in _jobs()]
    if todo or not os.path.exists(LIB):
        cmd = [NVCC] + ARCH + ["-shared", "-o", LIB] + objs
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError("link failed:\n%s\n%s" % (r.stdout, r.stderr))
    if force or not os.path.exists(CONTEXT_LIB) or os.path.getmtime(CONTEXT_LIB) < os.path.getmtime(CONTEXT_SRC):
        cmd = [NVCC] + ARCH + ["-O3", "-std=c++17", "-lineinfo", "-Xcompiler", "-fPIC", "-shared", "-o", CONTEXT_LIB, CONTEXT_SRC]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError("nvcc failed for %s:\n%s\n%s" % (CONTEXT_SRC, r.stdout, r.stderr))
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
