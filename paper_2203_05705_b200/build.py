"""Builds libard.so in-tree with nvcc for sm_100a (cross-compiles without a GPU).

    python -m paper_2203_05705_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import hashlib
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
OBJ = os.path.join(PKG, "build")
LIB = os.path.join(PKG, "libard.so")
SOURCES = ["api.cu", "sampler.cu", "gemm_cc.cu", "gemm_tc_sm100.cu", "aux_kernels.cu", "no_alloc.cu",
           "distribution_search.cu", "lstm_persistent.cu", "mlp_step.cu", "mlp_persistent.cu", "rows.cu", "blocks.cu", "dropout_schedule.cu"]
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
         "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]


def _sources():
    return [s for s in SOURCES if os.path.exists(os.path.join(CSRC, s))]


def _stale(target, deps):
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def _sha(paths, extra=""):
    h = hashlib.sha256(extra.encode())
    for p in paths:
        with open(p, "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def _object_is_current(obj, deps, flags):
    """An object counts only if it was made by this script from the sources as they are now: its side file holds
    the hash of the sources (and flags) it was compiled from and the hash of the object itself, so an object written
    by anything else (an experiment's build, an older checkout with newer time stamps) is compiled again."""
    key = obj + ".key"
    if not (os.path.exists(obj) and os.path.exists(key)):
        return False
    try:
        with open(key) as f:
            src_hash, obj_hash = f.read().split()
    except ValueError:
        return False
    return src_hash == _sha(deps, " ".join(flags)) and obj_hash == _sha([obj])


def build(force: bool = False, verbose: bool = False) -> str:
    os.makedirs(OBJ, exist_ok=True)
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith(".h")]
    headers.append(os.path.join(ROOT, "include", "ard.h"))
    jobs = []
    objs = []
    for src in _sources():
        s = os.path.join(CSRC, src)
        o = os.path.join(OBJ, src[:-3] + ".o")
        objs.append(o)
        deps = [s] + sorted(headers)
        if force or not _object_is_current(o, deps, FLAGS):
            cmd = [NVCC] + FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-c", s, "-o", o]
            jobs.append((cmd, o, deps))

    def run(cmd):
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError("nvcc failed:\n" + " ".join(cmd) + "\n" + r.stdout + r.stderr)
        return r.stderr

    def compile_one(job):
        cmd, o, deps = job
        out = run(cmd)
        with open(o + ".key", "w") as f:
            f.write(_sha(deps, " ".join(FLAGS)) + " " + _sha([o]))
        return out

    with ThreadPoolExecutor(max_workers=max(1, min(6, len(jobs)))) as ex:
        for out in ex.map(compile_one, jobs):
            if verbose and out:
                print(out)
    if jobs or force or _stale(LIB, objs):
        run([NVCC, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", LIB] + objs)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
