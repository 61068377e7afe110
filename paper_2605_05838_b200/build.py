"""Builds libmdn.so in-tree with nvcc for sm_100a (cross-compiles without a GPU).

    python -m paper_2605_05838_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import concurrent.futures
import glob
import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libmdn.so")
OBJ_DIR = os.path.join(PKG, "build")

# MDN_BUILD_DEBUG=1 in the environment of the BUILD compiles the debug knobs in (-DMDN_DEBUG: precision ablation
# switch and the per-chunk clock stamps of the chain kernels); the default library has none of them.
NVCC_FLAGS = (["-DMDN_DEBUG"] if os.environ.get("MDN_BUILD_DEBUG") == "1" else []) + ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr", "-I", os.path.join(ROOT, "include"), "-I", CSRC]


def _newer(path: str, deps) -> bool:
    if not os.path.exists(path):
        return False
    t = os.path.getmtime(path)
    return all(os.path.getmtime(d) <= t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    srcs = sorted(glob.glob(os.path.join(CSRC, "*.cu")))
    hdrs = sorted(glob.glob(os.path.join(CSRC, "*.cuh"))) + sorted(glob.glob(os.path.join(ROOT, "include", "*.h")))
    if not force and _newer(LIB, srcs + hdrs):
        write_build_info()
        return LIB
    os.makedirs(OBJ_DIR, exist_ok=True)

    def compile_one(src: str) -> str:
        obj = os.path.join(OBJ_DIR, os.path.basename(src)[:-3] + ".o")
        if force or not _newer(obj, [src] + hdrs):
            cmd = ["nvcc"] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-c", src, "-o", obj]
            r = subprocess.run(cmd, capture_output=True, text=True)
            if verbose or r.returncode != 0:
                sys.stderr.write(r.stdout + r.stderr)
            if r.returncode != 0:
                raise RuntimeError("nvcc failed for " + src)
        return obj

    with concurrent.futures.ThreadPoolExecutor(max_workers=8) as ex:
        objs = list(ex.map(compile_one, srcs))
    tmp = LIB + ".tmp.%d" % os.getpid()
    subprocess.run(["nvcc", "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp] + objs
                   + ["-lcudart", "-lcuda"], check=True)
    os.replace(tmp, LIB)
    write_build_info()
    return LIB


def write_build_info() -> None:
    """Leaves the source revision beside the library (a machine that receives the tree without its .git directory
    can still say which commit it runs): the short hash of HEAD and of the last commit of every profiles/ summary."""
    import json

    def git(*args):
        try:
            r = subprocess.run(["git", "-C", ROOT] + list(args), capture_output=True, text=True, timeout=10)
            return r.stdout.strip() if r.returncode == 0 and r.stdout.strip() else None
        except (OSError, subprocess.SubprocessError):
            return None

    head = git("rev-parse", "--short", "HEAD")
    if head is None:
        return
    dirty = bool(git("status", "--porcelain", "--untracked-files=no"))
    prof = {"profiles/" + os.path.basename(f): git("log", "-1", "--format=%h", "--", "profiles/" + os.path.basename(f))
            for f in glob.glob(os.path.join(ROOT, "profiles", "*.md"))}
    with open(os.path.join(PKG, "_build_info.json"), "w") as fh:
        json.dump({"git_hash": head + ("+" if dirty else ""), "profiles": prof}, fh)


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
