"""Builds the CUDA library in-tree with nvcc for sm_100a.

    python -m paper_2211_17192_b200.build [--force] [--verbose]

Each `csrc/*.cu` is compiled to an object under `build/` and the objects are
linked into `paper_2211_17192_b200/lib/libspecdecode.so`.  Nothing is cached
outside the repository, so the shared object travels with the tree.
"""

import argparse
import concurrent.futures
import hashlib
import os
import shutil
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG_DIR)
CSRC = os.path.join(PKG_DIR, "csrc")
INCLUDE = os.path.join(ROOT, "include")
OBJ_DIR = os.path.join(ROOT, "build", "obj")
LIB_DIR = os.path.join(PKG_DIR, "lib")
LIB_PATH = os.path.join(LIB_DIR, "libspecdecode.so")
DIGEST_PATH = LIB_PATH + ".sha256"

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC",
    "-I", INCLUDE, "-I", CSRC,
]


def _nvcc():
    path = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(path):
        raise RuntimeError("nvcc not found: the CUDA library cannot be built")
    return path


def _newest_header_mtime():
    newest = 0.0
    for folder in (CSRC, INCLUDE):
        for name in os.listdir(folder):
            if name.endswith((".cuh", ".h")):
                newest = max(newest, os.path.getmtime(os.path.join(folder, name)))
    return newest


def sources():
    return sorted(os.path.join(CSRC, n) for n in os.listdir(CSRC) if n.endswith(".cu"))


def source_digest():
    """Hash of every source, header and flag that goes into the library."""
    h = hashlib.sha256(" ".join(NVCC_FLAGS[:8]).encode())
    for folder in (CSRC, INCLUDE):
        for name in sorted(os.listdir(folder)):
            if name.endswith((".cu", ".cuh", ".h")):
                h.update(name.encode())
                with open(os.path.join(folder, name), "rb") as f:
                    h.update(f.read())
    return h.hexdigest()


def build(force=False, verbose=False):
    """Compile and link; returns the path of the shared library.  A library
    whose recorded source digest matches the tree is left alone."""
    digest = source_digest()
    if not force and not verbose and os.path.exists(LIB_PATH) and os.path.exists(DIGEST_PATH):
        with open(DIGEST_PATH) as f:
            if f.read().strip() == digest:
                return LIB_PATH
    os.makedirs(OBJ_DIR, exist_ok=True)
    os.makedirs(LIB_DIR, exist_ok=True)
    nvcc = _nvcc()
    header_time = _newest_header_mtime()
    jobs = []
    objects = []
    for src in sources():
        obj = os.path.join(OBJ_DIR, os.path.basename(src)[:-3] + ".o")
        objects.append(obj)
        stale = force or not os.path.exists(obj) or os.path.getmtime(obj) < max(os.path.getmtime(src), header_time)
        if stale:
            cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-c", src, "-o", obj]
            jobs.append(cmd)

    def run(cmd):
        res = subprocess.run(cmd, capture_output=True, text=True)
        return cmd, res

    with concurrent.futures.ThreadPoolExecutor(max_workers=min(8, max(1, len(jobs)))) as pool:
        for cmd, res in pool.map(run, jobs):
            if verbose or res.returncode != 0:
                sys.stderr.write(" ".join(cmd) + "\n" + res.stdout + res.stderr)
            if res.returncode != 0:
                raise RuntimeError("nvcc failed for " + cmd[-3])
    if jobs or not os.path.exists(LIB_PATH):
        cmd = [nvcc, "-shared", "-o", LIB_PATH] + objects + ["-gencode", "arch=compute_100a,code=sm_100a"]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            sys.stderr.write(res.stdout + res.stderr)
            raise RuntimeError("link failed")
    with open(DIGEST_PATH, "w") as f:
        f.write(digest + "\n")
    return LIB_PATH


if __name__ == "__main__":
    ap = argparse.ArgumentParser()
    ap.add_argument("--force", action="store_true")
    ap.add_argument("--verbose", action="store_true")
    args = ap.parse_args()
    print(build(force=args.force, verbose=args.verbose))
