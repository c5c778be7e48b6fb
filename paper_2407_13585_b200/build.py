"""Builds libacc.so (host library + sm_100a kernels) in-tree with nvcc.

    python -m paper_2407_13585_b200.build [--force] [--verbose] [--tests]

Objects go to <repo>/_build/, the library to paper_2407_13585_b200/libacc.so.
nvcc cross-compiles, so no GPU is needed to build.

Kernels are instantiated per cluster at build time, so a program whose clusters are not among
those of csrc/programs/ needs a library of its own instantiations: `build_kernel_library` compiles
a folder of such translation units (written by `python -m paper_2407_13585_b200.instantiate`)
into a shared object that registers its kernels with libacc.so when it is loaded
(`binding.load_kernel_library`).  --tests builds the one the test suite uses for its seeded
random programs, tests/libacc_test_kernels.so, from tests/programs/.
"""
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(ROOT, "_build")
LIB = os.path.join(HERE, "libacc.so")
TEST_SRC = os.path.join(ROOT, "tests", "programs")
TEST_LIB = os.path.join(ROOT, "tests", "libacc_test_kernels.so")

NVCC_FLAGS = [
    "-std=c++17", "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
    "--expt-relaxed-constexpr", "-fmad=false", "-Xcompiler", "-fPIC",
    "-I" + os.path.join(ROOT, "include"), "-I" + CSRC,
]


def _sources(top=CSRC):
    out = []
    for d, _, files in os.walk(top):
        for f in sorted(files):
            if f.endswith((".cu", ".cpp")):
                out.append(os.path.join(d, f))
    return sorted(out)


def _headers_mtime():
    m = os.path.getmtime(os.path.join(ROOT, "include", "acc.h"))
    for d, _, files in os.walk(CSRC):
        for f in files:
            if f.endswith((".h", ".cuh")):
                m = max(m, os.path.getmtime(os.path.join(d, f)))
    return max(m, os.path.getmtime(os.path.abspath(__file__)))


def _compile(src, obj, verbose):
    cmd = ["nvcc"] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-x", "cu", "-c", src, "-o", obj]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError("nvcc failed for %s\n%s\n%s" % (src, r.stdout, r.stderr))
    if verbose:
        sys.stderr.write(r.stderr)


def build(force=False, verbose=False):
    os.makedirs(OBJ, exist_ok=True)
    hdr = _headers_mtime()
    jobs, objs = [], []
    for src in _sources():
        obj = os.path.join(OBJ, os.path.relpath(src, CSRC).replace(os.sep, "_") + ".o")
        objs.append(obj)
        if force or not os.path.exists(obj) or os.path.getmtime(obj) < max(hdr, os.path.getmtime(src)):
            jobs.append((src, obj))
    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
        list(pool.map(lambda j: _compile(j[0], j[1], verbose), jobs))
    if jobs or not os.path.exists(LIB):
        cmd = ["nvcc", "-shared", "-o", LIB] + objs + ["-lcudart"]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError("link failed\n%s\n%s" % (r.stdout, r.stderr))
    return LIB


def build_kernel_library(src_dir, lib_path, force=False, verbose=False):
    """Compiles every .cu under src_dir into lib_path, a shared object of further kernel instantiations
    that resolves the registry and the launch helpers from libacc.so (found next to this file at run time)."""
    build(force=False, verbose=verbose)
    os.makedirs(OBJ, exist_ok=True)
    hdr = _headers_mtime()
    tag = os.path.basename(lib_path).replace(".so", "")
    jobs, objs = [], []
    for src in _sources(src_dir):
        obj = os.path.join(OBJ, tag + "_" + os.path.relpath(src, src_dir).replace(os.sep, "_") + ".o")
        objs.append(obj)
        if force or not os.path.exists(obj) or os.path.getmtime(obj) < max(hdr, os.path.getmtime(src)):
            jobs.append((src, obj))
    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
        list(pool.map(lambda j: _compile(j[0], j[1], verbose), jobs))
    if jobs or not os.path.exists(lib_path) or os.path.getmtime(lib_path) < os.path.getmtime(LIB):
        rpath = os.path.relpath(HERE, os.path.dirname(lib_path))
        cmd = ["nvcc", "-shared", "-o", lib_path] + objs + ["-L" + HERE, "-lacc", "-lcudart",
                                                           "-Xlinker", "-rpath", "-Xlinker", "$ORIGIN/" + rpath]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError("link failed\n%s\n%s" % (r.stdout, r.stderr))
    return lib_path


def build_test_kernels(force=False, verbose=False):
    return build_kernel_library(TEST_SRC, TEST_LIB, force, verbose)


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
    if "--tests" in sys.argv:
        print(build_test_kernels(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
