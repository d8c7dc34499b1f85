"""Builds libbtard.so (sm_100a) next to this file with nvcc.  Cross-compiles without a GPU."""
import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libbtard.so")


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _deps():
    return sources() + glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(CSRC, "*.cuh")) + \
        [os.path.join(os.path.dirname(HERE), "include", "btard.h")]


def up_to_date():
    return os.path.exists(LIB) and all(os.path.getmtime(LIB) >= os.path.getmtime(f) for f in _deps())


def build(force=False, verbose=False):
    """Compiles every translation unit on its own (in parallel) and links them into libbtard.so.  The
    objects live in a temporary folder; only the library stays."""
    if not force and up_to_date():
        return LIB
    import concurrent.futures
    import shutil
    import tempfile
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
             "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden"]
    if verbose:
        flags += ["-Xptxas", "-v"]
    work = tempfile.mkdtemp(prefix="btard_build_")
    try:
        def compile_one(src):
            obj = os.path.join(work, os.path.basename(src) + ".o")
            subprocess.run([nvcc] + flags + ["-c", "-o", obj, src], check=True)
            return obj
        with concurrent.futures.ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
            objs = list(pool.map(compile_one, sources()))
        tmp = LIB + ".tmp%d" % os.getpid()
        subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "--shared", "-cudart", "shared",
                        "-o", tmp] + objs, check=True)
        os.replace(tmp, LIB)
    finally:
        shutil.rmtree(work, ignore_errors=True)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
