"""Compile the CUDA library for sm_100a with nvcc into paper_1802_00150_b200/libamq_b200.so (in-tree).

    python -m paper_1802_00150_b200.build [--force] [-v] [--define NAME ...] [--lib FILE]

--define / --lib build a variant beside the product library (e.g. --define AMQ_PHASE_TIMING --lib
libamq_b200_phase.so: the batch-1 sequence kernel then records per-phase clock counts in its workspace status
block); the binding loads the file named by the environment variable AMQ_B200_LIBRARY instead of the product
library when that variable is set."""
import concurrent.futures
import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libamq_b200.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "-DAMQ_BUILD",
    "-I", os.path.join(ROOT, "include"), "-I", CSRC,
]


def _sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _deps_mtime():
    paths = glob.glob(os.path.join(CSRC, "*")) + glob.glob(os.path.join(ROOT, "include", "*.h"))
    return max(os.path.getmtime(p) for p in paths)


def build(force=False, verbose=False, defines=(), lib_name=None):
    srcs = _sources()
    lib = LIB if lib_name is None else os.path.join(HERE, lib_name)
    obj_dir = OBJ if lib_name is None else os.path.join(OBJ, os.path.splitext(lib_name)[0])
    flags = NVCC_FLAGS + ["-D" + d for d in defines]
    if not force and os.path.exists(lib) and os.path.getmtime(lib) >= _deps_mtime():
        return lib
    os.makedirs(obj_dir, exist_ok=True)
    hdr_mtime = max(os.path.getmtime(p) for p in glob.glob(os.path.join(CSRC, "*.cuh")) +
                    glob.glob(os.path.join(ROOT, "include", "*.h")))

    def compile_one(src):
        obj = os.path.join(obj_dir, os.path.basename(src)[:-3] + ".o")
        if not force and os.path.exists(obj) and os.path.getmtime(obj) >= max(os.path.getmtime(src), hdr_mtime):
            return obj
        cmd = ["nvcc"] + flags + (["-Xptxas", "-v"] if verbose else []) + ["-c", src, "-o", obj]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError("nvcc failed for %s:\n%s\n%s" % (src, res.stdout, res.stderr))
        if verbose:
            sys.stderr.write(res.stderr)
        return obj

    with concurrent.futures.ThreadPoolExecutor(max_workers=min(8, len(srcs))) as pool:
        objs = list(pool.map(compile_one, srcs))
    tmp = lib + ".tmp%d" % os.getpid()
    cmd = ["nvcc", "-shared", "-o", tmp] + objs + ["-lcudart"]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("link failed:\n%s\n%s" % (res.stdout, res.stderr))
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    argv = sys.argv[1:]
    defs = [argv[i + 1] for i, a in enumerate(argv) if a == "--define" and i + 1 < len(argv)]
    name = next((argv[i + 1] for i, a in enumerate(argv) if a == "--lib" and i + 1 < len(argv)), None)
    print(build(force="--force" in argv, verbose="-v" in argv, defines=defs, lib_name=name))
