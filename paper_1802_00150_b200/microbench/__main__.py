import os
import subprocess
import sys
import tempfile

HERE = os.path.dirname(os.path.abspath(__file__))


def main():
    out_dir = tempfile.mkdtemp(prefix="amq_microbench_")
    rc = 0
    for name in ("pipes", "mma_rate", "smem_store", "mma_with_stores", "exchange"):
        exe = os.path.join(out_dir, name)
        subprocess.check_call(["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-o", exe,
                               os.path.join(HERE, name + ".cu")])
        print("== %s" % name, flush=True)
        rc |= subprocess.call([exe])
    return rc


if __name__ == "__main__":
    sys.exit(main())
