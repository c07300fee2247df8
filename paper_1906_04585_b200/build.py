"""Build libgala.so (sm_100a) in-tree with nvcc.

`python -m paper_1906_04585_b200.build` or `build()`; the shared object is
written next to this file so that it travels with the source tree.
"""
import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libgala.so")
# The same sources with GALA_CROSS_CHECK defined: the only library in which the environment variable
# GALA_CONV_LEGACY selects the earlier convolution products (a second implementation that one test compares
# with the oracle).  Nothing but that test loads it.
CHECK_LIB = os.path.join(HERE, "libgala_check.so")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")

FLAGS = [
    "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
    "-Xcompiler", "-fPIC",
    "-I", os.path.join(ROOT, "include"), "-I", CSRC,
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale() -> bool:
    if not os.path.exists(LIB) or not os.path.exists(CHECK_LIB):
        return True
    t = min(os.path.getmtime(LIB), os.path.getmtime(CHECK_LIB))
    deps = sources() + glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(ROOT, "include", "*.h"))
    return any(os.path.getmtime(p) > t for p in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return LIB
    objs = []
    procs = []
    os.makedirs(os.path.join(HERE, "_build"), exist_ok=True)
    for src in sources():
        obj = os.path.join(HERE, "_build", os.path.basename(src) + ".o")
        objs.append(obj)
        cmd = [NVCC] + FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-c", src, "-o", obj]
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    api_src = os.path.join(CSRC, "api.cu")
    api_check = os.path.join(HERE, "_build", "api.cu.check.o")
    procs.append((api_src + " (cross-check)", subprocess.Popen(
        [NVCC] + FLAGS + ["-DGALA_CROSS_CHECK", "-c", api_src, "-o", api_check],
        stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    failed = False
    for src, p in procs:
        out, _ = p.communicate()
        if p.returncode != 0 or verbose:
            sys.stderr.write("== %s\n%s\n" % (os.path.basename(src), out))
        failed |= p.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    tmp = LIB + ".tmp.%d" % os.getpid()
    subprocess.check_call([NVCC, "-shared", "-o", tmp] + objs + ["-gencode", "arch=compute_100a,code=sm_100a"])
    os.replace(tmp, LIB)
    check_objs = [api_check if os.path.basename(o) == "api.cu.o" else o for o in objs]
    tmp = CHECK_LIB + ".tmp.%d" % os.getpid()
    subprocess.check_call([NVCC, "-shared", "-o", tmp] + check_objs + ["-gencode", "arch=compute_100a,code=sm_100a"])
    os.replace(tmp, CHECK_LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
