"""Compile the CUDA library in-tree: paper_1901_03040_b200/libqesgd.so (sm_100a).

The codec translation unit is built with -fmad=false so that no multiply-add of
the rounding chain is contracted; the logistic-regression unit keeps FMAs.
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libqesgd.so")
LIB_DEBUG = os.path.join(HERE, "libqesgd_debug.so")

ARCH = ["-gencode", "arch=compute_100a,code=sm_100a"]
COMMON = ["-O3", "-std=c++17", "-lineinfo", "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"),
          "-I", CSRC]
# (source, object name, extra flags): the codec is built once per code width, in parallel
UNITS = [
    ("qesgd_codec.cu", "qesgd_codec_2.o", ["-fmad=false", "-DQESGD_BITS=2"]),
    ("qesgd_codec.cu", "qesgd_codec_4.o", ["-fmad=false", "-DQESGD_BITS=4"]),
    ("qesgd_codec.cu", "qesgd_codec_8.o", ["-fmad=false", "-DQESGD_BITS=8"]),
    ("qesgd_lr.cu", "qesgd_lr.o", []),
    ("qesgd_lr_epoch.cu", "qesgd_lr_epoch.o", []),
    ("qesgd_api.cu", "qesgd_api.o", []),
]


def _nvcc():
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    raise RuntimeError("nvcc not found")


def _stale(target, sources):
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(s) > t for s in sources)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Builds libqesgd.so, or with debug=True libqesgd_debug.so: the same library compiled with
    -DQESGD_DEBUG (the codec kernels check their indices and set QESGD_STATUS_RANGE)."""
    os.makedirs(OBJ, exist_ok=True)
    headers = [os.path.join(CSRC, "qesgd_internal.h"), os.path.join(ROOT, "include", "qesgd.h"),
               os.path.abspath(__file__)]
    nvcc = _nvcc()
    objs = []
    procs = []
    lib = LIB_DEBUG if debug else LIB
    for name, objname, extra in UNITS:
        src = os.path.join(CSRC, name)
        if debug:
            objname, extra = "debug_" + objname, extra + ["-DQESGD_DEBUG"]
        obj = os.path.join(OBJ, objname)
        objs.append(obj)
        if force or _stale(obj, [src] + headers):
            cmd = [nvcc] + ARCH + COMMON + extra + (["-Xptxas", "-v"] if verbose else []) + ["-c", src, "-o", obj]
            procs.append((cmd, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    for cmd, p in procs:
        out, _ = p.communicate()
        if verbose or p.returncode != 0:
            sys.stderr.write(out)
        if p.returncode != 0:
            raise RuntimeError("nvcc failed: " + " ".join(cmd))
    if force or procs or _stale(lib, objs):
        cmd = [nvcc] + ARCH + ["-shared", "-o", lib] + objs
        subprocess.run(cmd, check=True)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
