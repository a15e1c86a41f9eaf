"""Builds libcacheback.so (the C-ABI library) in-tree with nvcc for sm_100a, and libcacheback_debug.so, the same sources
compiled with -DCB_DEBUG (range checks on indices taken from memory, guard areas behind the workspace regions)."""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
SO = os.path.join(HERE, "libcacheback.so")
SO_DEBUG = os.path.join(HERE, "libcacheback_debug.so")
SOURCES = ["cb_api.cu", "cb_table.cu", "cb_accept.cu", "cb_kv.cu", "cb_branches.cu", "cb_frozen.cu", "cb_frozen_build.cu", "cb_attn.cu", "cb_attn_tc.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]


def _stale(target, deps):
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def build(force=False, verbose=False, debug=False):
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    so, suffix, extra = (SO_DEBUG, ".dbg.o", ["-DCB_DEBUG"]) if debug else (SO, ".o", [])
    hdrs = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    hdrs.append(os.path.join(ROOT, "include", "cacheback.h"))
    objs = []
    procs = []
    for s in SOURCES:
        src = os.path.join(CSRC, s)
        obj = os.path.join(CSRC, s.replace(".cu", suffix))
        objs.append(obj)
        if force or _stale(obj, [src] + hdrs):
            cmd = [nvcc] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + ["-c", src, "-o", obj]
            procs.append((s, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    for s, p in procs:
        out, _ = p.communicate()
        if verbose or p.returncode != 0:
            sys.stderr.write(out)
        if p.returncode != 0:
            raise RuntimeError("nvcc failed on %s" % s)
    if force or procs or _stale(so, objs):
        tmp = so + ".tmp%d" % os.getpid()
        subprocess.check_call([nvcc, "-shared", "-o", tmp] + objs + ["-gencode", "arch=compute_100a,code=sm_100a"])
        os.replace(tmp, so)
    return so


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug=True))
