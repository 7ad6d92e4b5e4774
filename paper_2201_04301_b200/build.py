"""Compile the CUDA sources of this package into libgcada.so (in-tree).

    python -m paper_2201_04301_b200.build [--force] [--verbose] [--debug]

nvcc cross-compiles for sm_100a; no GPU is needed to build.
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libgcada.so")
DEBUG_LIB = os.path.join(HERE, "libgcada_dbg.so")
SOURCES = ["api.cu", "grad_linear.cu", "tail.cu", "mlp.cu", "mlp_bf16.cu", "noalloc.cu", "eval.cu", "linear_cluster.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC,-Wall,-Wno-unused-function", "--expt-relaxed-constexpr"]


def _newest_header():
    t = 0.0
    for root in (CSRC, os.path.join(HERE, "..", "include")):
        for f in os.listdir(root):
            if f.endswith((".h", ".cuh")):
                t = max(t, os.path.getmtime(os.path.join(root, f)))
    return t


def build(force=False, verbose=False, debug=False):
    """Compile libgcada.so, or with debug=True libgcada_dbg.so: the same sources with -DGCADA_DEBUG (every
    store position a kernel computes is checked against its buffer; a failed check raises an error word)."""
    nvcc = os.environ.get("NVCC", "nvcc")
    obj_dir = OBJ + ("_dbg" if debug else "")
    lib = DEBUG_LIB if debug else LIB
    flags = NVCC_FLAGS + (["-DGCADA_DEBUG"] if debug else [])
    os.makedirs(obj_dir, exist_ok=True)
    hdr_t = _newest_header()
    objs, rebuilt = [], False
    procs = []
    for src in SOURCES:
        s = os.path.join(CSRC, src)
        o = os.path.join(obj_dir, src.replace(".cu", ".o"))
        objs.append(o)
        if force or not os.path.exists(o) or os.path.getmtime(o) < max(os.path.getmtime(s), hdr_t):
            cmd = [nvcc, *flags, "-c", s, "-o", o]
            if verbose:
                cmd.insert(1, "-Xptxas=-v")
                print(" ".join(cmd), flush=True)
            procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
            rebuilt = True
    for src, pr in procs:
        out, _ = pr.communicate()
        if pr.returncode != 0:
            raise RuntimeError("nvcc failed on %s:\n%s" % (src, out))
        if verbose or out.strip():
            print(out)
    if rebuilt or not os.path.exists(lib):
        cmd = [nvcc, "-shared", "-o", lib, *objs, "-gencode", "arch=compute_100a,code=sm_100a"]
        r = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
        if r.returncode != 0:
            raise RuntimeError("link failed:\n%s" % r.stdout)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, debug="--debug" in sys.argv))
