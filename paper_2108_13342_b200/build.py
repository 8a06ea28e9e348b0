"""Builds libdnnf.so in-tree with nvcc for sm_100a (no JIT cache, no torch headers)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libdnnf.so")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = (["-DDNNF_TRACE"] if os.environ.get("DNNF_TRACE") else []) + os.environ.get("DNNF_EXTRA_NVCC_FLAGS", "").split() + ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
         "-Xcompiler", "-fPIC,-fvisibility=hidden,-Wall,-Wno-unused-function", "--expt-relaxed-constexpr",
         "-Xptxas", "-v"]


def sources():
    return sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cu", ".cpp")))


def _deps_of(obj, src):
    """Headers the object was built from (the compiler's dependency file of the last build); every header if unknown."""
    dfile = obj + ".d"
    if os.path.exists(dfile) and os.path.exists(obj) and os.path.getmtime(dfile) >= os.path.getmtime(obj) - 600:
        with open(dfile) as f:
            words = f.read().replace("\\\n", " ").split()
        deps = [w for w in words[1:] if not w.endswith(":") and (w.startswith(HERE) or w.startswith(os.path.join(HERE, "..")) or not os.path.isabs(w))]
        if deps:
            return [src] + deps
    return [src] + [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))] + \
           [os.path.join(HERE, "..", "include", "dnnf.h")]


def needs_build():
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(HERE, "..", "include", "dnnf.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force=False, verbose=False):
    if not force and not needs_build():
        return LIB
    objs = []
    odir = os.path.join(HERE, "build")
    os.makedirs(odir, exist_ok=True)
    procs = []
    for src in sources():
        obj = os.path.join(odir, os.path.basename(src) + ".o")
        objs.append(obj)
        deps = _deps_of(obj, src)
        if not force and os.path.exists(obj) and all(os.path.exists(d) and os.path.getmtime(obj) > os.path.getmtime(d) for d in deps):
            continue
        cmd = [NVCC, *FLAGS, "-MMD", "-MF", obj + ".d", "-x", "cu", "-c", src, "-o", obj]
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    log = []
    for src, p in procs:
        out, _ = p.communicate()
        log.append(f"== {os.path.basename(src)}\n{out}")
        if p.returncode != 0:
            sys.stderr.write("\n".join(log))
            raise RuntimeError(f"nvcc failed on {src}")
    with open(os.path.join(odir, "ptxas.log"), "a") as f:
        f.write("\n".join(log))
    if verbose:
        print("\n".join(log))
    cmd = [NVCC, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", LIB, *objs, "-Xlinker", "--exclude-libs,ALL"]
    subprocess.check_call(cmd)
    return LIB


if __name__ == "__main__":
    build(force="--force" in sys.argv, verbose="-v" in sys.argv)
    print(LIB)
