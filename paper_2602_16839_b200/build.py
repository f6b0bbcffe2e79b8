"""Builds libptenc.so (the C-ABI library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libptenc.so")
SOURCES = ["ptenc_api.cu", "ptenc_ring.cu", "ptenc_score.cu", "ptenc_encode.cu", "ptenc_encode_tc.cu", "ptenc_step_e1.cu", "ptenc_lora.cu", "ptenc_attn_generic.cu", "ptenc_attn_bf16.cu"]
HEADERS = [os.path.join(CSRC, "ptenc_internal.h"), os.path.join(ROOT, "include", "ptenc.h")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden", "--expt-relaxed-constexpr"]


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found: the ptenc CUDA library cannot be built")
    return exe


STAMP = os.path.join(PKG, "libptenc.flags")     # travels with the library, unlike the object folder


def _stamp(extra) -> str:
    return " ".join([*NVCC_FLAGS, *extra])


def needs_build(extra=()) -> bool:
    """True when the library is missing, older than a source, or was built with other flags than asked for now
    (so a library built with extra tunables is never mistaken for the default one)."""
    if not os.path.exists(LIB) or not os.path.exists(STAMP):
        return True
    with open(STAMP) as f:
        if f.read().strip() != _stamp(extra):
            return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in SOURCES] + HEADERS
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compiles the sources and links libptenc.so.  Extra nvcc flags (e.g. -DPTENC_ATTN_STAGES_128=8 to pin a tunable
    of the attention kernel for profiling) can be given in the environment variable PTENC_NVCC_FLAGS.  The flags of
    the last build are recorded beside the library; a build with other flags, or the default build after a flagged
    one, recompiles."""
    extra = os.environ.get("PTENC_NVCC_FLAGS", "").split()
    if not force and not needs_build(extra):
        return LIB
    objdir = os.path.join(PKG, "_build")
    os.makedirs(objdir, exist_ok=True)
    nvcc = _nvcc()
    procs = []
    for s in SOURCES:
        obj = os.path.join(objdir, s.replace(".cu", ".o"))
        cmd = [nvcc, *NVCC_FLAGS, *extra, "-I", os.path.join(ROOT, "include"), "-I", CSRC, "-c",
               os.path.join(CSRC, s), "-o", obj]
        if verbose:
            cmd.insert(1, "-Xptxas")
            cmd.insert(2, "-v")
        procs.append((s, obj, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
    objs = []
    for s, obj, p in procs:
        out, _ = p.communicate()
        if p.returncode != 0:
            raise RuntimeError(f"nvcc failed on {s}:\n{out}")
        if verbose:
            print(out)
        objs.append(obj)
    cmd = [nvcc, "-shared", "-o", LIB, *objs, "-gencode", "arch=compute_100a,code=sm_100a"]
    r = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
    if r.returncode != 0:
        raise RuntimeError(f"link failed:\n{r.stdout}")
    with open(STAMP, "w") as f:
        f.write(_stamp(extra) + "\n")
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
