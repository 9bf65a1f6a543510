"""Build libcdgrab.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libcdgrab.so")
# Diagnostic variants, built beside the product library and loaded instead of it when the
# environment variable CDGRAB_LIB names them:
#   --stamp  -DCDGRAB_STAMP  kernels record phase time stamps (libcdgrab_stamp.so)
#   --debug  -DCDGRAB_DEBUG  index checks and guard words around scratch (libcdgrab_debug.so)
VARIANTS = {"stamp": ("-DCDGRAB_STAMP", "libcdgrab_stamp.so"), "debug": ("-DCDGRAB_DEBUG", "libcdgrab_debug.so")}
SOURCES = ["api.cu", "kernels_generic.cu", "kernels_fma.cu", "kernels_umma.cu", "kernels_umma_f32.cu", "noalloc.cu", "herding.cu", "kernels_indep.cu", "kernels_block.cu", "kernels_literal.cu", "kernels_small.cu"]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC",
]


def _nvcc() -> str:
    cand = os.environ.get("NVCC")
    if cand:
        return cand
    if os.path.exists("/usr/local/cuda/bin/nvcc"):
        return "/usr/local/cuda/bin/nvcc"
    return "nvcc"


def needs_build(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(ROOT, "include", "cdgrab.h")]
    return any(os.path.getmtime(p) > t for p in deps)


def build(force: bool = False, verbose: bool = False, variant: str | None = None) -> str:
    """Compile every translation unit and link the shared library next to the package."""
    define, name = VARIANTS[variant] if variant else (None, os.path.basename(LIB))
    lib = os.path.join(HERE, name)
    if not force and not needs_build(lib):
        return lib
    objdir = os.path.join(HERE, "_build", variant or "release")
    os.makedirs(objdir, exist_ok=True)
    flags = list(NVCC_FLAGS) + ([define] if define else [])
    if verbose:
        flags += ["-Xptxas", "-v"]
    objs, procs = [], []
    for src in SOURCES:
        obj = os.path.join(objdir, src.replace(".cu", ".o"))
        cmd = [_nvcc(), *flags, "-I", os.path.join(ROOT, "include"), "-I", CSRC, "-c",
               os.path.join(CSRC, src), "-o", obj]
        procs.append((src, subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)))
        objs.append(obj)
    failed = False
    for src, p in procs:
        out, _ = p.communicate()
        if p.returncode != 0 or verbose:
            sys.stderr.write(f"--- nvcc {src} ---\n{out}\n")
        failed |= p.returncode != 0
    if failed:
        raise RuntimeError("nvcc failed")
    # cudart is linked statically (nvcc default); the driver API is reached through
    # cudaGetDriverEntryPoint, so the library has no link-time CUDA dependency
    subprocess.check_call([_nvcc(), "-shared", "-o", lib, *objs])
    return lib


if __name__ == "__main__":
    which = next((v for v in VARIANTS if "--" + v in sys.argv), None)
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, variant=which))
