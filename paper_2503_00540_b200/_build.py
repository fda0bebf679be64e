"""In-tree builds of the native libraries (nvcc for sm_100a, gcc for the host fillers).

The shared objects are written beside their sources so that they travel with the tree.
"""
import os
import subprocess
from typing import List

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
INCLUDE = os.path.join(ROOT, "include")
CSRC = os.path.join(PKG, "csrc")
SYNTH = os.path.join(PKG, "synth")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17", "-shared",
              "-Xcompiler", "-fPIC", "-Xptxas", "-v"]

LIBREKV = os.path.join(CSRC, "librekv.so")
LIBREKV_CHECKS = os.path.join(CSRC, "librekv_checks.so")   # the same sources with -DREKV_CHECKS (self-checking kernels)
LIBREKV_SAN = os.path.join(CSRC, "librekv_san.so")         # host code under AddressSanitizer + UBSan (test runs only)
LIBSYNTH_CPU = os.path.join(SYNTH, "librekv_synth_cpu.so")
LIBSYNTH_CUDA = os.path.join(SYNTH, "librekv_synth_cuda.so")


def _stale(target: str, deps: List[str]) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(d) > t for d in deps)


def _sources(folder: str, exts) -> List[str]:
    return sorted(os.path.join(folder, f) for f in os.listdir(folder) if f.endswith(tuple(exts)))


def build_synth(force: bool = False) -> None:
    hdr = os.path.join(SYNTH, "rekv_synth.h")
    src_c = os.path.join(SYNTH, "synth_cpu.c")
    if force or _stale(LIBSYNTH_CPU, [hdr, src_c]):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", LIBSYNTH_CPU, src_c])
    src_cu = os.path.join(SYNTH, "synth_cuda.cu")
    if force or _stale(LIBSYNTH_CUDA, [hdr, src_cu]):
        subprocess.check_call(["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-shared",
                               "-Xcompiler", "-fPIC", "-o", LIBSYNTH_CUDA, src_cu])


def build_librekv(force: bool = False, verbose: bool = False, checks: bool = False, sanitize: bool = False) -> str:
    """Builds csrc/librekv.so, or with checks=True csrc/librekv_checks.so: the same sources compiled with
    -DREKV_CHECKS, whose kernels test their index and address arithmetic and report a violation through the status
    word instead of making the access."""
    srcs = _sources(CSRC, (".cu",))
    deps = srcs + _sources(CSRC, (".cuh", ".h")) + _sources(INCLUDE, (".h",))
    target = LIBREKV_SAN if sanitize else (LIBREKV_CHECKS if checks else LIBREKV)
    if force or _stale(target, deps):
        extra = ["-DREKV_CHECKS"] if checks else []
        if sanitize:  # the host side of every translation unit (ABI plumbing, file I/O) instrumented; needs libasan preloaded
            extra += ["-Xcompiler", "-fsanitize=address,-fsanitize=undefined,-fno-sanitize-recover=undefined,-fno-omit-frame-pointer,-g"]
        cmd = ["nvcc"] + NVCC_FLAGS + extra + ["-I", INCLUDE, "-I", CSRC, "-o", target] + srcs
        env = {k: v for k, v in os.environ.items() if k != "LD_PRELOAD"}  # a preloaded sanitizer runtime is not for nvcc
        out = subprocess.run(cmd, capture_output=True, text=True, env=env)
        if verbose or out.returncode != 0:
            print(out.stdout)
            print(out.stderr)
        if out.returncode != 0:
            raise RuntimeError("nvcc failed building " + os.path.basename(target))
    return target


def build_all(force: bool = False, verbose: bool = False) -> None:
    build_synth(force)
    build_librekv(force, verbose)
    build_librekv(force, verbose, checks=True)
    build_librekv(force, verbose, sanitize=True)


if __name__ == "__main__":
    import sys
    build_all(force="--force" in sys.argv, verbose=True)
