"""Compile the C++ oracle into oracle/librekv_oracle.so (g++, OpenMP)."""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "rekv_oracle.cpp")
LIB = os.path.join(HERE, "librekv_oracle.so")
LIB_SAN = os.path.join(HERE, "librekv_oracle_san.so")   # the same source under AddressSanitizer + UBSan


def build(force: bool = False, sanitize: bool = False) -> str:
    """The oracle library; with sanitize=True (or ORACLE_SANITIZE=1 in the environment) the variant compiled with
    -fsanitize=address,undefined, to be loaded by a python that has the sanitizer runtime preloaded (the tests do)."""
    sanitize = sanitize or os.environ.get("ORACLE_SANITIZE", "") == "1"
    lib = LIB_SAN if sanitize else LIB
    if force or not os.path.exists(lib) or os.path.getmtime(lib) < os.path.getmtime(SRC):
        extra = ["-fsanitize=address,undefined", "-fno-sanitize-recover=undefined", "-fno-omit-frame-pointer", "-g"] if sanitize else []
        env = {k: v for k, v in os.environ.items() if k != "LD_PRELOAD"}  # a preloaded sanitizer runtime is not for g++
        subprocess.check_call(
            ["g++", "-std=c++17", "-O2", "-fopenmp", "-shared", "-fPIC"] + extra + ["-o", lib, SRC], env=env)
    return lib


def sanitizer_runtime() -> str:
    """Path of libasan.so as the compiler reports it (for LD_PRELOAD)."""
    return subprocess.check_output(["gcc", "-print-file-name=libasan.so"], text=True).strip()


if __name__ == "__main__":
    print(build(force=True))
