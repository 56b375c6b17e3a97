"""Build libtfe.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libtfe.so")
SOURCES = [os.path.join(CSRC, "tfe_api.cu"), os.path.join(CSRC, "tfe_head.cu"), os.path.join(CSRC, "tfe_mine.cu")]
DEPS = SOURCES + [os.path.join(CSRC, "tfe_kernels.cuh"), os.path.join(CSRC, "tfe_key.cuh"),
                  os.path.join(os.path.dirname(HERE), "include", "tfe.h")]
NVCC_FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-shared", "-Xcompiler", "-fPIC", "-cudart", "static"]


def build(force: bool = False, verbose: bool = False, defines=(), out: str | None = None) -> str:
    """Compile the library.  ``defines`` / ``out`` build a tuning variant next to the default one."""
    lib = out or LIB
    if (not force and os.path.exists(lib)
            and all(os.path.getmtime(lib) >= os.path.getmtime(d) for d in DEPS)):
        return lib
    nvcc = os.environ.get("NVCC", "nvcc")
    cmd = ([nvcc] + NVCC_FLAGS + [f"-D{d}" for d in defines] + (["-Xptxas", "-v"] if verbose else [])
           + SOURCES + ["-o", lib])
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    if verbose:
        print(res.stderr)
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
