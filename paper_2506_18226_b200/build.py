"""Builds libadsa.so (sm_100a) in-tree with nvcc.  No torch extension machinery is involved."""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libadsa.so")
SOURCES = ["adsa_api.cu", "adsa_pool.cu", "adsa_score_select.cu", "adsa_attn.cu", "adsa_step.cu", "adsa_pstep.cu", "adsa_wstep.cu", "adsa_prefill.cu", "adsa_attn_static.cu", "adsa_shell.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden"]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(_HERE, "..", "include", "adsa.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build_lib(force: bool = False, verbose: bool = False) -> str:
    """Compile every .cu of the library for sm_100a and link libadsa.so next to this file."""
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = LIB + f".tmp{os.getpid()}"
    # --threads: the sources are independent translation units, compiled side by side
    cmd = [nvcc, "--threads", str(min(len(SOURCES), os.cpu_count() or 1)), *NVCC_FLAGS, "-shared", "-o", tmp,
           *[os.path.join(CSRC, s) for s in SOURCES]]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.check_call(cmd)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    import sys
    print(build_lib(force=True, verbose="-v" in sys.argv))
