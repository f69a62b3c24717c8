"""Build the CUDA library (sm_100a only) into paper_2510_11958_b200/libdmtd_b200.so.

`python -m paper_2510_11958_b200.build` or build().  nvcc cross-compiles without a GPU.
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
LIB = os.path.join(HERE, "libdmtd_b200.so")
SOURCES = ["engine.cu"]
HEADERS = ["common.cuh", "kernels.cuh", "pass_common.cuh", "pass_stream.cuh", "pass_prologues.cuh",
           "pass_attention.cuh", "pass_attention_f32.cuh", "pass_kernel.cuh", "attention_kernel.cuh", "gemm_tc05.cuh"]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(HERE, "csrc", f) for f in SOURCES + HEADERS]
    deps.append(os.path.join(ROOT, "include", "dmtd.h"))
    return any(os.path.getmtime(d) > t for d in deps if os.path.exists(d))


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = LIB + f".tmp{os.getpid()}"
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
           "--use_fast_math" if False else "-DDMTD_NO_FAST_MATH", "-Xcompiler", "-fPIC", "-shared",
           "-I", os.path.join(ROOT, "include")]
    cmd += os.environ.get("DMTD_NVCC_FLAGS", "").split()      # e.g. -DDMTD_PASS_SLOTS=2 for an experiment
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(HERE, "csrc", f) for f in SOURCES] + ["-o", tmp]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        sys.stderr.write(r.stdout + r.stderr)
        raise RuntimeError("nvcc failed")
    if verbose:
        sys.stderr.write(r.stdout + r.stderr)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
