"""Compile the CPU oracle (plain C + OpenMP) into a shared library beside this file.

TEST INFRASTRUCTURE, NOT PRODUCT.  Run as `python -m oracle.build`, or call build().
The library name carries a hash of the host CPU's feature flags, so a copy built on
another machine is never loaded by mistake (it is compiled with -march=native).
"""
import hashlib
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))


def _host_tag() -> str:
    flags = ""
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags"):
                    flags = line
                    break
    except OSError:
        pass
    return hashlib.sha1(flags.encode()).hexdigest()[:10]


def lib_path() -> str:
    return os.path.join(HERE, f"libdmtd_oracle.{_host_tag()}.so")


def build(force: bool = False) -> str:
    src = os.path.join(HERE, "dmtd_oracle.c")
    hdr = os.path.join(HERE, "dmtd_oracle.h")
    lib = lib_path()
    if (not force and os.path.exists(lib)
            and os.path.getmtime(lib) >= max(os.path.getmtime(src), os.path.getmtime(hdr))):
        return lib
    tmp = lib + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O2", "-march=native", "-fopenmp", "-std=c11", "-Wall", "-Wextra", "-shared",
           "-fPIC", src, "-o", tmp, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force=True))
