"""Build the CUDA library (librmm.so) in-tree for sm_100a with nvcc.

``python -m paper_2201_13195_b200.build`` compiles csrc/rmm_api.cu into
paper_2201_13195_b200/librmm.so.  Cross-compiles without a GPU.
"""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "librmm.so")
SOURCES = ["rmm_api.cu"]


def _newest_source_mtime() -> float:
    m = 0.0
    for d in (CSRC, os.path.join(os.path.dirname(HERE), "include")):
        for f in os.listdir(d):
            m = max(m, os.path.getmtime(os.path.join(d, f)))
    return m


def nvcc_command(out: str, extra=()):
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    return [nvcc, "-std=c++17", "-O3", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
            "-Xcompiler", "-fPIC", "-shared", "--fmad=true", "--extended-lambda", "-diag-suppress", "20013,20015", "-o", out,
            *[os.path.join(CSRC, s) for s in SOURCES], *extra]


def build_trace(out: str) -> str:
    """A second library with the pass kernel's cycle accounting compiled in (-DRMM_PASS_TRACE): for profiling
    sessions only, never loaded by the package."""
    res = subprocess.run(nvcc_command(out, ["-DRMM_PASS_TRACE"]), capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("nvcc failed building the trace library")
    return out


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= _newest_source_mtime():
        return LIB
    cmd = nvcc_command(LIB + ".tmp", ["-Xptxas", "-v"] if verbose else [])
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed building librmm.so")
    os.replace(LIB + ".tmp", LIB)
    return LIB


if __name__ == "__main__":
    if "--trace" in sys.argv:
        print(build_trace(sys.argv[sys.argv.index("--trace") + 1]))
    else:
        print(build(force=True, verbose="-v" in sys.argv))
