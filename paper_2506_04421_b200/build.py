"""In-tree build of libhmar.so (nvcc, sm_100a only)."""
import os
import shutil
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG_DIR, "csrc")
LIB_PATH = os.environ.get("HMAR_LIBRARY") or os.path.join(PKG_DIR, "libhmar.so")
CHECKED_LIB_PATH = os.path.join(PKG_DIR, "libhmar_check.so")     # the same sources with -DHMAR_BOUNDS_CHECK (tests)
SOURCES = ["api.cu", "schedule.cpp", "simt_kernels.cu", "tc_dispatch.cu", "fwd_sm100.cu", "bwd_sm100.cu", "noalloc_bwd.cu", "step_small.cu", "recon.cu"]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--expt-relaxed-constexpr", "-Xcompiler", "-fPIC", "-Xcompiler", "-Wall", "-shared",
]


def _nvcc():
    path = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(path):
        raise RuntimeError("nvcc not found; the HMAR CUDA library cannot be built")
    return path


def needs_build(path=None):
    path = path or LIB_PATH
    if not os.path.exists(path):
        return True
    lib_time = os.path.getmtime(path)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    deps.append(os.path.join(PKG_DIR, "..", "include", "hmar.h"))
    return any(os.path.getmtime(d) > lib_time for d in deps)


def build(force=False, verbose=False, checked=False):
    """Compile every CUDA source of the library into paper_2506_04421_b200/libhmar.so, or, with `checked`, into
    libhmar_check.so: the build whose kernels compare every address they form with its tensor's extent."""
    target = CHECKED_LIB_PATH if checked else os.path.join(PKG_DIR, "libhmar.so")
    if not force and not needs_build(target):
        return target
    cmd = [_nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + (["-DHMAR_BOUNDS_CHECK"] if checked else [])
    cmd += [os.path.join(CSRC, s) for s in SOURCES] + ["-o", target]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("nvcc failed building libhmar.so")
    if verbose:
        sys.stderr.write(res.stdout + res.stderr)
    return target


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
