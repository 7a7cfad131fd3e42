"""Builds the CUDA library in-tree: paper_2507_18181_b200/libspecasr.so (sm_100a only)."""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
SOURCES = ["api.cu", "kernels_small.cu", "attention_tc.cu", "gemm_tcgen05.cu", "fused_stack.cu", "accept_static.cu", "top2.cu"]
CROSSCHECK_SOURCES = ["gemm_fma.cu", "attention.cu"]     # the plain-FMA engine: cross-check variant only
LIB = os.path.join(HERE, "libspecasr.so")
LIB_TRACE = os.path.join(HERE, "libspecasr_trace.so")      # same sources with -DSPECASR_TRACE (device-side trace)
LIB_CROSSCHECK = os.path.join(HERE, "libspecasr_crosscheck.so")   # + the plain-FMA engine (-DSPECASR_CROSSCHECK)


def _stale(lib=None) -> bool:
    lib = lib or LIB
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(HERE, "csrc", f) for f in os.listdir(os.path.join(HERE, "csrc"))]
    deps.append(os.path.join(ROOT, "include", "specasr.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, trace: bool = False, crosscheck: bool = False) -> str:
    """Builds libspecasr.so, or with trace=True the variant that can record the device-side trace, or with
    crosscheck=True the variant that also carries the plain-FMA projections and attention (a second engine used
    by tests to cross-check the tensor-core kernels and to run shapes those do not cover)."""
    lib = LIB_CROSSCHECK if crosscheck else (LIB_TRACE if trace else LIB)
    if not force and not _stale(lib):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-O3", "-std=c++17", "-shared", "-Xcompiler", "-fPIC", "-lineinfo",
           "-gencode", "arch=compute_100a,code=sm_100a",
           "-I", os.path.join(ROOT, "include"), "-I", os.path.join(HERE, "csrc")]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    if trace:
        cmd += ["-DSPECASR_TRACE"]
    if crosscheck:
        cmd += ["-DSPECASR_CROSSCHECK"]
    cmd += [os.path.join(HERE, "csrc", s) for s in SOURCES + (CROSSCHECK_SOURCES if crosscheck else [])]
    cmd += ["-o", lib, "-lcudart"]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("nvcc failed")
    if verbose:
        print(res.stdout + res.stderr)
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
