"""Builds the CUDA library in-tree: paper_2507_18181_b200/libspecasr.so (sm_100a only)."""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
SOURCES = ["api.cu", "kernels_small.cu", "attention.cu", "attention_tc.cu", "gemm_fma.cu", "gemm_tcgen05.cu", "fused_stack.cu", "accept_static.cu", "top2.cu"]
LIB = os.path.join(HERE, "libspecasr.so")
LIB_TRACE = os.path.join(HERE, "libspecasr_trace.so")      # same sources with -DSPECASR_TRACE (device-side trace)


def _stale(lib=None) -> bool:
    lib = lib or LIB
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(HERE, "csrc", f) for f in os.listdir(os.path.join(HERE, "csrc"))]
    deps.append(os.path.join(ROOT, "include", "specasr.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, trace: bool = False) -> str:
    """Builds libspecasr.so, or with trace=True the variant that can record the device-side trace."""
    lib = LIB_TRACE if trace else LIB
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
    cmd += [os.path.join(HERE, "csrc", s) for s in SOURCES]
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
