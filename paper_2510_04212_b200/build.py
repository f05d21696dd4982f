"""Build libattn_b200.so (the C-ABI library) in-tree with nvcc for sm_100a."""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libattn_b200.so")
SOURCES = [os.path.join(CSRC, "attn_api.cu")]
HEADERS = [os.path.join(CSRC, n) for n in ("ptx.cuh", "fwd_kernel.cuh", "bwd_kernel.cuh", "bwd_kernel_d64.cuh", "bwd_kernel_d128.cuh", "delta_dp_kernel.cuh", "selftest_kernel.cuh", "packed_copy_kernel.cuh", "quantize_v_kernel.cuh")] + [
    os.path.join(os.path.dirname(HERE), "include", "attn.h")]


def _nvcc():
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def is_stale():
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(f) > t for f in SOURCES + HEADERS)


def build(force=False, verbose=False):
    if not force and not is_stale():
        return LIB
    cmd = [_nvcc(), "-std=c++17", "-O3", "-lineinfo", "-shared", "-Xcompiler", "-fPIC",
           "-gencode", "arch=compute_100a,code=sm_100a",
           "-Xptxas", "-v" if verbose else "-warn-spills",
           *SOURCES, "-o", LIB + ".tmp"]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    if verbose:
        print(res.stdout + res.stderr)
    os.replace(LIB + ".tmp", LIB)
    return LIB


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
