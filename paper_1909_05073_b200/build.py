"""Builds libpconv.so (sm_100a) in-tree with nvcc.  `python -m paper_1909_05073_b200.build`."""
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libpconv.so")
DEV_LIB = os.path.join(HERE, "libpconv_dev.so")
# (fp32_peak.cu is a stand-alone measuring program, see build_peak)
SOURCES = ["pack.cu", "api.cu", "kernels_simple.cu", "kernels_tiled.cu", "kernels_tensor.cu", "project.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC"]


def generate():
    """Writes the generated PTX dispatch text (csrc/dispatch_s*.inc) next to the sources."""
    sys.path.insert(0, CSRC)
    try:
        import gen_dispatch
        gen_dispatch.main(CSRC)
    finally:
        sys.path.remove(CSRC)


def _stale(lib=None):
    lib = lib or LIB
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if not f.endswith(".inc")]
    deps.append(os.path.join(HERE, "..", "include", "pconv.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force=False, verbose=False, dev=False):
    """Compile the CUDA library if it is missing or older than its sources; returns its path.
    dev=True builds libpconv_dev.so instead: the same library with -DPCONV_DEV (the entry points
    of csrc/pconv_dev.h: phase timestamps of the tiled kernel, a launch plan forced through
    PCONV_FORCE_ZS / PCONV_FORCE_KS in the environment, and a bounded wait that can be made to
    run out for the tests of the give-up path)."""
    lib = DEV_LIB if dev else LIB
    if not force and not _stale(lib):
        return lib
    generate()
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = lib + ".tmp%d" % os.getpid()
    cmd = [nvcc] + NVCC_FLAGS + (["-DPCONV_DEV"] if dev else []) + \
          (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.check_call(cmd)
    os.replace(tmp, lib)
    return lib


def build_peak():
    """Compiles the stand-alone FP32-peak measurement (csrc/fp32_peak.cu) to ./fp32_peak."""
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    exe = os.path.join(HERE, "fp32_peak")
    subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-o", exe,
                           os.path.join(CSRC, "fp32_peak.cu")])
    return exe


if __name__ == "__main__":
    if "--peak" in sys.argv:
        print(build_peak())
        sys.exit(0)
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, dev="--dev" in sys.argv))
