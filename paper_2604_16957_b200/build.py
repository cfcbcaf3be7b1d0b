"""Build libtq.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

    python -m paper_2604_16957_b200.build [--force] [--verbose]
    python -m paper_2604_16957_b200.build --probe copies|math    # timing-probe builds of the decode kernel

The probe libraries (libtq_probe_copies.so, libtq_probe_math.so) are the same sources compiled with
-DTQ_PROBE_COPIES_ONLY / -DTQ_PROBE_MATH_ONLY: the fused decode kernel with its arithmetic, or its copies,
taken out.  They produce meaningless results and exist only to time (`bench.py --lib <path>`).
"""
import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
LIB = os.path.join(HERE, "libtq.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    # bit-exact quantiser: IEEE division / sqrt, no flush-to-zero, no fast-math; FMA contraction
    # is harmless because every quantiser operation is an explicit _rn intrinsic
    "-prec-div=true", "-prec-sqrt=true", "-ftz=false",
    "-Xcompiler", "-fPIC", "-shared", "-cudart", "static",
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(INCLUDE, "*.h"))
    return any(os.path.getmtime(p) > t for p in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-I", INCLUDE, "-I", CSRC, "-o", LIB] + sources()
    subprocess.run(cmd, check=True)
    return LIB


def build_probe(which: str) -> str:
    """Timing-probe build of the library: which = "copies" or "math"."""
    macro = {"copies": "TQ_PROBE_COPIES_ONLY", "math": "TQ_PROBE_MATH_ONLY"}[which]
    out = os.path.join(HERE, f"libtq_probe_{which}.so")
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    subprocess.run([nvcc] + NVCC_FLAGS + ["-D" + macro, "-I", INCLUDE, "-I", CSRC, "-o", out] + sources(), check=True)
    return out


if __name__ == "__main__":
    if "--probe" in sys.argv:
        print(build_probe(sys.argv[sys.argv.index("--probe") + 1]))
    else:
        print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
