"""Builds libgg_b200.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
BUILD = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libgg_b200.so")
SOURCES = ["gg_api.cu", "gg_stream.cu", "gg_tail_bf16.cu", "gg_tail_f32.cu", "gg_small_bf16.cu", "gg_team.cu", "gg_segment.cu", "gg_sample.cu", "gg_codes.cu", "gg_channels.cu", "gg_channels_f32.cu", "gg_noalloc.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", CSRC]


def _deps():
    hdrs = [os.path.join(ROOT, "include", "gg.h")]
    hdrs += [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    return hdrs


def _stale(target, sources):
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(s) > t for s in sources)


def build(force=False, verbose=False, ptxas_info=False, bounds=False):
    """Builds the library.  bounds=True builds libgg_b200_bounds.so instead: the same sources with -DGG_BOUNDS, whose
    streaming kernels count (and skip) every checked global access that would leave its buffer; run the GPU tests
    on it with GG_B200_LIB pointing at it."""
    build_dir = BUILD + ("_bounds" if bounds else "")
    lib = LIB.replace(".so", "_bounds.so") if bounds else LIB
    os.makedirs(build_dir, exist_ok=True)
    hdrs = _deps()
    objs, jobs = [], []
    for src in SOURCES:
        path = os.path.join(CSRC, src)
        obj = os.path.join(build_dir, src.replace(".cu", ".o"))
        objs.append(obj)
        if force or _stale(obj, [path] + hdrs):
            cmd = (["nvcc"] + NVCC_FLAGS + (["-DGG_BOUNDS"] if bounds else []) + (["-Xptxas", "-v"] if ptxas_info else []) +
                   ["-c", path, "-o", obj])
            jobs.append(cmd)

    def run(cmd):
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode != 0:
            raise RuntimeError("nvcc failed:\n" + " ".join(cmd) + "\n" + r.stdout + r.stderr)
        return r.stderr

    if jobs:
        with ThreadPoolExecutor(max_workers=4) as ex:
            for log in ex.map(run, jobs):
                if verbose or ptxas_info:
                    sys.stderr.write(log)
    if jobs or _stale(lib, objs):
        run(["nvcc", "-shared", "-o", lib] + objs + ["-lcudart"])
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose=True, ptxas_info="--ptxas" in sys.argv, bounds="--bounds" in sys.argv))
