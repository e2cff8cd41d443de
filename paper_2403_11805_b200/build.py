"""Compile csrc/*.cu into paper_2403_11805_b200/libllms.so with nvcc for sm_100a (in-tree build)."""
import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libllms.so")
# The checked build: the same library with a bounds check in front of every access the group-wise codec kernels make to
# the KV tensor and the swap buffer (csrc/codec.cu, LLMS_DEBUG_BOUNDS).  Only tests load it (LLMS_LIBRARY in the binding).
DEBUG_LIB = os.path.join(HERE, "libllms_debug.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--fmad=false",            # the record format fixes every rounding: fused operations are written out where wanted
    "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _newest_input():
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(ROOT, "include", "*.h"))
    return max(os.path.getmtime(p) for p in deps)


def nvcc_path():
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def build(force: bool = False, verbose: bool = False, debug_bounds: bool = False) -> str:
    """Compile every csrc/*.cu to an object (the files in parallel: the codec's template instantiations take most
    of the time) and link them into the shared library.  debug_bounds: also compile codec.cu a second time with its
    bounds checks and link the checked library from that object and the other files' ordinary ones."""
    fresh = os.path.exists(LIB) and os.path.getmtime(LIB) >= _newest_input()
    fresh_debug = not debug_bounds or (os.path.exists(DEBUG_LIB) and os.path.getmtime(DEBUG_LIB) >= _newest_input())
    if not force and fresh and fresh_debug:
        return LIB
    from concurrent.futures import ThreadPoolExecutor
    obj_dir = os.path.join(HERE, "_build")
    os.makedirs(obj_dir, exist_ok=True)
    compile_flags = [f for f in NVCC_FLAGS if f != "-shared"] + (["-Xptxas", "-v"] if verbose else [])

    def compile_one(job):
        src, suffix, extra = job
        obj = os.path.join(obj_dir, os.path.basename(src)[:-3] + suffix + ".o")
        subprocess.run([nvcc_path()] + compile_flags + extra + ["-c", src, "-o", obj], check=True)
        return obj

    jobs = [(src, "", []) for src in sources()]
    if debug_bounds:
        jobs.append((os.path.join(CSRC, "codec.cu"), "_debug", ["-DLLMS_DEBUG_BOUNDS"]))
    with ThreadPoolExecutor(max_workers=6) as pool:
        objects = list(pool.map(compile_one, jobs))
    plain = objects[:len(sources())]
    link = [nvcc_path(), "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o"]
    subprocess.run(link + [LIB + ".tmp"] + plain, check=True)
    os.replace(LIB + ".tmp", LIB)
    if debug_bounds:
        checked = [objects[-1] if os.path.basename(o) == "codec.o" else o for o in plain]
        subprocess.run(link + [DEBUG_LIB + ".tmp"] + checked, check=True)
        os.replace(DEBUG_LIB + ".tmp", DEBUG_LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug_bounds="--debug-bounds" in sys.argv))
