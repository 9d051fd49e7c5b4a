"""Compile libsjq.so (hand-written sm_100a CUDA kernels + C ABI) in-tree."""
from __future__ import annotations

import glob
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
LIB = os.path.join(HERE, "libsjq.so")
OBJ = os.path.join(HERE, "csrc", "obj")  # one object per translation unit, so that an edit recompiles only its own
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17", "-Xcompiler", "-fPIC"]


def sources() -> list[str]:
    return sorted(glob.glob(os.path.join(HERE, "csrc", "*.cu")))


def _headers() -> list[str]:
    return glob.glob(os.path.join(HERE, "csrc", "*.h")) + glob.glob(os.path.join(HERE, "csrc", "*.cuh")) + glob.glob(
        os.path.join(ROOT, "include", "*.h"))


def _object(src: str) -> str:
    return os.path.join(OBJ, os.path.splitext(os.path.basename(src))[0] + ".o")


def _stale(target: str, deps: list[str]) -> bool:
    return not os.path.exists(target) or any(os.path.getmtime(d) > os.path.getmtime(target) for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile the translation units that changed (all of them with force) in parallel, then link."""
    extra = os.environ.get("SJQ_NVCC_EXTRA", "").split()  # e.g. -D switches for kernel experiments
    headers = _headers()
    todo = [s for s in sources() if force or extra or _stale(_object(s), [s] + headers)]
    if not todo and not _stale(LIB, [_object(s) for s in sources()]):
        return LIB
    os.makedirs(OBJ, exist_ok=True)

    def compile_one(src: str) -> None:
        cmd = ["nvcc", *NVCC_FLAGS, *extra, "-I" + os.path.join(ROOT, "include"), "-c", src, "-o", _object(src)]
        if verbose:
            cmd[1:1] = ["-Xptxas", "-v"]
        subprocess.check_call(cmd, cwd=HERE)

    with ThreadPoolExecutor(max_workers=max(1, min(len(todo), os.cpu_count() or 1))) as pool:
        list(pool.map(compile_one, todo))
    subprocess.check_call(["nvcc", "-shared", *NVCC_FLAGS[:2], "-o", LIB, *[_object(s) for s in sources()]], cwd=HERE)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose=True))
