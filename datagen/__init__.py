"""Seeded synthetic inputs for the star-join workloads.

This package is the *input definition* shared by the CPU oracle's tests and the
CUDA path's tests and benchmark.  It contains no query arithmetic: only column
generators (host: C + OpenMP, device: a CUDA kernel, both evaluating the same
counter-based integer function) and plain-data workload descriptions.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
HOST_LIB = os.path.join(_HERE, "libsjqgen_host.so")
CUDA_LIB = os.path.join(_HERE, "libsjqgen_cuda.so")

UNIFORM_I32, UNIFORM_DIV_I32, DATE_FK_I32, SEQ_I32, DATE_KEY_I32, DATE_YEAR_I32, MIXKEY_I64, ZIPF_FK_I64 = range(8)
DATE_ROWS = 2556
_I64_KINDS = (MIXKEY_I64, ZIPF_FK_I64)


def _newer(target: str, sources: list[str]) -> bool:
    if not os.path.exists(target):
        return False
    t = os.path.getmtime(target)
    return all(os.path.getmtime(s) <= t for s in sources)


def build_host(force: bool = False) -> str:
    srcs = [os.path.join(_HERE, f) for f in ("sjq_gen_host.c", "sjq_gen_core.h", "sjq_gen.h")]
    if force or not _newer(HOST_LIB, srcs):
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-Wall", "-o", HOST_LIB, srcs[0]], cwd=_HERE
        )
    return HOST_LIB


def build_cuda(force: bool = False) -> str:
    srcs = [os.path.join(_HERE, f) for f in ("sjq_gen_cuda.cu", "sjq_gen_core.h", "sjq_gen.h")]
    if force or not _newer(CUDA_LIB, srcs):
        subprocess.check_call(
            ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-Xcompiler", "-fPIC",
             "-shared", "-o", CUDA_LIB, srcs[0]],
            cwd=_HERE,
        )
    return CUDA_LIB


_host = None
_cuda = None


def _host_lib():
    global _host
    if _host is None:
        lib = ctypes.CDLL(build_host())
        lib.sjq_gen_fill_host.restype = ctypes.c_int
        lib.sjq_gen_fill_host.argtypes = [
            ctypes.c_int, ctypes.c_uint64, ctypes.c_uint64, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64,
            ctypes.c_int64, ctypes.c_int64, ctypes.c_uint64, ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p,
        ]
        lib.sjq_gen_zipf_table.restype = ctypes.c_int
        lib.sjq_gen_zipf_table.argtypes = [ctypes.c_int64, ctypes.c_void_p]
        lib.sjq_gen_mix_host.restype = ctypes.c_uint64
        lib.sjq_gen_mix_host.argtypes = [ctypes.c_uint64]
        _host = lib
    return _host


def _cuda_lib():
    global _cuda
    if _cuda is None:
        if not os.path.exists(CUDA_LIB):
            build_cuda()
        lib = ctypes.CDLL(CUDA_LIB)
        lib.sjq_gen_fill_device.restype = ctypes.c_int
        lib.sjq_gen_fill_device.argtypes = [
            ctypes.c_int, ctypes.c_uint64, ctypes.c_uint64, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64,
            ctypes.c_int64, ctypes.c_int64, ctypes.c_uint64, ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p,
            ctypes.c_void_p,
        ]
        _cuda = lib
    return _cuda


def mix(z: int) -> int:
    return int(_host_lib().sjq_gen_mix_host(ctypes.c_uint64(z & 0xFFFFFFFFFFFFFFFF)))


_zipf_cache: dict[int, np.ndarray] = {}


def zipf_table(k: int) -> np.ndarray:
    """Cumulative integer weights floor(2^40/j), j = 1..k (uint64, host)."""
    if k not in _zipf_cache:
        cum = np.empty(k, dtype=np.uint64)
        rc = _host_lib().sjq_gen_zipf_table(k, cum.ctypes.data)
        if rc != 0:
            raise ValueError("bad zipf table size")
        _zipf_cache[k] = cum
    return _zipf_cache[k]


def fill_host(kind: int, seed: int, column: int, row0: int, n: int, a: int = 0, b: int = 0, div: int = 1,
              key_seed: int = 0, zipf_k: int = 0, out: np.ndarray | None = None) -> np.ndarray:
    dtype = np.int64 if kind in _I64_KINDS else np.int32
    if out is None:
        out = np.empty(n, dtype=dtype)
    assert out.dtype == dtype and out.size == n and out.flags["C_CONTIGUOUS"]
    cum = zipf_table(zipf_k) if kind == ZIPF_FK_I64 else None
    rc = _host_lib().sjq_gen_fill_host(kind, seed, column, row0, n, a, b, div, key_seed,
                                       cum.ctypes.data if cum is not None else None, zipf_k, out.ctypes.data)
    if rc != 0:
        raise ValueError(f"sjq_gen_fill_host failed ({rc})")
    return out


_zipf_dev_cache: dict[tuple, object] = {}


def fill_device(kind: int, seed: int, column: int, row0: int, n: int, a: int = 0, b: int = 0, div: int = 1,
                key_seed: int = 0, zipf_k: int = 0, device: str = "cuda:0"):
    """Generate a column straight into a torch CUDA tensor (same bytes as fill_host)."""
    import torch

    dtype = torch.int64 if kind in _I64_KINDS else torch.int32
    out = torch.empty(n, dtype=dtype, device=device)
    cum_ptr = None
    if kind == ZIPF_FK_I64:
        ck = (zipf_k, str(device))
        if ck not in _zipf_dev_cache:
            host = torch.from_numpy(zipf_table(zipf_k).view(np.int64))
            _zipf_dev_cache[ck] = host.to(device)
        cum_ptr = _zipf_dev_cache[ck].data_ptr()
    with torch.cuda.device(out.device):
        stream = torch.cuda.current_stream().cuda_stream
        rc = _cuda_lib().sjq_gen_fill_device(kind, seed, column, row0, n, a, b, div, key_seed, cum_ptr, zipf_k,
                                             out.data_ptr(), stream)
    if rc != 0:
        raise RuntimeError(f"sjq_gen_fill_device failed ({rc})")
    return out
