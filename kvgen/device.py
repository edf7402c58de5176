"""Device-side page generator (kvgen/gen.cu) behind a ctypes call; torch only carries memory."""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

from . import gen

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gen.cu")
_LIB = os.path.join(_HERE, "libkvgen.so")
_lib = None
_table = {}


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
                               "-Xcompiler", "-fPIC", "-shared", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB):
            raise RuntimeError("kvgen/libkvgen.so is missing: run __graft_entry__.build() first")
        _lib = C.CDLL(_LIB)
        _lib.kvgen_fill.restype = C.c_int
        _lib.kvgen_fill.argtypes = [C.c_void_p, C.c_uint64, C.c_uint64, C.c_uint64, C.c_void_p, C.c_void_p, C.c_uint64,
                                    C.c_uint32, C.c_void_p]
        _lib.kvgen_fill_runs.restype = C.c_int
        _lib.kvgen_fill_runs.argtypes = [C.c_void_p, C.c_uint64, C.c_uint64, C.c_uint64, C.c_uint32, C.c_void_p]
    return _lib


def fill(out, seed: int, first_pid: int, n_pages: int, scales_dev, pages_per_layer: int, n_kv_heads: int):
    """Writes pages [first_pid, first_pid + n_pages) into the torch CUDA tensor `out` (fp16/int16 bytes)."""
    import torch
    dev = out.device
    if dev not in _table:
        _table[dev] = torch.from_numpy(gen.normal_table()).to(dev)
    assert out.is_cuda and out.is_contiguous() and out.numel() * out.element_size() >= n_pages * 4096
    rc = _load().kvgen_fill(out.data_ptr(), first_pid, n_pages, int(gen.stream_key(seed)), _table[dev].data_ptr(),
                            scales_dev.data_ptr(), pages_per_layer, n_kv_heads, torch.cuda.current_stream().cuda_stream)
    if rc:
        raise RuntimeError(f"kvgen_fill failed: {rc}")


def fill_runs(out, seed: int, first_pid: int, n_pages: int, p256: int = gen.RUNS_P256):
    """Writes the piecewise-linear pages [first_pid, first_pid + n_pages) of gen.runs_pages into `out`."""
    import torch
    assert out.is_cuda and out.is_contiguous() and out.numel() * out.element_size() >= n_pages * 4096
    key = int(gen.stream_key(seed) ^ np.uint64(0x52554E53))
    rc = _load().kvgen_fill_runs(out.data_ptr(), first_pid, n_pages, key, p256, torch.cuda.current_stream().cuda_stream)
    if rc:
        raise RuntimeError(f"kvgen_fill_runs failed: {rc}")
