"""Device-side twin of the seeded generator (for workloads too large to generate on the host)."""
from __future__ import annotations

import ctypes as C
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "gen.cu")
SO = os.path.join(HERE, "libmatkv_inputs.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(SO) or os.path.getmtime(SO) < os.path.getmtime(SRC):
        nvcc = "/usr/local/cuda/bin/nvcc" if os.path.exists("/usr/local/cuda/bin/nvcc") else "nvcc"
        subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-shared",
                               "-Xcompiler", "-fPIC", "-o", SO, SRC])
    return SO


def fill_bf16(tensor, seed: int, stream: int, shift: int = 0, start: int = 0) -> None:
    """Fill a contiguous CUDA bf16 tensor with elements start..start+numel of the generator."""
    global _lib
    if _lib is None:
        if not os.path.exists(SO):
            raise ImportError(f"{SO} is missing: run matkv_inputs.device.build()")
        _lib = C.CDLL(SO)
        _lib.matkv_inputs_fill_bf16.restype = C.c_int
        _lib.matkv_inputs_fill_bf16.argtypes = [C.c_void_p, C.c_uint64, C.c_uint64, C.c_uint64, C.c_int, C.c_uint64,
                                                C.c_void_p]
    import torch
    assert tensor.is_cuda and tensor.is_contiguous() and tensor.element_size() == 2
    rc = _lib.matkv_inputs_fill_bf16(tensor.data_ptr(), tensor.numel(), seed, stream, shift, start,
                                     torch.cuda.current_stream().cuda_stream or None)
    if rc != 0:
        raise RuntimeError(f"generator launch failed: CUDA error {rc}")
