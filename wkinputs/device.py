"""Device side of the generators: fills torch CUDA tensors through libwkinputs.so (bit-identical to gen.py)."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

from . import gen

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libwkinputs.so")
_lib = None


def _load():
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: run `python -m paper_2605_22718_b200.build`")
        lib = C.CDLL(_LIB_PATH)
        u64 = C.c_uint64
        lib.wkin_fill_normal_bf16.restype = C.c_int
        lib.wkin_fill_normal_bf16.argtypes = [C.c_void_p, u64, u64, u64, u64, C.c_void_p]
        lib.wkin_fill_keys_bf16.restype = C.c_int
        lib.wkin_fill_keys_bf16.argtypes = [C.c_void_p, u64, u64, u64, u64, u64, u64, C.c_float, C.c_void_p]
        _lib = lib
    return _lib


def _check(rc: int) -> None:
    if rc != 0:
        raise RuntimeError(f"input generator launch failed (CUDA error {rc})")


def fill_normal_bf16(out: torch.Tensor, seed: int, stream_id: int, idx0: int) -> torch.Tensor:
    _check(_load().wkin_fill_normal_bf16(out.data_ptr(), seed, stream_id, idx0, out.numel(),
                                         torch.cuda.current_stream().cuda_stream))
    return out


def key_chunk(out: torch.Tensor, seed: int, layer: int, chunk: int, T: int, D: int, sigma: float, F: int = 3):
    """out: bf16 [F*T, D] on the device."""
    _check(_load().wkin_fill_keys_bf16(out.data_ptr(), seed, layer, F * chunk, F, T, D, sigma,
                                       torch.cuda.current_stream().cuda_stream))
    return out


def value_chunk(out: torch.Tensor, seed: int, layer: int, chunk: int, T: int, D: int, F: int = 3):
    return fill_normal_bf16(out, seed, gen.STREAM_V + layer, chunk * F * T * D)


def query(out: torch.Tensor, seed: int, layer: int, step: int, chunk: int):
    return fill_normal_bf16(out, seed, gen.STREAM_Q + layer * 64 + step, chunk * out.numel())


def to_device_bf16(bits: np.ndarray, device="cuda") -> torch.Tensor:
    """numpy uint16 bf16 bit patterns -> torch bf16 tensor on the device (same shape)."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).to(device)


def to_host_bits(t: torch.Tensor) -> np.ndarray:
    """torch bf16 tensor -> numpy uint16 bit patterns."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)
