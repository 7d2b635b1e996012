"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA path's tests and bench.

Holds input generation only (values as a pure function of ``(seed, buffer_id, index)``): none of the
transform's arithmetic lives here.  The host generator is plain C (``gen.c``), the device generator is a
small CUDA library of its own (``gen_cuda.cu``); both are compiled by :func:`build`.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
_HOST_SO = os.path.join(_DIR, "libsynth.so")
_CUDA_SO = os.path.join(_DIR, "libsynth_cuda.so")

BUF_MASTER, BUF_ADAM_M, BUF_ADAM_V, BUF_ROLLOUT = 0, 1, 2, 3
SEED_BASE = 0xD15A0000  # seed of config i is SEED_BASE + i


def _stale(so: str, srcs: list[str]) -> bool:
    return not os.path.exists(so) or any(os.path.getmtime(s) > os.path.getmtime(so) for s in srcs)


def build(cuda: bool = True, force: bool = False) -> None:
    src = os.path.join(_DIR, "gen.c")
    if force or _stale(_HOST_SO, [src]):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _HOST_SO, src])
    cu = os.path.join(_DIR, "gen_cuda.cu")
    if cuda and (force or _stale(_CUDA_SO, [cu])):
        subprocess.check_call(["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3",
                               "-shared", "-Xcompiler", "-fPIC", "-o", _CUDA_SO, cu])


_host = None
_cuda = None


def _h():
    global _host
    if _host is None:
        build(cuda=False)
        lib = ctypes.CDLL(_HOST_SO)
        u64, u32, p = ctypes.c_uint64, ctypes.c_uint32, ctypes.c_void_p
        lib.synth_bits.restype = u32
        lib.synth_bits.argtypes = [u64, u32, u64]
        for name in ("synth_fill_f32", "synth_fill_bf16"):
            getattr(lib, name).restype = None
            getattr(lib, name).argtypes = [p, u64, u32, u64, u64]
        for name in ("synth_at_f32", "synth_at_bf16"):
            getattr(lib, name).restype = None
            getattr(lib, name).argtypes = [p, u64, u32, p, u64]
        _host = lib
    return _host


def bits(seed: int, buffer_id: int, index: int) -> int:
    return int(_h().synth_bits(seed, buffer_id, index))


def fill_f32(seed: int, buffer_id: int, start: int, n: int, out: np.ndarray | None = None) -> np.ndarray:
    """uint32 bit patterns of fp32 elements start..start+n (written into ``out`` when given)."""
    if out is None:
        out = np.empty(n, dtype=np.uint32)
    assert out.dtype == np.uint32 and out.size == n and out.flags.c_contiguous
    _h().synth_fill_f32(out.ctypes.data, seed, buffer_id, start, n)
    return out


def at_f32(seed: int, buffer_id: int, idx: np.ndarray) -> np.ndarray:
    idx = np.ascontiguousarray(idx, dtype=np.uint64)
    out = np.empty(idx.size, dtype=np.uint32)
    _h().synth_at_f32(out.ctypes.data, seed, buffer_id, idx.ctypes.data, idx.size)
    return out.reshape(idx.shape)


def fill_bf16(seed: int, buffer_id: int, start: int, n: int) -> np.ndarray:
    out = np.empty(n, dtype=np.uint16)
    _h().synth_fill_bf16(out.ctypes.data, seed, buffer_id, start, n)
    return out


def at_bf16(seed: int, buffer_id: int, idx: np.ndarray) -> np.ndarray:
    idx = np.ascontiguousarray(idx, dtype=np.uint64)
    out = np.empty(idx.size, dtype=np.uint16)
    _h().synth_at_bf16(out.ctypes.data, seed, buffer_id, idx.ctypes.data, idx.size)
    return out.reshape(idx.shape)


def _c():
    global _cuda
    if _cuda is None:
        if not os.path.exists(_CUDA_SO):
            build(cuda=True)
        lib = ctypes.CDLL(_CUDA_SO)
        u64, u32, p = ctypes.c_uint64, ctypes.c_uint32, ctypes.c_void_p
        for name in ("synth_cuda_fill_f32", "synth_cuda_fill_bf16"):
            getattr(lib, name).restype = ctypes.c_int
            getattr(lib, name).argtypes = [p, u64, u32, u64, u64, p]
        lib.synth_cuda_mismatch_f32.restype = ctypes.c_int
        lib.synth_cuda_mismatch_f32.argtypes = [p, u64, u32, u64, u64, p, p]
        _cuda = lib
    return _cuda


def _stream_ptr(stream) -> int:
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def cuda_fill_f32(t, seed: int, buffer_id: int, start: int = 0, stream=None) -> None:
    """Fill a CUDA tensor viewed as fp32 words with generator elements start..start+t.numel()."""
    assert t.is_cuda and t.is_contiguous() and t.element_size() == 4
    rc = _c().synth_cuda_fill_f32(t.data_ptr(), seed, buffer_id, start, t.numel(), _stream_ptr(stream))
    if rc:
        raise RuntimeError(f"synth_cuda_fill_f32: cuda error {rc}")


def cuda_fill_bf16(t, seed: int, buffer_id: int, start: int = 0, stream=None) -> None:
    assert t.is_cuda and t.is_contiguous() and t.element_size() == 2
    rc = _c().synth_cuda_fill_bf16(t.data_ptr(), seed, buffer_id, start, t.numel(), _stream_ptr(stream))
    if rc:
        raise RuntimeError(f"synth_cuda_fill_bf16: cuda error {rc}")


def cuda_mismatch_f32(t, seed: int, buffer_id: int, start: int = 0) -> int:
    """Number of fp32 words of CUDA tensor ``t`` that differ from the generator's (regenerated by index)."""
    import torch
    assert t.is_cuda and t.is_contiguous() and t.element_size() == 4
    cnt = torch.zeros(1, dtype=torch.int64, device=t.device)
    rc = _c().synth_cuda_mismatch_f32(t.data_ptr(), seed, buffer_id, start, t.numel(), cnt.data_ptr(),
                                      _stream_ptr(None))
    if rc:
        raise RuntimeError(f"synth_cuda_mismatch_f32: cuda error {rc}")
    return int(cnt.item())
