"""TEST INFRASTRUCTURE -- not part of the product path.

ctypes wrapper around ``dr_oracle.c``, the plain CPU statement of the role-switch state transform
(layout map D1-D4, bf16 round-to-nearest-even cast D5, chunked staging D6, fp8 block scaling D7).  Only ``tests/``,
``__graft_entry__.smoke()`` and the bench's CPU-baseline / ``--impl reference`` legs may import this.
It shares no code with the CUDA library and never imports it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_DIR, "libdr_oracle.so")
_SRC = os.path.join(_DIR, "dr_oracle.c")


def build(force: bool = False) -> None:
    if force or not os.path.exists(_SO) or os.path.getmtime(_SRC) > os.path.getmtime(_SO):
        # -ffp-contract=off, no fast-math: fp32 divisions must round exactly once, as written
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-Wall", "-ffp-contract=off", "-shared", "-fPIC", "-o", _SO, _SRC,
                               "-lm"])


class _Spec(ctypes.Structure):
    _fields_ = [(n, ctypes.c_uint32) for n in (
        "n_layers", "hidden", "n_q_heads", "n_kv_heads", "head_dim", "ffn", "vocab",
        "n_experts", "moe_ffn", "tied", "qk_norm")]


class _Opts(ctypes.Structure):
    _fields_ = [(n, ctypes.c_uint32) for n in ("kv_replicate", "vocab_pad", "moe_tp", "moe_ep", "moe_ep_rank")]


_lib = None


def _l():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_SO)
        u64, i64, p = ctypes.c_uint64, ctypes.c_int64, ctypes.c_void_p
        lib.orc_cast_bf16.restype = ctypes.c_uint16
        lib.orc_cast_bf16.argtypes = [ctypes.c_uint32]
        lib.orc_cast_bf16_many.restype = None
        lib.orc_cast_bf16_many.argtypes = [p, p, u64]
        lib.orc_widen_bf16.restype = ctypes.c_uint32
        lib.orc_widen_bf16.argtypes = [ctypes.c_uint16]
        lib.orc_model_create.restype = p
        lib.orc_model_create.argtypes = [ctypes.POINTER(_Spec), u64, u64, u64, u64, u64, u64]
        lib.orc_model_create_ex.restype = p
        lib.orc_model_create_ex.argtypes = [ctypes.POINTER(_Spec), u64, u64, u64, u64, u64, u64, ctypes.POINTER(_Opts)]
        lib.orc_model_destroy.restype = None
        lib.orc_model_destroy.argtypes = [p]
        for n in ("orc_n_src", "orc_n_dst", "orc_flat_elems", "orc_shard_elems", "orc_arena_bytes"):
            getattr(lib, n).restype = u64
            getattr(lib, n).argtypes = [p]
        lib.orc_src_info.restype = ctypes.c_int
        lib.orc_src_info.argtypes = [p, u64, ctypes.c_char_p] + [ctypes.POINTER(u64)] * 3
        lib.orc_dst_info.restype = ctypes.c_int
        lib.orc_dst_info.argtypes = [p, u64, ctypes.c_char_p] + [ctypes.POINTER(u64)] * 3 + [ctypes.POINTER(i64)]
        lib.orc_map.restype = i64
        lib.orc_map.argtypes = [p, u64, u64, u64]
        lib.orc_map_rows.restype = ctypes.c_int
        lib.orc_map_rows.argtypes = [p, u64, u64, u64, p]
        lib.orc_forward.restype = ctypes.c_int
        lib.orc_forward.argtypes = [p, p, ctypes.c_int, u64, p, i64]
        lib.orc_inverse.restype = ctypes.c_int
        lib.orc_inverse.argtypes = [p, p, ctypes.c_int, u64, p]
        lib.orc_stage_out.restype = i64
        lib.orc_stage_out.argtypes = [p, p, u64, u64, u64, u64, p, p]
        lib.orc_stage_in.restype = i64
        lib.orc_stage_in.argtypes = [p, p, u64, p, u64, u64, p, p, p]
        lib.orc_cast_e4m3.restype = ctypes.c_uint8
        lib.orc_cast_e4m3.argtypes = [ctypes.c_uint32]
        lib.orc_e4m3_value.restype = ctypes.c_float
        lib.orc_e4m3_value.argtypes = [ctypes.c_uint8]
        lib.orc_fp8_layout.restype = u64
        lib.orc_fp8_layout.argtypes = [p, u64, ctypes.POINTER(ctypes.c_int), ctypes.POINTER(u64), ctypes.POINTER(u64)]
        lib.orc_forward_fp8.restype = ctypes.c_int
        lib.orc_forward_fp8.argtypes = [p, p, p, i64]
        lib.orc_inverse_fp8.restype = ctypes.c_int
        lib.orc_inverse_fp8.argtypes = [p, p, p, i64]
        lib.orc_restage_out.restype = None
        lib.orc_restage_out.argtypes = [p, u64, u64, u64, p]
        lib.orc_restage_in.restype = None
        lib.orc_restage_in.argtypes = [p, u64, u64, u64, p]
        _lib = lib
    return _lib


def cast_bf16(u: int) -> int:
    """D5 on one fp32 bit pattern."""
    return int(_l().orc_cast_bf16(u & 0xFFFFFFFF))


def cast_e4m3(u: int) -> int:
    """D7's fp32 -> e4m3 conversion on one bit pattern."""
    return int(_l().orc_cast_e4m3(u & 0xFFFFFFFF))


def e4m3_value(c: int) -> float:
    return float(_l().orc_e4m3_value(c & 0xFF))


def widen_bf16(b: int) -> int:
    return int(_l().orc_widen_bf16(b & 0xFFFF))


def cast_bf16_array(u: np.ndarray) -> np.ndarray:
    """D5 element by element (the scalar C function called in a loop)."""
    u = np.ascontiguousarray(u, dtype=np.uint32)
    out = np.empty(u.shape, dtype=np.uint16)
    _l().orc_cast_bf16_many(u.ctypes.data, out.ctypes.data, u.size)
    return out


@dataclass(frozen=True)
class SrcTensor:
    name: str
    rows: int
    cols: int
    flat_off: int


@dataclass(frozen=True)
class DstTensor:
    name: str
    rows: int
    cols: int
    arena_off: int
    alias_of: int


class Model:
    """Source (D1, D2) and rollout (D3) layouts of one model spec at (W, T, t)."""

    def __init__(self, spec: dict, *, align: int = 1, world: int = 1, tp: int = 1, tp_rank: int = 0,
                 elem_size: int = 2, arena_align: int = 256, kv_replicate: bool = False, vocab_pad: int = 0,
                 moe_tp: int = 1, moe_ep: int = 1, moe_ep_rank: int = 0):
        s = _Spec(**{k: int(spec.get(k, 0)) for k, _ in _Spec._fields_})
        o = _Opts(int(kv_replicate), vocab_pad, moe_tp, moe_ep, moe_ep_rank)
        self._h = _l().orc_model_create_ex(ctypes.byref(s), align, world, tp, tp_rank, elem_size, arena_align,
                                           ctypes.byref(o))
        if not self._h:
            raise ValueError("oracle: unsupported spec / layout")
        self.elem_size = elem_size
        self.world = world
        lib = _l()
        self.flat_elems = int(lib.orc_flat_elems(self._h))
        self.shard_elems = int(lib.orc_shard_elems(self._h))
        self.arena_bytes = int(lib.orc_arena_bytes(self._h))
        self.n_src = int(lib.orc_n_src(self._h))
        self.n_dst = int(lib.orc_n_dst(self._h))

    def __del__(self):
        if getattr(self, "_h", None) and _lib is not None:  # at interpreter exit the module may be gone already
            _lib.orc_model_destroy(self._h)
            self._h = None

    def src_tensors(self) -> list[SrcTensor]:
        out, name = [], ctypes.create_string_buffer(64)
        r, c, o = ctypes.c_uint64(), ctypes.c_uint64(), ctypes.c_uint64()
        for i in range(self.n_src):
            _l().orc_src_info(self._h, i, name, ctypes.byref(r), ctypes.byref(c), ctypes.byref(o))
            out.append(SrcTensor(name.value.decode(), r.value, c.value, o.value))
        return out

    def dst_tensors(self) -> list[DstTensor]:
        out, name = [], ctypes.create_string_buffer(64)
        r, c, o, a = ctypes.c_uint64(), ctypes.c_uint64(), ctypes.c_uint64(), ctypes.c_int64()
        for i in range(self.n_dst):
            _l().orc_dst_info(self._h, i, name, ctypes.byref(r), ctypes.byref(c), ctypes.byref(o), ctypes.byref(a))
            out.append(DstTensor(name.value.decode(), r.value, c.value, o.value, a.value))
        return out

    def map(self, i: int, row: int, col: int) -> int:
        return int(_l().orc_map(self._h, i, row, col))

    def map_rows(self, i: int, row0: int, nrows: int, cols: int) -> np.ndarray:
        out = np.empty((nrows, cols), dtype=np.int64)
        _l().orc_map_rows(self._h, i, row0, nrows, out.ctypes.data)
        return out

    def forward(self, src_u32: np.ndarray, arena_u8: np.ndarray, *, gathered: bool = True, rank: int = 0,
                only: int = -1) -> None:
        assert src_u32.dtype == np.uint32 and src_u32.flags.c_contiguous
        assert arena_u8.dtype == np.uint8 and arena_u8.flags.c_contiguous and arena_u8.size >= self.arena_bytes
        need = self.world * self.shard_elems if gathered else self.shard_elems
        assert src_u32.size >= min(need, self.flat_elems if gathered else need)
        _l().orc_forward(self._h, src_u32.ctypes.data, int(gathered), rank, arena_u8.ctypes.data, only)

    def fp8_layout(self):
        """(arena bytes, [(quantised, payload offset, scale offset)] per rollout tensor) of the fp8 arena (D7)."""
        out = []
        q, o, so = ctypes.c_int(), ctypes.c_uint64(), ctypes.c_uint64()
        total = 0
        for i in range(self.n_dst):
            total = int(_l().orc_fp8_layout(self._h, i, ctypes.byref(q), ctypes.byref(o), ctypes.byref(so)))
            out.append((bool(q.value), o.value, so.value))
        return total, out

    def forward_fp8(self, src_u32: np.ndarray, arena_u8: np.ndarray, only: int = -1) -> None:
        assert src_u32.dtype == np.uint32 and src_u32.flags.c_contiguous and src_u32.size >= self.flat_elems
        assert arena_u8.dtype == np.uint8 and arena_u8.size >= self.fp8_layout()[0]
        _l().orc_forward_fp8(self._h, src_u32.ctypes.data, arena_u8.ctypes.data, only)

    def inverse_fp8(self, arena_u8: np.ndarray, flat_u32: np.ndarray, only: int = -1) -> None:
        """Inverse of D7: codes times block scales (and widened bf16 tensors) back to their flat positions."""
        assert flat_u32.dtype == np.uint32 and flat_u32.flags.c_contiguous and flat_u32.size >= self.flat_elems
        assert arena_u8.dtype == np.uint8 and arena_u8.flags.c_contiguous and arena_u8.size >= self.fp8_layout()[0]
        _l().orc_inverse_fp8(self._h, arena_u8.ctypes.data, flat_u32.ctypes.data, only)

    def inverse(self, arena_u8: np.ndarray, flat_u32: np.ndarray, *, gathered: bool = True, rank: int = 0) -> None:
        assert flat_u32.dtype == np.uint32 and flat_u32.flags.c_contiguous
        assert arena_u8.dtype == np.uint8 and arena_u8.flags.c_contiguous and arena_u8.size >= self.arena_bytes
        _l().orc_inverse(self._h, arena_u8.ctypes.data, int(gathered), rank, flat_u32.ctypes.data)


def _ptr_array(bufs):
    arr = (ctypes.c_void_p * len(bufs))(*[b.ctypes.data for b in bufs])
    sizes = (ctypes.c_uint64 * len(bufs))(*[b.nbytes for b in bufs])
    return arr, sizes


def stage_out(bufs: list[np.ndarray], budget: int, chunk: int = 0, first_chunk: int = 0,
              sink: np.ndarray | None = None):
    """D6 stage-out of the byte stream bufs[0] | bufs[1] | ... ; returns (sink, chunk_sizes)."""
    total = sum(b.nbytes for b in bufs)
    if sink is None:
        sink = np.zeros(total, dtype=np.uint8)
    c = chunk or budget // 2 // 4096 * 4096
    n_chunks = -(-total // c) if c else 0
    sizes = np.zeros(max(n_chunks, 1), dtype=np.uint64)
    arr, nb = _ptr_array(bufs)
    n = _l().orc_stage_out(arr, nb, len(bufs), budget, chunk, first_chunk, sink.ctypes.data, sizes.ctypes.data)
    if n < 0:
        raise ValueError("oracle: budget cannot hold two slots")
    return sink, sizes[:n]


def stage_in(bufs: list[np.ndarray], source: np.ndarray, budget: int, chunk: int = 0, order=None, pieces=False):
    """D6 stage-in into bufs (in place), buffers restored in ``order``; returns (piece count, completion
    order), plus the walk itself as a list of (buffer, position, bytes) when ``pieces`` is set."""
    arr, nb = _ptr_array(bufs)
    o = (ctypes.c_uint32 * len(bufs))(*(order if order is not None else range(len(bufs))))
    done = (ctypes.c_uint32 * len(bufs))()
    c = chunk or budget // 2 // 4096 * 4096
    cap = sum(-(-b.nbytes // c) for b in bufs) if c else 0
    walk = np.zeros((max(cap, 1), 3), dtype=np.uint64)
    n = _l().orc_stage_in(arr, nb, len(bufs), o, budget, chunk, source.ctypes.data, done, walk.ctypes.data)
    if n < 0:
        raise ValueError("oracle: budget cannot hold two slots")
    if pieces:
        return int(n), list(done), [tuple(int(x) for x in row) for row in walk[:n]]
    return int(n), list(done)


def restage(old_shards: list[np.ndarray], n: int, w_new: int) -> list[np.ndarray]:
    """Old shards (world = len(old_shards)) -> new shards for world w_new, through a flat host image."""
    w_old = len(old_shards)
    image = np.zeros(n, dtype=np.uint32)
    for r, sh in enumerate(old_shards):
        assert sh.dtype == np.uint32 and sh.size == -(-n // w_old)
        _l().orc_restage_out(sh.ctypes.data, n, w_old, r, image.ctypes.data)
    out = []
    for q in range(w_new):
        new = np.empty(-(-n // w_new), dtype=np.uint32)
        _l().orc_restage_in(image.ctypes.data, n, w_new, q, new.ctypes.data)
        out.append(new)
    return out
