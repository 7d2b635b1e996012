"""ctypes binding for ``libdynaresize.so``: structures and functions named as in ``dynaresize.h``."""
from __future__ import annotations

import ctypes as C
import os

_DIR = os.path.dirname(os.path.abspath(__file__))
lib_path = os.path.join(_DIR, "libdynaresize.so")

DR_OK = 0
DR_ERR_INVALID, DR_ERR_UNSUPPORTED, DR_ERR_SIZE, DR_ERR_ALIGN, DR_ERR_NOMEM = -1, -2, -3, -4, -5
DR_ERR_CUDA, DR_ERR_BUDGET, DR_ERR_SINK, DR_ERR_TIMEOUT, DR_ERR_STATE = -6, -7, -8, -9, -10
DR_VERSION = 1
DR_SRC_FSDP_FLAT = 1
DR_DST_ROLLOUT_FUSED = 1
DR_F32, DR_BF16, DR_FP8_E4M3_B128 = 1, 2, 3
DR_MAX_STAGE_BUFS = 8
DR_STAGE_HOST_OFFSETS = 1
DR_STAGE_UNORDERED = 2
DR_STREAM_UNORDERED = 1
DR_STAGE_DIR_OUT, DR_STAGE_DIR_IN = 0, 1

EXPORTS = ["dr_plan_create", "dr_plan_create_host", "dr_plan_window_host", "dr_plan_query", "dr_plan_tensor", "dr_plan_segment",
           "dr_reshard", "dr_reshard_inverse", "dr_plan_group", "dr_reshard_groups", "dr_reshard_static", "dr_plan_ranges", "dr_reshard_push", "dr_reshard_stream", "dr_shard_range", "dr_stage_out", "dr_stage_in", "dr_stage_begin", "dr_stage_wait_buffer", "dr_stage_poll", "dr_stage_end", "dr_plan_destroy", "dr_strerror",
           "dr_last_error", "dr_probe_stream", "dr_host_copy", "dr_diag_bulk_wait_failures", "dr_diag_bulk_starve", "dr_ctl_create", "dr_ctl_observe", "dr_ctl_break_even", "dr_ctl_destroy"]

u8, u32, u64, i64, vp = C.c_uint8, C.c_uint32, C.c_uint64, C.c_int64, C.c_void_p


class dr_model_spec(C.Structure):
    _fields_ = [("struct_size", u32), ("version", u32), ("n_layers", u32), ("hidden", u32), ("n_q_heads", u32),
                ("n_kv_heads", u32), ("head_dim", u32), ("ffn", u32), ("vocab", u32), ("n_experts", u32),
                ("moe_ffn", u32), ("tied_embeddings", u8), ("qk_norm", u8), ("pad", u8 * 2)]


class dr_src_layout(C.Structure):
    _fields_ = [("struct_size", u32), ("kind", u32), ("dtype", u32), ("world", u32), ("rank", u32),
                ("gathered", u32), ("align_elems", u32)]


class dr_dst_layout(C.Structure):
    _fields_ = [("struct_size", u32), ("kind", u32), ("dtype", u32), ("moe_tp", u32), ("arena_align_bytes", u32),
                ("kv_replicate", u32), ("vocab_pad", u32), ("moe_ep", u32), ("moe_ep_rank", u32)]


class dr_plan_info(C.Structure):
    _fields_ = [(n, u64) for n in ("flat_elems", "shard_elems", "src_bytes", "dst_bytes", "n_tensors", "n_segments",
                                   "n_tiles", "elems_moved", "bytes_moved_fwd", "bytes_moved_inv",
                                   "quant_elems", "quant_blocks", "n_groups", "bulk_forward")]


class dr_group_desc(C.Structure):
    _fields_ = [("first_tensor", u32), ("n_tensors", u32), ("elems", u64), ("bytes_moved", u64)]


class dr_range(C.Structure):
    _fields_ = [("off", u64), ("bytes", u64)]


class dr_tensor_desc(C.Structure):
    _fields_ = [("name", C.c_char * 64), ("arena_off", u64), ("rows", u64), ("cols", u64), ("alias_of", i64),
                ("elem_size", u32), ("quantised", u32), ("scale_off", u64), ("scale_rows", u64), ("scale_cols", u64)]


class dr_segment_desc(C.Structure):
    _fields_ = [("dst_off", u64), ("src_off", u64), ("rows", u64), ("row_len", u64), ("src_row_stride", u64),
                ("dst_row_stride", u64), ("vector_bytes", u32), ("tensor", u32)]


dr_chunk_fn = C.CFUNCTYPE(C.c_int, vp, u64, u64, vp, u64)


class dr_stage_desc(C.Structure):
    _fields_ = [("struct_size", u32), ("n_bufs", u32), ("dev_ptr", vp * 8), ("bytes", u64 * 8), ("order", u32 * 8),
                ("budget_bytes", u64), ("chunk_bytes", u64), ("host_arena", vp), ("host_arena_bytes", u64),
                ("callback", dr_chunk_fn), ("user", vp), ("relay_dev", vp * 8), ("first_chunk", u64),
                ("wait_event", vp), ("ready_events", vp * 8), ("timeout_ms", u32), ("flags", u32),
                ("host_offset", u64 * 8), ("caller_stream", vp), ("done_event", vp)]


class dr_stage_stats(C.Structure):
    _fields_ = [("bytes", u64), ("chunks_done", u64), ("n_chunks", u64), ("elapsed_ms", C.c_double),
                ("link_gbs", C.c_double), ("pinned_high_water_bytes", u64), ("ready_ms", C.c_double * 8)]


class dr_stream_desc(C.Structure):
    _fields_ = [("struct_size", u32), ("flags", u32), ("host_src", vp), ("host_src_bytes", u64), ("dst_dev", vp),
                ("dst_bytes", u64), ("host_dst", vp), ("host_dst_bytes", u64), ("window_dev", vp), ("window_bytes", u64),
                ("chunk_bytes", u64), ("timeout_ms", u32), ("pad", u32), ("caller_stream", vp), ("wait_event", vp),
                ("done_event", vp)]


class dr_stream_stats(C.Structure):
    _fields_ = [("h2d_bytes", u64), ("d2h_bytes", u64), ("n_chunks", u64), ("kernels", u64), ("elapsed_ms", C.c_double)]


class dr_ctl_config(C.Structure):
    _fields_ = [("struct_size", u32), ("n_topologies", u32), ("initial", u32), ("consecutive", u32), ("dwell_steps", u32),
                ("cooldown_steps", u32), ("enter_threshold", C.c_double), ("exit_threshold", C.c_double)]


class DrError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {dr_strerror(status)} ({status}): {dr_last_error()}")


_lib = None


def lib() -> C.CDLL:
    """The loaded C-ABI library.  Raises if it has not been built: there is no other code path."""
    global _lib
    if _lib is None:
        if not os.path.exists(lib_path):
            raise ImportError(f"{lib_path} is missing: run `python -m paper_2607_22614_b200.build` "
                              "(the CUDA library is the only implementation)")
        L = C.CDLL(lib_path)
        P = C.POINTER
        L.dr_plan_create.argtypes = [P(dr_model_spec), P(dr_src_layout), P(dr_dst_layout), u32, u32, P(vp)]
        L.dr_plan_create_host.argtypes = L.dr_plan_create.argtypes
        L.dr_plan_window_host.argtypes = [vp, u64, u64, P(vp)]
        L.dr_plan_query.argtypes = [vp, P(dr_plan_info)]
        L.dr_plan_tensor.argtypes = [vp, u32, P(dr_tensor_desc)]
        L.dr_plan_segment.argtypes = [vp, u64, P(dr_segment_desc)]
        L.dr_reshard.argtypes = [vp, vp, u64, vp, u64, vp]
        L.dr_reshard_inverse.argtypes = [vp, vp, u64, vp, u64, vp]
        L.dr_reshard_static.argtypes = [vp, vp, u64, vp, u64, vp]
        L.dr_plan_ranges.argtypes = [vp, u64, P(dr_range), P(u64)]
        L.dr_reshard_push.argtypes = [vp, vp, u64, P(vp), u32, u64, vp]
        L.dr_plan_group.argtypes = [vp, u32, P(dr_group_desc)]
        L.dr_reshard_groups.argtypes = [vp, u32, u32, vp, u64, vp, u64, vp]
        L.dr_stage_out.argtypes = [vp, P(dr_stage_desc), P(dr_stage_stats)]
        L.dr_stage_in.argtypes = [vp, P(dr_stage_desc), P(dr_stage_stats)]
        L.dr_stage_begin.argtypes = [vp, P(dr_stage_desc), C.c_int, P(vp)]
        L.dr_stage_wait_buffer.argtypes = [vp, u32, u32]
        L.dr_stage_poll.argtypes = [vp, P(C.c_int)]
        L.dr_stage_end.argtypes = [vp, P(dr_stage_stats)]
        L.dr_reshard_stream.argtypes = [vp, P(dr_stream_desc), P(dr_stream_stats)]
        L.dr_plan_destroy.argtypes = [vp]
        L.dr_shard_range.argtypes = [u64, u32, u32, P(u64), P(u64), P(u64)]
        L.dr_probe_stream.argtypes = [u32, vp, vp, u64, vp]
        L.dr_host_copy.argtypes = [vp, vp, u64, u32]
        L.dr_diag_bulk_wait_failures.argtypes = [P(u64)]
        L.dr_diag_bulk_starve.argtypes = [C.c_int]
        L.dr_ctl_create.argtypes = [P(dr_ctl_config), P(vp)]
        L.dr_ctl_observe.argtypes = [vp, C.c_double, C.c_double, P(C.c_int32), P(u32)]
        L.dr_ctl_break_even.argtypes = [C.c_double, C.c_double, C.c_double, P(C.c_double)]
        L.dr_ctl_destroy.argtypes = [vp]
        for n in EXPORTS:
            getattr(L, n).restype = C.c_int
        L.dr_strerror.argtypes = [C.c_int]
        L.dr_strerror.restype = C.c_char_p
        L.dr_last_error.argtypes = []
        L.dr_last_error.restype = C.c_char_p
        _lib = L
    return _lib


# ---- struct helpers ----------------------------------------------------------------------------
def model_spec(spec: dict) -> dr_model_spec:
    return dr_model_spec(struct_size=C.sizeof(dr_model_spec), version=DR_VERSION, n_layers=spec["n_layers"],
                         hidden=spec["hidden"], n_q_heads=spec["n_q_heads"], n_kv_heads=spec["n_kv_heads"],
                         head_dim=spec["head_dim"], ffn=spec.get("ffn", 0), vocab=spec["vocab"],
                         n_experts=spec.get("n_experts", 0), moe_ffn=spec.get("moe_ffn", 0),
                         tied_embeddings=int(spec.get("tied", 0)), qk_norm=int(spec.get("qk_norm", 1)))


def src_layout(world=1, rank=0, gathered=True, align_elems=1) -> dr_src_layout:
    return dr_src_layout(struct_size=C.sizeof(dr_src_layout), kind=DR_SRC_FSDP_FLAT, dtype=DR_F32, world=world,
                         rank=rank, gathered=int(gathered), align_elems=align_elems)


def dst_layout(dtype=DR_BF16, arena_align_bytes=256, moe_tp=1, kv_replicate=False, vocab_pad=0, moe_ep=1,
               moe_ep_rank=0) -> dr_dst_layout:
    return dr_dst_layout(struct_size=C.sizeof(dr_dst_layout), kind=DR_DST_ROLLOUT_FUSED, dtype=dtype, moe_tp=moe_tp,
                         arena_align_bytes=arena_align_bytes, kv_replicate=int(kv_replicate), vocab_pad=vocab_pad,
                         moe_ep=moe_ep, moe_ep_rank=moe_ep_rank)


def _current_stream(stream):
    """cudaStream_t of `stream` (a torch stream, a raw handle, or None = torch's current stream)."""
    if stream is None:
        import torch
        # without a CUDA device the descriptor can still be built (argument checks); NULL = legacy default stream
        return torch.cuda.current_stream().cuda_stream if torch.cuda.is_available() else None
    return getattr(stream, "cuda_stream", stream)


def stage_desc(dev_ptrs, sizes, budget, chunk=0, order=None, host_arena=None, host_arena_bytes=0, callback=None,
               relay_dev=None, first_chunk=0, wait_event=None, ready_events=None, timeout_ms=0,
               host_offsets=None, caller_stream=None, done_event=None, unordered=False) -> dr_stage_desc:
    """Fill a dr_stage_desc.  caller_stream=None names torch's current stream: the call's first copy then waits
    for whatever has been enqueued there (the fills or kernels that produced the device buffers)."""
    d = dr_stage_desc()
    d.struct_size = C.sizeof(dr_stage_desc)
    d.n_bufs = len(dev_ptrs)
    for i, (p, n) in enumerate(zip(dev_ptrs, sizes)):
        d.dev_ptr[i] = p
        d.bytes[i] = n
    for i, o in enumerate(order if order is not None else range(len(dev_ptrs))):
        d.order[i] = o
    d.budget_bytes, d.chunk_bytes, d.first_chunk, d.timeout_ms = budget, chunk, first_chunk, timeout_ms
    d.host_arena, d.host_arena_bytes = host_arena, host_arena_bytes
    if callback is not None:
        d.callback = callback
    for i, p in enumerate(relay_dev or []):
        d.relay_dev[i] = p
    d.wait_event = wait_event
    for i, e in enumerate(ready_events or []):
        d.ready_events[i] = e
    if host_offsets is not None:
        d.flags |= DR_STAGE_HOST_OFFSETS
        for i, o in enumerate(host_offsets):
            d.host_offset[i] = o
    if unordered:
        d.flags |= DR_STAGE_UNORDERED
    else:
        d.caller_stream = _current_stream(caller_stream)
    d.done_event = done_event
    return d


# ---- the C calls, same names, status codes returned as-is ---------------------------------------
def dr_plan_create(spec, src, dst, tp, rank):
    h = vp()
    rc = lib().dr_plan_create(C.byref(spec), C.byref(src), C.byref(dst), tp, rank, C.byref(h))
    return rc, h


def dr_plan_create_host(spec, src, dst, tp, rank):
    h = vp()
    rc = lib().dr_plan_create_host(C.byref(spec), C.byref(src), C.byref(dst), tp, rank, C.byref(h))
    return rc, h


def dr_plan_window_host(plan, src_elem_lo, src_elem_hi):
    h = vp()
    return lib().dr_plan_window_host(plan, src_elem_lo, src_elem_hi, C.byref(h)), h


def dr_plan_query(plan):
    info = dr_plan_info()
    return lib().dr_plan_query(plan, C.byref(info)), info


def dr_plan_tensor(plan, i):
    t = dr_tensor_desc()
    return lib().dr_plan_tensor(plan, i, C.byref(t)), t


def dr_plan_segment(plan, i):
    s = dr_segment_desc()
    return lib().dr_plan_segment(plan, i, C.byref(s)), s


def dr_reshard(plan, src_dev, src_bytes, dst_dev, dst_bytes, cuda_stream):
    return lib().dr_reshard(plan, src_dev, src_bytes, dst_dev, dst_bytes, cuda_stream)


def dr_reshard_inverse(plan, rollout_dev, rollout_bytes, flat_dev, flat_bytes, cuda_stream):
    return lib().dr_reshard_inverse(plan, rollout_dev, rollout_bytes, flat_dev, flat_bytes, cuda_stream)


def dr_plan_group(plan, g):
    d = dr_group_desc()
    return lib().dr_plan_group(plan, g, C.byref(d)), d


def dr_reshard_groups(plan, first, count, src_dev, src_bytes, dst_dev, dst_bytes, cuda_stream):
    return lib().dr_reshard_groups(plan, first, count, src_dev, src_bytes, dst_dev, dst_bytes, cuda_stream)


def dr_plan_ranges(plan):
    """(status, [(off, bytes), ...]): the coalesced arena byte ranges the plan's repack writes."""
    n = u64()
    rc = lib().dr_plan_ranges(plan, 0, None, C.byref(n))
    if rc:
        return rc, []
    arr = (dr_range * max(n.value, 1))()
    rc = lib().dr_plan_ranges(plan, n.value, arr, C.byref(n))
    return rc, [(arr[i].off, arr[i].bytes) for i in range(n.value)]


def dr_reshard_push(plan, src_dev, src_bytes, dst_devs, dst_bytes, cuda_stream):
    arr = (vp * len(dst_devs))(*dst_devs)
    return lib().dr_reshard_push(plan, src_dev, src_bytes, arr, len(dst_devs), dst_bytes, cuda_stream)


def dr_reshard_static(plan, src_dev, src_bytes, dst_dev, dst_bytes, cuda_stream):
    """dr_reshard without any device allocation: the segment table goes into the library's fixed
    1 MiB table (at most 16 384 segments).  For workers whose memory pool owns the whole GPU, or whose
    switch must not be stalled by the device synchronisation that cudaMalloc / cudaFree imply."""
    return lib().dr_reshard_static(plan, src_dev, src_bytes, dst_dev, dst_bytes, cuda_stream)


def dr_stage_out(plan, desc):
    st = dr_stage_stats()
    return lib().dr_stage_out(plan, C.byref(desc), C.byref(st)), st


def dr_stage_in(plan, desc):
    st = dr_stage_stats()
    return lib().dr_stage_in(plan, C.byref(desc), C.byref(st)), st


def dr_stage_begin(plan, desc, direction):
    """Starts dr_stage_out / dr_stage_in on a thread of the library's own; returns (status, job handle)."""
    job = vp()
    return lib().dr_stage_begin(plan, C.byref(desc), direction, C.byref(job)), job


def dr_stage_wait_buffer(job, buffer, timeout_ms=0):
    return lib().dr_stage_wait_buffer(job, buffer, timeout_ms)


def dr_stage_poll(job):
    done = C.c_int(0)
    return lib().dr_stage_poll(job, C.byref(done)), bool(done.value)


def dr_stage_end(job):
    st = dr_stage_stats()
    return lib().dr_stage_end(job, C.byref(st)), st


def stream_desc(host_src, host_src_bytes, dst_dev, dst_bytes, window_dev, window_bytes, chunk_bytes=0, host_dst=None,
                host_dst_bytes=0, timeout_ms=0, caller_stream=None, wait_event=None, done_event=None,
                unordered=False) -> dr_stream_desc:
    """Fill a dr_stream_desc; caller_stream=None names torch's current stream (see stage_desc)."""
    return dr_stream_desc(struct_size=C.sizeof(dr_stream_desc), flags=DR_STREAM_UNORDERED if unordered else 0,
                          host_src=host_src, host_src_bytes=host_src_bytes,
                          dst_dev=dst_dev, dst_bytes=dst_bytes, host_dst=host_dst, host_dst_bytes=host_dst_bytes,
                          window_dev=window_dev, window_bytes=window_bytes, chunk_bytes=chunk_bytes, timeout_ms=timeout_ms,
                          caller_stream=None if unordered else _current_stream(caller_stream), wait_event=wait_event,
                          done_event=done_event)


def dr_reshard_stream(plan, desc):
    st = dr_stream_stats()
    return lib().dr_reshard_stream(plan, C.byref(desc), C.byref(st)), st


DR_PROBE_READ, DR_PROBE_WRITE, DR_PROBE_COPY, DR_PROBE_NARROW, DR_PROBE_WIDEN, DR_PROBE_NARROW4, DR_PROBE_WIDEN4 = range(7)


def dr_probe_stream(mode, a_dev, b_dev, n_bytes, cuda_stream):
    return lib().dr_probe_stream(mode, a_dev, b_dev, n_bytes, cuda_stream)


def dr_diag_bulk_wait_failures():
    n = u64()
    return lib().dr_diag_bulk_wait_failures(C.byref(n)), n.value


def dr_diag_bulk_starve(on):
    return lib().dr_diag_bulk_starve(int(on))


def dr_host_copy(dst_host, src_host, n_bytes, threads=0):
    return lib().dr_host_copy(dst_host, src_host, n_bytes, threads)


def dr_shard_range(flat_elems, world, rank):
    b, e, s = u64(), u64(), u64()
    rc = lib().dr_shard_range(flat_elems, world, rank, C.byref(b), C.byref(e), C.byref(s))
    return rc, b.value, e.value, s.value


def dr_ctl_create(n_topologies, initial=0, enter=0.2, exit=0.1, consecutive=3, dwell=5, cooldown=11):
    cfg = dr_ctl_config(struct_size=C.sizeof(dr_ctl_config), n_topologies=n_topologies, initial=initial,
                        consecutive=consecutive, dwell_steps=dwell, cooldown_steps=cooldown, enter_threshold=enter,
                        exit_threshold=exit)
    h = vp()
    return lib().dr_ctl_create(C.byref(cfg), C.byref(h)), h


def dr_ctl_observe(ctl, t_rollout, t_train):
    move, topo = C.c_int32(), u32()
    rc = lib().dr_ctl_observe(ctl, t_rollout, t_train, C.byref(move), C.byref(topo))
    return rc, move.value, topo.value


def dr_ctl_break_even(resize_cost_s, step_before_s, step_after_s):
    out = C.c_double()
    return lib().dr_ctl_break_even(resize_cost_s, step_before_s, step_after_s, C.byref(out)), out.value


def dr_ctl_destroy(ctl):
    return lib().dr_ctl_destroy(ctl)


def dr_plan_destroy(plan):
    return lib().dr_plan_destroy(plan)


def dr_strerror(status: int) -> str:
    return lib().dr_strerror(status).decode()


def dr_last_error() -> str:
    return lib().dr_last_error().decode()


# ---- convenience wrapper (raises instead of returning codes; still marshalling only) -------------
class StageJob:
    """A deferred stage call (dr_stage_begin): poll() tells whether the pump has returned, end() collects it."""

    def __init__(self, handle, desc):
        self.handle, self.desc = handle, desc

    def poll(self) -> bool:
        rc, done = dr_stage_poll(self.handle)
        if rc:
            raise DrError(rc, "dr_stage_poll")
        return done

    def wait_buffer(self, buffer: int, timeout_ms: int = 0) -> None:
        """Blocks until buffer `buffer` of a stage-in job is resident (dr_stage_wait_buffer)."""
        rc = dr_stage_wait_buffer(self.handle, buffer, timeout_ms)
        if rc:
            raise DrError(rc, "dr_stage_wait_buffer")

    def end(self):
        if self.handle is None:
            raise RuntimeError("job already ended")
        rc, st = dr_stage_end(self.handle)
        self.handle = None
        if rc:
            e = DrError(rc, "dr_stage_end")
            e.stats = st
            raise e
        return st


class Plan:
    """Owns one ``dr_plan``.  ``host_only=True`` builds the planner's tables without touching CUDA."""

    def __init__(self, spec: dict, *, world=1, rank=0, gathered=True, align_elems=1, tp=1, tp_rank=0,
                 dtype=DR_BF16, arena_align_bytes=256, host_only=False, moe_tp=1, kv_replicate=False, vocab_pad=0,
                 moe_ep=1, moe_ep_rank=0):
        create = dr_plan_create_host if host_only else dr_plan_create
        rc, self.handle = create(model_spec(spec), src_layout(world, rank, gathered, align_elems),
                                 dst_layout(dtype, arena_align_bytes, moe_tp, kv_replicate, vocab_pad, moe_ep,
                                            moe_ep_rank), tp, tp_rank)
        if rc:
            self.handle = None
            raise DrError(rc, "dr_plan_create")
        rc, self.info = dr_plan_query(self.handle)
        if rc:
            raise DrError(rc, "dr_plan_query")

    def window(self, src_elem_lo, src_elem_hi):
        """Host-only plan for the source window [lo, hi) (what one chunk of the streamed repack covers)."""
        rc, h = dr_plan_window_host(self.handle, src_elem_lo, src_elem_hi)
        if rc:
            raise DrError(rc, "dr_plan_window_host")
        w = Plan.__new__(Plan)
        w.handle = h
        rc, w.info = dr_plan_query(h)
        return w

    def close(self):
        if getattr(self, "handle", None):
            dr_plan_destroy(self.handle)
            self.handle = None

    __del__ = close

    def tensors(self):
        out = []
        for i in range(self.info.n_tensors):
            rc, t = dr_plan_tensor(self.handle, i)
            if rc:
                raise DrError(rc, "dr_plan_tensor")
            out.append(t)
        return out

    def segments(self):
        out = []
        for i in range(self.info.n_segments):
            rc, s = dr_plan_segment(self.handle, i)
            if rc:
                raise DrError(rc, "dr_plan_segment")
            out.append(s)
        return out

    _stream = staticmethod(_current_stream)

    def reshard(self, src, dst, stream=None):
        """src: CUDA tensor holding the flat fp32 buffer; dst: CUDA tensor holding the rollout arena."""
        rc = dr_reshard(self.handle, src.data_ptr(), src.numel() * src.element_size(), dst.data_ptr(),
                        dst.numel() * dst.element_size(), self._stream(stream))
        if rc:
            raise DrError(rc, "dr_reshard")

    def ranges(self):
        rc, out = dr_plan_ranges(self.handle)
        if rc:
            raise DrError(rc, "dr_plan_ranges")
        return out

    def reshard_push(self, src, dsts, stream=None):
        """Repack src and store the result into every arena of dsts (CUDA tensors, or raw device pointers with
        the plan's dst_bytes behind them)."""
        ptrs = [d.data_ptr() if hasattr(d, "data_ptr") else int(d) for d in dsts]
        nbytes = min([d.numel() * d.element_size() for d in dsts if hasattr(d, "numel")] or [self.info.dst_bytes])
        rc = dr_reshard_push(self.handle, src.data_ptr(), src.numel() * src.element_size(), ptrs, nbytes,
                             self._stream(stream))
        if rc:
            raise DrError(rc, "dr_reshard_push")

    def reshard_groups(self, first, count, src, dst, stream=None):
        """Repack only groups [first, first + count) (0: embed, l + 1: layer l, last: final norm and lm_head)."""
        rc = dr_reshard_groups(self.handle, first, count, src.data_ptr(), src.numel() * src.element_size(), dst.data_ptr(),
                               dst.numel() * dst.element_size(), self._stream(stream))
        if rc:
            raise DrError(rc, "dr_reshard_groups")

    def reshard_inverse(self, rollout, flat, stream=None):
        rc = dr_reshard_inverse(self.handle, rollout.data_ptr(), rollout.numel() * rollout.element_size(),
                                flat.data_ptr(), flat.numel() * flat.element_size(), self._stream(stream))
        if rc:
            raise DrError(rc, "dr_reshard_inverse")

    def reshard_stream(self, desc):
        rc, st = dr_reshard_stream(self.handle, desc)
        if rc:
            raise DrError(rc, "dr_reshard_stream")
        return st

    def stage_out(self, desc):
        rc, st = dr_stage_out(self.handle, desc)
        if rc:
            e = DrError(rc, "dr_stage_out")
            e.stats = st
            raise e
        return st

    def stage_in(self, desc):
        rc, st = dr_stage_in(self.handle, desc)
        if rc:
            e = DrError(rc, "dr_stage_in")
            e.stats = st
            raise e
        return st

    def stage_begin(self, desc, direction):
        """dr_stage_begin: the pump runs on the library's thread; returns a StageJob (keep `desc` and its buffers alive)."""
        rc, job = dr_stage_begin(self.handle, desc, direction)
        if rc:
            raise DrError(rc, "dr_stage_begin")
        return StageJob(job, desc)
