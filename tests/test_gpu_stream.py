"""GPU parity for the streamed repack: the flat source rests in pinned host memory and crosses the
link chunk by chunk through a small device window; arena ranges return to the host as they become
final.  Result on the device and on the host must be the oracle's forward, bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_22614_b200 as dr
from gpu_util import SENT8, dev, first_diff, make_source
from synth.configs import BRUTE, CONFIGS, MID

pytestmark = pytest.mark.gpu
B = dr.binding

CASES = [
    (MID[0]["spec"], dict(tp=2, tp_rank=1), 999_968, 2),                       # dense, strided segments, ragged chunks
    (MID[0]["spec"], dict(tp=1), 4 << 20, 3),                                   # contiguous, three slots
    (MID[2]["spec"], dict(tp=2, tp_rank=0), 1 << 20, 2),                        # MoE: arena order differs from flat order
    (MID[2]["spec"], dict(tp=4, tp_rank=3, moe_tp=4, moe_ep=2, moe_ep_rank=1, vocab_pad=64), 3 << 19, 2),
    (MID[1]["spec"], dict(tp=2, tp_rank=0, world=3, rank=1, gathered=False, align=4), 777_760, 2),  # shard-local source
    (BRUTE[0]["spec"], dict(tp=2, tp_rank=1, align=3), 64, 4),                  # scalar runs, 16-element chunks
    (CONFIGS[0]["spec"], dict(world=2, rank=0, gathered=False), 512 << 10, 2),
]


@pytest.mark.parametrize("spec,kw,chunk,slots", CASES, ids=[f"s{i}" for i in range(len(CASES))])
@pytest.mark.parametrize("dtype", [dr.DR_BF16, dr.DR_F32])
def test_streamed_repack_equals_oracle(spec, kw, chunk, slots, dtype):
    kw = dict(kw)
    world, rank, gathered, align = kw.pop("world", 1), kw.pop("rank", 0), kw.pop("gathered", True), kw.pop("align", 1)
    es = 2 if dtype == dr.DR_BF16 else 4
    om = oracle.Model(spec, align=align, world=world, elem_size=es, **kw)
    src = make_source(world * om.shard_elems, 77)
    local = src if gathered else src[rank * om.shard_elems:(rank + 1) * om.shard_elems].copy()
    want = np.full(om.arena_bytes, SENT8, dtype=np.uint8)
    om.forward(local, want, gathered=gathered, rank=rank)
    plan = dr.Plan(spec, world=world, rank=rank, gathered=gathered, align_elems=align, dtype=dtype, **kw)
    h_src = torch.from_numpy(local.view(np.int32)).pin_memory()
    h_dst = torch.full((om.arena_bytes,), SENT8, dtype=torch.uint8).pin_memory()
    arena = torch.full((om.arena_bytes,), SENT8, dtype=torch.uint8, device=dev())
    window = torch.empty(chunk * slots, dtype=torch.uint8, device=dev())
    d = dr.stream_desc(h_src.data_ptr(), local.nbytes, arena.data_ptr(), om.arena_bytes, window.data_ptr(), chunk * slots,
                       chunk_bytes=chunk, host_dst=h_dst.data_ptr(), host_dst_bytes=om.arena_bytes)
    for _ in range(2):  # the second call re-uses the per-chunk tables
        st = plan.reshard_stream(d)
        assert st.n_chunks == -(-local.nbytes // chunk) and st.h2d_bytes == local.nbytes
        assert st.d2h_bytes == om.arena_bytes
        assert first_diff(arena.cpu().numpy(), want) is None
        # the arena on the device started as sentinel, so the host copy (gaps included) equals it too
        assert first_diff(h_dst.numpy(), want) is None
    plan.close()


def test_streamed_repack_without_host_copy_and_argument_errors():
    spec = MID[1]["spec"]
    plan = dr.Plan(spec, tp=2, tp_rank=1)
    om = oracle.Model(spec, tp=2, tp_rank=1)
    src = make_source(om.flat_elems, 5)
    want = np.full(om.arena_bytes, SENT8, dtype=np.uint8)
    om.forward(src, want)
    h_src = torch.from_numpy(src.view(np.int32)).pin_memory()
    arena = torch.full((om.arena_bytes,), SENT8, dtype=torch.uint8, device=dev())
    window = torch.empty(4 << 20, dtype=torch.uint8, device=dev())
    mk = lambda **o: dr.stream_desc(**{**dict(host_src=h_src.data_ptr(), host_src_bytes=src.nbytes, dst_dev=arena.data_ptr(),
                                              dst_bytes=om.arena_bytes, window_dev=window.data_ptr(), window_bytes=4 << 20), **o})
    st = plan.reshard_stream(mk())            # default chunk = half the window
    assert st.d2h_bytes == 0 and st.n_chunks == -(-src.nbytes // (2 << 20))
    assert first_diff(arena.cpu().numpy(), want) is None
    assert dr.dr_reshard_stream(plan.handle, mk(chunk_bytes=3 << 20))[0] == B.DR_ERR_BUDGET
    assert dr.dr_reshard_stream(plan.handle, mk(chunk_bytes=1000))[0] == B.DR_ERR_INVALID       # not a multiple of 32
    assert dr.dr_reshard_stream(plan.handle, mk(host_src_bytes=src.nbytes - 4))[0] == B.DR_ERR_SIZE
    assert dr.dr_reshard_stream(plan.handle, mk(window_dev=window.data_ptr() + 8))[0] == B.DR_ERR_ALIGN
    host_plan = dr.Plan(spec, tp=2, tp_rank=1, host_only=True)
    assert dr.dr_reshard_stream(host_plan.handle, mk())[0] == B.DR_ERR_STATE
    plan.close()


def test_streamed_repack_is_ordered_after_pending_work_on_the_callers_stream():
    """The call's own streams are non-blocking, so the library orders them after the caller's stream on entry.
    A long queue of arena and window fills is still running on a side stream when the call begins; without the
    ordering the first repacked chunks would be overwritten by the late fills.  With a timing event recorded
    after the call returns we also check that the fills really were still pending when the call was made."""
    spec = MID[0]["spec"]
    plan = dr.Plan(spec)
    om = oracle.Model(spec)
    src = make_source(om.flat_elems, 9)
    want = np.full(om.arena_bytes, SENT8, dtype=np.uint8)
    om.forward(src, want)
    h_src = torch.from_numpy(src.view(np.int32)).pin_memory()
    chunk, slots = 1 << 20, 4
    side = torch.cuda.Stream()
    big = torch.empty(1 << 30, dtype=torch.uint8, device=dev())
    arena = big[:om.arena_bytes]
    window = torch.empty(chunk * slots, dtype=torch.uint8, device=dev())
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        for i in range(60):            # about 60 x 1 GiB of fills: tens of milliseconds of queued work
            big.fill_(i)
            window.fill_(i)
        big.fill_(SENT8)
        queued = torch.cuda.Event()
        queued.record()
        d = dr.stream_desc(h_src.data_ptr(), src.nbytes, arena.data_ptr(), om.arena_bytes, window.data_ptr(), chunk * slots,
                           chunk_bytes=chunk)   # caller_stream = torch's current stream = side
        still_pending = not queued.query()
        plan.reshard_stream(d)
    assert still_pending, "the fills finished before the call: the test did not exercise the ordering"
    assert first_diff(arena.cpu().numpy(), want) is None
    plan.close()


def test_no_bounded_device_wait_ran_out():
    """The repack kernels wait for their bulk copies on an mbarrier with an iteration limit and fall back to the
    register path if the wait runs out.  After everything this process has launched so far that must never have
    happened (a fallback would still give the right bytes, but would point at a broken pipeline)."""
    plan = dr.Plan(MID[0]["spec"])
    src = torch.zeros(plan.info.src_bytes // 4, dtype=torch.int32, device=dev())
    arena = torch.zeros(plan.info.dst_bytes, dtype=torch.uint8, device=dev())
    plan.reshard(src, arena)
    plan.reshard_inverse(arena, src)
    torch.cuda.synchronize()
    rc, n = dr.dr_diag_bulk_wait_failures()
    assert rc == 0 and n == 0
    plan.close()


def test_a_bulk_wait_that_runs_out_falls_back_to_the_register_path(monkeypatch):
    """With the test hook on, every tile of the bulk-copy kernel waits for bytes that never come: the wait gives up
    after about 50 ms, the counter goes up by one per tile, the tile is redone through registers and the arena is
    still the oracle's.  Nothing faults or hangs; with the hook off again the next call is an ordinary one."""
    import time
    spec = CONFIGS[0]["spec"]                                  # 1.98 M elements at TP = 1: 161 tiles, all resident at once
    om = oracle.Model(spec)
    src = make_source(om.flat_elems, 12)
    want = np.full(om.arena_bytes, SENT8, dtype=np.uint8)
    om.forward(src, want)
    monkeypatch.setenv("DR_FORWARD_KERNEL", "bulk")           # a plan this small would take the register kernel
    plan = dr.Plan(spec)
    assert plan.info.bulk_forward == 1
    s_dev = torch.from_numpy(src.view(np.int32)).to(dev())
    arena = torch.full((om.arena_bytes,), SENT8, dtype=torch.uint8, device=dev())
    torch.cuda.synchronize()
    rc, before = dr.dr_diag_bulk_wait_failures()
    assert rc == 0 and dr.dr_diag_bulk_starve(1) == 0
    try:
        t0 = time.perf_counter()
        plan.reshard(s_dev, arena)
        torch.cuda.synchronize()
        took = time.perf_counter() - t0
    finally:
        assert dr.dr_diag_bulk_starve(0) == 0
    rc, after = dr.dr_diag_bulk_wait_failures()
    assert first_diff(arena.cpu().numpy(), want) is None
    assert after - before == plan.info.n_tiles and 0.05 < took < 5.0
    arena.fill_(SENT8)
    plan.reshard(s_dev, arena)                                  # hook off: the ordinary path, no new failures
    torch.cuda.synchronize()
    assert first_diff(arena.cpu().numpy(), want) is None
    assert dr.dr_diag_bulk_wait_failures()[1] == after
    plan.close()
