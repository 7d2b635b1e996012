"""GPU tests of the threading rules the header states: a plan is immutable for the dr_reshard* calls, which may
run concurrently from several threads on different streams; dr_stage_* calls on one plan are serialised inside
the library; the repack and the staging pump may run on the same plan from two threads at once.  The foreign
calls release the interpreter lock, so the threads below really overlap.  Results are compared with the oracle."""
import threading

import numpy as np
import pytest
import torch

import oracle
import paper_2607_22614_b200 as dr
import synth
from gpu_util import SENT8, dev, first_diff, make_source
from synth.configs import CONFIGS, MID

pytestmark = pytest.mark.gpu


def _run(threads):
    errs = []

    def wrap(fn):
        def go():
            try:
                fn()
            except BaseException as e:  # noqa: BLE001 - reported by the test below
                errs.append(e)
        return go

    ts = [threading.Thread(target=wrap(f)) for f in threads]
    for t in ts:
        t.start()
    for t in ts:
        t.join(timeout=120)
    assert not any(t.is_alive() for t in ts), "a thread did not finish"
    if errs:
        raise errs[0]


def test_one_plan_repacks_from_four_threads_on_four_streams():
    spec = MID[1]["spec"]
    om = oracle.Model(spec, tp=2, tp_rank=1)
    plan = dr.Plan(spec, tp=2, tp_rank=1)
    n_threads, rounds = 4, 12
    srcs = [make_source(om.shard_elems, 100 + i) for i in range(n_threads)]
    wants = []
    for s in srcs:
        w = np.full(om.arena_bytes, SENT8, dtype=np.uint8)
        om.forward(s, w)
        wants.append(w)
    backs_want = []
    for w in wants:
        b = np.full(om.shard_elems, 0xDEADBEEF, dtype=np.uint32)
        om.inverse(w, b)
        backs_want.append(b)
    d_src = [torch.from_numpy(s.view(np.int32)).to(dev()) for s in srcs]
    d_arena = [torch.full((om.arena_bytes,), SENT8, dtype=torch.uint8, device=dev()) for _ in range(n_threads)]
    d_back = [torch.full((om.shard_elems,), 0xDEADBEEF - (1 << 32), dtype=torch.int32, device=dev()) for _ in range(n_threads)]
    streams = [torch.cuda.Stream() for _ in range(n_threads)]
    torch.cuda.synchronize()

    def worker(i):
        def go():
            with torch.cuda.stream(streams[i]):
                for _ in range(rounds):
                    d_arena[i].fill_(SENT8)
                    plan.reshard(d_src[i], d_arena[i])
                    plan.reshard_inverse(d_arena[i], d_back[i])
            streams[i].synchronize()
        return go

    _run([worker(i) for i in range(n_threads)])
    for i in range(n_threads):
        assert first_diff(d_arena[i].cpu().numpy(), wants[i]) is None
        assert np.array_equal(d_back[i].cpu().numpy().view(np.uint32), backs_want[i])
    plan.close()


def test_stage_calls_on_one_plan_from_two_threads_are_serialised_and_exact():
    plan = dr.Plan(CONFIGS[0]["spec"], world=2, rank=0, gathered=False)
    n = 9_000_001
    host = [synth.fill_f32(200 + i, synth.BUF_ADAM_M, 0, -(-n // 4)).view(np.uint8)[:n].copy() for i in range(2)]
    devs = [torch.from_numpy(h).to(dev()) for h in host]
    images = [np.full(n + 32, 0x5A, dtype=np.uint8) for _ in range(2)]
    backs = [torch.zeros(n, dtype=torch.uint8, device=dev()) for _ in range(2)]
    torch.cuda.synchronize()
    stats = [None, None]

    def worker(i):
        def go():
            # different ring geometries, so that the shared ring is re-cut between the interleaved calls
            budget, chunk = ((4 << 20, 1 << 20), (6 << 20, 3 << 20))[i]
            for _ in range(4):
                out = plan.stage_out(dr.stage_desc([devs[i].data_ptr()], [n], budget=budget, chunk=chunk,
                                                   host_arena=images[i].ctypes.data, host_arena_bytes=n, unordered=True))
                assert out.bytes == n and out.chunks_done == out.n_chunks == -(-n // chunk)
                back = plan.stage_in(dr.stage_desc([backs[i].data_ptr()], [n], budget=budget, chunk=chunk,
                                                   host_arena=images[i].ctypes.data, host_arena_bytes=n, unordered=True))
                assert back.bytes == n
                stats[i] = out
        return go

    _run([worker(0), worker(1)])
    torch.cuda.synchronize()
    for i in range(2):
        budget, chunk = ((4 << 20, 1 << 20), (6 << 20, 3 << 20))[i]
        want, sizes = oracle.stage_out([host[i]], budget, chunk)
        assert stats[i].n_chunks == len(sizes)
        assert np.array_equal(images[i][:n], want) and (images[i][n:] == 0x5A).all()
        assert torch.equal(backs[i], devs[i])
    plan.close()


def test_repack_on_one_thread_while_another_stages_out_of_the_same_plan():
    """The overlap of Sec. 3.3 driven from two threads: both only read the master buffer."""
    spec = MID[0]["spec"]
    om = oracle.Model(spec)
    plan = dr.Plan(spec)
    src = make_source(om.shard_elems, 31)
    want = np.full(om.arena_bytes, SENT8, dtype=np.uint8)
    om.forward(src, want)
    master = torch.from_numpy(src.view(np.int32)).to(dev())
    arena = torch.full((om.arena_bytes,), SENT8, dtype=torch.uint8, device=dev())
    image = np.zeros(4 * om.shard_elems, dtype=np.uint8)
    side = torch.cuda.Stream()
    torch.cuda.synchronize()

    def repack():
        with torch.cuda.stream(side):
            for _ in range(50):
                plan.reshard(master, arena)
        side.synchronize()

    def stage():
        for _ in range(3):
            st = plan.stage_out(dr.stage_desc([master.data_ptr()], [4 * om.shard_elems], budget=2 << 20,
                                              host_arena=image.ctypes.data, host_arena_bytes=image.size, unordered=True))
            assert st.bytes == 4 * om.shard_elems

    _run([repack, stage])
    assert first_diff(arena.cpu().numpy(), want) is None
    assert np.array_equal(image.view(np.uint32), src)
    plan.close()
