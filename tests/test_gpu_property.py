"""GPU property test: random small shapes, layouts and variants through dr_reshard, dr_reshard_inverse and
dr_reshard_stream, each compared with the oracle bit for bit (deterministic example sequence)."""
import numpy as np
import pytest
import torch
from hypothesis import HealthCheck, given, settings

import oracle
import paper_2607_22614_b200 as dr
from gpu_util import SENT8, dev, first_diff
from test_planner_property import cases

pytestmark = pytest.mark.gpu


@settings(max_examples=60, deadline=None, derandomize=True, database=None, suppress_health_check=list(HealthCheck))
@given(cases())
def test_random_plans_on_the_gpu(c):
    es = 2 if c["dtype"] == dr.DR_BF16 else 4
    om = oracle.Model(c["spec"], align=c["align"], world=c["world"], tp=c["tp"], tp_rank=c["tp_rank"], elem_size=es,
                      arena_align=c["arena_align"], **c["opts"])
    plan = dr.Plan(c["spec"], world=c["world"], rank=c["rank"], gathered=c["gathered"], align_elems=c["align"], tp=c["tp"],
                   tp_rank=c["tp_rank"], dtype=c["dtype"], arena_align_bytes=c["arena_align"], **c["opts"])
    S, W, r, g = om.shard_elems, c["world"], c["rank"], c["gathered"]
    rng = np.random.default_rng(om.flat_elems * 31 + W)
    full = rng.integers(0, 1 << 32, size=W * S, dtype=np.uint64).astype(np.uint32)
    local = full if g else full[r * S:(r + 1) * S].copy()
    n_arena = max(om.arena_bytes, 32)
    want = np.full(n_arena, SENT8, dtype=np.uint8)
    om.forward(local, want, gathered=g, rank=r)
    src = torch.from_numpy(local.view(np.int32)).to(dev())
    arena = torch.full((n_arena,), SENT8, dtype=torch.uint8, device=dev())
    plan.reshard(src, arena)
    torch.cuda.synchronize()
    assert first_diff(arena.cpu().numpy(), want) is None
    # inverse of the oracle's arena into a sentinel-filled flat buffer
    wflat = np.full(local.size, 0xDEADBEEF, dtype=np.uint32)
    om.inverse(want, wflat, gathered=g, rank=r)
    flat = torch.full((local.size,), 0xDEADBEEF - (1 << 32), dtype=torch.int32, device=dev())
    plan.reshard_inverse(torch.from_numpy(want).to(dev()), flat)
    torch.cuda.synchronize()
    assert first_diff(flat.cpu().numpy().view(np.uint32), wflat) is None
    # streamed repack of the same source: 96-byte chunks through a 3-slot window
    if local.nbytes >= 32:
        h_src = torch.from_numpy(np.concatenate([local, np.zeros(8, dtype=np.uint32)]).view(np.int32)).pin_memory()
        h_dst = torch.full((n_arena,), SENT8, dtype=torch.uint8).pin_memory()
        arena2 = torch.full((n_arena,), SENT8, dtype=torch.uint8, device=dev())
        window = torch.empty(96 * 3, dtype=torch.uint8, device=dev())
        d = dr.stream_desc(h_src.data_ptr(), local.nbytes, arena2.data_ptr(), n_arena, window.data_ptr(), 96 * 3,
                           chunk_bytes=96, host_dst=h_dst.data_ptr(), host_dst_bytes=n_arena)
        plan.reshard_stream(d)
        assert first_diff(arena2.cpu().numpy(), want) is None
        assert first_diff(h_dst.numpy()[:om.arena_bytes], want[:om.arena_bytes]) is None
    plan.close()


from hypothesis import strategies as st  # noqa: E402
import ctypes as C  # noqa: E402


@st.composite
def staging_cases(draw):
    n = draw(st.integers(1, 4))
    sizes = [draw(st.integers(0, 150_000)) for _ in range(n)]
    if sum(sizes) == 0:
        sizes[0] = 777
    chunk = draw(st.integers(1, 70_000))
    slots = draw(st.integers(2, 4))
    sink = draw(st.sampled_from(["pageable", "pinned", "callback", "scattered"]))
    order = draw(st.permutations(list(range(n))))
    return dict(sizes=sizes, chunk=chunk, budget=chunk * slots + draw(st.integers(0, chunk - 1)), sink=sink, order=list(order))


@settings(max_examples=40, deadline=None, derandomize=True, database=None, suppress_health_check=list(HealthCheck))
@given(staging_cases())
def test_random_staging_geometries(c):
    """Random buffer sizes (odd byte counts included), chunk sizes, slot counts, sinks and restore orders:
    the host image is the oracle's, stage-in restores every byte."""
    from synth.configs import CONFIGS
    plan = dr.Plan(CONFIGS[0]["spec"])
    rng = np.random.default_rng(sum(c["sizes"]) + c["chunk"])
    host = [rng.integers(0, 256, size=n, dtype=np.uint64).astype(np.uint8) for n in c["sizes"]]
    devs = [torch.from_numpy(h).to(dev()) if h.size else torch.zeros(1, dtype=torch.uint8, device=dev()) for h in host]
    ptrs = [t.data_ptr() for t in devs]
    total = sum(c["sizes"])
    want, csz = oracle.stage_out(host, c["budget"], c["chunk"])
    kw = dict(budget=c["budget"], chunk=c["chunk"])
    offsets = None
    if c["sink"] == "callback":
        got = np.zeros(total, dtype=np.uint8)
        seen = []

        @dr.dr_chunk_fn
        def sink(user, k, off, ptr, n):
            seen.append((k, n))
            C.memmove(got.ctypes.data + off, ptr, n)
            return 0

        st_out = plan.stage_out(dr.stage_desc(ptrs, c["sizes"], callback=sink, **kw))
        assert [n for _, n in seen] == [int(x) for x in csz] and [k for k, _ in seen] == list(range(len(csz)))
        image = torch.from_numpy(got)
    else:
        if c["sink"] == "scattered":  # buffers rest in reverse order, 64 bytes apart
            offsets, pos = [0] * len(host), 0
            for i in reversed(range(len(host))):
                offsets[i] = pos
                pos += c["sizes"][i] + 64
            image = torch.full((pos,), 0x5A, dtype=torch.uint8)
        else:
            image = torch.full((total + 64,), 0x5A, dtype=torch.uint8)
        if c["sink"] == "pinned":
            image = image.pin_memory()
        st_out = plan.stage_out(dr.stage_desc(ptrs, c["sizes"], host_arena=image.data_ptr(), host_arena_bytes=image.numel(),
                                              host_offsets=offsets, **kw))
        if offsets is None:
            assert np.array_equal(image.numpy()[:total], want) and (image.numpy()[total:] == 0x5A).all()
        else:
            for i, h in enumerate(host):
                assert np.array_equal(image.numpy()[offsets[i]:offsets[i] + h.size], h)
                assert (image.numpy()[offsets[i] + h.size:offsets[i] + h.size + 64] == 0x5A).all()
    assert st_out.n_chunks == st_out.chunks_done == len(csz) and st_out.bytes == total
    back = [torch.zeros_like(t) for t in devs]
    asked = []
    if c["sink"] == "callback":
        @dr.dr_chunk_fn
        def source(user, k, off, ptr, n):
            asked.append((k, off, n))
            C.memmove(ptr, want.ctypes.data + off, n)
            return 0
        st_in = plan.stage_in(dr.stage_desc([t.data_ptr() for t in back], c["sizes"], callback=source, order=c["order"], **kw))
    else:
        st_in = plan.stage_in(dr.stage_desc([t.data_ptr() for t in back], c["sizes"], host_arena=image.data_ptr(),
                                            host_arena_bytes=image.numel(), host_offsets=offsets, order=c["order"], **kw))
    ob = [np.zeros(n, dtype=np.uint8) for n in c["sizes"]]
    pieces, done, walk = oracle.stage_in(ob, want, c["budget"], c["chunk"], c["order"], pieces=True)
    assert st_in.chunks_done == st_in.n_chunks == pieces and done == c["order"]
    if c["sink"] == "callback":  # the pieces the engine asked for are the oracle's walk, in its order
        prefix = np.concatenate([[0], np.cumsum(c["sizes"])])
        assert asked == [(i, int(prefix[b]) + pos, nb) for i, (b, pos, nb) in enumerate(walk)]
    # buffers became resident in the asked order (empty buffers never report a time)
    ready = [st_in.ready_ms[b] for b in c["order"] if c["sizes"][b]]
    assert all(x > 0 for x in ready) and ready == sorted(ready)
    for b, h, o in zip(back, host, ob):
        assert np.array_equal(b.cpu().numpy()[:h.size], h) and np.array_equal(o, h)
    plan.close()
