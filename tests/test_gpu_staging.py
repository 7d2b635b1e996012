"""GPU parity for the chunked staging engine: byte-exact against the oracle's staging model on every
sink (pageable arena, pinned arena, callback, relay), chunk geometry, resume after an injected
failure, weights-first ordering, and overlap with the repack."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
import paper_2607_22614_b200 as dr
import synth
from gpu_util import dev, to_dev_u32
from synth.configs import CONFIGS, MID, MiB

pytestmark = pytest.mark.gpu
B = dr.binding


def _state(n_elems, seed, bufs=(synth.BUF_ADAM_M, synth.BUF_ADAM_V)):
    host = [synth.fill_f32(seed, b, 0, n_elems) for b in bufs]
    return host, [to_dev_u32(h) for h in host]


@pytest.fixture(scope="module")
def plan():
    p = dr.Plan(CONFIGS[0]["spec"], world=2, rank=0, gathered=False)
    yield p
    p.close()


def test_tiny_workload_stage_out_and_in_pageable_arena(plan):
    """Adam m and v of rank 0's shard, 1 MiB budget: 16 chunks of 512 KiB through a two-slot ring."""
    S = plan.info.shard_elems
    host, devs = _state(S, synth.SEED_BASE)
    want_sink, want_sizes = oracle.stage_out([h.view(np.uint8) for h in host], 1 * MiB)
    arena = np.zeros(want_sink.size + 64, dtype=np.uint8)
    arena[-64:] = 0x5A
    d = dr.stage_desc([t.data_ptr() for t in devs], [4 * S, 4 * S], budget=1 * MiB, host_arena=arena.ctypes.data,
                      host_arena_bytes=want_sink.size)
    st = plan.stage_out(d)
    assert np.array_equal(arena[:-64], want_sink) and (arena[-64:] == 0x5A).all()
    assert st.n_chunks == st.chunks_done == len(want_sizes) == 16
    assert st.bytes == want_sink.size == 7_903_232
    assert 0 < st.pinned_high_water_bytes <= 1 * MiB
    # stage back in, v first this time
    back = [torch.zeros_like(t) for t in devs]
    d = dr.stage_desc([t.data_ptr() for t in back], [4 * S, 4 * S], budget=1 * MiB, order=[1, 0],
                      host_arena=arena.ctypes.data, host_arena_bytes=want_sink.size)
    st = plan.stage_in(d)
    ob = [np.zeros(4 * S, dtype=np.uint8) for _ in host]
    pieces, done = oracle.stage_in(ob, want_sink, 1 * MiB, order=[1, 0])
    assert st.chunks_done == st.n_chunks == pieces and done == [1, 0]
    for t, h, o in zip(back, host, ob):
        assert np.array_equal(t.cpu().numpy().view(np.uint32), h) and np.array_equal(o.view(np.uint32), h)
    assert 0 < st.ready_ms[1] <= st.ready_ms[0]  # buffer 1 was asked for first and is resident first


def test_pinned_arena_is_copied_to_directly(plan):
    S = 300_000
    host, devs = _state(S, 3, bufs=(0, 1, 2))
    total = 12 * S
    pinned = torch.zeros(total, dtype=torch.uint8).pin_memory()
    d = dr.stage_desc([t.data_ptr() for t in devs], [4 * S] * 3, budget=256 * 1024, chunk=64 * 1024,
                      host_arena=pinned.data_ptr(), host_arena_bytes=total)
    st = plan.stage_out(d)
    assert st.pinned_high_water_bytes == 0 and st.n_chunks == -(-total // (64 * 1024))
    assert np.array_equal(pinned.numpy(), np.concatenate([h.view(np.uint8) for h in host]))
    back = [torch.zeros_like(t) for t in devs]
    d = dr.stage_desc([t.data_ptr() for t in back], [4 * S] * 3, budget=256 * 1024, chunk=64 * 1024,
                      host_arena=pinned.data_ptr(), host_arena_bytes=total)
    plan.stage_in(d)
    assert all(torch.equal(a, b) for a, b in zip(back, devs))


def test_callback_sink_failure_and_resume(plan):
    sizes = [100_000, 3, 250_001]  # odd sizes: chunks straddle buffers, ragged tail
    rng = np.random.default_rng(0)
    host = [rng.integers(0, 256, size=n, dtype=np.uint64).astype(np.uint8) for n in sizes]
    devs = [torch.from_numpy(h).to(dev()) for h in host]
    want, sizes_k = oracle.stage_out(host, 64 * 1024, 16 * 1024)
    got = np.zeros_like(want)
    calls = []
    fail_at = [5]

    @dr.dr_chunk_fn
    def sink(user, k, off, ptr, n):
        if k == fail_at[0]:
            return 1
        calls.append((k, off, n))
        C.memmove(got.ctypes.data + off, ptr, n)
        return 0

    d = dr.stage_desc([t.data_ptr() for t in devs], sizes, budget=64 * 1024, chunk=16 * 1024, callback=sink)
    rc, st = dr.dr_stage_out(plan.handle, d)
    assert rc == B.DR_ERR_SINK and st.chunks_done == 5 and "callback" in dr.dr_last_error()
    assert [c[0] for c in calls] == [0, 1, 2, 3, 4]
    assert np.array_equal(got[:5 * 16 * 1024], want[:5 * 16 * 1024])
    fail_at[0] = -1
    d.first_chunk = st.chunks_done
    rc, st2 = dr.dr_stage_out(plan.handle, d)
    assert rc == 0 and st2.chunks_done == st2.n_chunks == len(sizes_k)
    assert [c[0] for c in calls] == list(range(len(sizes_k)))
    assert [c[2] for c in calls] == [int(x) for x in sizes_k]
    assert np.array_equal(got, want)

    # stage-in from a callback source: the pieces asked for, in order, are the oracle's walk (buffer 2 first,
    # every buffer cut on its own, no piece straddling two buffers)
    asked = []

    @dr.dr_chunk_fn
    def source(user, k, off, ptr, n):
        asked.append((k, off, n))
        C.memmove(ptr, want.ctypes.data + off, n)
        return 0

    back = [torch.zeros_like(t) for t in devs]
    d = dr.stage_desc([t.data_ptr() for t in back], sizes, budget=64 * 1024, chunk=16 * 1024, callback=source,
                      order=[2, 0, 1])
    st = plan.stage_in(d)
    assert all(torch.equal(a, b) for a, b in zip(back, devs))
    ob = [np.zeros(n, dtype=np.uint8) for n in sizes]
    n_pieces, done, walk = oracle.stage_in(ob, want, 64 * 1024, 16 * 1024, order=[2, 0, 1], pieces=True)
    prefix = np.concatenate([[0], np.cumsum(sizes)])
    assert asked == [(i, int(prefix[b]) + pos, nb) for i, (b, pos, nb) in enumerate(walk)]
    assert st.n_chunks == n_pieces and done == [2, 0, 1]
    assert [b for b, _, _ in walk][:16] == [2] * 16      # 250 001 bytes of buffer 2 = 16 pieces, before anything else


def test_stage_in_failure_reports_the_pieces_done_and_resumes_from_there(plan):
    """A source callback that fails at piece 6: the call stops with DR_ERR_SINK, reports six pieces done (those are
    on the device, byte-exact), and a second call with first_chunk = 6 asks for exactly the remaining pieces of the
    oracle's walk and completes the state."""
    sizes = [70_001, 30_000, 55_555]
    rng = np.random.default_rng(9)
    host = [rng.integers(0, 256, size=n, dtype=np.uint64).astype(np.uint8) for n in sizes]
    stream = np.concatenate(host)
    prefix = np.concatenate([[0], np.cumsum(sizes)])
    order, chunk = [1, 2, 0], 16 * 1024
    asked, fail_at = [], [6]

    @dr.dr_chunk_fn
    def source(user, k, off, ptr, n):
        if k == fail_at[0]:
            return 7
        asked.append((k, off, n))
        C.memmove(ptr, stream.ctypes.data + off, n)
        return 0

    back = [torch.full((n,), 0xEE, dtype=torch.uint8, device=dev()) for n in sizes]
    d = dr.stage_desc([t.data_ptr() for t in back], sizes, budget=4 * chunk, chunk=chunk, callback=source, order=order)
    rc, st = dr.dr_stage_in(plan.handle, d)
    assert rc == B.DR_ERR_SINK and st.chunks_done == 6 and "piece 6" in dr.dr_last_error()
    ob = [np.zeros(n, dtype=np.uint8) for n in sizes]
    n_pieces, _, walk = oracle.stage_in(ob, stream, 4 * chunk, chunk, order=order, pieces=True)
    torch.cuda.synchronize()
    for b, pos, nb in walk[:6]:                       # what was reported done is there
        assert np.array_equal(back[b][pos:pos + nb].cpu().numpy(), host[b][pos:pos + nb])
    fail_at[0] = -1
    d.first_chunk = st.chunks_done
    rc, st2 = dr.dr_stage_in(plan.handle, d)
    assert rc == 0 and st2.chunks_done == st2.n_chunks == n_pieces
    assert asked == [(i, int(prefix[b]) + pos, nb) for i, (b, pos, nb) in enumerate(walk)]
    assert all(np.array_equal(t.cpu().numpy(), h) for t, h in zip(back, host))


def test_relay_sink_moves_state_to_other_device_buffers(plan):
    S = 1_000_003
    host, devs = _state(S, 11, bufs=(0, 1))
    relay = [torch.zeros_like(t) for t in devs]
    d = dr.stage_desc([t.data_ptr() for t in devs], [4 * S] * 2, budget=1 * MiB, chunk=128 * 1024,
                      relay_dev=[t.data_ptr() for t in relay])
    st = plan.stage_out(d)
    assert st.bytes == 8 * S and st.pinned_high_water_bytes == 1 * MiB
    assert all(torch.equal(a, b) for a, b in zip(relay, devs))


def test_ready_events_and_overlap_with_the_repack():
    """The repack kernel is enqueued first, then stage-out runs on the side stream while it executes;
    both only read the master buffer.  Stage-in then records the caller's events per buffer."""
    spec = MID[0]["spec"]
    p = dr.Plan(spec)
    N = p.info.flat_elems
    master = torch.empty(N, dtype=torch.int32, device=dev())
    synth.cuda_fill_f32(master, 5, synth.BUF_MASTER)
    m = torch.empty(N, dtype=torch.int32, device=dev())
    synth.cuda_fill_f32(m, 5, synth.BUF_ADAM_M)
    arena = torch.zeros(p.info.dst_bytes, dtype=torch.uint8, device=dev())
    produced = torch.cuda.Event()
    produced.record()
    host = np.zeros(8 * N, dtype=np.uint8)
    p.reshard(master, arena)
    d = dr.stage_desc([master.data_ptr(), m.data_ptr()], [4 * N] * 2, budget=8 * MiB, host_arena=host.ctypes.data,
                      host_arena_bytes=host.size, wait_event=produced.cuda_event)
    st = p.stage_out(d)
    torch.cuda.synchronize()
    assert np.array_equal(host.view(np.uint32)[:N], synth.fill_f32(5, synth.BUF_MASTER, 0, N))
    assert np.array_equal(host.view(np.uint32)[N:], synth.fill_f32(5, synth.BUF_ADAM_M, 0, N))
    om = oracle.Model(spec)
    want = np.zeros(om.arena_bytes, dtype=np.uint8)
    om.forward(host.view(np.uint32)[:N].copy(), want)
    assert np.array_equal(arena.cpu().numpy(), want)
    # stage-in: weights first, one event per buffer
    back = [torch.zeros_like(master), torch.zeros_like(m)]
    evs = [torch.cuda.Event(), torch.cuda.Event()]
    for e in evs:
        e.record()
    d = dr.stage_desc([t.data_ptr() for t in back], [4 * N] * 2, budget=8 * MiB, host_arena=host.ctypes.data,
                      host_arena_bytes=host.size, order=[0, 1], ready_events=[e.cuda_event for e in evs])
    st = p.stage_in(d)
    evs[0].synchronize()
    evs[1].synchronize()
    assert torch.equal(back[0], master) and torch.equal(back[1], m)
    assert 0 < st.ready_ms[0] <= st.ready_ms[1]
    p.close()


def test_staging_argument_errors(plan):
    t = torch.zeros(1024, dtype=torch.int32, device=dev())
    host = np.zeros(4096, dtype=np.uint8)
    mk = lambda **kw: dr.stage_desc([t.data_ptr()], [4096], **kw)
    assert dr.dr_stage_out(plan.handle, mk(budget=4096, chunk=4096, host_arena=host.ctypes.data, host_arena_bytes=4096))[0] == B.DR_ERR_BUDGET
    assert dr.dr_stage_out(plan.handle, mk(budget=8192, chunk=4096, host_arena=host.ctypes.data, host_arena_bytes=100))[0] == B.DR_ERR_SIZE
    assert dr.dr_stage_out(plan.handle, mk(budget=8192, chunk=4096))[0] == B.DR_ERR_INVALID
    assert dr.dr_stage_in(plan.handle, mk(budget=8192, chunk=4096, host_arena=host.ctypes.data, host_arena_bytes=4096, order=[3]))[0] == B.DR_ERR_INVALID


def test_wait_that_runs_out_returns_timeout_and_the_transfer_resumes(plan):
    """A 1 ms bound on a 256 MiB copy (about 5 ms on the link) must run out: the call reports
    DR_ERR_TIMEOUT with the chunks that did complete, the context stays usable, and resuming from
    chunks_done with a normal bound delivers the same bytes."""
    n = 256 * MiB
    t = torch.empty(n // 4 * 3, dtype=torch.int32, device=dev())
    synth.cuda_fill_f32(t, 17, synth.BUF_ADAM_M)
    pinned = torch.zeros(3 * n, dtype=torch.uint8).pin_memory()
    d = dr.stage_desc([t.data_ptr()], [3 * n], budget=2 * n, chunk=n, host_arena=pinned.data_ptr(),
                      host_arena_bytes=3 * n, timeout_ms=1)
    rc, st = dr.dr_stage_out(plan.handle, d)
    assert rc == B.DR_ERR_TIMEOUT and st.chunks_done < st.n_chunks == 3
    assert "timed out" in dr.dr_last_error()
    d.timeout_ms = 0
    d.first_chunk = st.chunks_done
    rc, st2 = dr.dr_stage_out(plan.handle, d)
    assert rc == 0 and st2.chunks_done == 3
    torch.cuda.synchronize()
    assert np.array_equal(pinned.numpy().view(np.uint32), synth.fill_f32(17, synth.BUF_ADAM_M, 0, 3 * n // 4))


def _split(flat, w):
    s = -(-flat.size // w)
    padded = np.concatenate([flat, np.full(w * s - flat.size, 0xDEAD, dtype=np.uint32)])
    return [a.copy() for a in np.split(padded, w)]


@pytest.mark.parametrize("n,w_old,w_new,pinned", [(3_000_001, 6, 4, True), (3_000_001, 4, 6, False), (1_000_000, 3, 5, False)])
def test_reshard_state_across_world_sizes_through_one_host_image(plan, n, w_old, w_new, pinned):
    """Six training GPUs become four (the paper's 6:2 -> 4:4 resize): every old rank stages its shard of
    master, m and v out to its place in a flat host image, every new rank stages its own range back in.
    Ranks run one after the other on this GPU; the result must be the oracle's re-sharding."""
    kinds = (synth.BUF_MASTER, synth.BUF_ADAM_M, synth.BUF_ADAM_V)
    flats = [synth.fill_f32(23, k, 0, n) for k in kinds]
    image = torch.zeros(3 * 4 * n, dtype=torch.uint8)
    if pinned:
        image = image.pin_memory()
    for r in range(w_old):
        rc, lo, hi, s_old = dr.dr_shard_range(n, w_old, r)
        assert rc == 0
        shards = [to_dev_u32(_split(f, w_old)[r]) for f in flats]
        d = dr.stage_desc([t.data_ptr() for t in shards], [4 * (hi - lo)] * 3, budget=1 * MiB, chunk=256 * 1024,
                          host_arena=image.data_ptr(), host_arena_bytes=image.numel(),
                          host_offsets=[4 * (k * n + lo) for k in range(3)])
        st = plan.stage_out(d)
        assert st.bytes == 12 * (hi - lo)
    want = [oracle.restage(_split(f, w_old), n, w_new) for f in flats]
    for q in range(w_new):
        rc, lo, hi, s_new = dr.dr_shard_range(n, w_new, q)
        new = [torch.zeros(s_new, dtype=torch.int32, device=dev()) for _ in kinds]
        d = dr.stage_desc([t.data_ptr() for t in new], [4 * (hi - lo)] * 3, budget=1 * MiB, chunk=256 * 1024,
                          host_arena=image.data_ptr(), host_arena_bytes=image.numel(),
                          host_offsets=[4 * (k * n + lo) for k in range(3)], order=[0, 1, 2])
        st = plan.stage_in(d)
        assert 0 < st.ready_ms[0] <= st.ready_ms[1] <= st.ready_ms[2] or hi == lo
        for k in range(3):
            assert np.array_equal(new[k].cpu().numpy().view(np.uint32), want[k][q])


def test_part_of_the_new_shard_already_on_this_gpu_moves_through_the_relay(plan):
    """Old rank 1 of 6 becomes new rank 1 of 4: the overlap of the two ranges never rests on the host."""
    n = 2_400_000
    flat = synth.fill_f32(29, synth.BUF_MASTER, 0, n)
    _, olo, ohi, _ = dr.dr_shard_range(n, 6, 1)
    _, nlo, nhi, s_new = dr.dr_shard_range(n, 4, 1)
    lo, hi = max(olo, nlo), min(ohi, nhi)
    assert lo < hi
    old = to_dev_u32(flat[olo:ohi].copy())
    new = torch.zeros(s_new, dtype=torch.int32, device=dev())
    d = dr.stage_desc([old.data_ptr() + 4 * (lo - olo)], [4 * (hi - lo)], budget=1 * MiB, chunk=128 * 1024,
                      relay_dev=[new.data_ptr() + 4 * (lo - nlo)])
    plan.stage_out(d)
    got = new.cpu().numpy().view(np.uint32)
    assert np.array_equal(got[lo - nlo:hi - nlo], flat[lo:hi])
    assert (got[:lo - nlo] == 0).all() and (got[hi - nlo:] == 0).all()


def _cut(begin, end, lo, hi):
    """[begin, end) cut at the overlap [lo, hi) it contains: (a, e, inside the overlap) pieces, empty ones dropped."""
    if hi <= lo:
        return [(begin, end, False)] if end > begin else []
    return [(a, e, inside) for a, e, inside in ((begin, lo, False), (lo, hi, True), (hi, end, False)) if e > a]


@pytest.mark.parametrize("n,w_old,w_new,pinned", [(2_400_001, 6, 4, False), (2_400_001, 6, 4, True), (1_000_003, 4, 6, False)])
def test_ranks_that_stay_relay_what_they_hold_and_rest_the_remainder_in_one_call(plan, n, w_old, w_new, pinned):
    """A change of the training world size in which GPU i is old rank i and (if i < w_new) new rank i.  Each GPU
    makes ONE stage-out call over master, m and v: the part of its old shard that lies inside its new range is
    relayed into the new buffers, the rest goes to its place in the flat host image.  One stage-in call then
    fetches what the new range still lacks.  The new shards must be the oracle's re-sharding (padding zero)."""
    kinds = (synth.BUF_MASTER, synth.BUF_ADAM_M, synth.BUF_ADAM_V)
    flats = [synth.fill_f32(53, k, 0, n) for k in kinds]
    want = [oracle.restage(_split(f, w_old), n, w_new) for f in flats]
    image = torch.zeros(3 * 4 * n, dtype=torch.uint8)
    if pinned:
        image = image.pin_memory()
    new_bufs = {}
    for i in range(w_old):                                   # every old rank, one after the other on this GPU
        _, olo, ohi, _ = dr.dr_shard_range(n, w_old, i)
        old = [to_dev_u32(_split(f, w_old)[i]) for f in flats]
        ptrs, sizes, relay, offs = [], [], [], []
        if i < w_new:
            _, nlo, nhi, s_new = dr.dr_shard_range(n, w_new, i)
            new_bufs[i] = [torch.zeros(s_new, dtype=torch.int32, device=dev()) for _ in kinds]
            lo, hi = max(olo, nlo), min(ohi, nhi)
        else:
            lo = hi = nlo = 0
        for k in range(3):                                   # up to three pieces of the old shard per state buffer
            for a, e, keep in _cut(olo, ohi, lo, hi):
                ptrs.append(old[k].data_ptr() + 4 * (a - olo))
                sizes.append(4 * (e - a))
                relay.append(new_bufs[i][k].data_ptr() + 4 * (a - nlo) if keep else None)
                offs.append(4 * (k * n + a))
        assert len(ptrs) <= dr.DR_MAX_STAGE_BUFS
        d = dr.stage_desc(ptrs, sizes, budget=1 * MiB, chunk=128 * 1024, host_arena=image.data_ptr(),
                          host_arena_bytes=image.numel(), host_offsets=offs, relay_dev=relay)
        st = plan.stage_out(d)
        assert st.bytes == 12 * (ohi - olo) and st.chunks_done == st.n_chunks
    for i in range(w_new):                                   # each new rank fetches what it does not hold yet
        _, nlo, nhi, s_new = dr.dr_shard_range(n, w_new, i)
        if i < w_old:
            _, olo, ohi, _ = dr.dr_shard_range(n, w_old, i)
            lo, hi = max(olo, nlo), min(ohi, nhi)
        else:                                                # a GPU that joins training holds nothing yet
            lo = hi = nlo
            new_bufs[i] = [torch.zeros(s_new, dtype=torch.int32, device=dev()) for _ in kinds]
        ptrs, sizes, offs = [], [], []
        for k in range(3):
            for a, e, held in _cut(nlo, nhi, lo, hi):
                if not held:
                    ptrs.append(new_bufs[i][k].data_ptr() + 4 * (a - nlo))
                    sizes.append(4 * (e - a))
                    offs.append(4 * (k * n + a))
        if ptrs:
            plan.stage_in(dr.stage_desc(ptrs, sizes, budget=1 * MiB, chunk=128 * 1024, host_arena=image.data_ptr(),
                                        host_arena_bytes=image.numel(), host_offsets=offs))
        for k in range(3):
            assert np.array_equal(new_bufs[i][k].cpu().numpy().view(np.uint32), want[k][i]), (i, k)


@pytest.mark.parametrize("chunk,slots", [(2_500_001, 3), (1 << 20, 5), (32 << 20, 3), (7 << 20, 8)])
def test_pageable_arena_with_chunks_of_several_host_copy_tasks(plan, chunk, slots):
    """Chunks larger than the 1 MiB host-copy task, of odd sizes, straddling buffers: the worker threads behind
    the pump cut them into tasks.  Rings of at most 64 MiB are filled with ordinary stores on the way in, larger
    ones (the 3 x 32 MiB case) with non-temporal stores.  The image is the oracle's concatenation and stage-in
    (v first) restores every byte."""
    sizes = [50_000_003, 4_099, 71_000_001]
    host = [synth.fill_f32(61 + i, synth.BUF_ADAM_M, 0, -(-n // 4)).view(np.uint8)[:n].copy() for i, n in enumerate(sizes)]
    devs = [torch.from_numpy(h).to(dev()) for h in host]
    total = sum(sizes)
    image = np.full(total + 64, 0x5A, dtype=np.uint8)
    d = dr.stage_desc([t.data_ptr() for t in devs], sizes, budget=chunk * slots, chunk=chunk, host_arena=image.ctypes.data,
                      host_arena_bytes=total)
    st = plan.stage_out(d)
    assert st.n_chunks == st.chunks_done == -(-total // chunk) and st.bytes == total
    assert st.pinned_high_water_bytes == chunk * slots
    assert np.array_equal(image[:total], np.concatenate(host)) and (image[total:] == 0x5A).all()
    back = [torch.zeros_like(t) for t in devs]
    d = dr.stage_desc([t.data_ptr() for t in back], sizes, budget=chunk * slots, chunk=chunk, host_arena=image.ctypes.data,
                      host_arena_bytes=total, order=[2, 0, 1])
    st = plan.stage_in(d)
    assert st.chunks_done == st.n_chunks == sum(-(-n // chunk) for n in sizes) and st.bytes == total
    assert all(torch.equal(a, b) for a, b in zip(back, devs))
    assert 0 < st.ready_ms[2] <= st.ready_ms[0] <= st.ready_ms[1]


def test_no_chunk_size_given_takes_the_small_ring_where_bytes_pass_through_it(plan):
    """chunk_bytes = 0 means budget / 2, except where the bytes pass through the ring (pageable arena, relay target) and
    budget / 2 is large: then 4 MiB chunks on the way out and 8 MiB pieces on the way in, in a ring of at most 64 MiB.
    A pinned arena and a callback keep budget / 2."""
    sizes = [60_000_003, 4_099, 41_000_001]
    host = [synth.fill_f32(71 + i, synth.BUF_ADAM_V, 0, -(-n // 4)).view(np.uint8)[:n].copy() for i, n in enumerate(sizes)]
    devs = [torch.from_numpy(h).to(dev()) for h in host]
    total = sum(sizes)
    budget = 256 * MiB
    image = np.full(total + 64, 0x5A, dtype=np.uint8)
    st = plan.stage_out(dr.stage_desc([t.data_ptr() for t in devs], sizes, budget=budget, host_arena=image.ctypes.data,
                                      host_arena_bytes=total))
    assert st.n_chunks == st.chunks_done == -(-total // (4 * MiB)) and st.bytes == total
    assert st.pinned_high_water_bytes == 64 * MiB
    assert np.array_equal(image[:total], np.concatenate(host)) and (image[total:] == 0x5A).all()
    back = [torch.zeros_like(t) for t in devs]
    st = plan.stage_in(dr.stage_desc([t.data_ptr() for t in back], sizes, budget=budget, host_arena=image.ctypes.data,
                                     host_arena_bytes=total, order=[1, 2, 0]))
    assert st.chunks_done == st.n_chunks == sum(-(-n // (8 * MiB)) for n in sizes) and st.bytes == total
    assert st.pinned_high_water_bytes == 64 * MiB
    assert all(torch.equal(a, b) for a, b in zip(back, devs))
    # relay: the same small chunks
    relay = [torch.zeros_like(t) for t in devs]
    st = plan.stage_out(dr.stage_desc([t.data_ptr() for t in devs], sizes, budget=budget,
                                      relay_dev=[t.data_ptr() for t in relay]))
    assert st.n_chunks == -(-total // (4 * MiB)) and st.pinned_high_water_bytes == 64 * MiB
    torch.cuda.synchronize()
    assert all(torch.equal(a, b) for a, b in zip(relay, devs))
    # a pinned arena is copied to directly, in chunks of budget / 2; a small budget keeps budget / 2 everywhere
    pinned = torch.empty(total, dtype=torch.uint8, pin_memory=True)
    st = plan.stage_out(dr.stage_desc([t.data_ptr() for t in devs], sizes, budget=budget, host_arena=pinned.data_ptr(),
                                      host_arena_bytes=total))
    assert st.n_chunks == -(-total // (budget // 2)) and np.array_equal(pinned.numpy(), np.concatenate(host))
    st = plan.stage_out(dr.stage_desc([t.data_ptr() for t in devs], sizes, budget=6 * MiB, host_arena=image.ctypes.data,
                                      host_arena_bytes=total))
    assert st.n_chunks == -(-total // (3 * MiB)) and st.pinned_high_water_bytes == 6 * MiB


def test_host_offset_errors(plan):
    t = torch.zeros(2048, dtype=torch.int32, device=dev())
    host = np.zeros(16384, dtype=np.uint8)
    mk = lambda offs, nbytes=host.size: dr.stage_desc([t.data_ptr(), t.data_ptr() + 4096], [4096, 4096], budget=8192, chunk=4096,
                                                      host_arena=host.ctypes.data, host_arena_bytes=nbytes, host_offsets=offs)
    assert dr.dr_stage_out(plan.handle, mk([0, 2048]))[0] == B.DR_ERR_INVALID      # regions overlap
    assert dr.dr_stage_out(plan.handle, mk([0, 14000]))[0] == B.DR_ERR_SIZE        # runs past the arena
    assert dr.dr_stage_out(plan.handle, mk([8192, 0]))[0] == 0                     # any order of regions is fine


def test_pinned_ring_allocation_failure_is_reported_and_the_plan_stays_usable(plan):
    """A budget no machine can pin: the ring allocation fails on the host side, the call returns an
    out-of-memory (or CUDA) error, nothing was copied, and the same plan still works afterwards."""
    t = torch.arange(4096, dtype=torch.int32, device=dev())
    host = np.zeros(16384, dtype=np.uint8)
    d = dr.stage_desc([t.data_ptr()], [16384], budget=1 << 47, chunk=1 << 46, host_arena=host.ctypes.data,
                      host_arena_bytes=host.size)
    rc, st = dr.dr_stage_out(plan.handle, d)
    assert rc in (B.DR_ERR_NOMEM, B.DR_ERR_CUDA) and st.bytes == 0
    assert (host == 0).all()
    d = dr.stage_desc([t.data_ptr()], [16384], budget=8192, chunk=4096, host_arena=host.ctypes.data, host_arena_bytes=host.size)
    assert plan.stage_out(d).bytes == 16384
    assert np.array_equal(host.view(np.int32), np.arange(4096, dtype=np.int32))
    # and a kernel launch after the failed allocation sees no stale error
    p2 = dr.Plan(MID[2]["spec"])
    src = torch.zeros(p2.info.src_bytes // 4, dtype=torch.int32, device=dev())
    arena = torch.zeros(p2.info.dst_bytes, dtype=torch.uint8, device=dev())
    p2.reshard(src, arena)
    torch.cuda.synchronize()
    p2.close()


def test_stage_in_and_out_are_ordered_after_pending_work_on_the_callers_stream(plan):
    """The pump copies on the plan's own non-blocking streams.  On entry it makes them wait for what the caller
    has already enqueued on caller_stream, so a fill of the target buffer that is still running cannot land
    after the first host-to-device copy, and a stage-out cannot read a buffer that is still being produced.
    The queue of fills is long enough to be still running when the calls are made (checked with an event)."""
    n = 1 << 22                                          # 4 Mi words of state at the head of a 1 GiB buffer
    host = synth.fill_f32(31, synth.BUF_ADAM_M, 0, n)
    pinned = torch.from_numpy(host.view(np.int32)).pin_memory()
    side = torch.cuda.Stream()
    big = torch.empty(1 << 28, dtype=torch.int32, device=dev())
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        for i in range(80):
            big.fill_(i)
        queued = torch.cuda.Event()
        queued.record()
        d = dr.stage_desc([big.data_ptr()], [4 * n], budget=8 * MiB, chunk=1 * MiB, host_arena=pinned.data_ptr(),
                          host_arena_bytes=4 * n)       # caller_stream defaults to the current stream: side
        pending_in = not queued.query()
        plan.stage_in(d)
    assert pending_in, "the fills finished before the call: the test did not exercise the ordering"
    got = big[:n].cpu().numpy().view(np.uint32)
    assert np.array_equal(got, host)
    assert int(big[n]) == 79                             # the rest of the buffer holds the last fill
    # stage-out: the buffer is produced by the tail of a long queue; the image must hold the final values
    out = torch.zeros(4 * n, dtype=torch.uint8).pin_memory()
    with torch.cuda.stream(side):
        for i in range(80):
            big.fill_(i)
        synth.cuda_fill_f32(big[:n], 37, synth.BUF_ADAM_V, stream=side)
        queued = torch.cuda.Event()
        queued.record()
        d = dr.stage_desc([big.data_ptr()], [4 * n], budget=8 * MiB, chunk=1 * MiB, host_arena=out.data_ptr(),
                          host_arena_bytes=4 * n, caller_stream=side)
        pending_out = not queued.query()
        plan.stage_out(d)
    assert pending_out
    assert np.array_equal(out.numpy().view(np.uint32), synth.fill_f32(37, synth.BUF_ADAM_V, 0, n))


def test_done_event_and_unordered_flag(plan):
    """done_event is recorded after the last copy; DR_STAGE_UNORDERED skips the entry ordering (the caller has
    synchronised)."""
    n = 300_000
    host, devs = _state(n, 41, bufs=(1,))
    torch.cuda.synchronize()
    image = np.zeros(4 * n, dtype=np.uint8)
    done = torch.cuda.Event()
    d = dr.stage_desc([devs[0].data_ptr()], [4 * n], budget=1 * MiB, host_arena=image.ctypes.data, host_arena_bytes=4 * n,
                      unordered=True, done_event=done.cuda_event)
    assert d.flags & B.DR_STAGE_UNORDERED and not d.caller_stream
    plan.stage_out(d)
    assert done.query()                                   # the call blocks until its copies are complete
    assert np.array_equal(image.view(np.uint32), host[0])


def test_deferred_stage_in_weights_first_while_the_caller_goes_on(plan):
    """dr_stage_begin / dr_stage_end (Sec. 3.3: only the weights at the transition, optimizer state deferred): the pump
    runs on the library's thread; the caller waits on the host for the weights alone (dr_stage_wait_buffer), works on
    them, and collects the job later.  The ordering point is taken at begin: the zero-fills queued before it cannot land
    late.  The ready events are recorded as in the blocking call; once the job has ended they have all completed."""
    sizes = [24_000_004, 64_000_004, 64_000_004]
    host = [synth.fill_f32(81 + i, synth.BUF_ADAM_M, 0, n // 4).view(np.uint8).copy() for i, n in enumerate(sizes)]
    total = sum(sizes)
    image = torch.empty(total, dtype=torch.uint8, pin_memory=True)
    image.numpy()[:] = np.concatenate(host)
    back = [torch.empty(n, dtype=torch.uint8, device=dev()) for n in sizes]
    big = torch.empty(1 << 28, dtype=torch.int32, device=dev())
    for _ in range(8):
        big.fill_(1)                       # keeps the stream busy while begin is called
    for b in back:
        b.zero_()
    ready = [torch.cuda.Event() for _ in sizes]
    d = dr.stage_desc([b.data_ptr() for b in back], sizes, budget=8 * MiB, host_arena=image.data_ptr(),
                      host_arena_bytes=total, order=[0, 1, 2], ready_events=[e.cuda_event for e in ready])
    job = plan.stage_begin(d, dr.DR_STAGE_DIR_IN)
    job.wait_buffer(0)                                         # the weights: resident, usable by anything enqueued from here on
    doubled = back[0].to(torch.int32) * 2                      # the caller's work on them
    job.wait_buffer(1, timeout_ms=30000)
    st = job.end()
    assert all(e.query() for e in ready)
    torch.cuda.synchronize()
    assert st.bytes == total and st.chunks_done == st.n_chunks
    assert 0 < st.ready_ms[0] <= st.ready_ms[1] <= st.ready_ms[2] <= st.elapsed_ms
    assert all(np.array_equal(b.cpu().numpy(), h) for b, h in zip(back, host))
    assert np.array_equal(doubled.cpu().numpy(), host[0].astype(np.int32) * 2)


def test_deferred_stage_out_reports_a_failing_sink_at_end_and_jobs_on_one_plan_run_in_turn(plan):
    n = 6_000_000
    host = [synth.fill_f32(91 + i, synth.BUF_ADAM_V, 0, n // 4).view(np.uint8).copy() for i in range(2)]
    devs = [torch.from_numpy(h).to(dev()) for h in host]
    images = [np.zeros(n, dtype=np.uint8) for _ in range(2)]
    torch.cuda.synchronize()
    descs = [dr.stage_desc([devs[i].data_ptr()], [n], budget=2 * MiB, chunk=MiB, host_arena=images[i].ctypes.data,
                           host_arena_bytes=n) for i in range(2)]
    jobs = [plan.stage_begin(descs[i], dr.DR_STAGE_DIR_OUT) for i in range(2)]   # both started; the plan serialises them
    stats = [j.end() for j in jobs]
    assert all(j.handle is None for j in jobs)
    for i in range(2):
        assert stats[i].bytes == n and np.array_equal(images[i], host[i])

    seen = []

    def sink(user, k, off, ptr, nbytes):
        seen.append(k)
        return 1 if k == 3 else 0

    cb = B.dr_chunk_fn(sink)
    job = plan.stage_begin(dr.stage_desc([devs[0].data_ptr()], [n], budget=2 * MiB, chunk=MiB, callback=cb), dr.DR_STAGE_DIR_OUT)
    with pytest.raises(dr.DrError) as w:
        job.wait_buffer(0)                                    # not a stage-in job
    assert w.value.status == B.DR_ERR_INVALID
    with pytest.raises(dr.DrError) as e:
        job.end()
    assert e.value.status == B.DR_ERR_SINK and e.value.stats.chunks_done == 3 and seen == [0, 1, 2, 3]
    assert "callback" in dr.dr_last_error()
    # a stage-in whose source fails: the wait for a buffer that will not arrive ends with the job's own error
    back = torch.zeros(n, dtype=torch.uint8, device=dev())

    def source(user, k, off, ptr, nbytes):
        return 1 if k == 2 else 0

    cb2 = B.dr_chunk_fn(source)
    job = plan.stage_begin(dr.stage_desc([back.data_ptr()], [n], budget=2 * MiB, chunk=MiB, callback=cb2), dr.DR_STAGE_DIR_IN)
    with pytest.raises(dr.DrError) as w:
        job.wait_buffer(0, timeout_ms=30000)
    assert w.value.status == B.DR_ERR_SINK
    with pytest.raises(dr.DrError) as e:
        job.end()
    assert e.value.status == B.DR_ERR_SINK and e.value.stats.chunks_done == 2
    # errors that need nothing started are reported by begin itself
    bad = dr.stage_desc([devs[0].data_ptr()], [n], budget=MiB, chunk=MiB, host_arena=images[0].ctypes.data, host_arena_bytes=n)
    assert dr.dr_stage_begin(plan.handle, bad, dr.DR_STAGE_DIR_OUT)[0] == B.DR_ERR_BUDGET
    assert dr.dr_stage_begin(plan.handle, descs[0], 7)[0] == B.DR_ERR_INVALID
