"""Pins for the oracle's staging model (D6): the sink is the concatenation, chunk count and sizes,
stage-in inverts stage-out, resume, budget rule, completion order."""
import numpy as np
import pytest

import oracle


def _bufs(sizes, seed=0):
    rng = np.random.default_rng(seed)
    return [rng.integers(0, 256, size=n, dtype=np.uint64).astype(np.uint8) for n in sizes]


@pytest.mark.parametrize("sizes,budget,chunk", [
    ((10000, 10000), 8192, 0),          # default chunk = budget/2; a chunk straddles the boundary
    ((12345, 1, 777), 3000, 1000),      # three slots, ragged tail
    ((4096,), 8192, 4096),              # exactly one chunk
    ((5000, 0, 5000), 8192, 4096),      # an empty buffer in the middle
])
def test_stage_out_is_concatenation_and_stage_in_inverts_it(sizes, budget, chunk):
    bufs = _bufs(sizes)
    sink, csz = oracle.stage_out(bufs, budget, chunk)
    cat = np.concatenate(bufs)
    assert np.array_equal(sink, cat)
    c = chunk or budget // 2 // 4096 * 4096
    assert len(csz) == -(-cat.size // c)
    assert (csz[:-1] == c).all() and csz[-1] == cat.size - c * (len(csz) - 1)
    back = [np.zeros_like(b) for b in bufs]
    order = list(range(len(bufs)))[::-1]
    pieces, done = oracle.stage_in(back, sink, budget, chunk, order)
    assert all(np.array_equal(a, b) for a, b in zip(back, bufs))
    assert done == order
    assert pieces == sum(-(-n // c) for n in sizes)


def test_tiny_workload_chunking_matches_the_quoted_figures():
    # Adam m and v of rank 0's shard of the tiny model, 1 MiB budget: 16 chunks, last of 38 912 bytes,
    # chunk 7 straddles the m | v boundary.
    shard_bytes = 987_904 * 4
    bufs = _bufs((shard_bytes, shard_bytes), 1)
    sink, csz = oracle.stage_out(bufs, 1 << 20)
    assert len(csz) == 16 and csz[-1] == 38_912 and (csz[:-1] == 512 * 1024).all()
    assert 7 * 512 * 1024 < shard_bytes < 8 * 512 * 1024
    assert np.array_equal(sink, np.concatenate(bufs))


def test_stage_in_walks_buffers_in_order_in_pieces_that_never_straddle_hand_written():
    """The walk of stage-in, written out by hand.  Tiny workload: Adam m and v of 3 951 616 bytes each
    (7 x 524 288 + 281 600), 1 MiB budget, v asked for first: eight pieces of v, then eight of m."""
    shard_bytes = 987_904 * 4
    assert shard_bytes == 7 * 524_288 + 281_600
    bufs = _bufs((shard_bytes, shard_bytes), 2)
    back = [np.zeros_like(b) for b in bufs]
    n, done, walk = oracle.stage_in(back, np.concatenate(bufs), 1 << 20, order=[1, 0], pieces=True)
    expected = [
        (1, 0, 524_288), (1, 524_288, 524_288), (1, 1_048_576, 524_288), (1, 1_572_864, 524_288),
        (1, 2_097_152, 524_288), (1, 2_621_440, 524_288), (1, 3_145_728, 524_288), (1, 3_670_016, 281_600),
        (0, 0, 524_288), (0, 524_288, 524_288), (0, 1_048_576, 524_288), (0, 1_572_864, 524_288),
        (0, 2_097_152, 524_288), (0, 2_621_440, 524_288), (0, 3_145_728, 524_288), (0, 3_670_016, 281_600),
    ]
    assert n == 16 and walk == expected and done == [1, 0]
    assert all(np.array_equal(a, b) for a, b in zip(back, bufs))
    # three buffers of 5, 0 and 3 bytes, pieces of 2 bytes, order 2, 0, 1: the empty buffer has no piece
    bufs = _bufs((5, 0, 3), 4)
    back = [np.zeros_like(b) for b in bufs]
    n, done, walk = oracle.stage_in(back, np.concatenate(bufs), 4, 2, order=[2, 0, 1], pieces=True)
    assert walk == [(2, 0, 2), (2, 2, 1), (0, 0, 2), (0, 2, 2), (0, 4, 1)] and n == 5 and done == [2, 0, 1]
    assert all(np.array_equal(a, b) for a, b in zip(back, bufs))


def test_stage_in_walk_properties_on_random_geometries():
    """Whatever the sizes: pieces of one buffer are consecutive and cover it from 0 upwards without gaps,
    none is longer than the chunk, buffers appear in the asked order, nothing straddles."""
    rng = np.random.default_rng(8)
    for _ in range(40):
        k = int(rng.integers(1, 5))
        sizes = [int(rng.integers(0, 5000)) for _ in range(k)]
        chunk = int(rng.integers(1, 1500))
        order = [int(x) for x in rng.permutation(k)]
        bufs = _bufs(sizes, 5)
        back = [np.zeros_like(b) for b in bufs]
        n, done, walk = oracle.stage_in(back, np.concatenate(bufs) if sum(sizes) else np.zeros(1, np.uint8), 3 * chunk, chunk,
                                        order=order, pieces=True)
        assert done == order
        seen_order, cursor = [], {}
        for b, pos, nb in walk:
            if not seen_order or seen_order[-1] != b:
                assert b not in seen_order          # a buffer's pieces are consecutive
                seen_order.append(b)
            assert pos == cursor.get(b, 0) and 0 < nb <= chunk and pos + nb <= sizes[b]
            cursor[b] = pos + nb
        assert seen_order == [b for b in order if sizes[b]]
        assert all(cursor.get(b, 0) == sizes[b] for b in range(k))
        assert all(np.array_equal(a, b) for a, b in zip(back, bufs))


def test_resume_from_a_failed_chunk_gives_the_same_bytes():
    bufs = _bufs((9000, 7000), 3)
    full, csz = oracle.stage_out(bufs, 4096, 1024)
    k = 5
    partial = np.zeros_like(full)
    partial[:k * 1024] = full[:k * 1024]          # chunks < k were delivered before the failure
    sink, _ = oracle.stage_out(bufs, 4096, 1024, first_chunk=k, sink=partial)
    assert np.array_equal(sink, full)


def test_budget_must_hold_two_slots():
    bufs = _bufs((100,))
    with pytest.raises(ValueError):
        oracle.stage_out(bufs, 1000, 600)
    with pytest.raises(ValueError):
        oracle.stage_out(bufs, 4096)  # default chunk rounds down to 0


@pytest.mark.parametrize("n,w_old,w_new", [(1000, 6, 4), (1001, 4, 6), (17, 3, 5), (4096, 2, 8), (5, 8, 3)])
def test_restage_across_world_sizes_is_split_of_the_concatenation(n, w_old, w_new):
    """The new shards are what numpy's own split of the (zero padded) flat buffer gives."""
    rng = np.random.default_rng(n)
    flat = rng.integers(1, 1 << 32, size=n, dtype=np.uint64).astype(np.uint32)
    s_old, s_new = -(-n // w_old), -(-n // w_new)
    padded_old = np.concatenate([flat, np.full(w_old * s_old - n, 0xDEAD, dtype=np.uint32)])  # old padding is garbage
    old = [a.copy() for a in np.split(padded_old, w_old)]
    new = oracle.restage(old, n, w_new)
    padded_new = np.concatenate([flat, np.zeros(w_new * s_new - n, dtype=np.uint32)])
    for got, want in zip(new, np.split(padded_new, w_new)):
        assert np.array_equal(got, want)
    assert np.array_equal(np.concatenate(new)[:n], flat)
