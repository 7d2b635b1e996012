"""Pins for the oracle's inverse map and shard-local mode: round trips and union-of-shards."""
import numpy as np
import pytest

import oracle
from synth.configs import BRUTE, MID

SENT = 0xDEADBEEF


def _rand_words(n, seed, nan_free=True):
    rng = np.random.default_rng(seed)
    u = rng.integers(0, 1 << 32, size=n, dtype=np.uint64).astype(np.uint32)
    if nan_free:
        nan = (u & 0x7FFFFFFF) > 0x7F800000
        u[nan] &= 0x807FFFFF
    return u


@pytest.mark.parametrize("cfg", BRUTE + MID[:1], ids=lambda c: c["name"])
@pytest.mark.parametrize("A,W", [(1, 1), (4, 3)])
def test_inverse_of_forward_is_identity_on_layout_only_plans(cfg, A, W):
    spec, T = cfg["spec"], 2
    ms = [oracle.Model(spec, align=A, world=W, tp=T, tp_rank=t, elem_size=4) for t in range(T)]
    n = ms[0].shard_elems * W
    x = _rand_words(n, 5, nan_free=False)
    back = np.full(n, SENT, dtype=np.uint32)
    for m in ms:
        arena = np.zeros(m.arena_bytes, dtype=np.uint8)
        m.forward(x, arena)
        m.inverse(arena, back)
    real = np.zeros(n, dtype=bool)
    for t in ms[0].src_tensors():
        real[t.flat_off:t.flat_off + t.rows * t.cols] = True
    assert np.array_equal(back[real], x[real])       # every parameter restored bit for bit
    assert (back[~real] == SENT).all()               # padding never written


def test_bf16_round_trip_is_widen_of_cast_and_forward_inverts_inverse():
    spec = MID[1]["spec"]
    m = oracle.Model(spec, tp=1, elem_size=2)
    x = _rand_words(m.flat_elems, 9)
    arena = np.zeros(m.arena_bytes, dtype=np.uint8)
    m.forward(x, arena)
    back = np.full(m.flat_elems, SENT, dtype=np.uint32)
    m.inverse(arena, back)
    want = ((x.astype(np.uint64) + 0x7FFF + ((x >> 16) & 1)) >> 16).astype(np.uint32) << 16  # cast pinned elsewhere
    assert np.array_equal(back, want)
    # forward(inverse(y)) == y for a NaN-free bf16 arena
    rng = np.random.default_rng(2)
    y = rng.integers(0, 256, size=m.arena_bytes, dtype=np.uint64).astype(np.uint8)
    h = y.view(np.uint16)
    nan = ((h & 0x7F80) == 0x7F80) & ((h & 0x7F) != 0)
    h[nan] &= 0xFF00
    flat = np.zeros(m.flat_elems, dtype=np.uint32)
    m.inverse(y, flat)
    y2 = np.zeros_like(y)
    m.forward(flat, y2)
    for d in m.dst_tensors():
        if d.alias_of < 0:
            sl = slice(d.arena_off, d.arena_off + d.rows * d.cols * 2)
            assert np.array_equal(y[sl], y2[sl])


@pytest.mark.parametrize("cfg", BRUTE + MID[1:], ids=lambda c: c["name"])
def test_union_of_shard_local_forwards_is_the_gathered_forward(cfg):
    spec = cfg["spec"]
    for W in (2, 3, 5):
        m = oracle.Model(spec, world=W, tp=2, tp_rank=1, elem_size=2)
        S = m.shard_elems
        x = _rand_words(W * S, 4)
        want = np.full(m.arena_bytes, 0xA5, dtype=np.uint8)
        m.forward(x, want)
        got = np.full(m.arena_bytes, 0xA5, dtype=np.uint8)
        touched = np.zeros(m.arena_bytes, dtype=np.int32)
        for r in range(W):
            one = np.full(m.arena_bytes, 0xA5, dtype=np.uint8)
            m.forward(x[r * S:(r + 1) * S].copy(), one, gathered=False, rank=r)
            m.forward(x[r * S:(r + 1) * S].copy(), got, gathered=False, rank=r)
            probe = np.zeros(m.arena_bytes, dtype=np.uint8)
            m.forward(np.full(S, 0x3F803F80, dtype=np.uint32), probe, gathered=False, rank=r)
            touched += probe != 0
        assert np.array_equal(got, want)
        assert touched.max() == 1  # no rollout byte is produced by two shards


def test_shard_local_inverse_writes_only_its_shard():
    spec = MID[2]["spec"]
    W = 4
    m = oracle.Model(spec, world=W, tp=2, tp_rank=0, elem_size=2)
    S = m.shard_elems
    rng = np.random.default_rng(8)
    arena = rng.integers(0, 120, size=m.arena_bytes, dtype=np.uint64).astype(np.uint8)  # NaN-free bf16
    full = np.full(W * S, SENT, dtype=np.uint32)
    m.inverse(arena, full)
    for r in range(W):
        shard = np.full(S, SENT, dtype=np.uint32)
        m.inverse(arena, shard, gathered=False, rank=r)
        assert np.array_equal(shard, full[r * S:(r + 1) * S])
