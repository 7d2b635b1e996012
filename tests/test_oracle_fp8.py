"""Pins for the oracle's fp8 block-scaled cast (D7): the e4m3 conversion against torch's float8_e4m3fn
and against the format's definition, the block quantisation against torch amax / divide / convert."""
import numpy as np
import pytest
import torch

import oracle
from synth.configs import BRUTE, MID
from torch_layout import named_params, rollout_state

F8 = torch.float8_e4m3fn
QUANT = ("qkv", "o", "gate_up", "down", "w13", "w2")


def _f32_bits(x):
    return np.asarray(x, dtype=np.float32).view(np.uint32)


def test_all_codes_decode_like_torch_and_round_trip():
    codes = np.arange(256, dtype=np.uint8)
    tv = torch.from_numpy(codes).view(F8).to(torch.float32).numpy()
    for c in codes:
        v = oracle.e4m3_value(int(c))
        if (c & 0x7F) == 0x7F:
            assert np.isnan(v) and np.isnan(tv[c])
            continue
        assert v == tv[c]
        want = int(c) if v != 0 else int(c) & 0x80
        assert oracle.cast_e4m3(int(_f32_bits(v))) == want
    assert oracle.e4m3_value(0x7E) == 448.0 and oracle.e4m3_value(0x08) == 2.0 ** -6 and oracle.e4m3_value(0x01) == 2.0 ** -9


def test_conversion_matches_torch_on_in_range_values_and_ties():
    rng = np.random.default_rng(0)
    x = np.concatenate([
        rng.normal(0, 100, 50_000), rng.normal(0, 1, 50_000), rng.normal(0, 0.01, 50_000),
        rng.uniform(-448, 448, 50_000)]).astype(np.float32)
    x = x[np.abs(x) <= 448]
    # every midpoint between neighbouring codes (exact ties), both signs
    vals = np.array(sorted(v for v in (oracle.e4m3_value(c) for c in range(0x7F))), dtype=np.float64)
    mids = ((vals[:-1] + vals[1:]) / 2).astype(np.float32)
    x = np.concatenate([x, mids, -mids, np.nextafter(mids, np.float32(0)), np.nextafter(mids, np.float32(1e9))])
    want = torch.from_numpy(x).to(F8).view(torch.uint8).numpy()
    got = np.array([oracle.cast_e4m3(int(b)) for b in x.view(np.uint32)], dtype=np.uint8)
    assert np.array_equal(got, want)
    # a tie goes to the code with an even mantissa
    for m, lo, hi in zip(mids[:40], vals[:40], vals[1:41]):
        c = oracle.cast_e4m3(int(_f32_bits(m)))
        assert c & 1 == 0 and oracle.e4m3_value(c) in (np.float32(lo), np.float32(hi))


def test_saturation_nan_and_tiny_values():
    assert oracle.cast_e4m3(int(_f32_bits(449.0))) == 0x7E
    assert oracle.cast_e4m3(int(_f32_bits(-1e30))) == 0xFE
    assert oracle.cast_e4m3(0x7F800000) == 0x7E and oracle.cast_e4m3(0xFF800000) == 0xFE   # infinities saturate
    assert oracle.cast_e4m3(0x7FC00000) == 0x7F and oracle.cast_e4m3(0xFFC00001) == 0x7F   # NaN
    assert oracle.cast_e4m3(int(_f32_bits(2.0 ** -10))) == 0x00          # tie between 0 and 2^-9 -> even (0)
    assert oracle.cast_e4m3(int(_f32_bits(1.5 * 2.0 ** -9))) == 0x02     # tie between codes 1 and 2 -> even (2)
    assert oracle.cast_e4m3(int(_f32_bits(-0.0))) == 0x80
    assert oracle.cast_e4m3(int(_f32_bits(464.0))) == 0x7E


def _torch_block_quant(x):
    """x: 2-D float32 tensor -> (uint8 codes, float32 scales) with torch ops on 128 x 128 blocks."""
    rows, cols = x.shape
    nbr, nbc = -(-rows // 128), -(-cols // 128)
    q = torch.empty(rows, cols, dtype=torch.uint8)
    s = torch.empty(nbr, nbc, dtype=torch.float32)
    for bi in range(nbr):
        for bj in range(nbc):
            blk = x[bi * 128:(bi + 1) * 128, bj * 128:(bj + 1) * 128]
            amax = blk.abs().amax()
            scale = amax / torch.tensor(448.0, dtype=torch.float32)
            recip = torch.tensor(448.0, dtype=torch.float32) / amax
            if amax == 0:
                scale = recip = torch.tensor(1.0)
            s[bi, bj] = scale
            q[bi * 128:(bi + 1) * 128, bj * 128:(bj + 1) * 128] = (blk * recip).to(F8).view(torch.uint8)
    return q, s


@pytest.mark.parametrize("spec,T", [(MID[1]["spec"], 2), (MID[2]["spec"], 2), (dict(BRUTE[0]["spec"], ffn=12), 2)],
                         ids=["mid-dense-tied", "mid-moe", "brute"])
def test_block_quantised_forward_equals_torch(spec, T):
    n = oracle.Model(spec).flat_elems
    rng = np.random.default_rng(5)
    vals = (rng.standard_normal(n) * 0.02).astype(np.float32)
    vals[rng.integers(0, n, 50)] = 0.0
    params = named_params(spec, torch.from_numpy(vals))
    for t in range(T):
        m = oracle.Model(spec, tp=T, tp_rank=t, arena_align=64)
        total, lay = m.fp8_layout()
        arena = np.full(total, 0xEE, dtype=np.uint8)
        m.forward_fp8(vals.view(np.uint32), arena)
        want = rollout_state(spec, params, T, t)
        pos = 0
        for d, (qz, off, soff) in zip(m.dst_tensors(), lay):
            if d.alias_of >= 0:
                continue
            assert qz == (d.name.split(".")[-1] in QUANT)
            assert off % 64 == 0 and off >= pos
            w = want[d.name].reshape(d.rows, d.cols)
            if not qz:
                got = arena[off:off + d.rows * d.cols * 2].view(np.uint16)
                assert np.array_equal(got, w.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16).ravel())
                pos = off + d.rows * d.cols * 2
                continue
            q, s = _torch_block_quant(w)
            assert np.array_equal(arena[off:off + d.rows * d.cols], q.numpy().ravel()), d.name
            nb = s.numel()
            assert soff % 64 == 0 and soff >= off + d.rows * d.cols
            assert np.array_equal(arena[soff:soff + 4 * nb].view(np.float32), s.numpy().ravel()), d.name
            pos = soff + 4 * nb
        assert total == pos


def test_zero_block_gets_unit_scale_and_nan_is_skipped_by_amax():
    spec = dict(BRUTE[0]["spec"], ffn=12)
    m = oracle.Model(spec, arena_align=64)
    src = np.zeros(m.flat_elems, dtype=np.uint32)
    total, lay = m.fp8_layout()
    arena = np.full(total, 0xEE, dtype=np.uint8)
    m.forward_fp8(src, arena)
    for d, (qz, off, soff) in zip(m.dst_tensors(), lay):
        if qz:
            assert (arena[off:off + d.rows * d.cols] == 0).all()
            assert arena[soff:soff + 4].view(np.float32)[0] == 1.0
    src[:] = _f32_bits(0.5)
    src[::7] = 0x7FC00000
    m.forward_fp8(src, arena)
    for d, (qz, off, soff) in zip(m.dst_tensors(), lay):
        if qz:
            body = arena[off:off + d.rows * d.cols]
            assert set(np.unique(body)) <= {0x7E, 0x7F}                  # 0.5 * (448 / 0.5) = 448; NaN stays NaN
            assert arena[soff:soff + 4].view(np.float32)[0] == np.float32(0.5) / np.float32(448)
