"""Pins for the oracle's fp8 block-scaled cast (D7): the e4m3 conversion against torch's float8_e4m3fn
and against the format's definition; the block quantisation against torch amax / divide / convert and,
without repeating any formula, against what quantisation has to guarantee (the code is a nearest e4m3
value of x / scale found by brute force over all codes in float64, zeros stay zeros, the block maximum
lands on 448, tiny blocks stay finite); the inverse against an exact float64 product."""
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
            scale = (amax / torch.tensor(448.0, dtype=torch.float32)).clamp(min=2.0 ** -126)
            s[bi, bj] = scale
            q[bi * 128:(bi + 1) * 128, bj * 128:(bj + 1) * 128] = (blk / scale).to(F8).view(torch.uint8)
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


def _blocks(m, arena, lay):
    """(name, rows, cols, codes[rows, cols], scales[nbr, nbc]) of every quantised rollout tensor."""
    for d, (qz, off, soff) in zip(m.dst_tensors(), lay):
        if qz and d.alias_of < 0:
            nbr, nbc = -(-d.rows // 128), -(-d.cols // 128)
            yield (d.name, d.rows, d.cols, arena[off:off + d.rows * d.cols].reshape(d.rows, d.cols),
                   arena[soff:soff + 4 * nbr * nbc].view(np.float32).reshape(nbr, nbc))


# every finite e4m3 value, from torch's own decoding of the 256 codes
_CODE_VALUES = torch.arange(256, dtype=torch.uint8).view(F8).to(torch.float64).numpy()
_FINITE = np.sort(_CODE_VALUES[np.isfinite(_CODE_VALUES) & (_CODE_VALUES >= 0)])


def _check_quantisation_guarantees(spec, T, t, vals, expect_unclamped=True):
    """What any correct block quantiser must deliver, checked in float64 with no reference to how the oracle
    computes it: every code is a nearest representable value of x / scale (brute force over the codes),
    zeros keep code 0, the block's largest magnitude decodes to 448 * scale, nothing is NaN."""
    m = oracle.Model(spec, tp=T, tp_rank=t, arena_align=64)
    total, lay = m.fp8_layout()
    arena = np.full(total, 0xEE, dtype=np.uint8)
    m.forward_fp8(vals.view(np.uint32), arena)
    params = named_params(spec, torch.from_numpy(vals))
    want = rollout_state(spec, params, T, t)
    n_blocks = 0
    for name, rows, cols, codes, scales in _blocks(m, arena, lay):
        x = want[name].reshape(rows, cols).numpy().astype(np.float64)
        sc = np.repeat(np.repeat(scales.astype(np.float64), 128, 0), 128, 1)[:rows, :cols]
        assert np.isfinite(scales).all() and (scales >= 2.0 ** -126).all(), name
        y = x / sc                                                   # exact enough: float64
        v = _CODE_VALUES[codes]
        assert np.isfinite(v).all(), f"{name}: a NaN code for a finite input"
        assert (np.sign(v) == np.sign(y))[(v != 0)].all()
        # distance to the chosen code vs distance to the best code, with the fp32 division's rounding as slack
        ay = np.minimum(np.abs(y), 448.0)
        k = np.clip(np.searchsorted(_FINITE, ay), 1, _FINITE.size - 1)
        best = np.minimum(np.abs(ay - _FINITE[k - 1]), np.abs(ay - _FINITE[k]))
        assert (np.abs(ay - np.abs(v)) <= best + ay * 2.0 ** -22).all(), name
        assert (codes[x == 0] & 0x7F == 0).all(), f"{name}: a zero did not stay zero"
        for bi in range(scales.shape[0]):
            for bj in range(scales.shape[1]):
                blk = np.abs(x[bi * 128:(bi + 1) * 128, bj * 128:(bj + 1) * 128])
                vb = np.abs(v[bi * 128:(bi + 1) * 128, bj * 128:(bj + 1) * 128])
                n_blocks += 1
                if scales[bi, bj] > 2.0 ** -126:
                    assert vb.flat[blk.argmax()] == 448.0, name      # the block maximum uses the whole range
                    assert abs(scales[bi, bj] * 448.0 / blk.max() - 1) < 2.0 ** -22
                else:                                                # held at 2^-126 only where amax / 448 is below it
                    assert not expect_unclamped and blk.max() / 448.0 <= 2.0 ** -126 * (1 + 2.0 ** -22)
                # dequantised error: at most half a code step (relative 1/16 in the normal range, 2^-10 below)
                err = np.abs(vb * scales[bi, bj] - blk)
                assert (err <= np.maximum(blk / 16, scales[bi, bj] * 2.0 ** -10) * (1 + 1e-6)).all(), name
    assert n_blocks > 0


@pytest.mark.parametrize("spec,T", [(MID[1]["spec"], 2), (MID[2]["spec"], 2), (dict(BRUTE[0]["spec"], ffn=12), 2)],
                         ids=["mid-dense-tied", "mid-moe", "brute"])
def test_quantisation_guarantees_on_weight_like_values(spec, T):
    n = oracle.Model(spec).flat_elems
    rng = np.random.default_rng(11)
    vals = (rng.standard_normal(n) * 0.02).astype(np.float32)
    vals[rng.integers(0, n, n // 50)] = 0.0
    for t in range(T):
        _check_quantisation_guarantees(spec, T, t, vals)


def test_blocks_of_subnormals_with_embedded_zeros_stay_finite_and_zeros_stay_zero():
    """amax / 448 underflows here: the scale is held at the smallest normal fp32, nothing turns into NaN,
    zeros keep code 0 and the dequantised error stays below half a step of the (clamped) scale."""
    spec = MID[1]["spec"]
    n = oracle.Model(spec).flat_elems
    rng = np.random.default_rng(12)
    for sigma in (1e-41, 3e-39, 1e-35):                  # subnormal / around FLT_MIN / scale just above FLT_MIN
        vals = (rng.standard_normal(n) * sigma).astype(np.float32)
        vals[rng.integers(0, n, n // 10)] = 0.0
        _check_quantisation_guarantees(spec, 1, 0, vals, expect_unclamped=sigma > 1e-36)
    m = oracle.Model(spec, arena_align=64)
    total, lay = m.fp8_layout()
    arena = np.full(total, 0xEE, dtype=np.uint8)
    vals = (rng.standard_normal(n) * 1e-41).astype(np.float32)
    m.forward_fp8(vals.view(np.uint32), arena)
    for name, rows, cols, codes, scales in _blocks(m, arena, lay):
        assert (scales == np.float32(2.0 ** -126)).all() and (codes & 0x7F <= 4).all()   # |x| / 2^-126 stays below 2^-7


def test_zero_block_nan_and_infinity():
    spec = dict(BRUTE[0]["spec"], ffn=12)
    m = oracle.Model(spec, arena_align=64)
    src = np.zeros(m.flat_elems, dtype=np.uint32)
    total, lay = m.fp8_layout()
    arena = np.full(total, 0xEE, dtype=np.uint8)
    m.forward_fp8(src, arena)
    for name, rows, cols, codes, scales in _blocks(m, arena, lay):
        assert (codes == 0).all() and (scales == np.float32(2.0 ** -126)).all()   # all-zero block: codes 0, a usable scale
    src[:] = _f32_bits(0.5)
    src[::7] = 0x7FC00000
    m.forward_fp8(src, arena)
    for name, rows, cols, codes, scales in _blocks(m, arena, lay):
        assert set(np.unique(codes)) <= {0x7E, 0x7F}                  # NaN is skipped by amax and stays NaN; 0.5 -> 448
        assert (scales == np.float32(0.5) / np.float32(448)).all()
    src[:] = _f32_bits(3.0)
    src[::5] = 0x7F800000                                             # +Inf in every block
    src[1::5] = 0xFF800000
    m.forward_fp8(src, arena)
    for name, rows, cols, codes, scales in _blocks(m, arena, lay):
        assert (scales == np.finfo(np.float32).max).all()             # the scale stays finite
        assert set(np.unique(codes)) <= {0x00, 0x7E, 0xFE}            # infinities saturate, finite values vanish


@pytest.mark.parametrize("spec,T", [(MID[2]["spec"], 2), (dict(BRUTE[0]["spec"], ffn=12), 1)], ids=["mid-moe", "brute"])
def test_inverse_fp8_is_the_exactly_rounded_product_of_code_value_and_scale(spec, T):
    """value(code) * scale has at most 28 significant bits, so float64 holds it exactly and one conversion to
    float32 rounds it once: that is the expected word.  bf16 tensors are widened; unmapped words are kept."""
    rng = np.random.default_rng(3)
    for t in range(T):
        m = oracle.Model(spec, tp=T, tp_rank=t, arena_align=64)
        total, lay = m.fp8_layout()
        arena = rng.integers(0, 256, size=total, dtype=np.uint64).astype(np.uint8)        # every code, NaN codes too
        for name, rows, cols, codes, scales in _blocks(m, arena, lay):
            scales[...] = np.exp(rng.uniform(-20, 5, scales.shape)).astype(np.float32)
        flat = np.full(m.flat_elems, 0xDEADBEEF, dtype=np.uint32)
        m.inverse_fp8(arena, flat)
        seen = np.zeros(m.flat_elems, dtype=bool)
        for i, (d, (qz, off, soff)) in enumerate(zip(m.dst_tensors(), lay)):
            if d.alias_of >= 0:
                continue
            f = m.map_rows(i, 0, d.rows, d.cols)
            ok = f >= 0
            seen[f[ok]] = True
            if not qz:
                b = arena[off:off + d.rows * d.cols * 2].view(np.uint16).reshape(d.rows, d.cols)
                assert np.array_equal(flat[f[ok]], b[ok].astype(np.uint32) << 16)
                continue
            codes = arena[off:off + d.rows * d.cols].reshape(d.rows, d.cols)
            nbr, nbc = -(-d.rows // 128), -(-d.cols // 128)
            sc = arena[soff:soff + 4 * nbr * nbc].view(np.float32).reshape(nbr, nbc).astype(np.float64)
            sc = np.repeat(np.repeat(sc, 128, 0), 128, 1)[:d.rows, :d.cols]
            with np.errstate(invalid="ignore"):
                want = (_CODE_VALUES[codes] * sc).astype(np.float32)
            got = flat[f[ok]].view(np.float32)
            nan = np.isnan(want[ok])
            assert np.array_equal(got[~nan].view(np.uint32), want[ok][~nan].view(np.uint32)), d.name
            assert (flat[f[ok]][nan] == 0x7FC00000).all()
        assert (flat[~seen] == 0xDEADBEEF).all()
