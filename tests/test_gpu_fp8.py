"""GPU parity for the fp8 block-scaled rollout cast: payload bytes and fp32 scales must equal the
oracle's bit for bit, on seeded weights with special values, odd shapes, MoE layouts, and on sampled
tensors of the full-size Qwen3-8B-shaped workload."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_22614_b200 as dr
import synth
from gpu_util import SENT8, dev, first_diff, make_source, to_dev_u32
from synth.configs import BRUTE, CONFIGS, MID, seed_of

pytestmark = pytest.mark.gpu
B = dr.binding


def _run(spec, tp, t, src, arena_align=256, **opts):
    om = oracle.Model(spec, tp=tp, tp_rank=t, arena_align=arena_align, **opts)
    total, lay = om.fp8_layout()
    want = np.full(total, SENT8, dtype=np.uint8)
    om.forward_fp8(src, want)
    plan = dr.Plan(spec, tp=tp, tp_rank=t, dtype=dr.DR_FP8_E4M3_B128, arena_align_bytes=arena_align, **opts)
    assert plan.info.dst_bytes == total
    arena = torch.full((total,), SENT8, dtype=torch.uint8, device=dev())
    plan.reshard(to_dev_u32(src), arena)
    torch.cuda.synchronize()
    return arena.cpu().numpy(), want, plan, om, lay


CASES = [(MID[0]["spec"], 2, {}), (MID[1]["spec"], 4, dict(vocab_pad=64)), (MID[2]["spec"], 2, {}),
         (MID[2]["spec"], 4, dict(moe_tp=4, moe_ep=2, moe_ep_rank=1)), (MID[0]["spec"], 16, dict(kv_replicate=True)),
         (dict(BRUTE[0]["spec"], ffn=12), 2, {}), (BRUTE[2]["spec"], 1, {})]


@pytest.mark.parametrize("spec,T,opts", CASES, ids=[f"q{i}" for i in range(len(CASES))])
def test_fp8_forward_matches_oracle(spec, T, opts):
    n = oracle.Model(spec).flat_elems
    for t in sorted({0, T - 1}):
        src = make_source(n, 60 + t)  # sigma 0.02 weights with ties, infinities, NaNs, subnormals sprinkled in
        got, want, plan, _, _ = _run(spec, T, t, src, **opts)
        assert first_diff(got, want) is None
        plan.close()


def test_fp8_special_blocks():
    spec = MID[1]["spec"]
    om = oracle.Model(spec)
    n = om.flat_elems
    rng = np.random.default_rng(1)
    src = np.zeros(n, dtype=np.uint32)                                # all-zero blocks: scale 1, codes 0
    got, want, plan, _, _ = _run(spec, 1, 0, src)
    assert first_diff(got, want) is None
    src = rng.integers(0, 1 << 32, size=n, dtype=np.uint64).astype(np.uint32)  # every bit pattern incl. NaN / Inf / huge
    got, want, _, _, _ = _run(spec, 1, 0, src)
    assert first_diff(got, want) is None
    src = (rng.standard_normal(n) * 1e-41).astype(np.float32).view(np.uint32)  # subnormal weights: tiny scales
    got, want, _, _, _ = _run(spec, 1, 0, src)
    assert first_diff(got, want) is None
    plan.close()


@pytest.mark.parametrize("misalign", [16, 48])
def test_fp8_sixteen_byte_aligned_bases_take_the_narrow_path(misalign):
    """Bases that are 16- but not 32-byte aligned are legal: the quantisation kernel then reads with 128-bit
    loads instead of 256-bit ones and produces the same bytes."""
    spec = MID[0]["spec"]
    om = oracle.Model(spec, tp=2, tp_rank=1)
    total, _ = om.fp8_layout()
    src = make_source(om.flat_elems, 71)
    want = np.full(total, SENT8, dtype=np.uint8)
    om.forward_fp8(src, want)
    plan = dr.Plan(spec, tp=2, tp_rank=1, dtype=dr.DR_FP8_E4M3_B128)
    pad = misalign // 4
    s_buf = torch.zeros(src.size + pad, dtype=torch.int32, device=dev())
    s_dev = s_buf[pad:]
    s_dev.copy_(torch.from_numpy(src.view(np.int32)))
    a_buf = torch.full((256 + misalign + total + 256,), SENT8, dtype=torch.uint8, device=dev())
    a_dev = a_buf[256 + misalign:256 + misalign + total]
    assert s_dev.data_ptr() % 32 == 16 and a_dev.data_ptr() % 32 == 16
    plan.reshard(s_dev, a_dev)
    torch.cuda.synchronize()
    assert first_diff(a_dev.cpu().numpy(), want) is None
    assert (a_buf[:256 + misalign] == SENT8).all() and (a_buf[256 + misalign + total:] == SENT8).all()
    # a base that is not even 16-byte aligned is refused on the host, before any launch
    s = torch.cuda.current_stream().cuda_stream
    assert dr.dr_reshard(plan.handle, s_dev.data_ptr() + 4, 4 * src.size, a_dev.data_ptr(), total, s) == B.DR_ERR_ALIGN
    plan.close()


def test_fp8_unsupported_calls():
    spec = MID[2]["spec"]
    plan = dr.Plan(spec, dtype=dr.DR_FP8_E4M3_B128)
    src = torch.zeros(plan.info.src_bytes // 4, dtype=torch.int32, device=dev())
    arena = torch.zeros(plan.info.dst_bytes, dtype=torch.uint8, device=dev())
    s = torch.cuda.current_stream().cuda_stream
    assert dr.dr_reshard_static(plan.handle, src.data_ptr(), plan.info.src_bytes, arena.data_ptr(), plan.info.dst_bytes, s) == B.DR_ERR_UNSUPPORTED
    plan.close()


INV_CASES = [(MID[2]["spec"], 2, 1, {}, 0), (MID[1]["spec"], 4, 3, dict(vocab_pad=64), 0), (dict(BRUTE[0]["spec"], ffn=12), 2, 0, {}, 0),
             (MID[0]["spec"], 2, 0, {}, 16), (MID[2]["spec"], 4, 1, dict(moe_tp=4, moe_ep=2, moe_ep_rank=1), 0)]


@pytest.mark.parametrize("spec,T,t,opts,misalign", INV_CASES, ids=[f"i{i}" for i in range(len(INV_CASES))])
def test_fp8_inverse_matches_oracle(spec, T, t, opts, misalign):
    """Rollout -> Training from an fp8 arena: codes times block scales (one fp32 multiplication) and widened bf16
    tensors at their flat positions, every other word untouched.  The arena holds every code (NaN codes too)
    and scales over a wide range, including a NaN, an infinity and a zero scale."""
    om = oracle.Model(spec, tp=T, tp_rank=t, **opts)
    total, lay = om.fp8_layout()
    rng = np.random.default_rng(17)
    arena = rng.integers(0, 256, size=total, dtype=np.uint64).astype(np.uint8)
    k = 0
    for d, (qz, off, soff) in zip(om.dst_tensors(), lay):
        if qz and d.alias_of < 0:
            nb = (-(-d.rows // 128)) * (-(-d.cols // 128))
            sc = np.exp(rng.uniform(-40, 20, nb)).astype(np.float32)
            for special in (np.nan, np.inf, 0.0, 2.0 ** -140):
                sc[k % nb] = special
                k += 7
            arena[soff:soff + 4 * nb] = sc.view(np.uint8)
    want = np.full(om.flat_elems, 0xDEADBEEF, dtype=np.uint32)
    om.inverse_fp8(arena, want)
    plan = dr.Plan(spec, tp=T, tp_rank=t, dtype=dr.DR_FP8_E4M3_B128, **opts)
    assert plan.info.dst_bytes == total and plan.info.src_bytes == 4 * om.flat_elems
    pad = misalign // 4
    f_buf = torch.full((om.flat_elems + pad + 64,), 0xDEADBEEF - (1 << 32), dtype=torch.int32, device=dev())
    flat = f_buf[pad:pad + om.flat_elems]
    a_buf = torch.zeros(total + misalign, dtype=torch.uint8, device=dev())
    a_dev = a_buf[misalign:]
    a_dev.copy_(torch.from_numpy(arena))
    plan.reshard_inverse(a_dev, flat)
    torch.cuda.synchronize()
    assert first_diff(flat.cpu().numpy().view(np.uint32), want) is None
    assert (f_buf[:pad] == 0xDEADBEEF - (1 << 32)).all() and (f_buf[pad + om.flat_elems:] == 0xDEADBEEF - (1 << 32)).all()
    plan.close()


def test_fp8_forward_then_inverse_is_within_half_a_code_step_of_the_weights():
    """Dequantised weights: |code * scale - x| <= |x| / 16 (half an e4m3 step) or half a subnormal step."""
    spec = MID[0]["spec"]
    om = oracle.Model(spec)
    src = synth.fill_f32(5, synth.BUF_MASTER, 0, om.flat_elems)
    plan = dr.Plan(spec, dtype=dr.DR_FP8_E4M3_B128)
    arena = torch.zeros(plan.info.dst_bytes, dtype=torch.uint8, device=dev())
    back = torch.zeros(om.flat_elems, dtype=torch.float32, device=dev())
    plan.reshard(to_dev_u32(src), arena)
    plan.reshard_inverse(arena, back)
    torch.cuda.synchronize()
    x, y = src.view(np.float32).astype(np.float64), back.cpu().numpy().astype(np.float64)
    lin = np.zeros(om.flat_elems, dtype=bool)
    for s_ in om.src_tensors():
        if s_.name.split(".")[-1] in ("q", "k", "v", "o", "gate", "up", "down"):
            lin[s_.flat_off:s_.flat_off + s_.rows * s_.cols] = True
    amax = np.abs(x[lin]).max()
    assert (np.abs(y[lin] - x[lin]) <= np.maximum(np.abs(x[lin]) / 16, amax / 448 * 2.0 ** -10) * (1 + 1e-6)).all()
    # bf16 tensors: half a bf16 step (half a subnormal step, 2^-134, for the generator's subnormal ties)
    assert (np.abs(y[~lin] - x[~lin]) <= np.maximum(np.abs(x[~lin]) * 2.0 ** -8, 2.0 ** -134)).all()
    plan.close()


def test_fp8_groups_give_the_whole_plan_result():
    spec = MID[2]["spec"]
    om = oracle.Model(spec, tp=2, tp_rank=1)
    total, _ = om.fp8_layout()
    src = make_source(om.flat_elems, 19)
    want = np.full(total, SENT8, dtype=np.uint8)
    om.forward_fp8(src, want)
    plan = dr.Plan(spec, tp=2, tp_rank=1, dtype=dr.DR_FP8_E4M3_B128)
    s_dev = to_dev_u32(src)
    arena = torch.full((total,), SENT8, dtype=torch.uint8, device=dev())
    n_groups = plan.info.n_groups
    moved = 0
    for g in reversed(range(n_groups)):            # any order
        plan.reshard_groups(g, 1, s_dev, arena)
        rc, gd = dr.dr_plan_group(plan.handle, g)
        moved += gd.bytes_moved
    torch.cuda.synchronize()
    assert first_diff(arena.cpu().numpy(), want) is None and moved == plan.info.bytes_moved_fwd
    # one layer alone writes only that layer's tensors
    arena.fill_(SENT8)
    plan.reshard_groups(1, 1, s_dev, arena)
    torch.cuda.synchronize()
    got = arena.cpu().numpy()
    tens = plan.tensors()
    rc, gd = dr.dr_plan_group(plan.handle, 1)
    lo = tens[gd.first_tensor].arena_off
    hi = tens[gd.first_tensor + gd.n_tensors].arena_off
    assert (got[:lo] == SENT8).all() and (got[hi:] == SENT8).all()
    assert first_diff(got[lo:hi], want[lo:hi]) is None
    plan.close()


def test_fp8_full_size_qwen3_8b_sampled_tensors():
    free, _ = torch.cuda.mem_get_info()
    if free < 50e9:
        pytest.skip("needs 50 GB of device memory")
    cfg = CONFIGS[2]
    seed = seed_of(2)
    plan = dr.Plan(cfg["spec"], dtype=dr.DR_FP8_E4M3_B128)
    om = oracle.Model(cfg["spec"])
    total, lay = om.fp8_layout()
    assert plan.info.dst_bytes == total
    src = torch.empty(plan.info.src_bytes // 4, dtype=torch.int32, device=dev())
    synth.cuda_fill_f32(src, seed, synth.BUF_MASTER)
    arena = torch.full((total,), SENT8, dtype=torch.uint8, device=dev())
    plan.reshard(src, arena)
    torch.cuda.synchronize()
    # the oracle on whole tensors of layers 0 and 35; only those layers' sources are generated on the host
    flat = np.empty(om.flat_elems, dtype=np.uint32)   # lazily committed
    want = np.empty(total, dtype=np.uint8)
    srcs = om.src_tensors()
    dst = om.dst_tensors()
    for layer in (0, 35):
        names = [s for s in srcs if s.name.startswith(f"layers.{layer}.")]
        lo = min(s.flat_off for s in names)
        hi = max(s.flat_off + s.rows * s.cols for s in names)
        flat[lo:hi] = synth.fill_f32(seed, synth.BUF_MASTER, lo, hi - lo)
        for i, d in enumerate(dst):
            if not d.name.startswith(f"layers.{layer}."):
                continue
            om.forward_fp8(flat, want, only=i)
            qz, off, soff = lay[i]
            nbytes = d.rows * d.cols * (1 if qz else 2)
            assert torch.equal(arena[off:off + nbytes].cpu(), torch.from_numpy(want[off:off + nbytes])), d.name
            if qz:
                nb = 4 * (-(-d.rows // 128)) * (-(-d.cols // 128))
                assert torch.equal(arena[soff:soff + nb].cpu(), torch.from_numpy(want[soff:soff + nb])), d.name
    plan.close()
