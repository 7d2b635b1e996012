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
    assert dr.dr_reshard_inverse(plan.handle, arena.data_ptr(), plan.info.dst_bytes, src.data_ptr(), plan.info.src_bytes, s) == B.DR_ERR_UNSUPPORTED
    assert dr.dr_reshard_static(plan.handle, src.data_ptr(), plan.info.src_bytes, arena.data_ptr(), plan.info.dst_bytes, s) == B.DR_ERR_UNSUPPORTED
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
