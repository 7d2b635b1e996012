"""The allocation-free repack entry point, dr_reshard_static, against dr_reshard.

Some users of this library cannot allocate device memory when a GPU switches role: their framework's
memory pool already owns the whole GPU, or a cudaMalloc would stall the staging copies running beside
the repack.  For them the segment table sits in a fixed table inside the library.  This test calls the
entry point through the C ABI, twice in a row with different plans (so that entries left over from the
first call would show), and requires the output to equal dr_reshard's bit for bit.
"""
import numpy as np
import pytest
import torch

import paper_2607_22614_b200 as dr
from synth.configs import BRUTE, MID

pytestmark = pytest.mark.gpu
B = dr.binding


def _both(spec, tp, tp_rank, src, dtype=dr.DR_BF16):
    dev = src.device
    ref_plan = dr.Plan(spec, tp=tp, tp_rank=tp_rank, dtype=dtype)          # table in cudaMalloc'ed memory
    host_plan = dr.Plan(spec, tp=tp, tp_rank=tp_rank, dtype=dtype, host_only=True)  # no device memory at all
    n = ref_plan.info.dst_bytes
    want = torch.full((n,), 0xA5, dtype=torch.uint8, device=dev)
    got = torch.full((n,), 0xA5, dtype=torch.uint8, device=dev)
    ref_plan.reshard(src, want)
    s = torch.cuda.current_stream().cuda_stream
    rc = dr.dr_reshard_static(host_plan.handle, src.data_ptr(), src.numel() * 4, got.data_ptr(), n, s)
    assert rc == 0, dr.dr_last_error()
    return got, want, ref_plan, host_plan


def test_static_table_repack_equals_dr_reshard_on_two_calls_in_a_row():
    dev = torch.device("cuda:0")
    spec = MID[0]["spec"]
    probe = dr.Plan(spec, host_only=True)
    g = torch.Generator(device="cpu").manual_seed(3)
    src = torch.randint(-2**31, 2**31 - 1, (probe.info.flat_elems,), dtype=torch.int32, generator=g).to(dev)
    probe.close()
    # first call: TP rank 1 of 2 (226-ish segments); second call: TP 1 (fewer, differently placed segments)
    got1, want1, a1, b1 = _both(spec, 2, 1, src)
    got2, want2, a2, b2 = _both(spec, 1, 0, src)
    torch.cuda.synchronize()
    assert torch.equal(got1, want1)
    assert torch.equal(got2, want2)
    assert not torch.equal(got1[:1 << 20], got2[:1 << 20]) or a1.info.dst_bytes != a2.info.dst_bytes
    # and once more the first plan, now after a different table was resident
    got3, want3, a3, b3 = _both(spec, 2, 1, src)
    torch.cuda.synchronize()
    assert torch.equal(got3, want1)
    for p in (a1, b1, a2, b2, a3, b3):
        p.close()


def test_static_table_handles_scalar_runs_and_layout_only_plans():
    dev = torch.device("cuda:0")
    spec = BRUTE[2]["spec"]
    probe = dr.Plan(spec, host_only=True)
    src = torch.arange(probe.info.flat_elems, dtype=torch.int32, device=dev)
    probe.close()
    for dtype in (dr.DR_BF16, dr.DR_F32):
        got, want, a, b = _both(spec, 2, 0, src, dtype)
        torch.cuda.synchronize()
        assert torch.equal(got, want)
        a.close()
        b.close()


def test_static_table_rejects_oversized_plans_and_bad_buffers():
    dev = torch.device("cuda:0")
    big = dict(n_layers=80, hidden=64, n_q_heads=2, n_kv_heads=2, head_dim=8, ffn=0, vocab=64, n_experts=128, moe_ffn=8,
               tied=0, qk_norm=1)
    p = dr.Plan(big, arena_align_bytes=16, align_elems=3, host_only=True)  # odd alignment: nothing merges
    assert p.info.n_segments > 16384
    src = torch.zeros(p.info.src_bytes // 4, dtype=torch.int32, device=dev)
    dst = torch.full((p.info.dst_bytes,), 7, dtype=torch.uint8, device=dev)
    s = torch.cuda.current_stream().cuda_stream
    assert dr.dr_reshard_static(p.handle, src.data_ptr(), p.info.src_bytes, dst.data_ptr(), p.info.dst_bytes, s) == B.DR_ERR_SIZE
    assert "16384" in dr.dr_last_error()
    p.close()
    q = dr.Plan(MID[2]["spec"], host_only=True)
    src = torch.zeros(q.info.src_bytes // 4, dtype=torch.int32, device=dev)
    dst = torch.full((q.info.dst_bytes,), 7, dtype=torch.uint8, device=dev)
    assert dr.dr_reshard_static(q.handle, src.data_ptr(), q.info.src_bytes - 4, dst.data_ptr(), q.info.dst_bytes, s) == B.DR_ERR_SIZE
    assert dr.dr_reshard_static(q.handle, src.data_ptr() + 4, q.info.src_bytes, dst.data_ptr(), q.info.dst_bytes, s) == B.DR_ERR_ALIGN
    torch.cuda.synchronize()
    assert (dst == 7).all()
    q.close()
