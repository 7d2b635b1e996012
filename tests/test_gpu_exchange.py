"""GPU parity for the exchange fused into the repack (dr_reshard_push): every FSDP rank repacks its own shard
and stores the pieces into all rollout arenas in the same kernel.  The ranks run one after the other on this
GPU and the "peers'" arenas are buffers of this GPU, which is enough to prove the bytes: the kernel neither
waits on nor signals anything, so no interplay between ranks exists beyond what lands in memory.  After all
ranks have pushed, every arena must equal the oracle's gathered forward, gaps untouched."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_22614_b200 as dr
from gpu_util import SENT8, dev, first_diff, make_source
from synth.configs import BRUTE, CONFIGS, MID

pytestmark = pytest.mark.gpu
B = dr.binding

CASES = [(MID[0]["spec"], 2, 1, 3, 1, dr.DR_BF16, 3, 0), (MID[1]["spec"], 2, 0, 2, 4, dr.DR_BF16, 2, 0),
         (MID[2]["spec"], 2, 1, 4, 1, dr.DR_BF16, 8, 0), (MID[0]["spec"], 1, 0, 5, 1, dr.DR_F32, 2, 0),
         (BRUTE[0]["spec"], 2, 1, 3, 3, dr.DR_BF16, 4, 0), (BRUTE[2]["spec"], 1, 0, 2, 1, dr.DR_F32, 3, 0),
         (CONFIGS[0]["spec"], 1, 0, 2, 1, dr.DR_BF16, 2, 0), (MID[0]["spec"], 2, 0, 3, 1, dr.DR_BF16, 3, 16)]


@pytest.mark.parametrize("spec,T,t,W,A,dtype,n_dst,misalign", CASES, ids=[f"p{i}" for i in range(len(CASES))])
def test_all_ranks_push_and_every_arena_holds_the_gathered_forward(spec, T, t, W, A, dtype, n_dst, misalign):
    es = 2 if dtype == dr.DR_BF16 else 4
    om = oracle.Model(spec, align=A, world=W, tp=T, tp_rank=t, elem_size=es)
    S = om.shard_elems
    src = make_source(W * S, 123)
    want = np.full(om.arena_bytes, SENT8, dtype=np.uint8)
    om.forward(src, want, gathered=True)
    G = 256
    bufs = [torch.full((G + misalign + om.arena_bytes + G,), SENT8, dtype=torch.uint8, device=dev()) for _ in range(n_dst)]
    arenas = [b[G + misalign:G + misalign + om.arena_bytes] for b in bufs]
    for r in range(W):
        plan = dr.Plan(spec, world=W, rank=r, gathered=False, align_elems=A, tp=T, tp_rank=t, dtype=dtype)
        shard = torch.from_numpy(src[r * S:(r + 1) * S].copy().view(np.int32)).to(dev())
        plan.reshard_push(shard, arenas)
        torch.cuda.synchronize()
        if r == 0:  # after one rank: exactly that plan's ranges are written, in every arena
            one = np.full(om.arena_bytes, SENT8, dtype=np.uint8)
            om.forward(src[:S].copy(), one, gathered=False, rank=0)
            for a in arenas:
                assert first_diff(a.cpu().numpy(), one) is None
        plan.close()
    for a, b in zip(arenas, bufs):
        assert first_diff(a.cpu().numpy(), want) is None
        assert (b[:G + misalign] == SENT8).all() and (b[G + misalign + om.arena_bytes:] == SENT8).all()


def test_push_into_one_arena_is_dr_reshard_and_argument_errors():
    spec = MID[1]["spec"]
    plan = dr.Plan(spec, tp=2, tp_rank=1)
    n = plan.info.src_bytes // 4
    src = torch.from_numpy(make_source(n, 7).view(np.int32)).to(dev())
    a = torch.full((plan.info.dst_bytes,), SENT8, dtype=torch.uint8, device=dev())
    b = torch.full((plan.info.dst_bytes,), SENT8, dtype=torch.uint8, device=dev())
    plan.reshard(src, a)
    plan.reshard_push(src, [b])
    torch.cuda.synchronize()
    assert torch.equal(a, b)
    s = torch.cuda.current_stream().cuda_stream
    nb = plan.info.dst_bytes
    assert dr.dr_reshard_push(plan.handle, src.data_ptr(), 4 * n, [], nb, s) == B.DR_ERR_INVALID
    assert dr.dr_reshard_push(plan.handle, src.data_ptr(), 4 * n, [a.data_ptr()] * 9, nb, s) == B.DR_ERR_INVALID
    assert dr.dr_reshard_push(plan.handle, src.data_ptr(), 4 * n, [a.data_ptr(), None], nb, s) == B.DR_ERR_INVALID
    assert dr.dr_reshard_push(plan.handle, src.data_ptr(), 4 * n, [a.data_ptr(), b.data_ptr() + 8], nb, s) == B.DR_ERR_ALIGN
    assert dr.dr_reshard_push(plan.handle, src.data_ptr(), 4 * n, [a.data_ptr(), b.data_ptr()], nb - 1, s) == B.DR_ERR_SIZE
    q = dr.Plan(spec, dtype=dr.DR_FP8_E4M3_B128)
    qa = torch.zeros(q.info.dst_bytes, dtype=torch.uint8, device=dev())
    assert dr.dr_reshard_push(q.handle, src.data_ptr(), 4 * n, [qa.data_ptr()], q.info.dst_bytes, s) == B.DR_ERR_UNSUPPORTED
    host = dr.Plan(spec, tp=2, tp_rank=1, host_only=True)
    assert dr.dr_reshard_push(host.handle, src.data_ptr(), 4 * n, [a.data_ptr()], nb, s) == B.DR_ERR_STATE
    torch.cuda.synchronize()
    assert torch.equal(a, b)
    for p in (plan, q, host):
        p.close()


def test_push_into_an_arena_owned_by_another_process():
    """Two processes on this GPU play FSDP ranks 0 and 1.  Rank 0 (this process) owns a rollout arena and hands it
    to rank 1 through CUDA IPC; rank 1 repacks its shard and pushes the pieces into that arena, which it reaches
    only through the IPC mapping, as it would reach a peer GPU's arena.  The processes are ordered on the host
    (rank 1 synchronises and reports before rank 0 reads), no kernel waits for another.  After rank 0's own push the
    arena must equal the oracle's gathered forward."""
    import torch.multiprocessing as mp

    import synth
    from push_peer_worker import run

    spec, W, T, t, seed = MID[0]["spec"], 2, 2, 1, 4242
    om = oracle.Model(spec, world=W, tp=T, tp_rank=t)
    S = om.shard_elems
    arena = torch.full((om.arena_bytes,), SENT8, dtype=torch.uint8, device=dev())
    torch.cuda.synchronize()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    child = ctx.Process(target=run, args=(arena, spec, W, T, t, seed, q))
    child.start()
    try:
        status, n_ranges, digest = q.get(timeout=300)
    finally:
        child.join(timeout=60)
        if child.is_alive():
            child.kill()
    assert status == "ok", n_ranges
    # what rank 1 left in this process's memory: exactly its plan's ranges, everything else still sentinel
    flat = synth.fill_f32(seed, synth.BUF_MASTER, 0, W * S)
    after_one = np.full(om.arena_bytes, SENT8, dtype=np.uint8)
    om.forward(flat[S:2 * S].copy(), after_one, gathered=False, rank=1)
    assert first_diff(arena.cpu().numpy(), after_one) is None
    assert digest == int(after_one.astype(np.int64).sum()) and n_ranges > 0
    plan = dr.Plan(spec, world=W, rank=0, gathered=False, tp=T, tp_rank=t)
    plan.reshard_push(torch.from_numpy(flat[:S].copy().view(np.int32)).to(dev()), [arena])
    torch.cuda.synchronize()
    want = np.full(om.arena_bytes, SENT8, dtype=np.uint8)
    om.forward(flat, want, gathered=True)
    assert first_diff(arena.cpu().numpy(), want) is None
    plan.close()
    del arena
    torch.cuda.ipc_collect()
