"""GPU parity: dr_reshard / dr_reshard_inverse through the C ABI against the CPU oracle, bit for bit,
on seeded inputs that span many tiles, ragged tails, unaligned runs and every special value."""
import numpy as np
import pytest
import torch

import oracle
import paper_2607_22614_b200 as dr
import synth
from gpu_util import SENT8, arena_dev, dev, first_diff, forward_both, make_source, special_values, to_dev_u32
from synth.configs import BRUTE, CONFIGS, MID

pytestmark = pytest.mark.gpu


FWD = []
for cfg in BRUTE:
    for T in (1, 2):
        for (W, g, A) in ((1, True, 1), (3, True, 4), (3, False, 1), (2, False, 16)):
            for dt in (dr.DR_BF16, dr.DR_F32):
                FWD.append((cfg, T, W, g, A, dt))
for cfg in MID + [CONFIGS[0]]:
    for (T, W, g, A, dt) in ((1, 1, True, 1, dr.DR_BF16), (2, 1, True, 1, dr.DR_BF16), (2, 3, False, 1, dr.DR_BF16),
                            (4 if cfg["spec"]["n_kv_heads"] % 4 == 0 else 2, 2, False, 4, dr.DR_BF16),
                            (2, 1, True, 1, dr.DR_F32), (1, 5, False, 3, dr.DR_F32)):
        FWD.append((cfg, T, W, g, A, dt))


@pytest.mark.parametrize("cfg,T,W,gathered,A,dtype", FWD,
                         ids=[f"{c[0]['name']}-tp{c[1]}-w{c[2]}-g{int(c[3])}-a{c[4]}-d{c[5]}" for c in FWD])
def test_forward_matches_oracle(cfg, T, W, gathered, A, dtype):
    for t in range(T):
        for r in ((W - 1,) if gathered else range(W)):
            got, want, plan, _, _ = forward_both(cfg["spec"], world=W, rank=r, gathered=gathered, align=A, tp=T,
                                                 tp_rank=t, dtype=dtype, seed=7 + t)
            assert first_diff(got, want) is None  # includes sentinel bytes in gaps and uncovered elements
            plan.close()


@pytest.mark.parametrize("misalign", [16, 48])
@pytest.mark.parametrize("dtype", [dr.DR_BF16, dr.DR_F32])
def test_sixteen_byte_aligned_bases_take_the_narrow_path(misalign, dtype):
    got, want, plan, _, _ = forward_both(MID[0]["spec"], tp=2, tp_rank=1, dtype=dtype, misalign=misalign)
    assert first_diff(got, want) is None
    plan.close()


# A MoE shape whose column-sliced (strided) attention output is under 2 % of the elements.  Plans of that kind with
# 2^28 elements or more run the kernel that brings tiles in with the TMA unit's bulk copies; the tests ask for that
# kernel on this small shape through the library's override, strided rows and run tails included.
MOE32 = dict(MID[2]["spec"], n_experts=32)


@pytest.fixture
def bulk_kernel(monkeypatch):
    monkeypatch.setenv("DR_FORWARD_KERNEL", "bulk")


@pytest.mark.parametrize("kw", [dict(tp=2, tp_rank=1), dict(tp=2, tp_rank=0, world=3, rank=1, gathered=False),
                                dict(tp=2, tp_rank=1, align=4, dtype=dr.DR_F32), dict(tp=2, tp_rank=0, misalign=16),
                                dict(tp=4, tp_rank=3, world=5, gathered=True, align=16)],
                         ids=["tp2", "shard-local", "f32-align4", "base16", "tp4-w5"])
def test_bulk_copy_kernel_with_strided_rows_tails_and_shard_cuts(kw, bulk_kernel):
    kw = dict(kw)
    got, want, plan, om, _ = forward_both(MOE32, seed=91, **kw)
    assert plan.info.bulk_forward == 1
    assert any(s.rows > 1 for s in plan.segments())          # column-sliced segments are there
    assert first_diff(got, want) is None
    plan.close()
    # the dense TP = 1 plans of the other mid-size shapes, and one with 30 % strided elements, through the same kernel
    for cfg, more in ((MID[0], {}), (MID[1], {}), (MID[0], dict(tp=2, tp_rank=1))):
        got, want, plan, _, _ = forward_both(cfg["spec"], seed=92, **more)
        assert plan.info.bulk_forward == 1 and first_diff(got, want) is None
        plan.close()


def test_which_plans_take_the_bulk_copy_kernel(monkeypatch):
    """Large plans with next to no strided work take it; small plans and plans with column-sliced matrices do not."""
    monkeypatch.delenv("DR_FORWARD_KERNEL", raising=False)
    want = {0: 0, 1: 0, 2: 1, 3: 0, 4: 1}   # tiny: small; 1.7B at TP=2 and 14B at TP=4: 27-31 % strided
    for i, cfg in enumerate(CONFIGS):
        p = dr.Plan(cfg["spec"], world=cfg["world"], rank=cfg["rank"], gathered=cfg["gathered"], tp=cfg["tp"],
                    tp_rank=cfg["tp_rank"], host_only=True)
        assert p.info.bulk_forward == want[i], i
        p.close()
    monkeypatch.setenv("DR_FORWARD_KERNEL", "register")
    p = dr.Plan(CONFIGS[2]["spec"], host_only=True)
    assert p.info.bulk_forward == 0
    p.close()


def test_cast_special_values_in_hardware():
    """Every hand-picked pattern (ties, carries, overflow, subnormals, NaNs) through the vector path and,
    via an odd-sized spec, through the scalar path."""
    sp = special_values()
    for cfg in (MID[2], BRUTE[0]):
        om = oracle.Model(cfg["spec"])
        src = np.resize(sp, om.flat_elems).astype(np.uint32)
        got, want, plan, _, _ = forward_both(cfg["spec"], src=src)
        assert first_diff(got, want) is None
        plan.close()
    # all 65536 high halves x tie / near-tie low halves, as one big "embedding"
    spec = dict(MID[2]["spec"], vocab=4096 * 6 // 8, hidden=128, n_layers=0, n_q_heads=1, n_kv_heads=1, head_dim=8,
                tied=1)
    highs = np.arange(1 << 16, dtype=np.uint32) << 16
    pats = np.concatenate([highs | np.uint32(lo) for lo in (0x0000, 0x0001, 0x7FFF, 0x8000, 0x8001, 0xFFFF)])
    om = oracle.Model(spec)
    assert om.flat_elems >= pats.size
    src = np.resize(pats, om.flat_elems).astype(np.uint32)
    got, want, plan, _, _ = forward_both(spec, src=src)
    assert first_diff(got, want) is None
    plan.close()


def test_union_of_shards_fills_the_arena_like_a_gathered_call():
    cfg = CONFIGS[0]  # tiny, world 2: rank 0 alone, then rank 1 into the same arena
    spec, W = cfg["spec"], cfg["world"]
    om = oracle.Model(spec, world=W)
    src = make_source(W * om.shard_elems, 5)
    full = np.full(om.arena_bytes, SENT8, dtype=np.uint8)
    om.forward(src, full)
    arena = arena_dev(om.arena_bytes)
    for r in range(W):
        plan = dr.Plan(spec, world=W, rank=r, gathered=False)
        shard = to_dev_u32(src[r * om.shard_elems:(r + 1) * om.shard_elems].copy())
        plan.reshard(shard, arena)
        torch.cuda.synchronize()
        if r == 0:
            one = np.full(om.arena_bytes, SENT8, dtype=np.uint8)
            om.forward(src[:om.shard_elems].copy(), one, gathered=False, rank=0)
            assert first_diff(arena.cpu().numpy(), one) is None
            assert plan.info.elems_moved == 987_904
        plan.close()
    assert first_diff(arena.cpu().numpy(), full) is None


INV = [(BRUTE[0], 2, 3, False, 4, dr.DR_BF16), (BRUTE[2], 2, 1, True, 1, dr.DR_F32), (MID[0], 2, 1, True, 1, dr.DR_BF16),
       (MID[1], 2, 3, False, 1, dr.DR_BF16), (MID[2], 1, 2, False, 16, dr.DR_F32), (MID[0], 4, 4, False, 1, dr.DR_BF16),
       (CONFIGS[0], 1, 2, False, 1, dr.DR_BF16)]


@pytest.mark.parametrize("cfg,T,W,gathered,A,dtype", INV,
                         ids=[f"{c[0]['name']}-tp{c[1]}-w{c[2]}-g{int(c[3])}-a{c[4]}-d{c[5]}" for c in INV])
def test_inverse_matches_oracle(cfg, T, W, gathered, A, dtype):
    es = 2 if dtype == dr.DR_BF16 else 4
    spec = cfg["spec"]
    for t in range(T):
        om = oracle.Model(spec, align=A, world=W, tp=T, tp_rank=t, elem_size=es)
        arena = synth.fill_bf16(3, synth.BUF_ROLLOUT, 0, om.arena_bytes // 2).view(np.uint8)
        if es == 2:  # sprinkle NaN, Inf and subnormal bf16 patterns: widening is a bit copy
            h = arena.view(np.uint16)
            h[::97] = np.resize(np.array([0x7FC0, 0xFF81, 0x7F80, 0x0001, 0x8000, 0x7FFF], dtype=np.uint16), h[::97].size)
        for r in ((0,) if gathered else range(W)):
            n = W * om.shard_elems if gathered else om.shard_elems
            want = np.full(n, 0xDEADBEEF, dtype=np.uint32)
            om.inverse(arena, want, gathered=gathered, rank=r)
            plan = dr.Plan(spec, world=W, rank=r, gathered=gathered, align_elems=A, tp=T, tp_rank=t, dtype=dtype)
            flat = torch.full((n,), 0xDEADBEEF - (1 << 32), dtype=torch.int32, device=dev())
            a_dev = torch.from_numpy(arena).to(dev())
            plan.reshard_inverse(a_dev, flat)
            torch.cuda.synchronize()
            assert first_diff(flat.cpu().numpy().view(np.uint32), want) is None
            plan.close()


def test_round_trip_on_layout_only_plan_is_identity():
    spec = MID[0]["spec"]
    T = 2
    om = oracle.Model(spec, tp=T, elem_size=4)
    src = make_source(om.flat_elems, 21)
    s_dev = to_dev_u32(src)
    back = torch.zeros_like(s_dev)
    for t in range(T):
        plan = dr.Plan(spec, tp=T, tp_rank=t, dtype=dr.DR_F32)
        arena = arena_dev(plan.info.dst_bytes)
        plan.reshard(s_dev, arena)
        plan.reshard_inverse(arena, back)
        torch.cuda.synchronize()
        plan.close()
    assert torch.equal(back, s_dev)


def test_argument_errors_are_found_before_launch():
    spec = MID[2]["spec"]
    plan = dr.Plan(spec)
    src = torch.zeros(plan.info.src_bytes // 4, dtype=torch.int32, device=dev())
    arena = arena_dev(plan.info.dst_bytes)
    B = dr.binding
    s = torch.cuda.current_stream().cuda_stream
    assert dr.dr_reshard(plan.handle, src.data_ptr(), plan.info.src_bytes - 4, arena.data_ptr(), plan.info.dst_bytes, s) == B.DR_ERR_SIZE
    assert dr.dr_reshard(plan.handle, src.data_ptr(), plan.info.src_bytes, arena.data_ptr(), plan.info.dst_bytes - 1, s) == B.DR_ERR_SIZE
    assert dr.dr_reshard(plan.handle, src.data_ptr() + 4, plan.info.src_bytes, arena.data_ptr(), plan.info.dst_bytes, s) == B.DR_ERR_ALIGN
    assert dr.dr_reshard(plan.handle, None, plan.info.src_bytes, arena.data_ptr(), plan.info.dst_bytes, s) == B.DR_ERR_INVALID
    assert dr.dr_reshard_inverse(plan.handle, arena.data_ptr(), 10, src.data_ptr(), plan.info.src_bytes, s) == B.DR_ERR_SIZE
    assert "small" in dr.dr_last_error()
    torch.cuda.synchronize()
    assert (arena.cpu().numpy() == SENT8).all()  # nothing ran
    plan.close()


def test_device_generator_equals_host_generator():
    n = 3_000_001
    for buf in (synth.BUF_MASTER, synth.BUF_ADAM_M, synth.BUF_ADAM_V):
        t = torch.empty(n, dtype=torch.int32, device=dev())
        synth.cuda_fill_f32(t, 99, buf, start=12345)
        assert np.array_equal(t.cpu().numpy().view(np.uint32), synth.fill_f32(99, buf, 12345, n))
        assert synth.cuda_mismatch_f32(t, 99, buf, start=12345) == 0
        t[77] += 1
        assert synth.cuda_mismatch_f32(t, 99, buf, start=12345) == 1
    h = torch.empty(n, dtype=torch.int16, device=dev())
    synth.cuda_fill_bf16(h, 99, synth.BUF_ROLLOUT, start=5)
    assert np.array_equal(h.cpu().numpy().view(np.uint16), synth.fill_bf16(99, synth.BUF_ROLLOUT, 5, n))


VARIANTS = [
    (dict(BRUTE[0]["spec"], ffn=12), 4, dict(kv_replicate=True, vocab_pad=8)),
    (MID[0]["spec"], 16, dict(kv_replicate=True)),
    (dict(MID[1]["spec"], tied=0), 2, dict(vocab_pad=1024)),
    (BRUTE[2]["spec"], 2, dict(moe_tp=2)),
    (MID[2]["spec"], 4, dict(moe_tp=4, moe_ep=2, moe_ep_rank=0, vocab_pad=64)),
    (MID[2]["spec"], 8, dict(kv_replicate=True, moe_ep=4, moe_ep_rank=3)),
]


@pytest.mark.parametrize("spec,T,opts", VARIANTS, ids=[f"v{i}" for i in range(len(VARIANTS))])
def test_layout_variants_forward_and_inverse_match_oracle(spec, T, opts):
    """KV-head replication, vocabulary padding, expert tensor / expert parallelism: forward into a
    sentinel-filled arena (padding rows must keep the sentinel), then the inverse of that arena."""
    for t in sorted({0, T // 2, T - 1}):
        for (W, g) in ((1, True), (3, False)):
            r = W - 1
            got, want, plan, om, src = forward_both(spec, world=W, rank=r, gathered=g, tp=T, tp_rank=t, seed=40 + t, **opts)
            assert first_diff(got, want) is None
            n = W * om.shard_elems if g else om.shard_elems
            wflat = np.full(n, 0xDEADBEEF, dtype=np.uint32)
            om.inverse(want, wflat, gathered=g, rank=r)
            flat = torch.full((n,), 0xDEADBEEF - (1 << 32), dtype=torch.int32, device=dev())
            plan.reshard_inverse(torch.from_numpy(got).to(dev()), flat)
            torch.cuda.synchronize()
            assert first_diff(flat.cpu().numpy().view(np.uint32), wflat) is None
            plan.close()


def test_empty_plan_launches_nothing_and_touches_nothing():
    spec = dict(n_layers=0, hidden=4, n_q_heads=1, n_kv_heads=1, head_dim=2, ffn=4, vocab=2, tied=1, qk_norm=1)
    p = dr.Plan(spec, world=16, rank=15, gathered=False)
    src = torch.zeros(8, dtype=torch.int32, device=dev())
    arena = arena_dev(max(p.info.dst_bytes, 16))
    p.reshard(src, arena)
    p.reshard_inverse(arena, src)
    torch.cuda.synchronize()
    assert (arena.cpu().numpy() == SENT8).all() and (src.cpu().numpy() == 0).all()
    p.close()


def test_one_plan_on_two_streams_at_once():
    """A plan is immutable: two repacks of different sources run concurrently on two streams."""
    spec = MID[0]["spec"]
    plan = dr.Plan(spec, tp=2, tp_rank=0)
    om = oracle.Model(spec, tp=2, tp_rank=0)
    srcs = [make_source(om.flat_elems, s) for s in (91, 92)]
    wants = []
    for s in srcs:
        w = np.full(om.arena_bytes, SENT8, dtype=np.uint8)
        om.forward(s, w)
        wants.append(w)
    devs = [to_dev_u32(s) for s in srcs]
    arenas = [arena_dev(om.arena_bytes) for _ in srcs]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    torch.cuda.synchronize()
    for _ in range(3):
        for d, a, st in zip(devs, arenas, streams):
            plan.reshard(d, a, stream=st)
    torch.cuda.synchronize()
    for a, w in zip(arenas, wants):
        assert first_diff(a.cpu().numpy(), w) is None
    plan.close()


def test_repack_and_inverse_replay_from_a_cuda_graph():
    """dr_reshard / dr_reshard_inverse only enqueue kernels, so a switch can be captured once and replayed."""
    spec = MID[2]["spec"]
    plan = dr.Plan(spec, tp=2, tp_rank=1)
    om = oracle.Model(spec, tp=2, tp_rank=1)
    src = to_dev_u32(make_source(om.flat_elems, 93))
    arena = arena_dev(om.arena_bytes)
    back = torch.full((om.flat_elems,), 0x5A5A5A5A, dtype=torch.int32, device=dev())
    plan.reshard(src, arena)          # warm-up outside the capture (module load)
    torch.cuda.synchronize()
    arena.fill_(SENT8)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        plan.reshard(src, arena)      # enqueued on the capturing stream (the current stream inside the context)
        plan.reshard_inverse(arena, back)
    torch.cuda.synchronize()
    assert (arena.cpu().numpy() == SENT8).all()   # capture enqueues nothing
    for seed in (94, 95):             # new weights in the same buffers, same graph
        host = make_source(om.flat_elems, seed)
        src.copy_(torch.from_numpy(host.view(np.int32)))
        graph.replay()
        torch.cuda.synchronize()
        want = np.full(om.arena_bytes, SENT8, dtype=np.uint8)
        om.forward(host, want)
        assert first_diff(arena.cpu().numpy(), want) is None
        wflat = np.full(om.flat_elems, 0x5A5A5A5A, dtype=np.uint32)
        om.inverse(want, wflat)
        assert first_diff(back.cpu().numpy().view(np.uint32), wflat) is None
    plan.close()


@pytest.mark.parametrize("spec,kw", [(MID[0]["spec"], dict(tp=2, tp_rank=1)), (MID[2]["spec"], dict(tp=1)),
                                     (MID[1]["spec"], dict(world=3, rank=1, gathered=False, tp=2, tp_rank=0)),
                                     (BRUTE[1]["spec"], dict(tp=2, tp_rank=0, align=3))],
                         ids=["dense-tp2", "moe", "shard-local-tied", "brute-tied"])
def test_groups_in_any_order_build_up_the_full_repack(spec, kw):
    """One layer at a time, in a shuffled order: after every call the arena holds exactly the oracle's tensors
    of the groups done so far and the sentinel everywhere else; at the end it is dr_reshard's result."""
    kw = dict(kw)
    world, rank, gathered, align = kw.pop("world", 1), kw.pop("rank", 0), kw.pop("gathered", True), kw.pop("align", 1)
    om = oracle.Model(spec, align=align, world=world, **kw)
    full = make_source(world * om.shard_elems, 123)
    local = full if gathered else full[rank * om.shard_elems:(rank + 1) * om.shard_elems].copy()
    plan = dr.Plan(spec, world=world, rank=rank, gathered=gathered, align_elems=align, **kw)
    src = to_dev_u32(local)
    arena = arena_dev(om.arena_bytes)
    want = np.full(om.arena_bytes, SENT8, dtype=np.uint8)
    order = np.random.default_rng(5).permutation(plan.info.n_groups)
    for g in order:
        rc, d = dr.dr_plan_group(plan.handle, int(g))
        for i in range(d.first_tensor, d.first_tensor + d.n_tensors):
            om.forward(local, want, gathered=gathered, rank=rank, only=i)
        plan.reshard_groups(int(g), 1, src, arena)
        torch.cuda.synchronize()
        assert first_diff(arena.cpu().numpy(), want) is None
    ref = arena_dev(om.arena_bytes)
    plan.reshard(src, ref)
    torch.cuda.synchronize()
    assert torch.equal(ref, arena)
    # several groups in one call, and the argument checks
    arena2 = arena_dev(om.arena_bytes)
    half = plan.info.n_groups // 2
    plan.reshard_groups(0, half, src, arena2)
    plan.reshard_groups(half, plan.info.n_groups - half, src, arena2)
    torch.cuda.synchronize()
    assert torch.equal(ref, arena2)
    s = torch.cuda.current_stream().cuda_stream
    bad = dr.dr_reshard_groups(plan.handle, 1, plan.info.n_groups, src.data_ptr(), src.numel() * 4, arena.data_ptr(), arena.numel(), s)
    assert bad == dr.binding.DR_ERR_INVALID
    plan.close()


def test_the_bulk_copy_kernel_replays_from_a_cuda_graph_too(bulk_kernel):
    """The kernel that moves tiles with bulk copies (dynamic shared memory, mbarrier) is captured and replayed like the
    register kernel: each replay repacks whatever the source buffer holds at that time."""
    spec, kw = MOE32, dict(tp=2, tp_rank=0)
    om = oracle.Model(spec, **kw)
    plan = dr.Plan(spec, **kw)
    assert plan.info.bulk_forward == 1
    src = torch.zeros(om.shard_elems, dtype=torch.int32, device=dev())
    arena = arena_dev(om.arena_bytes)
    back = torch.zeros(om.shard_elems, dtype=torch.int32, device=dev())
    plan.reshard(src, arena)            # an ordinary call first
    plan.reshard_inverse(arena, back)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):           # captures what is enqueued on torch's current (capturing) stream
        plan.reshard(src, arena)
        plan.reshard_inverse(arena, back)
    for seed in (3, 4):
        host = make_source(om.shard_elems, seed)
        src.copy_(torch.from_numpy(host.view(np.int32)))
        arena.fill_(SENT8)
        back.fill_(0x5A5A5A5A)
        g.replay()
        torch.cuda.synchronize()
        want = np.full(om.arena_bytes, SENT8, dtype=np.uint8)
        om.forward(host, want)
        assert first_diff(arena.cpu().numpy(), want) is None
        want_back = np.full(om.shard_elems, 0x5A5A5A5A, dtype=np.uint32)
        om.inverse(want, want_back)
        assert np.array_equal(back.cpu().numpy().view(np.uint32), want_back)
    plan.close()
