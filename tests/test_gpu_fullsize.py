"""GPU parity at the full sizes of the five workloads, in the launch configuration bench.py times.

cfg 1 is compared whole against the oracle (the oracle finishes it in seconds).  cfg 2-4 are too big
for that: they are checked on sampled outputs that the oracle computes one by one, on whole small
tensors, on row blocks at the edges of the big tensors, and by counting what the call touched."""
import os

import numpy as np
import pytest
import torch

import oracle
import paper_2607_22614_b200 as dr
import synth
from synth.configs import CONFIGS, seed_of

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _need(gb):
    import gc
    gc.collect()
    torch.cuda.empty_cache()  # memory cached by earlier tests counts as free
    free, _ = torch.cuda.mem_get_info()
    if free < gb * 1e9:
        pytest.skip(f"needs {gb} GB of free device memory, {free / 1e9:.0f} GB free")


def _models(cfg, world=None, rank=None, gathered=None):
    world = cfg["world"] if world is None else world
    rank = cfg["rank"] if rank is None else rank
    gathered = cfg["gathered"] if gathered is None else gathered
    plan = dr.Plan(cfg["spec"], world=world, rank=rank, gathered=gathered, tp=cfg["tp"], tp_rank=cfg["tp_rank"])
    om = oracle.Model(cfg["spec"], world=world, tp=cfg["tp"], tp_rank=cfg["tp_rank"])
    assert plan.info.dst_bytes == om.arena_bytes and plan.info.flat_elems == cfg["flat_elems"]
    return plan, om


def _sample_positions(om, n, rng):
    """Random (tensor, row, col) weighted by tensor size, plus every element of the small tensors of three
    layers and 2-row blocks at the top and bottom of every big tensor of the first and last layer."""
    dst = [(i, d) for i, d in enumerate(om.dst_tensors()) if d.alias_of < 0]
    sizes = np.array([d.rows * d.cols for _, d in dst], dtype=np.float64)
    pick = rng.choice(len(dst), size=n, p=sizes / sizes.sum())
    ti = np.array([dst[k][0] for k in pick])
    rows = np.array([rng.integers(0, dst[k][1].rows) for k in pick])
    cols = np.array([rng.integers(0, dst[k][1].cols) for k in pick])
    extra = []
    L = max(1, sum(1 for _, d in dst if d.name.endswith(".in_norm")))
    for i, d in dst:
        layer = int(d.name.split(".")[1]) if d.name.startswith("layers.") else -1
        if d.rows * d.cols <= 8192 and layer in (-1, 0, L // 2, L - 1):
            r, c = np.divmod(np.arange(d.rows * d.cols), d.cols)
            extra.append((np.full(r.size, i), r, c))
        elif layer in (-1, 0, L - 1):
            for r0 in (0, d.rows - 2):
                r = np.repeat(np.arange(r0, r0 + 2), d.cols)
                c = np.tile(np.arange(d.cols), 2)
                extra.append((np.full(r.size, i), r, c))
    ti = np.concatenate([ti] + [e[0] for e in extra])
    rows = np.concatenate([rows] + [e[1] for e in extra])
    cols = np.concatenate([cols] + [e[2] for e in extra])
    return ti, rows, cols


def _oracle_flat_index(om, ti, rows, cols):
    return np.array([om.map(int(i), int(r), int(c)) for i, r, c in zip(ti, rows, cols)], dtype=np.int64)


def _arena_slots(om, ti, rows, cols):
    dst = om.dst_tensors()
    off = np.array([dst[i].arena_off for i in ti], dtype=np.int64) // 2
    ncol = np.array([dst[i].cols for i in ti], dtype=np.int64)
    return off + rows * ncol + cols


def test_cfg1_whole_arena_equals_oracle():
    """Qwen3-1.7B-shaped, gathered flat buffer, TP=2 rank 0: every byte of the 1.72 GB arena."""
    _need(12)
    cfg = CONFIGS[1]
    plan, om = _models(cfg)
    seed = seed_of(1)
    src = torch.empty(plan.info.src_bytes // 4, dtype=torch.int32, device=DEV)
    synth.cuda_fill_f32(src, seed, synth.BUF_MASTER)
    arena = torch.full((plan.info.dst_bytes,), 0xA5, dtype=torch.uint8, device=DEV)
    plan.reshard(src, arena)
    torch.cuda.synchronize()
    got = arena.cpu().numpy()
    del src, arena
    flat = synth.fill_f32(seed, synth.BUF_MASTER, 0, om.world * om.shard_elems)
    want = np.full(om.arena_bytes, 0xA5, dtype=np.uint8)
    om.forward(flat, want)
    assert np.array_equal(got, want)
    assert plan.info.elems_moved == 860_349_440
    plan.close()


def test_cfg2_sampled_outputs():
    """Qwen3-8B-shaped, TP=1: 8.19 G elements, 49 GB moved per launch."""
    _need(55)
    cfg = CONFIGS[2]
    plan, om = _models(cfg)
    seed = seed_of(2)
    src = torch.empty(plan.info.src_bytes // 4, dtype=torch.int32, device=DEV)
    synth.cuda_fill_f32(src, seed, synth.BUF_MASTER)
    arena = torch.full((plan.info.dst_bytes,), 0xA5, dtype=torch.uint8, device=DEV)
    plan.reshard(src, arena)
    torch.cuda.synchronize()
    rng = np.random.default_rng(2)
    ti, rows, cols = _sample_positions(om, 200_000, rng)
    f = _oracle_flat_index(om, ti, rows, cols)
    want = oracle.cast_bf16_array(synth.at_f32(seed, synth.BUF_MASTER, f))
    slots = torch.from_numpy(_arena_slots(om, ti, rows, cols)).to(DEV)
    got = arena.view(torch.int16)[slots].cpu().numpy().view(np.uint16)
    assert np.array_equal(got, want)
    # at TP=1 every arena byte is written: the sentinel pattern (not a value the generator can produce) is gone
    assert int((arena.view(torch.int16) == (0xA5A5 - 65536)).sum()) == 0
    plan.close()


def test_cfg3_inverse_shard_local_sampled_and_counted():
    """Qwen3-14B-shaped, Rollout -> Training: TP=4 rank 1 arena scattered into FSDP shard 1 of 4."""
    _need(26)
    cfg = CONFIGS[3]
    plan, om = _models(cfg)
    seed = seed_of(3)
    S, r = plan.info.shard_elems, cfg["rank"]
    arena = torch.empty(plan.info.dst_bytes // 2, dtype=torch.int16, device=DEV)
    synth.cuda_fill_bf16(arena, seed, synth.BUF_ROLLOUT)
    sent = 0xDEADBEEF - (1 << 32)
    flat = torch.full((S,), sent, dtype=torch.int32, device=DEV)
    plan.reshard_inverse(arena, flat)
    torch.cuda.synchronize()
    # every word the call wrote is a widened bf16 (low half zero), so counting non-sentinel words counts writes
    assert int((flat != sent).sum()) == plan.info.elems_moved
    rng = np.random.default_rng(3)
    ti, rows, cols = _sample_positions(om, 300_000, rng)
    f = _oracle_flat_index(om, ti, rows, cols)
    inside = (f >= r * S) & (f < (r + 1) * S)
    assert 0.15 < inside.mean() < 0.5
    slots = _arena_slots(om, ti, rows, cols)
    want = synth.at_bf16(seed, synth.BUF_ROLLOUT, slots[inside]).astype(np.uint32) << 16
    got = flat[torch.from_numpy(f[inside] - r * S).to(DEV)].cpu().numpy().view(np.uint32)
    assert np.array_equal(got, want)
    plan.close()


def test_cfg4_moe_two_half_shards_sampled():
    """Qwen3-30B-A3B-shaped MoE: run as two shard-local halves into one arena (it does not fit whole)."""
    _need(125)
    cfg = CONFIGS[4]
    seed = seed_of(4)
    om = oracle.Model(cfg["spec"], world=2, tp=cfg["tp"], tp_rank=cfg["tp_rank"])
    S = om.shard_elems
    arena = torch.full((om.arena_bytes,), 0xA5, dtype=torch.uint8, device=DEV)
    shard = torch.empty(S, dtype=torch.int32, device=DEV)
    moved = 0
    for half in (0, 1):
        plan, _ = _models(cfg, world=2, rank=half, gathered=False)
        synth.cuda_fill_f32(shard, seed, synth.BUF_MASTER, start=half * S)
        plan.reshard(shard, arena)
        torch.cuda.synchronize()
        moved += plan.info.elems_moved
        plan.close()
    assert moved == 29_767_972_864
    rng = np.random.default_rng(4)
    ti, rows, cols = _sample_positions(om, 200_000, rng)
    f = _oracle_flat_index(om, ti, rows, cols)
    want = oracle.cast_bf16_array(synth.at_f32(seed, synth.BUF_MASTER, f))
    slots = torch.from_numpy(_arena_slots(om, ti, rows, cols)).to(DEV)
    got = arena.view(torch.int16)[slots].cpu().numpy().view(np.uint16)
    assert np.array_equal(got, want)


def _host_room_gb():
    with open("/proc/meminfo") as f:
        for line in f:
            if line.startswith("MemAvailable:"):
                return int(line.split()[1]) / 1e6
    return 0


def test_cfg2_whole_arena_equals_oracle():
    """All 8.19 G elements of the Qwen3-8B-shaped switch against the oracle (needs about 70 GB of host memory)."""
    _need(55)
    if _host_room_gb() < 90:
        pytest.skip("needs 90 GB of free host memory")
    cfg = CONFIGS[2]
    plan, om = _models(cfg)
    seed = seed_of(2)
    src = torch.empty(plan.info.src_bytes // 4, dtype=torch.int32, device=DEV)
    synth.cuda_fill_f32(src, seed, synth.BUF_MASTER)
    arena = torch.full((plan.info.dst_bytes,), 0xA5, dtype=torch.uint8, device=DEV)
    plan.reshard(src, arena)
    torch.cuda.synchronize()
    del src
    flat = synth.fill_f32(seed, synth.BUF_MASTER, 0, om.flat_elems)
    want = np.full(om.arena_bytes, 0xA5, dtype=np.uint8)
    om.forward(flat, want)
    del flat
    got = arena.cpu().numpy()
    assert np.array_equal(got, want)
    plan.close()


def test_cfg3_whole_shard_equals_oracle_inverse():
    """The complete Rollout -> Training result of the Qwen3-14B-shaped workload: every word of FSDP shard 1 of 4,
    written or not, against the oracle's inverse."""
    _need(26)
    if _host_room_gb() < 50:
        pytest.skip("needs 50 GB of free host memory")
    cfg = CONFIGS[3]
    plan, om = _models(cfg)
    seed = seed_of(3)
    S, r = plan.info.shard_elems, cfg["rank"]
    arena = torch.empty(plan.info.dst_bytes // 2, dtype=torch.int16, device=DEV)
    synth.cuda_fill_bf16(arena, seed, synth.BUF_ROLLOUT)
    sent = 0xDEADBEEF - (1 << 32)
    flat = torch.full((S,), sent, dtype=torch.int32, device=DEV)
    plan.reshard_inverse(arena, flat)
    torch.cuda.synchronize()
    del arena
    h_arena = synth.fill_bf16(seed, synth.BUF_ROLLOUT, 0, om.arena_bytes // 2).view(np.uint8)
    want = np.full(S, 0xDEADBEEF, dtype=np.uint32)
    om.inverse(h_arena, want, gathered=False, rank=r)
    assert np.array_equal(flat.cpu().numpy().view(np.uint32), want)
    plan.close()


def test_cfg4_whole_arena_equals_oracle_streamed_by_layer():
    """All 29.8 G elements of the Qwen3-30B-A3B-shaped MoE switch.  Neither the 122 GB source nor the 59.5 GB
    arena is held on the host: the oracle runs tensor by tensor on lazily committed mappings, one layer's
    source at a time, and each rollout tensor is compared and released."""
    import mmap
    _need(125)
    if _host_room_gb() < 24:
        pytest.skip("needs 24 GB of free host memory")
    cfg = CONFIGS[4]
    seed = seed_of(4)
    om = oracle.Model(cfg["spec"], world=2, tp=cfg["tp"], tp_rank=cfg["tp_rank"])
    S = om.shard_elems
    arena = torch.full((om.arena_bytes,), 0xA5, dtype=torch.uint8, device=DEV)
    shard = torch.empty(S, dtype=torch.int32, device=DEV)
    for half in (0, 1):
        plan, _ = _models(cfg, world=2, rank=half, gathered=False)
        synth.cuda_fill_f32(shard, seed, synth.BUF_MASTER, start=half * S)
        plan.reshard(shard, arena)
        torch.cuda.synchronize()
        plan.close()
    del shard
    page = mmap.PAGESIZE
    mm_src = mmap.mmap(-1, -(-4 * 2 * S // page) * page)
    mm_dst = mmap.mmap(-1, -(-om.arena_bytes // page) * page)
    flat = np.frombuffer(mm_src, dtype=np.uint32)
    want = np.frombuffer(mm_dst, dtype=np.uint8)

    def release(mm, lo, hi):  # give whole pages inside [lo, hi) back
        a, b = -(-lo // page) * page, hi // page * page
        if b > a:
            mm.madvise(mmap.MADV_DONTNEED, a, b - a)

    srcs = om.src_tensors()
    dst = om.dst_tensors()
    groups = ["embed"] + [f"layers.{l}." for l in range(cfg["spec"]["n_layers"])] + ["final_norm", "lm_head"]

    def check_group(g):
        """Generate the group's source, run the oracle on its rollout tensors, compare with the GPU arena, release."""
        mine = [s for s in srcs if s.name == g or (g.endswith(".") and s.name.startswith(g))]
        lo = min(s.flat_off for s in mine)
        hi = max(s.flat_off + s.rows * s.cols for s in mine)
        synth.fill_f32(seed, synth.BUF_MASTER, lo, hi - lo, out=flat[lo:hi])
        n = 0
        for i, d in enumerate(dst):
            if d.alias_of >= 0 or not (d.name == g or (g.endswith(".") and d.name.startswith(g))):
                continue
            nbytes = d.rows * d.cols * 2
            want[d.arena_off:d.arena_off + nbytes] = 0xA5
            om.forward(flat, want, gathered=True, only=i)
            got = arena[d.arena_off:d.arena_off + nbytes].cpu().numpy()
            assert np.array_equal(got, want[d.arena_off:d.arena_off + nbytes]), d.name
            release(mm_dst, d.arena_off, d.arena_off + nbytes)
            n += d.rows * d.cols
        release(mm_src, 4 * lo, 4 * hi)
        return n

    # the groups are independent: several run at once on the host cores (the oracle itself stays single-threaded)
    from concurrent.futures import ThreadPoolExecutor
    with ThreadPoolExecutor(max_workers=min(6, os.cpu_count() or 1)) as ex:
        checked = sum(ex.map(check_group, groups))
    assert checked == 29_767_972_864
    del flat, want


def test_cfg1_streamed_repack_equals_resident_repack():
    """The 6.9 GB source of the Qwen3-1.7B-shaped workload streamed from pinned host memory through a 512 MiB
    window: the arena on the device and its copy on the host equal the resident dr_reshard result
    (itself compared whole with the oracle above)."""
    _need(12)
    cfg = CONFIGS[1]
    plan, om = _models(cfg)
    seed = seed_of(1)
    src = torch.empty(plan.info.src_bytes // 4, dtype=torch.int32, device=DEV)
    synth.cuda_fill_f32(src, seed, synth.BUF_MASTER)
    ref = torch.full((plan.info.dst_bytes,), 0xA5, dtype=torch.uint8, device=DEV)
    plan.reshard(src, ref)
    h_src = torch.empty(plan.info.src_bytes, dtype=torch.uint8, pin_memory=True)
    h_src.copy_(src.view(torch.uint8))
    del src
    h_dst = torch.zeros(plan.info.dst_bytes, dtype=torch.uint8, pin_memory=True)
    arena = torch.full((plan.info.dst_bytes,), 0xA5, dtype=torch.uint8, device=DEV)
    window = torch.empty(512 << 20, dtype=torch.uint8, device=DEV)
    st = plan.reshard_stream(dr.stream_desc(h_src.data_ptr(), plan.info.src_bytes, arena.data_ptr(), plan.info.dst_bytes,
                                            window.data_ptr(), 512 << 20, chunk_bytes=64 << 20, host_dst=h_dst.data_ptr(),
                                            host_dst_bytes=plan.info.dst_bytes))
    assert st.n_chunks == -(-plan.info.src_bytes // (64 << 20)) and st.d2h_bytes == plan.info.dst_bytes
    assert torch.equal(arena, ref)
    assert torch.equal(h_dst, ref.cpu())
    plan.close()


def test_cfg1_eight_ranks_push_into_two_arenas_equals_oracle():
    """The Qwen3-1.7B-shaped flat buffer cut into its eight FSDP shards: every rank repacks its own shard and
    stores the pieces into two rollout arenas with dr_reshard_push (ranks one after the other on this GPU).
    Both arenas must equal the oracle's gathered forward, all 1.72 GB of each."""
    _need(14)
    cfg = CONFIGS[1]
    _, om = _models(cfg)
    seed = seed_of(1)
    S = om.shard_elems
    arenas = [torch.full((om.arena_bytes,), 0xA5, dtype=torch.uint8, device=DEV) for _ in range(2)]
    shard = torch.empty(S, dtype=torch.int32, device=DEV)
    moved = 0
    for r in range(cfg["world"]):
        plan = dr.Plan(cfg["spec"], world=cfg["world"], rank=r, gathered=False, tp=cfg["tp"], tp_rank=cfg["tp_rank"])
        synth.cuda_fill_f32(shard, seed, synth.BUF_MASTER, start=r * S)
        plan.reshard_push(shard, arenas)
        moved += plan.info.elems_moved
        torch.cuda.synchronize()
        plan.close()
    assert moved == 860_349_440
    flat = synth.fill_f32(seed, synth.BUF_MASTER, 0, om.world * S)
    want = np.full(om.arena_bytes, 0xA5, dtype=np.uint8)
    om.forward(flat, want)
    for a in arenas:
        assert np.array_equal(a.cpu().numpy(), want)


def test_cfg2_fp8_inverse_full_size_sampled_tensors():
    """Qwen3-8B-shaped fp8 arena (random codes, scales of weight-like size) back to the 32.8 GB flat buffer:
    the oracle's inverse on every tensor of layers 0 and 35 (the layers' whole flat ranges are compared)."""
    _need(50)
    cfg = CONFIGS[2]
    plan = dr.Plan(cfg["spec"], dtype=dr.DR_FP8_E4M3_B128)
    om = oracle.Model(cfg["spec"])
    total, lay = om.fp8_layout()
    assert plan.info.dst_bytes == total
    arena = torch.empty(total, dtype=torch.uint8, device=DEV)
    synth.cuda_fill_bf16(arena[:total // 2 * 2].view(torch.int16), seed_of(2), synth.BUF_ROLLOUT)   # every byte value occurs
    dst = om.dst_tensors()
    rng = np.random.default_rng(4)
    for d, (qz, off, soff) in zip(dst, lay):                      # sane block scales for the quantised tensors
        if qz and d.alias_of < 0:
            nb = (-(-d.rows // 128)) * (-(-d.cols // 128))
            sc = np.exp(rng.uniform(-12, -6, nb)).astype(np.float32)
            arena[soff:soff + 4 * nb] = torch.from_numpy(sc.view(np.uint8)).to(DEV)
    flat = torch.full((om.flat_elems,), 0x5A5A5A5A, dtype=torch.int32, device=DEV)
    plan.reshard_inverse(arena, flat)
    torch.cuda.synchronize()
    host_arena = np.empty(total, dtype=np.uint8)                   # lazily committed; only the tested tensors are filled
    want = np.empty(om.flat_elems, dtype=np.uint32)
    srcs = {s.name: s for s in om.src_tensors()}
    for layer in (0, 35):
        names = [n for n in srcs if n.startswith(f"layers.{layer}.")]
        lo = min(srcs[n].flat_off for n in names)
        hi = max(srcs[n].flat_off + srcs[n].rows * srcs[n].cols for n in names)
        want[lo:hi] = 0x5A5A5A5A
        for i, (d, (qz, off, soff)) in enumerate(zip(dst, lay)):
            if d.name.startswith(f"layers.{layer}."):
                nbytes = d.rows * d.cols * (1 if qz else 2)
                host_arena[off:off + nbytes] = arena[off:off + nbytes].cpu().numpy()
                if qz:
                    nb = 4 * (-(-d.rows // 128)) * (-(-d.cols // 128))
                    host_arena[soff:soff + nb] = arena[soff:soff + nb].cpu().numpy()
                om.inverse_fp8(host_arena, want, only=i)   # the oracle's loop over this rollout tensor alone
        got = flat[lo:hi].cpu().numpy().view(np.uint32)
        assert np.array_equal(got, want[lo:hi]), layer
    plan.close()
