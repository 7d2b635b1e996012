"""Host logic of the CUDA library, checked without a GPU: the planner's segment table expanded to a
per-element map must be the oracle's map; sizes, tensor descriptors and error codes."""
import ctypes as C
import re
import os

import numpy as np
import pytest

import oracle
import paper_2607_22614_b200 as dr
from synth.configs import BRUTE, CONFIGS, MID

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def expand(plan, es):
    """flat index (relative to the buffer the call receives) of every arena element slot the
    segment table writes; -1 elsewhere.  Also checks that no slot is written twice."""
    n_slots = plan.info.dst_bytes // es
    m = np.full(n_slots, -1, dtype=np.int64)
    moved = 0
    for s in plan.segments():
        assert s.dst_off % es == 0
        rows = np.arange(s.rows, dtype=np.int64)[:, None]
        cols = np.arange(s.row_len, dtype=np.int64)[None, :]
        d = (s.dst_off // es + rows * s.dst_row_stride + cols).ravel()
        f = (s.src_off + rows * s.src_row_stride + cols).ravel()
        assert (m[d] == -1).all(), "two segments write the same arena element"
        m[d] = f
        moved += s.rows * s.row_len
        if s.vector_bytes:
            assert s.row_len % 8 == 0 and s.dst_off % (8 * es) == 0 and (s.src_off * 4) % s.vector_bytes == 0
            if s.rows > 1:
                assert (s.src_row_stride * 4) % s.vector_bytes == 0 and s.dst_row_stride % 8 == 0
    assert moved == plan.info.elems_moved
    return m


def oracle_map(om, es, gathered, rank):
    n_slots = om.arena_bytes // es
    m = np.full(n_slots, -1, dtype=np.int64)
    lo, hi = rank * om.shard_elems, (rank + 1) * om.shard_elems
    for i, d in enumerate(om.dst_tensors()):
        if d.alias_of >= 0:
            continue
        f = om.map_rows(i, 0, d.rows, d.cols).ravel()
        if not gathered:
            f = np.where((f >= lo) & (f < hi), f - lo, -1)
        m[d.arena_off // es:d.arena_off // es + f.size] = f
    return m


CASES = []
for cfg in BRUTE:
    for T in (1, 2):
        for (W, gathered, A) in ((1, True, 1), (3, True, 4), (3, False, 1), (2, False, 16), (5, False, 3)):
            for dtype in (dr.DR_BF16, dr.DR_F32):
                CASES.append((cfg["name"], cfg["spec"], T, W, gathered, A, dtype))
for cfg in MID + [CONFIGS[0]]:
    CASES.append((cfg["name"], cfg["spec"], 2, 1, True, 1, dr.DR_BF16))
    CASES.append((cfg["name"], cfg["spec"], 2, 3, False, 1, dr.DR_BF16))
    CASES.append((cfg["name"], cfg["spec"], 1, 2, False, 4, dr.DR_F32))


@pytest.mark.parametrize("name,spec,T,W,gathered,A,dtype", CASES,
                         ids=[f"{c[0]}-tp{c[2]}-w{c[3]}-g{int(c[4])}-a{c[5]}-d{c[6]}" for c in CASES])
def test_segment_table_is_the_oracle_map(name, spec, T, W, gathered, A, dtype):
    es = 2 if dtype == dr.DR_BF16 else 4
    for t in range(T):
        for r in (range(W) if not gathered else (0,)):
            p = dr.Plan(spec, world=W, rank=r, gathered=gathered, align_elems=A, tp=T, tp_rank=t, dtype=dtype,
                        arena_align_bytes=64, host_only=True)
            om = oracle.Model(spec, align=A, world=W, tp=T, tp_rank=t, elem_size=es, arena_align=64)
            assert p.info.flat_elems == om.flat_elems and p.info.shard_elems == om.shard_elems
            assert p.info.dst_bytes == om.arena_bytes
            assert p.info.src_bytes == 4 * (W * om.shard_elems if gathered else om.shard_elems)
            assert p.info.bytes_moved_fwd == p.info.elems_moved * (4 + es) == p.info.bytes_moved_inv
            assert np.array_equal(expand(p, es), oracle_map(om, es, gathered, r))
            for a, b in zip(p.tensors(), om.dst_tensors()):
                assert (a.name.decode(), a.arena_off, a.rows, a.cols, a.alias_of) == \
                       (b.name, b.arena_off, b.rows, b.cols, b.alias_of)
            p.close()


def test_full_size_plans_match_quoted_sizes():
    quoted_moved = {"tiny": 987_904, "qwen3-1.7b": 860_349_440, "qwen3-8b": 8_190_735_360,
                    "qwen3-30b-a3b": 29_767_972_864}
    for cfg in CONFIGS:
        p = dr.Plan(cfg["spec"], world=cfg["world"], rank=cfg["rank"], gathered=cfg["gathered"], tp=cfg["tp"],
                    tp_rank=cfg["tp_rank"], host_only=True)
        om = oracle.Model(cfg["spec"], world=cfg["world"], tp=cfg["tp"], tp_rank=cfg["tp_rank"])
        assert p.info.flat_elems == cfg["flat_elems"] and p.info.dst_bytes == om.arena_bytes
        if cfg["name"] in quoted_moved:
            assert p.info.elems_moved == quoted_moved[cfg["name"]]
        segs = p.segments()
        assert all(s.vector_bytes == 32 for s in segs)  # the benchmark shapes never need the scalar path
        # sampled elements of sampled segments agree with the oracle's single-element map
        rng = np.random.default_rng(1)
        dst = om.dst_tensors()
        lo = 0 if cfg["gathered"] else cfg["rank"] * om.shard_elems
        starts = np.array([d.arena_off if d.alias_of < 0 else -1 for d in dst])
        own = np.flatnonzero(starts >= 0)
        for s in [segs[i] for i in rng.integers(0, len(segs), size=min(60, len(segs)))]:
            for _ in range(20):
                i, j = int(rng.integers(0, s.rows)), int(rng.integers(0, s.row_len))
                byte = s.dst_off + (i * s.dst_row_stride + j) * 2
                ti = int(own[np.searchsorted(starts[own], byte, side="right") - 1])  # merged runs span tensors
                d = dst[ti]
                slot = (byte - d.arena_off) // 2
                assert slot < d.rows * d.cols
                assert om.map(ti, slot // d.cols, slot % d.cols) == lo + s.src_off + i * s.src_row_stride + j
        p.close()


def test_plans_far_larger_than_the_workloads_keep_64_bit_arithmetic_and_segment_limits():
    """A 70B-class dense shape (6.9e10 elements) and a 235B-class MoE shape (2.3e11 elements): element counts
    equal the closed form, every segment stays inside the buffers and below the per-segment unit limit, and
    sampled elements agree with the oracle's map.  Host only: nothing is allocated."""
    shapes = [dict(n_layers=80, hidden=8192, n_q_heads=64, n_kv_heads=8, head_dim=128, ffn=28672, vocab=128256,
                   n_experts=0, moe_ffn=0, tied=0, qk_norm=0),
              dict(n_layers=94, hidden=4096, n_q_heads=64, n_kv_heads=4, head_dim=128, ffn=0, vocab=151936,
                   n_experts=128, moe_ffn=1536, tied=0, qk_norm=1)]
    for spec, T in zip(shapes, (8, 4)):
        H, hd, nq, nkv, V, L = (spec[k] for k in ("hidden", "head_dim", "n_q_heads", "n_kv_heads", "vocab", "n_layers"))
        mlp = 3 * H * spec["ffn"] if not spec["n_experts"] else spec["n_experts"] * H + 3 * spec["n_experts"] * H * spec["moe_ffn"]
        closed = 2 * V * H + L * (2 * H + 2 * hd * spec["qk_norm"] + 2 * H * nq * hd + 2 * H * nkv * hd + mlp) + H
        p = dr.Plan(spec, world=16, rank=5, gathered=True, tp=T, tp_rank=T - 1, host_only=True)
        assert p.info.flat_elems == closed > (1 << 36)
        om = oracle.Model(spec, world=16, tp=T, tp_rank=T - 1)
        assert p.info.dst_bytes == om.arena_bytes and p.info.src_bytes == 4 * 16 * om.shard_elems
        segs = p.segments()
        n_src = p.info.src_bytes // 4
        assert sum(s.rows * s.row_len for s in segs) == p.info.elems_moved
        for s in segs:
            assert s.src_off + (s.rows - 1) * s.src_row_stride + s.row_len <= n_src
            assert s.dst_off + ((s.rows - 1) * s.dst_row_stride + s.row_len) * 2 <= p.info.dst_bytes
            assert s.rows * -(-s.row_len // 8) < (1 << 32)
        dst = om.dst_tensors()
        starts = np.array([d.arena_off if d.alias_of < 0 else -1 for d in dst])
        own = np.flatnonzero(starts >= 0)
        rng = np.random.default_rng(2)
        for s in [segs[i] for i in rng.integers(0, len(segs), size=40)] + [segs[0], segs[-1]]:
            for _ in range(5):
                i, j = int(rng.integers(0, s.rows)), int(rng.integers(0, s.row_len))
                byte = s.dst_off + (i * s.dst_row_stride + j) * 2
                ti = int(own[np.searchsorted(starts[own], byte, side="right") - 1])
                d = dst[ti]
                slot = (byte - d.arena_off) // 2
                assert om.map(ti, slot // d.cols, slot % d.cols) == s.src_off + i * s.src_row_stride + j
        p.close()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "dynaresize.h")).read()
    declared = set(re.findall(r"\b(dr_[a-z_]+)\s*\(", header)) - {"dr_chunk_fn"}
    assert declared == set(dr.EXPORTS)
    L = C.CDLL(dr.lib_path)
    for name in declared:
        assert getattr(L, name) is not None


def test_struct_sizes_match_the_header_layout():
    assert C.sizeof(dr.dr_model_spec) == 48 and C.sizeof(dr.dr_src_layout) == 28 and C.sizeof(dr.dr_dst_layout) == 36
    assert C.sizeof(dr.dr_stage_desc) == 448 and C.sizeof(dr.dr_stream_desc) == 112 and C.sizeof(dr.dr_stage_stats) == 112 and C.sizeof(dr.dr_plan_info) == 112 and C.sizeof(dr.dr_tensor_desc) == 128 and C.sizeof(dr.dr_segment_desc) == 56


def test_error_codes():
    spec = BRUTE[0]["spec"]
    with pytest.raises(dr.DrError) as e:
        dr.Plan(spec, tp=4, host_only=True)
    assert e.value.status == dr.binding.DR_ERR_UNSUPPORTED
    with pytest.raises(dr.DrError) as e:
        dr.Plan(spec, tp=2, tp_rank=2, host_only=True)
    assert e.value.status == dr.binding.DR_ERR_INVALID
    with pytest.raises(dr.DrError) as e:
        dr.Plan(spec, arena_align_bytes=24, host_only=True)
    assert e.value.status == dr.binding.DR_ERR_INVALID
    s = dr.model_spec(spec)
    s.version = 99
    rc, h = dr.dr_plan_create_host(s, dr.src_layout(), dr.dst_layout(), 1, 0)
    assert rc == dr.binding.DR_ERR_INVALID and not h
    rc, h = dr.dr_plan_create_host(dr.model_spec(spec), dr.src_layout(), dr.dst_layout(moe_tp=2), 1, 0)
    assert rc == dr.binding.DR_ERR_UNSUPPORTED
    # a host-only plan answers queries but refuses to launch or stage
    p = dr.Plan(spec, host_only=True)
    assert dr.dr_reshard(p.handle, 16, 1 << 30, 32, 1 << 30, None) == dr.binding.DR_ERR_STATE
    d = dr.stage_desc([16], [4096], budget=1 << 20, host_arena=4096, host_arena_bytes=4096)
    rc, _ = dr.dr_stage_out(p.handle, d)
    assert rc == dr.binding.DR_ERR_STATE
    d = dr.stage_desc([16], [4096], budget=4096, chunk=4096, host_arena=4096, host_arena_bytes=4096)
    rc, _ = dr.dr_stage_out(p.handle, d)
    assert rc == dr.binding.DR_ERR_BUDGET
    # the deferred form checks the same things before it starts anything
    rc, job = dr.dr_stage_begin(p.handle, d, dr.DR_STAGE_DIR_OUT)
    assert rc == dr.binding.DR_ERR_BUDGET and not job
    d = dr.stage_desc([16], [4096], budget=1 << 20, host_arena=4096, host_arena_bytes=4096)
    assert dr.dr_stage_begin(p.handle, d, dr.DR_STAGE_DIR_IN)[0] == dr.binding.DR_ERR_STATE
    assert dr.dr_stage_begin(p.handle, d, 2)[0] == dr.binding.DR_ERR_INVALID
    assert dr.dr_stage_end(None)[0] == dr.binding.DR_ERR_INVALID and dr.dr_stage_poll(None)[0] == dr.binding.DR_ERR_INVALID
    assert dr.dr_plan_tensor(p.handle, 10_000)[0] == dr.binding.DR_ERR_INVALID
    assert "budget" in dr.dr_strerror(dr.binding.DR_ERR_BUDGET)
    assert dr.dr_plan_destroy(None) == 0


def test_host_copy_workers_copy_every_byte():
    """The staging engine's host-copy workers (1 MiB tasks taken by several threads), run on their own through
    dr_host_copy: odd sizes, sizes below and above one task, one and many threads, unaligned ends."""
    rng = np.random.default_rng(0)
    for n, threads in ((0, 2), (1, 1), (4097, 3), ((1 << 20) - 1, 2), ((1 << 20) + 1, 16), (5 * (1 << 20) + 12345, 4), (33_333_333, 0)):
        src = rng.integers(0, 256, size=n + 64, dtype=np.uint64).astype(np.uint8)
        dst = np.full(n + 128, 0x5A, dtype=np.uint8)
        rc = dr.dr_host_copy(dst.ctypes.data + 31, src.ctypes.data + 7, n, threads)
        assert rc == 0
        assert np.array_equal(dst[31:31 + n], src[7:7 + n])
        assert (dst[:31] == 0x5A).all() and (dst[31 + n:] == 0x5A).all()
    assert dr.dr_host_copy(None, 4096, 16, 1) == dr.binding.DR_ERR_INVALID


def test_shard_range():
    assert dr.dr_shard_range(1000, 6, 0) == (0, 0, 167, 167)
    assert dr.dr_shard_range(1000, 6, 5) == (0, 835, 1000, 167)      # last shard holds 165 real elements
    assert dr.dr_shard_range(5, 8, 4) == (0, 4, 5, 1)
    assert dr.dr_shard_range(5, 8, 7) == (0, 5, 5, 1)                # all padding
    assert dr.dr_shard_range(5, 8, 8)[0] == dr.binding.DR_ERR_INVALID
    assert dr.dr_shard_range(5, 0, 0)[0] == dr.binding.DR_ERR_INVALID
    for n, w in ((1_975_808, 2), (14_768_307_200, 4), (17, 3)):
        ends = [dr.dr_shard_range(n, w, r)[1:3] for r in range(w)]
        assert ends[0][0] == 0 and ends[-1][1] == n and all(a[1] == b[0] for a, b in zip(ends, ends[1:]))


VARIANTS = [
    (dict(BRUTE[0]["spec"], ffn=12), 4, dict(kv_replicate=True, vocab_pad=8)),
    (MID[0]["spec"], 16, dict(kv_replicate=True)),
    (MID[1]["spec"], 4, dict(vocab_pad=64)),
    (dict(MID[1]["spec"], tied=0), 2, dict(vocab_pad=1024)),
    (BRUTE[2]["spec"], 2, dict(moe_tp=2)),
    (BRUTE[2]["spec"], 2, dict(moe_ep=2, moe_ep_rank=1)),
    (MID[2]["spec"], 4, dict(moe_tp=4, moe_ep=2, moe_ep_rank=0, vocab_pad=64)),
    (MID[2]["spec"], 8, dict(kv_replicate=True, moe_ep=4, moe_ep_rank=3)),
]


@pytest.mark.parametrize("spec,T,opts", VARIANTS, ids=[f"v{i}" for i in range(len(VARIANTS))])
@pytest.mark.parametrize("W,gathered", [(1, True), (3, False)])
def test_layout_variants_segment_table_is_the_oracle_map(spec, T, opts, W, gathered):
    for t in sorted({0, 1, T - 1}):
        r = W - 1
        p = dr.Plan(spec, world=W, rank=r, gathered=gathered, tp=T, tp_rank=t, arena_align_bytes=64, host_only=True, **opts)
        om = oracle.Model(spec, world=W, tp=T, tp_rank=t, arena_align=64, **opts)
        assert p.info.dst_bytes == om.arena_bytes
        assert np.array_equal(expand(p, 2), oracle_map(om, 2, gathered, r))
        for a, b in zip(p.tensors(), om.dst_tensors()):
            assert (a.name.decode(), a.arena_off, a.rows, a.cols, a.alias_of) == (b.name, b.arena_off, b.rows, b.cols, b.alias_of)
        p.close()


def test_layout_variant_errors():
    E = dr.binding
    for kw, tp, want in ((dict(), 4, E.DR_ERR_UNSUPPORTED), (dict(kv_replicate=True), 3, E.DR_ERR_UNSUPPORTED)):
        with pytest.raises(dr.DrError) as e:
            dr.Plan(MID[0]["spec"] if tp == 3 else dict(BRUTE[0]["spec"], ffn=12), tp=tp, host_only=True, **kw)
        assert e.value.status == want
    with pytest.raises(dr.DrError) as e:
        dr.Plan(BRUTE[2]["spec"], tp=2, moe_ep=3, host_only=True)
    assert e.value.status == E.DR_ERR_UNSUPPORTED
    with pytest.raises(dr.DrError) as e:
        dr.Plan(BRUTE[2]["spec"], tp=2, moe_ep=2, moe_ep_rank=2, host_only=True)
    assert e.value.status == E.DR_ERR_INVALID
    with pytest.raises(dr.DrError) as e:
        dr.Plan(MID[2]["spec"], tp=4, moe_tp=2, host_only=True)
    assert e.value.status == E.DR_ERR_UNSUPPORTED


@pytest.mark.parametrize("spec,T,opts", [(MID[0]["spec"], 2, {}), (MID[2]["spec"], 2, dict(moe_ep=2, moe_ep_rank=1)),
                                         (dict(BRUTE[0]["spec"], ffn=12), 2, {}), (CONFIGS[2]["spec"], 1, {})],
                         ids=["mid-dense", "mid-moe-ep", "brute", "qwen3-8b"])
def test_fp8_plan_layout_matches_oracle(spec, T, opts):
    for t in range(T):
        p = dr.Plan(spec, tp=T, tp_rank=t, dtype=dr.DR_FP8_E4M3_B128, arena_align_bytes=64, host_only=True, **opts)
        om = oracle.Model(spec, tp=T, tp_rank=t, arena_align=64, **opts)
        total, lay = om.fp8_layout()
        assert p.info.dst_bytes == total
        q_elems = q_blocks = 0
        for a, b, (qz, off, soff) in zip(p.tensors(), om.dst_tensors(), lay):
            assert (a.name.decode(), a.rows, a.cols, a.alias_of, bool(a.quantised), a.arena_off) == \
                   (b.name, b.rows, b.cols, b.alias_of, qz and b.alias_of < 0 or qz, off)
            if qz:
                assert a.elem_size == 1 and a.scale_off == soff
                assert (a.scale_rows, a.scale_cols) == (-(-b.rows // 128), -(-b.cols // 128))
                q_elems += b.rows * b.cols
                q_blocks += a.scale_rows * a.scale_cols
            elif b.alias_of < 0:
                assert a.elem_size == 2
        assert (p.info.quant_elems, p.info.quant_blocks) == (q_elems, q_blocks)
        copied = p.info.elems_moved - q_elems
        assert p.info.bytes_moved_fwd == copied * 6 + q_elems * 5 + q_blocks * 4
        # the copy segments cover exactly the non-quantised tensors
        assert sum(s.rows * s.row_len for s in p.segments()) == copied == \
            sum(b.rows * b.cols for b, (qz, _, _) in zip(om.dst_tensors(), lay) if not qz and b.alias_of < 0)
        p.close()


def test_fp8_plan_restrictions():
    E = dr.binding
    with pytest.raises(dr.DrError) as e:
        dr.Plan(MID[0]["spec"], world=2, rank=0, gathered=False, dtype=dr.DR_FP8_E4M3_B128, host_only=True)
    assert e.value.status == E.DR_ERR_UNSUPPORTED
    p = dr.Plan(MID[0]["spec"], world=2, rank=1, gathered=True, dtype=dr.DR_FP8_E4M3_B128, host_only=True)
    assert p.info.quant_blocks > 0


def test_plan_with_nothing_to_move():
    """More ranks than elements: the last shards hold only padding, the plan is empty and still valid."""
    spec = dict(n_layers=0, hidden=4, n_q_heads=1, n_kv_heads=1, head_dim=2, ffn=4, vocab=2, tied=1, qk_norm=1)
    full = dr.Plan(spec, host_only=True)
    assert full.info.flat_elems == 12
    p = dr.Plan(spec, world=16, rank=15, gathered=False, host_only=True)
    assert p.info.shard_elems == 1 and p.info.n_segments == 0 and p.info.n_tiles == 0 and p.info.elems_moved == 0
    assert p.info.dst_bytes == full.info.dst_bytes


@pytest.mark.parametrize("spec,kw,chunk", [
    (MID[0]["spec"], dict(tp=2, tp_rank=1), 2_499_992), (MID[2]["spec"], dict(tp=2, tp_rank=0, moe_ep=2, moe_ep_rank=1), 1_000_003),
    (BRUTE[0]["spec"], dict(tp=2, tp_rank=1, align_elems=3), 16), (MID[1]["spec"], dict(world=3, rank=1, gathered=False, tp=2), 600_001),
    (BRUTE[2]["spec"], dict(dtype=dr.DR_F32), 7)], ids=["dense-tp2", "moe-ep", "brute", "shard-local", "brute-moe-f32"])
def test_source_windows_partition_the_plan(spec, kw, chunk):
    """The per-chunk plans of the streamed repack: together they write exactly what the whole plan writes, each
    from inside its own window, and nothing twice."""
    es = 4 if kw.get("dtype") == dr.DR_F32 else 2
    p = dr.Plan(spec, arena_align_bytes=64, host_only=True, **kw)
    whole = expand(p, es)
    n_src = p.info.src_bytes // 4
    union = np.full_like(whole, -1)
    moved = 0
    for lo in range(0, n_src, chunk):
        hi = min(lo + chunk, n_src)
        w = p.window(lo, hi)
        assert w.info.src_bytes == 4 * (hi - lo) and w.info.dst_bytes == p.info.dst_bytes
        m = expand(w, es)                      # indices relative to the window
        hit = m >= 0
        assert (m[hit] < hi - lo).all()
        assert (union[hit] == -1).all()        # no arena element comes from two windows
        union[hit] = m[hit] + lo
        moved += w.info.elems_moved
        w.close()
    assert np.array_equal(union, whole) and moved == p.info.elems_moved
    assert dr.dr_plan_window_host(p.handle, 5, 5)[0] == dr.binding.DR_ERR_INVALID
    assert dr.dr_plan_window_host(p.handle, 0, n_src + 1)[0] == dr.binding.DR_ERR_INVALID
    p.close()


def test_groups_partition_the_plan():
    for cfg, kw in ((CONFIGS[2], {}), (CONFIGS[4], {}), (MID[1], dict(world=3, rank=2, gathered=False, tp=2)),
                    (BRUTE[2], dict(tp=2, tp_rank=1))):
        kw = dict(kw)
        if "world" in cfg and not kw:
            kw = dict(world=cfg["world"], rank=cfg["rank"], gathered=cfg["gathered"], tp=cfg["tp"], tp_rank=cfg["tp_rank"])
        p = dr.Plan(cfg["spec"], host_only=True, **kw)
        L = cfg["spec"]["n_layers"]
        assert p.info.n_groups == L + 2
        names = [t.name.decode() for t in p.tensors()]
        nxt, elems = 0, 0
        for g in range(p.info.n_groups):
            rc, d = dr.dr_plan_group(p.handle, g)
            assert rc == 0 and d.first_tensor == nxt and d.bytes_moved == d.elems * 6
            mine = names[d.first_tensor:d.first_tensor + d.n_tensors]
            if g == 0:
                assert mine == ["embed"]
            elif g <= L:
                assert mine and all(n.startswith(f"layers.{g - 1}.") for n in mine)
            else:
                assert mine == ["final_norm", "lm_head"]
            nxt += d.n_tensors
            elems += d.elems
        assert nxt == len(names) and elems == p.info.elems_moved
        assert dr.dr_plan_group(p.handle, p.info.n_groups)[0] == dr.binding.DR_ERR_INVALID
        p.close()
