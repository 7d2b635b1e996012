"""Pins for the oracle's layout map (D1-D4): closed-form counts, reconstruction with torch CPU
chunk/cat, brute-force coverage on tiny specs, and agreement of its two formulations."""
import numpy as np
import pytest
import torch

import oracle
from synth.configs import BRUTE, CONFIGS, MID
from torch_layout import named_params, rollout_state


def closed_form(s):
    H, hd = s["hidden"], s["head_dim"]
    mlp = 3 * H * s["ffn"] if s["n_experts"] == 0 else s["n_experts"] * H + 3 * s["n_experts"] * H * s["moe_ffn"]
    per = 2 * H + (2 * hd if s["qk_norm"] else 0) + 2 * H * s["n_q_heads"] * hd + 2 * H * s["n_kv_heads"] * hd + mlp
    return s["vocab"] * H * (2 - s["tied"]) + s["n_layers"] * per + H


def test_flat_counts_match_published_totals(golden):
    want = {r[0]: int(r[1]) for r in golden("param_counts.txt")}
    for cfg in CONFIGS:
        m = oracle.Model(cfg["spec"], world=cfg["world"], tp=cfg["tp"], tp_rank=cfg["tp_rank"])
        assert m.flat_elems == want[cfg["name"]] == closed_form(cfg["spec"]) == cfg["flat_elems"]
        assert m.shard_elems == -(-m.flat_elems // cfg["world"])
        src = m.src_tensors()
        assert sum(t.rows * t.cols for t in src) == m.flat_elems
        offs = np.array([t.flat_off for t in src])
        assert (np.diff(offs) == np.array([t.rows * t.cols for t in src[:-1]])).all()  # align 1: dense packing


def test_rollout_counts_per_rank():
    for cfg in CONFIGS:
        s, T = cfg["spec"], cfg["tp"]
        H, hd = s["hidden"], s["head_dim"]
        if s["n_experts"] == 0:
            mlp = 3 * H * s["ffn"] // T
        else:
            mlp = s["n_experts"] * H + 3 * s["n_experts"] * H * s["moe_ffn"]
        per = 2 * H + 2 * hd + (2 * H * s["n_q_heads"] * hd + 2 * H * s["n_kv_heads"] * hd) // T + mlp
        want = s["vocab"] // T * H * (2 - s["tied"]) + s["n_layers"] * per + H
        for t in range(T):
            m = oracle.Model(s, tp=T, tp_rank=t)
            got = sum(d.rows * d.cols for d in m.dst_tensors() if d.alias_of < 0)
            assert got == want
    # the destination sizes quoted for the five workloads
    quoted = {"qwen3-1.7b": 860_349_440, "qwen3-14b": 3_692_395_520, "qwen3-30b-a3b": 29_767_972_864}
    for cfg in CONFIGS:
        if cfg["name"] in quoted:
            m = oracle.Model(cfg["spec"], tp=cfg["tp"], tp_rank=cfg["tp_rank"])
            assert sum(d.rows * d.cols for d in m.dst_tensors() if d.alias_of < 0) == quoted[cfg["name"]]


def _arena_tensor(m, arena, d, dtype):
    n = d.rows * d.cols
    return arena[d.arena_off:d.arena_off + n * dtype().itemsize].view(dtype).reshape(d.rows, d.cols)


CASES = [(c["name"], c["spec"], T) for c in BRUTE + MID for T in (1, 2)] + [("tiny", CONFIGS[0]["spec"], 1),
                                                                            ("tiny", CONFIGS[0]["spec"], 2)]


@pytest.mark.parametrize("name,spec,T", CASES, ids=[f"{n}-tp{T}" for n, _, T in CASES])
def test_forward_equals_torch_chunk_cat(name, spec, T):
    """fp32 layout-only plan with source value = its own flat index: every rollout element names its
    origin, and must be where torch's chunk/cat puts it."""
    N = closed_form(spec)
    iota = torch.arange(N, dtype=torch.int32)
    params = named_params(spec, iota)
    covered = np.zeros(N, dtype=np.int64)
    for t in range(T):
        m = oracle.Model(spec, tp=T, tp_rank=t, elem_size=4, arena_align=64)
        assert m.flat_elems == N
        arena = np.full(m.arena_bytes, 0xEE, dtype=np.uint8)
        m.forward(iota.numpy().view(np.uint32), arena)
        want = rollout_state(spec, params, T, t)
        written = np.zeros(m.arena_bytes, dtype=bool)
        for i, d in enumerate(m.dst_tensors()):
            if d.alias_of >= 0:
                assert spec["tied"] and d.name == "lm_head" and m.dst_tensors()[d.alias_of].name == "embed"
                continue
            got = _arena_tensor(m, arena, d, np.int32)
            w = want[d.name].reshape(d.rows, d.cols).numpy()
            assert np.array_equal(got, w), d.name
            assert d.arena_off % 64 == 0
            written[d.arena_off:d.arena_off + d.rows * d.cols * 4] = True
            np.add.at(covered, got.ravel(), 1)
            # the single-element map agrees with the loop formulation
            fm = m.map_rows(i, 0, d.rows, d.cols)
            assert np.array_equal(fm, got)
        assert (arena[~written] == 0xEE).all()  # arena gaps untouched
    # over all ranks: sliced positions exactly once, replicated (norms, router, experts) exactly T times
    rep = np.ones(N, dtype=np.int64)
    for n, p in params.items():
        leaf = n.split(".")[-1]
        if leaf.endswith("norm") or leaf == "router" or ".experts." in n:
            rep[p.flatten().numpy()] = T
    assert np.array_equal(covered, rep)


def test_slices_concatenate_to_the_full_tensors():
    spec, T = MID[0]["spec"], 4
    N = closed_form(spec)
    vals = torch.arange(N, dtype=torch.int32)
    params = named_params(spec, vals)
    ranks = []
    for t in range(T):
        m = oracle.Model(spec, tp=T, tp_rank=t, elem_size=4)
        arena = np.zeros(m.arena_bytes, dtype=np.uint8)
        m.forward(vals.numpy().view(np.uint32), arena)
        ranks.append({d.name: torch.from_numpy(_arena_tensor(m, arena, d, np.int32).copy()) for d in m.dst_tensors()})
    hd = spec["head_dim"]
    nq, nkv = spec["n_q_heads"] * hd // T, spec["n_kv_heads"] * hd // T
    F = spec["ffn"] // T
    assert torch.equal(torch.cat([r["embed"] for r in ranks]), params["embed"])
    assert torch.equal(torch.cat([r["lm_head"] for r in ranks]), params["lm_head"])
    for l in range(spec["n_layers"]):
        p = f"layers.{l}."
        assert torch.equal(torch.cat([r[p + "qkv"][:nq] for r in ranks]), params[p + "q"])
        assert torch.equal(torch.cat([r[p + "qkv"][nq:nq + nkv] for r in ranks]), params[p + "k"])
        assert torch.equal(torch.cat([r[p + "qkv"][nq + nkv:] for r in ranks]), params[p + "v"])
        assert torch.equal(torch.cat([r[p + "gate_up"][:F] for r in ranks]), params[p + "gate"])
        assert torch.equal(torch.cat([r[p + "gate_up"][F:] for r in ranks]), params[p + "up"])
        assert torch.equal(torch.cat([r[p + "o"] for r in ranks], dim=1), params[p + "o"])
        assert torch.equal(torch.cat([r[p + "down"] for r in ranks], dim=1), params[p + "down"])


def test_alignment_padding_and_tail():
    """align_elems > 1 inserts gaps that no rollout element maps to; W not dividing N pads the tail."""
    spec = BRUTE[0]["spec"]
    for A in (4, 16):
        m = oracle.Model(spec, align=A, world=3, elem_size=4)
        src = m.src_tensors()
        assert all(t.flat_off % A == 0 for t in src)
        assert all(b.flat_off >= a.flat_off + a.rows * a.cols and b.flat_off - (a.flat_off + a.rows * a.cols) < A
                   for a, b in zip(src, src[1:]))
        assert m.flat_elems == src[-1].flat_off + src[-1].rows * src[-1].cols
        assert m.shard_elems == -(-m.flat_elems // 3)
        hit = np.zeros(m.flat_elems, dtype=bool)
        for i, d in enumerate(m.dst_tensors()):
            f = m.map_rows(i, 0, d.rows, d.cols)
            assert not hit[f.ravel()].any()  # injective
            hit[f.ravel()] = True
        real = np.zeros(m.flat_elems, dtype=bool)
        for t in src:
            real[t.flat_off:t.flat_off + t.rows * t.cols] = True
        assert np.array_equal(hit, real)  # padding never mapped, every real element mapped (T = 1)


def test_bf16_forward_is_the_cast_of_the_layout_only_forward():
    spec = MID[2]["spec"]
    N = closed_form(spec)
    rng = np.random.default_rng(3)
    src = rng.integers(0, 1 << 32, size=N, dtype=np.uint64).astype(np.uint32)
    m4 = oracle.Model(spec, tp=2, tp_rank=1, elem_size=4)
    m2 = oracle.Model(spec, tp=2, tp_rank=1, elem_size=2)
    a4 = np.zeros(m4.arena_bytes, dtype=np.uint8)
    a2 = np.zeros(m2.arena_bytes, dtype=np.uint8)
    m4.forward(src, a4)
    m2.forward(src, a2)
    for d4, d2 in zip(m4.dst_tensors(), m2.dst_tensors()):
        if d4.alias_of >= 0:
            continue
        x = _arena_tensor(m4, a4, d4, np.uint32)
        y = _arena_tensor(m2, a2, d2, np.uint16)
        nan = (x & 0x7FFFFFFF) > 0x7F800000
        t = torch.from_numpy(x.view(np.float32).copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        assert np.array_equal(y[~nan], t[~nan]) and (y[nan] == 0x7FFF).all()


def test_unsupported_divisibility_is_rejected():
    spec = dict(BRUTE[0]["spec"])
    with pytest.raises(ValueError):
        oracle.Model(spec, tp=4)  # 2 kv heads cannot be split 4 ways: no replication
    with pytest.raises(ValueError):
        oracle.Model(spec, tp=3)


VARIANTS = [
    # (spec, tp, options)
    (dict(BRUTE[0]["spec"], ffn=12), 4, dict(kv_replicate=True, vocab_pad=8)),   # 2 kv heads on 4 ranks; vocab 6 -> 8
    (MID[0]["spec"], 16, dict(kv_replicate=True)),                               # 8 kv heads on 16 ranks
    (MID[1]["spec"], 4, dict(vocab_pad=64)),                                     # vocab 5000 -> 5056, tied
    (dict(MID[1]["spec"], tied=0), 2, dict(vocab_pad=1024)),                     # last rank partly padding
    (BRUTE[2]["spec"], 2, dict(moe_tp=2)),                                       # expert FFN sliced
    (BRUTE[2]["spec"], 2, dict(moe_ep=2, moe_ep_rank=1)),                        # expert block 1 of 2
    (MID[2]["spec"], 4, dict(moe_tp=4, moe_ep=2, moe_ep_rank=0, vocab_pad=64)),
    (MID[2]["spec"], 8, dict(kv_replicate=True, moe_ep=4, moe_ep_rank=3)),
]


@pytest.mark.parametrize("spec,T,opts", VARIANTS, ids=[f"v{i}" for i in range(len(VARIANTS))])
def test_layout_variants_equal_torch_chunk_cat(spec, T, opts):
    N = closed_form(spec)
    iota = torch.arange(N, dtype=torch.int32)
    params = named_params(spec, iota)
    for t in sorted({0, 1, T // 2, T - 1}):
        m = oracle.Model(spec, tp=T, tp_rank=t, elem_size=4, arena_align=64, **opts)
        arena = np.full(m.arena_bytes, 0xFF, dtype=np.uint8)  # int32 -1 wherever nothing is written
        m.forward(iota.numpy().view(np.uint32), arena)
        want = rollout_state(spec, params, T, t, fill=-1, **opts)
        for i, d in enumerate(m.dst_tensors()):
            if d.alias_of >= 0:
                continue
            got = _arena_tensor(m, arena, d, np.int32)
            w = want[d.name].reshape(d.rows, d.cols).numpy()
            assert np.array_equal(got, w), (d.name, t)
            assert np.array_equal(m.map_rows(i, 0, d.rows, d.cols), got)  # unmapped padding rows are -1 in both
        # inverse restores exactly what forward read
        back = np.full(N, 0x7E7E7E7E, dtype=np.uint32)
        m.inverse(arena, back)
        hit = back != 0x7E7E7E7E
        assert np.array_equal(back[hit], iota.numpy().view(np.uint32)[hit])
        mapped = np.concatenate([m.map_rows(i, 0, d.rows, d.cols).ravel()
                                 for i, d in enumerate(m.dst_tensors()) if d.alias_of < 0])
        assert hit.sum() == np.unique(mapped[mapped >= 0]).size


def test_variant_divisibility_rules():
    with pytest.raises(ValueError):
        oracle.Model(BRUTE[0]["spec"], tp=4)                              # needs kv_replicate
    with pytest.raises(ValueError):
        oracle.Model(MID[0]["spec"], tp=3, kv_replicate=True)             # 3 is not a multiple of 8 kv heads
    with pytest.raises(ValueError):
        oracle.Model(MID[1]["spec"], tp=16)                               # vocab 5000 needs padding for 16 ranks
    with pytest.raises(ValueError):
        oracle.Model(BRUTE[2]["spec"], tp=2, moe_ep=3)                    # 4 experts, 3 blocks
    with pytest.raises(ValueError):
        oracle.Model(BRUTE[2]["spec"], tp=4, kv_replicate=True, moe_tp=2) # moe_tp is 1 or tp
