"""Helpers for the GPU parity tests: run the CUDA path through the C ABI, run the oracle on the same
seeded inputs, compare bit for bit."""
import numpy as np
import torch

import oracle
import paper_2607_22614_b200 as dr
import synth

SENT8 = 0xA5


def dev():
    return torch.device("cuda:0")


def to_dev_u32(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(a.view(np.int32)).to(dev())


def arena_dev(nbytes: int, fill=SENT8) -> torch.Tensor:
    return torch.full((nbytes,), fill, dtype=torch.uint8, device=dev())


def special_values() -> np.ndarray:
    """Bit patterns that exercise ties, carries, overflow, subnormals, infinities and NaNs."""
    from conftest import read_golden
    vals = [int(r[0], 16) for r in read_golden("cast_rne.txt")]
    vals += [0x7FFFFFFF, 0xFFFFFFFF, 0x7FBFFFFF, 0x00000000, 0x00010000, 0x0000FFFF, 0x807FFFFF, 0x7F000000]
    return np.array(vals, dtype=np.uint32)


def make_source(n: int, seed: int, with_specials: bool = True) -> np.ndarray:
    src = synth.fill_f32(seed, synth.BUF_MASTER, 0, n)
    if with_specials:
        sp = special_values()
        rng = np.random.default_rng(seed)
        pos = rng.integers(0, n, size=min(n, 40 * sp.size))
        src[pos] = np.resize(sp, pos.size)
    return src


def forward_both(spec, *, world=1, rank=0, gathered=True, align=1, tp=1, tp_rank=0, dtype=dr.DR_BF16,
                 arena_align=256, src=None, seed=1, arena_init=None, misalign=0, **opts):
    """Returns (gpu arena bytes, oracle arena bytes, plan, oracle model, src) for one forward call."""
    es = 2 if dtype == dr.DR_BF16 else 4
    om = oracle.Model(spec, align=align, world=world, tp=tp, tp_rank=tp_rank, elem_size=es, arena_align=arena_align,
                      **opts)
    n_src = world * om.shard_elems if gathered else om.shard_elems
    if src is None:
        src = make_source(world * om.shard_elems, seed)
    local = src if gathered else src[rank * om.shard_elems:(rank + 1) * om.shard_elems].copy()
    assert local.size == n_src
    want = np.full(om.arena_bytes, SENT8, dtype=np.uint8) if arena_init is None else arena_init[0].copy()
    om.forward(local, want, gathered=gathered, rank=rank)
    plan = dr.Plan(spec, world=world, rank=rank, gathered=gathered, align_elems=align, tp=tp, tp_rank=tp_rank,
                   dtype=dtype, arena_align_bytes=arena_align, **opts)
    assert plan.info.dst_bytes == om.arena_bytes and plan.info.src_bytes == 4 * n_src
    # misalign > 0 shifts both device buffers by that many bytes (a multiple of 16) off their 256-byte
    # allocation boundary, which forces the 128-bit access path
    pad = misalign // 4
    s_buf = torch.zeros(n_src + pad, dtype=torch.int32, device=dev())
    s_dev = s_buf[pad:]
    s_dev.copy_(torch.from_numpy(local.view(np.int32)))
    # guard bands of 256 sentinel bytes on both sides of the arena: a write outside the arena would show there
    G = 256
    a_buf = arena_dev(G + misalign + om.arena_bytes + G)
    a_dev = a_buf[G + misalign:G + misalign + om.arena_bytes]
    if arena_init is not None:
        a_dev.copy_(arena_init[1])
    plan.reshard(s_dev, a_dev)
    torch.cuda.synchronize()
    got = a_dev.cpu().numpy()
    assert (a_buf[:G + misalign].cpu().numpy() == SENT8).all() and (a_buf[G + misalign + om.arena_bytes:].cpu().numpy() == SENT8).all()
    return got, want, plan, om, src


def first_diff(a, b):
    d = np.flatnonzero(a != b)
    return None if d.size == 0 else (int(d[0]), int(d.size))
