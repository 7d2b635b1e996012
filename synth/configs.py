"""The five benchmark workloads: model shapes, source/destination layouts and staging budgets.

Shapes only (Qwen3-class decoders); the weights themselves come from the seeded generator.  Sizes in
"MB"/"GB" of the workload descriptions are read as MiB/GiB for budgets and chunk sizes.
"""
from __future__ import annotations

MiB, GiB = 1 << 20, 1 << 30


def _spec(L, H, nq, nkv, hd, F, V, tied, E=0, Fm=0):
    return dict(n_layers=L, hidden=H, n_q_heads=nq, n_kv_heads=nkv, head_dim=hd, ffn=F, vocab=V,
                n_experts=E, moe_ffn=Fm, tied=int(tied), qk_norm=1)


CONFIGS = [
    dict(name="tiny", spec=_spec(2, 256, 4, 2, 64, 688, 1024, False),
         world=2, rank=0, gathered=False, tp=1, tp_rank=0, direction="fwd",
         stage=("m", "v"), budget=1 * MiB, flat_elems=1_975_808),
    dict(name="qwen3-1.7b", spec=_spec(28, 2048, 16, 8, 128, 6144, 151936, True),
         world=8, rank=3, gathered=True, tp=2, tp_rank=0, direction="fwd",
         stage=(), budget=0, flat_elems=1_720_574_976),
    dict(name="qwen3-8b", spec=_spec(36, 4096, 32, 8, 128, 12288, 151936, False),
         world=1, rank=0, gathered=True, tp=1, tp_rank=0, direction="fwd",
         stage=("master", "m", "v"), budget=2 * GiB, flat_elems=8_190_735_360),
    dict(name="qwen3-14b", spec=_spec(40, 5120, 40, 8, 128, 17408, 151936, False),
         world=4, rank=1, gathered=False, tp=4, tp_rank=1, direction="inv",
         stage=("master", "m", "v"), budget=4 * GiB, flat_elems=14_768_307_200),
    dict(name="qwen3-30b-a3b", spec=_spec(48, 2048, 32, 4, 128, 0, 151936, False, E=128, Fm=768),
         world=1, rank=0, gathered=True, tp=2, tp_rank=1, direction="fwd",
         stage=(), budget=0, flat_elems=30_532_122_624),
]

# Small specs whose whole element map can be enumerated by brute force (odd sizes on purpose:
# nothing is a multiple of the vector width, several tensors start at unaligned offsets).
BRUTE = [
    dict(name="brute-dense", spec=dict(_spec(1, 12, 4, 2, 3, 10, 6, False))),
    dict(name="brute-dense-tied", spec=dict(_spec(2, 12, 4, 2, 3, 10, 6, True))),
    dict(name="brute-moe", spec=dict(_spec(2, 8, 4, 2, 4, 0, 6, False, E=4, Fm=6))),
]

# A mid-size dense spec and a mid-size MoE spec: large enough to span many tiles and ragged tails,
# small enough for the CPU oracle to finish in seconds.
MID = [
    dict(name="mid-dense", spec=_spec(3, 1024, 16, 8, 64, 2816, 8192, False)),
    dict(name="mid-dense-tied", spec=_spec(2, 768, 12, 4, 64, 2048, 5000, True)),
    dict(name="mid-moe", spec=_spec(2, 512, 8, 4, 64, 0, 4096, False, E=8, Fm=192)),
]


def seed_of(cfg_index: int) -> int:
    return 0xD15A0000 + cfg_index
