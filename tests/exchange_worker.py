"""Worker for the world-size-2 gloo test of the exchange step: every rank repacks its own FSDP shard with the
oracle (standing in for its GPU), packs the arena ranges its shard-local plan lists, all-gathers the packed
pieces, and unpacks the other ranks' pieces at the ranges their plans list.  The arena must then equal the
oracle's gathered forward."""
import json
import os
import sys

import numpy as np
import torch
import torch.distributed as dist

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import oracle  # noqa: E402
import paper_2607_22614_b200 as dr  # noqa: E402
from synth.configs import MID  # noqa: E402
import synth  # noqa: E402

dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
spec, T, t = MID[0]["spec"], 2, 1
om = oracle.Model(spec, world=world, tp=T, tp_rank=t)
flat = synth.fill_f32(99, synth.BUF_MASTER, 0, world * om.shard_elems)       # every rank can regenerate any shard
mine = flat[rank * om.shard_elems:(rank + 1) * om.shard_elems].copy()
arena = np.full(om.arena_bytes, 0xA5, dtype=np.uint8)
om.forward(mine, arena, gathered=False, rank=rank)                            # the local repack

# topology-scoped metadata, computed once per (world, tp, rank): every rank's send list
plans = [dr.Plan(spec, world=world, rank=r, gathered=False, tp=T, tp_rank=t, host_only=True) for r in range(world)]
ranges = [p.ranges() for p in plans]
sizes = [sum(n for _, n in rr) for rr in ranges]
packed = np.concatenate([arena[o:o + n] for o, n in ranges[rank]]) if ranges[rank] else np.zeros(0, np.uint8)
assert packed.size == sizes[rank]
pad = max(sizes)
send = torch.zeros(pad, dtype=torch.uint8)
send[:packed.size] = torch.from_numpy(packed)
recv = [torch.zeros(pad, dtype=torch.uint8) for _ in range(world)]
dist.all_gather(recv, send)
received = 0
for r in range(world):
    if r == rank:
        continue
    buf, pos = recv[r].numpy(), 0
    for o, n in ranges[r]:
        arena[o:o + n] = buf[pos:pos + n]
        pos += n
    received += pos
want = np.full(om.arena_bytes, 0xA5, dtype=np.uint8)
om.forward(flat, want, gathered=True)
mapped = np.zeros(om.arena_bytes, dtype=bool)
for rr in ranges:
    for o, n in rr:
        mapped[o:o + n] = True
out = {"rank": rank, "equal_to_gathered_oracle": bool(np.array_equal(arena, want)),
       "sentinel_gaps_intact": bool((arena[~mapped] == 0xA5).all()), "received_bytes": int(received),
       "mapped_bytes": int(mapped.sum())}
for p in plans:
    p.close()
gathered = [None] * world
dist.all_gather_object(gathered, out)
dist.barrier()
dist.destroy_process_group()
if rank == 0:  # one writer: lines of two processes could interleave
    for o in gathered:
        print(json.dumps(o), flush=True)
