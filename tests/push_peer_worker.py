"""Child process of the cross-process push test: it plays FSDP rank 1.  The parent's rollout arena arrives as a CUDA
tensor shared through CUDA IPC (torch.multiprocessing does the handle exchange), i.e. as memory this process did not
allocate and reaches through a peer mapping; the child repacks its own shard and stores the pieces into its own arena
and into the parent's with one dr_reshard_push, synchronises, and reports."""
import os
import sys

import numpy as np
import torch

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def run(parent_arena, spec, world, tp, tp_rank, seed, result_queue):
    import paper_2607_22614_b200 as dr
    import synth
    try:
        torch.cuda.set_device(0)
        plan = dr.Plan(spec, world=world, rank=1, gathered=False, tp=tp, tp_rank=tp_rank)
        S = plan.info.shard_elems
        shard = torch.empty(S, dtype=torch.int32, device="cuda:0")
        synth.cuda_fill_f32(shard, seed, synth.BUF_MASTER, start=S)           # rank 1's elements of the flat buffer
        own = torch.full((plan.info.dst_bytes,), 0xA5, dtype=torch.uint8, device="cuda:0")
        plan.reshard_push(shard, [own, parent_arena])
        torch.cuda.synchronize()                                               # the pieces are in the parent's memory
        ranges = plan.ranges()
        digest = int(own.to(torch.int64).sum().item())
        plan.close()
        result_queue.put(("ok", len(ranges), digest))
    except Exception as exc:  # reported to the parent, which fails the test
        result_queue.put(("error", repr(exc), 0))
