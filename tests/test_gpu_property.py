"""GPU property test: random small shapes, layouts and variants through dr_reshard, dr_reshard_inverse and
dr_reshard_stream, each compared with the oracle bit for bit (deterministic example sequence)."""
import numpy as np
import pytest
import torch
from hypothesis import HealthCheck, given, settings

import oracle
import paper_2607_22614_b200 as dr
from gpu_util import SENT8, dev, first_diff
from test_planner_property import cases

pytestmark = pytest.mark.gpu


@settings(max_examples=60, deadline=None, derandomize=True, suppress_health_check=list(HealthCheck))
@given(cases())
def test_random_plans_on_the_gpu(c):
    es = 2 if c["dtype"] == dr.DR_BF16 else 4
    om = oracle.Model(c["spec"], align=c["align"], world=c["world"], tp=c["tp"], tp_rank=c["tp_rank"], elem_size=es,
                      arena_align=c["arena_align"], **c["opts"])
    plan = dr.Plan(c["spec"], world=c["world"], rank=c["rank"], gathered=c["gathered"], align_elems=c["align"], tp=c["tp"],
                   tp_rank=c["tp_rank"], dtype=c["dtype"], arena_align_bytes=c["arena_align"], **c["opts"])
    S, W, r, g = om.shard_elems, c["world"], c["rank"], c["gathered"]
    rng = np.random.default_rng(om.flat_elems * 31 + W)
    full = rng.integers(0, 1 << 32, size=W * S, dtype=np.uint64).astype(np.uint32)
    local = full if g else full[r * S:(r + 1) * S].copy()
    n_arena = max(om.arena_bytes, 32)
    want = np.full(n_arena, SENT8, dtype=np.uint8)
    om.forward(local, want, gathered=g, rank=r)
    src = torch.from_numpy(local.view(np.int32)).to(dev())
    arena = torch.full((n_arena,), SENT8, dtype=torch.uint8, device=dev())
    plan.reshard(src, arena)
    torch.cuda.synchronize()
    assert first_diff(arena.cpu().numpy(), want) is None
    # inverse of the oracle's arena into a sentinel-filled flat buffer
    wflat = np.full(local.size, 0xDEADBEEF, dtype=np.uint32)
    om.inverse(want, wflat, gathered=g, rank=r)
    flat = torch.full((local.size,), 0xDEADBEEF - (1 << 32), dtype=torch.int32, device=dev())
    plan.reshard_inverse(torch.from_numpy(want).to(dev()), flat)
    torch.cuda.synchronize()
    assert first_diff(flat.cpu().numpy().view(np.uint32), wflat) is None
    # streamed repack of the same source: 96-byte chunks through a 3-slot window
    if local.nbytes >= 32:
        h_src = torch.from_numpy(np.concatenate([local, np.zeros(8, dtype=np.uint32)]).view(np.int32)).pin_memory()
        h_dst = torch.full((n_arena,), SENT8, dtype=torch.uint8).pin_memory()
        arena2 = torch.full((n_arena,), SENT8, dtype=torch.uint8, device=dev())
        window = torch.empty(96 * 3, dtype=torch.uint8, device=dev())
        d = dr.stream_desc(h_src.data_ptr(), local.nbytes, arena2.data_ptr(), n_arena, window.data_ptr(), 96 * 3,
                           chunk_bytes=96, host_dst=h_dst.data_ptr(), host_dst_bytes=n_arena)
        plan.reshard_stream(d)
        assert first_diff(arena2.cpu().numpy(), want) is None
        assert first_diff(h_dst.numpy()[:om.arena_bytes], want[:om.arena_bytes]) is None
    plan.close()
