"""The exchange that follows the local repack (weight synchronisation between roles), as far as CPU ranks
can prove it: the per-rank arena byte ranges from the planner are exactly what the oracle's element map
covers for that shard, they partition the gathered result over the FSDP ranks, and two gloo ranks that
repack their own shards with the oracle and all-gather those ranges end up with the gathered oracle arena."""
import json
import os
import subprocess
import sys

import numpy as np
import pytest

import oracle
import paper_2607_22614_b200 as dr
from synth.configs import BRUTE, CONFIGS, MID
from test_planner_host import oracle_map

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CASES = [(BRUTE[0]["spec"], 2, 1, 3, 1, dr.DR_BF16), (BRUTE[0]["spec"], 1, 0, 5, 3, dr.DR_F32),
         (BRUTE[1]["spec"], 2, 0, 8, 16, dr.DR_F32), (BRUTE[2]["spec"], 2, 0, 4, 4, dr.DR_BF16),
         (CONFIGS[0]["spec"], 1, 0, 2, 1, dr.DR_BF16), (MID[2]["spec"], 2, 1, 3, 1, dr.DR_BF16)]


def _mask(ranges, nbytes):
    m = np.zeros(nbytes, dtype=np.int32)
    prev_end = -1
    for off, n in ranges:
        assert n > 0 and off > prev_end, "ranges must be ascending, non-empty and not touching (coalesced)"
        prev_end = off + n
        m[off:off + n] += 1
    return m


@pytest.mark.parametrize("spec,T,t,W,A,dtype", CASES, ids=[f"x{i}" for i in range(len(CASES))])
def test_rank_ranges_are_the_bytes_the_oracle_map_covers_and_partition_the_gathered_arena(spec, T, t, W, A, dtype):
    es = 2 if dtype == dr.DR_BF16 else 4
    om = oracle.Model(spec, align=A, world=W, tp=T, tp_rank=t, elem_size=es)
    full = dr.Plan(spec, world=W, gathered=True, align_elems=A, tp=T, tp_rank=t, dtype=dtype, host_only=True)
    full_mask = _mask(full.ranges(), om.arena_bytes)
    want_full = np.repeat(oracle_map(om, es, True, 0) >= 0, es).astype(np.int32)
    assert np.array_equal(full_mask[:want_full.size], want_full) and not full_mask[want_full.size:].any()
    union = np.zeros(om.arena_bytes, dtype=np.int32)
    total = 0
    for r in range(W):
        p = dr.Plan(spec, world=W, rank=r, gathered=False, align_elems=A, tp=T, tp_rank=t, dtype=dtype, host_only=True)
        rr = p.ranges()
        m = _mask(rr, om.arena_bytes)
        want = np.repeat(oracle_map(om, es, False, r) >= 0, es).astype(np.int32)
        assert np.array_equal(m[:want.size], want)                   # exactly the bytes this shard produces
        assert sum(n for _, n in rr) == p.info.elems_moved * es
        union += m
        total += p.info.elems_moved
        p.close()
    assert np.array_equal(union, full_mask)                           # disjoint over ranks, union = gathered
    assert total == full.info.elems_moved
    full.close()


def test_ranges_call_contract():
    p = dr.Plan(MID[0]["spec"], tp=2, tp_rank=1, host_only=True)
    n = dr.binding.u64()
    assert dr.lib().dr_plan_ranges(p.handle, 0, None, n) == 0 and n.value == len(p.ranges()) > 0
    two = (dr.dr_range * 2)()
    assert dr.lib().dr_plan_ranges(p.handle, 2, two, n) == 0                # a short buffer gets the first entries
    assert (two[0].off, two[0].bytes) == p.ranges()[0] and (two[1].off, two[1].bytes) == p.ranges()[1]
    assert dr.lib().dr_plan_ranges(p.handle, 2, None, n) == dr.binding.DR_ERR_INVALID
    p.close()
    q = dr.Plan(MID[0]["spec"], dtype=dr.DR_FP8_E4M3_B128, host_only=True)
    assert dr.dr_plan_ranges(q.handle)[0] == dr.binding.DR_ERR_UNSUPPORTED
    q.close()
    # TP = 1 dense plan: everything is one contiguous run per gap-free stretch, so there are few ranges
    p = dr.Plan(CONFIGS[2]["spec"], host_only=True)
    r = p.ranges()
    assert sum(n for _, n in r) == 2 * p.info.elems_moved and len(r) <= p.info.n_tensors
    p.close()


def test_two_gloo_ranks_repack_their_shards_and_all_gather_the_ranges():
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", "29613", os.path.join("tests", "exchange_worker.py")]
    r = subprocess.run(cmd, cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-3000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 2 and {l["rank"] for l in lines} == {0, 1}
    for l in lines:
        assert l["equal_to_gathered_oracle"] and l["sentinel_gaps_intact"] and l["received_bytes"] > 0
    # what crossed the "wire" is the other rank's share of the mapped bf16 bytes, half of gathering fp32
    assert lines[0]["received_bytes"] + lines[1]["received_bytes"] == lines[0]["mapped_bytes"]
