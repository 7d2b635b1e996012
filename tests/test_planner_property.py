"""Property test of the planner: for random small model shapes, layouts and variants, the segment table
expanded element by element is the oracle's map, no arena element is written twice, and every access
stays inside the buffers the plan asks for."""
import numpy as np
from hypothesis import HealthCheck, given, settings, strategies as st

import oracle
import paper_2607_22614_b200 as dr
from test_planner_host import expand, oracle_map


@st.composite
def cases(draw):
    tp = draw(st.sampled_from([1, 2, 4]))
    moe = draw(st.booleans())
    kv_rep = draw(st.booleans()) and tp > 1
    nkv = draw(st.sampled_from([1, 2])) if kv_rep else tp * draw(st.integers(1, 2))
    if kv_rep and tp % nkv:
        nkv = 1
    hd = draw(st.integers(1, 9))
    spec = dict(n_layers=draw(st.integers(0, 2)), hidden=draw(st.integers(1, 24)), n_q_heads=tp * draw(st.integers(1, 2)),
                n_kv_heads=nkv, head_dim=hd, ffn=0 if moe else tp * draw(st.integers(1, 9)),
                vocab=draw(st.integers(1, 20)), n_experts=draw(st.sampled_from([2, 4])) if moe else 0,
                moe_ffn=tp * draw(st.integers(1, 5)) if moe else 0, tied=int(draw(st.booleans())), qk_norm=int(draw(st.booleans())))
    opts = dict(kv_replicate=kv_rep, vocab_pad=tp * draw(st.integers(1, 4)))
    if moe:
        ep = draw(st.sampled_from([1, 2]))
        opts.update(moe_tp=draw(st.sampled_from([1, tp])), moe_ep=ep, moe_ep_rank=draw(st.integers(0, ep - 1)))
    world = draw(st.integers(1, 5))
    return dict(spec=spec, tp=tp, tp_rank=draw(st.integers(0, tp - 1)), world=world, rank=draw(st.integers(0, world - 1)),
                gathered=draw(st.booleans()), align=draw(st.sampled_from([1, 1, 3, 4, 8])),
                dtype=draw(st.sampled_from([dr.DR_BF16, dr.DR_F32])), arena_align=draw(st.sampled_from([16, 64, 256])), opts=opts)


@settings(max_examples=400, deadline=None, derandomize=True, database=None, suppress_health_check=[HealthCheck.too_slow])
@given(cases())
def test_random_plans_equal_the_oracle_map(c):
    es = 2 if c["dtype"] == dr.DR_BF16 else 4
    om = oracle.Model(c["spec"], align=c["align"], world=c["world"], tp=c["tp"], tp_rank=c["tp_rank"], elem_size=es,
                      arena_align=c["arena_align"], **c["opts"])
    p = dr.Plan(c["spec"], world=c["world"], rank=c["rank"], gathered=c["gathered"], align_elems=c["align"], tp=c["tp"],
                tp_rank=c["tp_rank"], dtype=c["dtype"], arena_align_bytes=c["arena_align"], host_only=True, **c["opts"])
    assert p.info.dst_bytes == om.arena_bytes and p.info.flat_elems == om.flat_elems
    assert np.array_equal(expand(p, es), oracle_map(om, es, c["gathered"], c["rank"]))
    n_src = p.info.src_bytes // 4
    for s in p.segments():
        assert s.src_off + (s.rows - 1) * s.src_row_stride + s.row_len <= n_src
        assert s.dst_off + ((s.rows - 1) * s.dst_row_stride + s.row_len) * es <= p.info.dst_bytes
    p.close()
