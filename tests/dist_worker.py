"""Worker for the world-size-2 gloo test: the bench's multi-process plumbing, on CPU."""
import json
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import bench  # noqa: E402

ctx = bench.Dist("gloo")
ctx.barrier()
slowest = ctx.max(10.0 + 5.0 * ctx.rank)          # rank r "took" 10 + 5 r ms
value = bench.whole_job_gbs(ctx.world, 1_000_000_000, 4, slowest)
ctx.close()
if ctx.rank == 0:
    print(json.dumps({"world": ctx.world, "slowest_ms": slowest, "value": value}))
