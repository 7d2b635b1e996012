#!/usr/bin/env python
"""Benchmark of the role-switch state transform on B200.

One step = the device-resident transform of one whole model in both switch directions through the
C ABI: ``dr_reshard`` (Training -> Rollout: un-flatten, fuse, TP-slice, cast to bf16) followed by
``dr_reshard_inverse`` (Rollout -> Training).  ``value`` is the algorithmic bytes of those two calls
over the device time of K steps.  The same run also measures, outside the K-step loop because they
are bound by the host link and take seconds: chunked stage-out / stage-in of the fp32 master and Adam
state, the switch latencies, the end-to-end number with host buffers, and the CPU oracle on a bounded
sample.  Prints one JSON line on rank 0.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--cfg I] [--impl reference]
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "role-switch transform GB/s (% of HBM peak); stage-out/in GB/s; switch ms"
GiB = 1 << 30
MiB = 1 << 20
# DRAM bytes per element (dram__bytes_read.sum + dram__bytes_write.sum over elements moved) of the forward
# kernel, from the committed ncu capture summary of this kernel (a 654 M-element case of the
# same kernel; traffic grows in proportion to the elements, so it is scaled to the launch timed here).
NCU_DRAM_BYTES_PER_ELEMENT_FWD = 5.949


def load_peaks():
    """Measured HBM copy bandwidth of this machine's B200s (generated file), else the stated fallback."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def mem_available_bytes() -> int:
    with open("/proc/meminfo") as f:
        for line in f:
            if line.startswith("MemAvailable:"):
                return int(line.split()[1]) * 1024
    return 0


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.path = None

    def _lines(self) -> int:
        try:
            with open(self.path) as f:
                return sum(1 for _ in f)
        except OSError:
            return 0

    def start(self):
        """Starts nvidia-smi and waits (at most 5 s) for its first line: the tool needs a few hundred milliseconds to
        come up, which is longer than a short timed region.  Call before the warm-up steps."""
        fd, self.path = tempfile.mkstemp(suffix=".csv")
        os.close(fd)
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None
            return
        t0 = time.time()
        while self._lines() == 0 and time.time() - t0 < 5 and self.proc.poll() is None:
            time.sleep(0.02)

    def mark(self):
        """The timed region starts here: earlier samples are not used."""
        self.first = self._lines() if self.proc is not None else 0

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.06)  # one more sample period, so that the region's last sample is written
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as f:
            for k, line in enumerate(f):
                if k < getattr(self, "first", 0):
                    continue
                p = [x.strip() for x in line.split(",")]
                if len(p) < 7:
                    continue
                try:
                    sm.append(float(p[0]))
                    mx.append(float(p[1]))
                except ValueError:
                    continue
                for n, v in zip(names, p[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
        os.unlink(self.path)
        sm.sort()
        # the load is bursty: the median of the upper half is the clock while kernels ran
        busy = sm[len(sm) // 2:] if sm else []
        return {"sm_mhz": busy[len(busy) // 2] if busy else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


class Dist:
    """One process per GPU under torchrun (RANK / LOCAL_RANK / WORLD_SIZE / MASTER_* from the environment).
    The path has no exchange step, so the process group only carries the barrier and the max-over-ranks of
    the timings; `backend="gloo"` runs the same plumbing on CPU for the tests."""

    def __init__(self, backend: str = "nccl", device=None):
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        self.device = device
        self.backend = backend
        if self.world > 1:
            import torch.distributed as dist
            kw = {"device_id": device} if backend == "nccl" and device is not None else {}
            dist.init_process_group(backend, **kw)

    def barrier(self):
        import torch
        if self.world > 1:
            import torch.distributed as dist
            dist.barrier()
        if self.backend == "nccl":
            torch.cuda.synchronize()

    def max(self, x: float) -> float:
        if self.world == 1:
            return x
        import torch
        import torch.distributed as dist
        t = torch.tensor([x], dtype=torch.float64, device=self.device if self.backend == "nccl" else "cpu")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def close(self):
        if self.world > 1:
            import torch.distributed as dist
            dist.barrier()
            dist.destroy_process_group()


def whole_job_gbs(world: int, bytes_per_rank_step: int, steps: int, max_ms_over_ranks: float) -> float:
    """Replicas only: every rank moves the same bytes; the job's rate is all ranks' bytes over the slowest rank's time."""
    return world * bytes_per_rank_step * steps / max_ms_over_ranks / 1e6


def workload_name(cfg) -> str:
    return (f"cfg{cfg['index']} {cfg['name']}: fp32 flat master -> bf16 rollout arena at TP={cfg['tp']} "
            f"rank {cfg['tp_rank']}, and back")


def median(xs):
    s = sorted(xs)
    return s[len(s) // 2]


# ------------------------------------------------------------------------------------------------
# CPU oracle legs (the only places this file touches oracle/)
# ------------------------------------------------------------------------------------------------
def oracle_sample(cfg, seconds: float, max_layers: int = 1 << 30):
    """Times the oracle's forward transform, as it stands, on whole rollout tensors of the workload:
    embed is skipped (4.7 GB of source), layers are taken in order until `seconds` have elapsed.
    The source values come from the seeded generator (its time is not counted).  Returns
    (GB/s on the same 6 B/element accounting, elements, seconds, description)."""
    import numpy as np

    import oracle
    import synth

    om = oracle.Model(cfg["spec"], world=cfg["world"], tp=cfg["tp"], tp_rank=cfg["tp_rank"])
    srcs = {s.name: s for s in om.src_tensors()}
    dst = om.dst_tensors()
    # a lazily committed view of the whole flat buffer: only the sampled layers are ever touched
    flat = np.empty(om.world * om.shard_elems, dtype=np.uint32)
    arena = np.empty(om.arena_bytes, dtype=np.uint8)
    seed = synth.SEED_BASE + cfg["index"]
    elems, spent, layers = 0, 0.0, 0
    for layer in range(min(max_layers, cfg["spec"]["n_layers"])):
        names = [n for n in srcs if n.startswith(f"layers.{layer}.")]
        lo = min(srcs[n].flat_off for n in names)
        hi = max(srcs[n].flat_off + srcs[n].rows * srcs[n].cols for n in names)
        flat[lo:hi] = synth.fill_f32(seed, synth.BUF_MASTER, lo, hi - lo)
        for i, d in enumerate(dst):
            if d.name.startswith(f"layers.{layer}.") and d.alias_of < 0:
                arena[d.arena_off:d.arena_off + d.rows * d.cols * 2].fill(0)  # commit the output pages before timing
                t0 = time.perf_counter()
                om.forward(flat, arena, gathered=True, only=i)
                spent += time.perf_counter() - t0
                elems += d.rows * d.cols
        layers += 1
        if spent >= seconds:
            break
    gbs = elems * 6 / spent / 1e9
    return gbs, elems, spent, f"forward transform of rollout layers 0..{layers - 1} of {cfg['name']} ({elems} elements)"


def oracle_sample_all_cores(cfg, layers: int = 8):
    """The same oracle, one thread per rollout tensor over all host cores (the C loop releases the GIL):
    layers 0..layers-1 of the workload.  Returns (GB/s, threads, elements, seconds)."""
    from concurrent.futures import ThreadPoolExecutor

    import numpy as np

    import oracle
    import synth

    om = oracle.Model(cfg["spec"], world=cfg["world"], tp=cfg["tp"], tp_rank=cfg["tp_rank"])
    srcs = {s.name: s for s in om.src_tensors()}
    flat = np.empty(om.world * om.shard_elems, dtype=np.uint32)
    arena = np.empty(om.arena_bytes, dtype=np.uint8)
    seed = synth.SEED_BASE + cfg["index"]
    layers = min(layers, cfg["spec"]["n_layers"])
    work = []
    for layer in range(layers):
        names = [n for n in srcs if n.startswith(f"layers.{layer}.")]
        lo = min(srcs[n].flat_off for n in names)
        hi = max(srcs[n].flat_off + srcs[n].rows * srcs[n].cols for n in names)
        synth.fill_f32(seed, synth.BUF_MASTER, lo, hi - lo, out=flat[lo:hi])
        for i, d in enumerate(om.dst_tensors()):
            if d.name.startswith(f"layers.{layer}.") and d.alias_of < 0:
                arena[d.arena_off:d.arena_off + d.rows * d.cols * 2].fill(0)  # commit the output pages before timing
                work.append((i, d.rows * d.cols))
    work.sort(key=lambda w: -w[1])  # big tensors first
    threads = os.cpu_count() or 1
    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=threads) as ex:
        list(ex.map(lambda w: om.forward(flat, arena, gathered=True, only=w[0]), work))
    spent = time.perf_counter() - t0
    elems = sum(w[1] for w in work)
    return elems * 6 / spent / 1e9, threads, elems, spent


def run_reference(args, cfg):
    """--impl reference: the oracle on this machine's host cores, each step a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    per_step = max(1.0, min(10.0, 120.0 / max(1, args.steps + args.warmup)))
    for _ in range(args.warmup):
        oracle_sample(cfg, per_step, max_layers=1)
    t_total, e_total, desc = 0.0, 0, ""
    for _ in range(args.steps):
        _, elems, spent, desc = oracle_sample(cfg, per_step, max_layers=1)
        t_total += spent
        e_total += elems
    gbs = e_total * 6 / t_total / 1e9
    line = {"impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_total / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32->bf16", "data": "synthetic",
            "config": {"workload": workload_name(cfg), "step": "oracle forward transform of one layer's rollout tensors "
                       "(bounded sample of the workload)"},
            "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": desc},
            "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def duplex_model_ms(h2d_bytes, d2h_bytes, h2d_alone_gbs, h2d_duplex_gbs, d2h_duplex_gbs):
    """Time of a transfer of h2d_bytes in and d2h_bytes out over a link that runs the two directions at the duplex rates
    while both are busy and the remaining direction at its own rate afterwards (rates in GB/s = bytes / ns)."""
    t_out = d2h_bytes / d2h_duplex_gbs  # ns
    t_in_beside = h2d_bytes / h2d_duplex_gbs
    if t_in_beside <= t_out:
        return t_out / 1e6
    return (t_out + (h2d_bytes - t_out * h2d_duplex_gbs) / h2d_alone_gbs) / 1e6


def engine_copy_threads() -> int:
    """The staging engine's worker count on this machine (its rule, restated for the report)."""
    env = os.environ.get("DR_COPY_THREADS", "")
    if env.isdigit() and 1 <= int(env) <= 64:
        return int(env)
    n = os.cpu_count() or 1
    return max(1, min(16, n - 2 if n > 4 else n))


def run_all(args):
    """The per-workload table: each workload in a process of its own (device memory is returned in between)."""
    for i in range(5):
        cmd = [sys.executable, os.path.abspath(__file__), "--cfg", str(i), "--steps", str(args.steps), "--warmup",
               str(args.warmup), "--no-cpu", "--no-others"] + (["--no-staging"] if args.no_staging or i == 4 else [])
        r = subprocess.run(cmd, capture_output=True, text=True)
        lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
        if r.returncode or not lines:
            print(json.dumps({"cfg": i, "error": (r.stderr or r.stdout)[-300:]}))
            continue
        d = json.loads(lines[-1])
        st = d.get("staging", {})
        print(json.dumps({"cfg": i, "workload": d["config"]["workload"], "value": d["value"],
                          "forward_gbs": d["forward"]["gbs_avg"], "forward_ms": d["forward"]["ms_avg"],
                          "inverse_gbs": d.get("inverse", {}).get("gbs_avg"), "frac_of_measured_peak": d["roofline"]["frac"],
                          "fp8_forward_gbs": d.get("fp8_forward", {}).get("gbs_avg"),
                          "stage_out_gbs": st.get("stage_out_gbs"), "stage_in_gbs": st.get("stage_in_gbs"),
                          "e2e_gbs": d.get("e2e", {}).get("value"), "switch_ms": d.get("switch_ms")}), flush=True)


# ------------------------------------------------------------------------------------------------
# CUDA path
# ------------------------------------------------------------------------------------------------
def quick_transform(i, dev, peak, steps=10, warmup=3):
    """Device-resident forward (and, where a second flat buffer fits, inverse) transform of workload i, timed per
    launch with CUDA events: the per-workload figures that accompany the default workload's line."""
    import torch

    import paper_2607_22614_b200 as dr
    import synth
    from synth.configs import CONFIGS

    cfg = dict(CONFIGS[i], index=i)
    seed = synth.SEED_BASE + i
    kw = dict(tp=cfg["tp"], tp_rank=cfg["tp_rank"])
    free_b, _ = torch.cuda.mem_get_info()
    probe = dr.Plan(cfg["spec"], world=cfg["world"], rank=cfg["rank"], gathered=cfg["gathered"], host_only=True, **kw)
    halves = 2 if cfg["gathered"] and probe.info.src_bytes + probe.info.dst_bytes > free_b * 0.92 else 1
    probe.close()
    if halves == 2:  # does not fit beside its arena: two shard-local halves, back to back, into the same arena
        plans = [dr.Plan(cfg["spec"], world=2, rank=r, gathered=False, **kw) for r in (0, 1)]
    else:
        plans = [dr.Plan(cfg["spec"], world=cfg["world"], rank=cfg["rank"], gathered=cfg["gathered"], **kw)]
    info = plans[0].info
    n_src = info.src_bytes // 4
    base = cfg["rank"] * info.shard_elems if not cfg["gathered"] else 0
    master = torch.empty(n_src, dtype=torch.int32, device=dev)
    synth.cuda_fill_f32(master, seed, synth.BUF_MASTER, start=base)
    arena = torch.empty(info.dst_bytes, dtype=torch.uint8, device=dev)
    synth.cuda_fill_bf16(arena.view(torch.int16), seed, synth.BUF_ROLLOUT)
    do_inverse = halves == 1 and free_b > (2 * info.src_bytes + info.dst_bytes) * 1.05
    flat_back = torch.empty(n_src, dtype=torch.int32, device=dev) if do_inverse else None
    fwd, inv = [], []
    for it in range(warmup + steps):
        ev = []
        for h, p in enumerate(plans):
            if halves == 2:
                synth.cuda_fill_f32(master, seed, synth.BUF_MASTER, start=h * info.shard_elems)
            ev.append(torch.cuda.Event(enable_timing=True)); ev[-1].record()
            p.reshard(master, arena)
            ev.append(torch.cuda.Event(enable_timing=True)); ev[-1].record()
        if do_inverse:
            plans[0].reshard_inverse(arena, flat_back)
            ev.append(torch.cuda.Event(enable_timing=True)); ev[-1].record()
        torch.cuda.synchronize()
        if it >= warmup:
            fwd.append(sum(ev[2 * h].elapsed_time(ev[2 * h + 1]) for h in range(halves)))
            if do_inverse:
                inv.append(ev[-2].elapsed_time(ev[-1]))
    b_fwd = sum(p.info.bytes_moved_fwd for p in plans)
    b_inv = plans[0].info.bytes_moved_inv
    f_ms = sum(fwd) / len(fwd)
    out = {"cfg": i, "workload": workload_name(cfg), "elements": int(sum(p.info.elems_moved for p in plans)),
           "passes": halves, "segments": int(sum(p.info.n_segments for p in plans)), "steps": steps,
           "forward_gbs": b_fwd / f_ms / 1e6, "forward_ms": f_ms, "forward_ms_best": min(fwd),
           "forward_frac_of_measured_peak": b_fwd / f_ms / 1e6 / peak, "forward_frac_of_nominal_8000": b_fwd / f_ms / 1e6 / 8000.0}
    if inv:
        i_ms = sum(inv) / len(inv)
        out.update({"inverse_gbs": b_inv / i_ms / 1e6, "inverse_ms": i_ms,
                    "inverse_frac_of_measured_peak": b_inv / i_ms / 1e6 / peak})
    if info.src_bytes < (64 << 20):
        out["note"] = "working set fits L2: a latency figure, not a bandwidth one"
    for p in plans:
        p.close()
    del master, arena, flat_back
    torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--cfg", type=int, default=2, help="workload index 0..4 (default: Qwen3-8B-shaped, the paper's model)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-staging", action="store_true", help="skip the host-link sections")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle baseline")
    ap.add_argument("--no-fp8", action="store_true", help="skip the fp8 block-quantised variant")
    ap.add_argument("--no-others", action="store_true", help="skip the short device-only runs of the other workloads")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--layers", type=int, default=0, help="profiling aid: override the layer count (smaller case)")
    ap.add_argument("--vocab", type=int, default=0, help="profiling aid: override the vocabulary size")
    ap.add_argument("--profile", action="store_true", help="profiling aid: allow fewer than 3 warm-up steps")
    ap.add_argument("--all", action="store_true", help="run the five workloads one after the other (one process each) "
                                                       "and print one summary line per workload")
    args = ap.parse_args()
    if args.impl == "ours" and not args.profile:
        args.warmup = max(args.warmup, 3)

    from synth.configs import CONFIGS
    cfg = dict(CONFIGS[args.cfg], index=args.cfg)
    if args.layers or args.vocab:
        cfg["spec"] = dict(cfg["spec"], n_layers=args.layers or cfg["spec"]["n_layers"],
                           vocab=args.vocab or cfg["spec"]["vocab"])
        cfg["name"] += f" (reduced: {cfg['spec']['n_layers']} layers, vocab {cfg['spec']['vocab']})"
    if args.all:
        run_all(args)
        return
    if args.impl == "reference":
        run_reference(args, cfg)
        return

    import numpy as np
    import torch

    import paper_2607_22614_b200 as dr
    import synth

    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    ctx = Dist("nccl", dev)
    world, rank = ctx.world, ctx.rank
    barrier, max_over_ranks = ctx.barrier, ctx.max

    peak, peak_kind = load_peaks()
    seed = synth.SEED_BASE + args.cfg
    inverse_dir = cfg["direction"] == "inv"

    # cfg 4 does not fit beside its arena as one buffer: two shard-local halves, back to back
    free_b, _ = torch.cuda.mem_get_info()
    probe = dr.Plan(cfg["spec"], world=cfg["world"], rank=cfg["rank"], gathered=cfg["gathered"], tp=cfg["tp"],
                    tp_rank=cfg["tp_rank"], host_only=True)
    halves = 1
    if probe.info.src_bytes * (1 if args.cfg == 4 else 2) + probe.info.dst_bytes > free_b * 0.92 and cfg["gathered"]:
        halves = 2
    probe.close()
    if halves == 2:
        plans = [dr.Plan(cfg["spec"], world=2, rank=r, gathered=False, tp=cfg["tp"], tp_rank=cfg["tp_rank"]) for r in (0, 1)]
    else:
        plans = [dr.Plan(cfg["spec"], world=cfg["world"], rank=cfg["rank"], gathered=cfg["gathered"], tp=cfg["tp"],
                         tp_rank=cfg["tp_rank"])]
    t0 = time.perf_counter()  # plan compile (host) + table upload: prepared ahead of a switch, not on its critical path
    dr.Plan(cfg["spec"], world=cfg["world"], rank=cfg["rank"], gathered=cfg["gathered"], tp=cfg["tp"],
            tp_rank=cfg["tp_rank"]).close()
    plan_create_ms = (time.perf_counter() - t0) * 1e3
    info = plans[0].info
    n_src = info.src_bytes // 4
    bytes_fwd = sum(p.info.bytes_moved_fwd for p in plans)
    bytes_inv = sum(p.info.bytes_moved_inv for p in plans)

    master = torch.empty(n_src, dtype=torch.int32, device=dev)
    base = cfg["rank"] * info.shard_elems if not cfg["gathered"] else 0
    synth.cuda_fill_f32(master, seed, synth.BUF_MASTER, start=base)
    arena = torch.empty(info.dst_bytes, dtype=torch.uint8, device=dev)
    if inverse_dir:
        synth.cuda_fill_bf16(arena.view(torch.int16), seed, synth.BUF_ROLLOUT)
    do_inverse = halves == 1 and free_b > (2 * info.src_bytes + info.dst_bytes) * 1.05
    flat_back = torch.empty(n_src, dtype=torch.int32, device=dev) if do_inverse else None
    torch.cuda.synchronize()

    def step(events=None):
        for hi, p in enumerate(plans):
            if halves == 2:
                synth.cuda_fill_f32(master, seed, synth.BUF_MASTER, start=hi * info.shard_elems)
            if events is not None:
                events.append(torch.cuda.Event(enable_timing=True))
                events[-1].record()
            p.reshard(master, arena)
            if events is not None:
                events.append(torch.cuda.Event(enable_timing=True))
                events[-1].record()
        if do_inverse:
            plans[0].reshard_inverse(arena, flat_back)
            if events is not None:
                events.append(torch.cuda.Event(enable_timing=True))
                events[-1].record()

    sampler = ClockSampler(local)
    sampler.start()
    for _ in range(args.warmup):
        step()
    barrier()
    evs = []
    wall0 = torch.cuda.Event(enable_timing=True)
    wall1 = torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.mark()
    wall0.record()
    for _ in range(args.steps):
        step(evs)
    wall1.record()
    barrier()
    clocks = sampler.stop()
    per = len(evs) // args.steps
    fwd_ms, inv_ms = [], []
    for s in range(args.steps):
        e = evs[s * per:(s + 1) * per]
        if halves == 2:
            fwd_ms.append(e[0].elapsed_time(e[1]) + e[2].elapsed_time(e[3]))
        else:
            fwd_ms.append(e[0].elapsed_time(e[1]))
            if do_inverse:
                inv_ms.append(e[1].elapsed_time(e[2]))
    if halves == 2:
        total_ms = sum(fwd_ms)  # the generator refills between halves are not part of the transform
    else:
        total_ms = wall0.elapsed_time(wall1)
    total_ms = max_over_ranks(total_ms)
    step_bytes = bytes_fwd + (bytes_inv if do_inverse else 0)
    value = whole_job_gbs(world, step_bytes, args.steps, total_ms)
    fwd_avg = sum(fwd_ms) / len(fwd_ms)
    ach = bytes_fwd / fwd_avg / 1e6

    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32->bf16", "data": "synthetic",
        "config": {"workload": workload_name(cfg),
                   "step": "dr_reshard + dr_reshard_inverse" if do_inverse else "dr_reshard",
                   "elements": int(info.elems_moved if halves == 1 else sum(p.info.elems_moved for p in plans)),
                   "bytes_per_step": int(step_bytes), "l2": "inputs larger than L2 (no flush needed)",
                   "passes": halves, "parallelism": "replicas only" if world > 1 else "1 GPU",
                   "segments": int(info.n_segments), "tiles": int(info.n_tiles), "plan_create_ms": plan_create_ms},
        "clocks": clocks,
        "gpu_launches": args.steps * (len(plans) + (1 if do_inverse else 0)),
        "forward": {"gbs_avg": ach, "gbs_best": bytes_fwd / min(fwd_ms) / 1e6, "ms_avg": fwd_avg, "ms_best": min(fwd_ms),
                    "ms_median": median(fwd_ms), "frac_of_measured_peak": ach / peak, "frac_of_nominal_8000": ach / 8000.0},
        "roofline": {"bound": "hbm", "kernel": "reshard_kernel<2,false> (dr_reshard), bulk-copy form" if plans[0].info.bulk_forward else "reshard_kernel<2,false> (dr_reshard), register form", "achieved": ach, "peak": peak,
                     "peak_kind": f"{peak_kind} copy bandwidth (burst)", "unit": "GB/s", "frac": ach / peak,
                     "traffic": None, "algorithmic_bytes": int(bytes_fwd // len(plans))},
    }
    if inv_ms:
        ia = sum(inv_ms) / len(inv_ms)
        line["inverse"] = {"gbs_avg": bytes_inv / ia / 1e6, "gbs_best": bytes_inv / min(inv_ms) / 1e6, "ms_avg": ia,
                           "ms_best": min(inv_ms), "ms_median": median(inv_ms),
                           "frac_of_measured_peak": bytes_inv / ia / 1e6 / peak}
    line["roofline"]["traffic"] = NCU_DRAM_BYTES_PER_ELEMENT_FWD * (bytes_fwd // 6 // len(plans)) if cfg["spec"] else None
    line["roofline"]["traffic_source"] = "ncu capture of a 654 M-element case of the same kernel, scaled by elements"

    # where the arena is the flat buffer cast in place (TP = 1, dense packing), check the timed output against
    # torch's own float32 -> bfloat16 on two 64 Mi-element windows
    if halves == 1 and info.dst_bytes == 2 * n_src and not inverse_dir:
        plans[0].reshard(master, arena)
        w = min(n_src, 1 << 26)
        ok = True
        for lo in (0, n_src - w):
            ok &= torch.equal(arena.view(torch.bfloat16)[lo:lo + w], master.view(torch.float32)[lo:lo + w].to(torch.bfloat16))
        line["config"]["output_equals_torch_cast_on_windows"] = bool(ok)

    # Ceilings measured in this run: trivial contiguous streaming kernels in the repack's own launch shape
    # (dr_probe_stream), one per read : write mix.  The forward repack is a 2 : 1 stream (4 B read, 2 B written),
    # the inverse map a 1 : 2 stream; torch's own copy and reduction are given for context.
    TILE = 49152
    if halves == 1 and n_src >= (1 << 28):
        nb = min(info.src_bytes, info.dst_bytes, 8 << 30) // TILE * TILE   # bytes of the wider side
        s0 = torch.cuda.current_stream().cuda_stream

        def best(fn, nbytes, reps=7):
            ts = []
            for i in range(reps + 2):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(); fn(); e1.record(); torch.cuda.synchronize()
                if i >= 2:
                    ts.append(e0.elapsed_time(e1))
            return nbytes / min(ts) / 1e6

        def probe(mode, a, b, n):
            rc = dr.dr_probe_stream(mode, a, b, n, s0)
            if rc:
                raise dr.DrError(rc, "dr_probe_stream")

        mp, ap = master.data_ptr(), arena.data_ptr()
        ceil = {"bytes_wider_side": int(nb),
                "read_gbs": best(lambda: probe(dr.binding.DR_PROBE_READ, mp, None, nb), nb),
                "write_gbs": best(lambda: probe(dr.binding.DR_PROBE_WRITE, None, ap, nb), nb),
                "copy_1to1_gbs": best(lambda: probe(dr.binding.DR_PROBE_COPY, mp, ap, nb), 2 * nb),
                "narrow_2to1_gbs": best(lambda: probe(dr.binding.DR_PROBE_NARROW, mp, ap, nb), nb * 3 // 2)}
        ceil["narrow_4to1_gbs"] = best(lambda: probe(dr.binding.DR_PROBE_NARROW4, mp, ap, nb), nb * 5 // 4)
        if flat_back is not None:
            ceil["widen_1to2_gbs"] = best(lambda: probe(dr.binding.DR_PROBE_WIDEN, ap, flat_back.data_ptr(), nb), nb * 3 // 2)
            ceil["widen_1to4_gbs"] = best(lambda: probe(dr.binding.DR_PROBE_WIDEN4, ap, flat_back.data_ptr(), nb), nb * 5 // 4)
        w = min(n_src, 1 << 30)
        ceil["torch_read_sum_gbs"] = best(lambda: master.view(torch.float32)[:w].sum(), 4 * w, reps=3)
        if info.dst_bytes >= 2 * w:
            ceil["torch_copy_gbs"] = best(lambda: arena.view(torch.bfloat16)[:w].copy_(master.view(torch.bfloat16)[:w]), 4 * w, reps=3)
        line["context_ceilings"] = ceil
        line["roofline"]["same_run_ceiling_for_this_mix"] = ceil["narrow_2to1_gbs"]
        line["roofline"]["frac_of_same_run_ceiling"] = ach / ceil["narrow_2to1_gbs"]
        if inv_ms and "widen_1to2_gbs" in ceil:
            line["inverse"]["same_run_ceiling_for_this_mix"] = ceil["widen_1to2_gbs"]
            line["inverse"]["frac_of_same_run_ceiling"] = line["inverse"]["gbs_avg"] / ceil["widen_1to2_gbs"]
    line["roofline"]["frac_of_nominal_8000"] = ach / 8000.0

    del flat_back
    torch.cuda.empty_cache()

    # the fp8 variant of the same switch: linear weights as e4m3 with one scale per 128 x 128 block
    if cfg["gathered"] and halves == 1 and not args.no_fp8:
        qplan = dr.Plan(cfg["spec"], world=cfg["world"], rank=cfg["rank"], gathered=True, tp=cfg["tp"],
                        tp_rank=cfg["tp_rank"], dtype=dr.DR_FP8_E4M3_B128)
        qarena = torch.empty(qplan.info.dst_bytes, dtype=torch.uint8, device=dev)
        for _ in range(args.warmup):
            qplan.reshard(master, qarena)
        qe = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
        qe[0].record()
        for i in range(args.steps):
            qplan.reshard(master, qarena)
            qe[i + 1].record()
        torch.cuda.synchronize()
        qms = [qe[i].elapsed_time(qe[i + 1]) for i in range(args.steps)]
        qavg = sum(qms) / len(qms)
        qb = qplan.info.bytes_moved_fwd
        line["fp8_forward"] = {"what": "dr_reshard with dtype DR_FP8_E4M3_B128 (copy kernel for bf16 tensors + block-quantisation "
                                       "kernel), same source", "bytes": int(qb), "quant_elems": int(qplan.info.quant_elems),
                               "quant_blocks": int(qplan.info.quant_blocks), "gbs_avg": qb / qavg / 1e6,
                               "gbs_best": qb / min(qms) / 1e6, "ms_avg": qavg, "ms_best": min(qms),
                               "frac_of_measured_peak": qb / qavg / 1e6 / peak, "frac_of_nominal_8000": qb / qavg / 1e6 / 8000.0,
                               "algorithmic_bytes_per_quant_elem": 5}
        c41 = line.get("context_ceilings", {}).get("narrow_4to1_gbs")
        if c41:
            line["fp8_forward"].update({"same_run_ceiling_for_this_mix": c41, "frac_of_same_run_ceiling": qb / qavg / 1e6 / c41})
        # and back: value(code) * scale to the flat fp32 positions (bf16 tensors widened), where a second flat buffer fits
        free_q, _ = torch.cuda.mem_get_info()
        if free_q > info.src_bytes * 1.05:
            qflat = torch.empty(n_src, dtype=torch.int32, device=dev)
            for _ in range(args.warmup):
                qplan.reshard_inverse(qarena, qflat)
            qe = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
            qe[0].record()
            for i in range(args.steps):
                qplan.reshard_inverse(qarena, qflat)
                qe[i + 1].record()
            torch.cuda.synchronize()
            ims = [qe[i].elapsed_time(qe[i + 1]) for i in range(args.steps)]
            iavg, ib = sum(ims) / len(ims), qplan.info.bytes_moved_inv
            # round trip on a window of a quantised tensor: |code * scale - x| <= |x| / 16 or half a subnormal code step
            t1 = [t for t in qplan.tensors() if t.quantised][0]
            line["fp8_inverse"] = {"what": "dr_reshard_inverse on the same plan (widening kernel + dequantisation kernel)",
                                   "bytes": int(ib), "gbs_avg": ib / iavg / 1e6, "gbs_best": ib / min(ims) / 1e6, "ms_avg": iavg,
                                   "ms_best": min(ims), "frac_of_measured_peak": ib / iavg / 1e6 / peak,
                                   "frac_of_nominal_8000": ib / iavg / 1e6 / 8000.0, "first_quantised_tensor": t1.name.decode()}
            c14 = line.get("context_ceilings", {}).get("widen_1to4_gbs")
            if c14:
                line["fp8_inverse"].update({"same_run_ceiling_for_this_mix": c14, "frac_of_same_run_ceiling": ib / iavg / 1e6 / c14})
            del qflat
        qplan.close()
        del qarena
        torch.cuda.empty_cache()

    # the exchange fused into the repack, as far as one GPU can time it: rank 0 of a world of two repacks its shard
    # and stores the pieces into two arenas of this GPU (the second stands for a peer's; over NVLink the stores to it
    # would be bound by the link instead of HBM)
    if cfg["gathered"] and halves == 1 and not args.no_fp8:
        xplan = dr.Plan(cfg["spec"], world=2, rank=0, gathered=False, tp=cfg["tp"], tp_rank=cfg["tp_rank"])
        free_x, _ = torch.cuda.mem_get_info()
        if free_x > info.dst_bytes * 1.1:
            arena2 = torch.empty(info.dst_bytes, dtype=torch.uint8, device=dev)
            shard = master[:xplan.info.src_bytes // 4]
            for _ in range(args.warmup):
                xplan.reshard_push(shard, [arena, arena2])
            xe = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
            xe[0].record()
            for i in range(args.steps):
                xplan.reshard_push(shard, [arena, arena2])
                xe[i + 1].record()
            torch.cuda.synchronize()
            xms = [xe[i].elapsed_time(xe[i + 1]) for i in range(args.steps)]
            xavg = sum(xms) / len(xms)
            xb = xplan.info.elems_moved * (4 + 2 * 2)
            same = bool(torch.equal(arena[:1 << 24], arena2[:1 << 24]))
            line["exchange_local"] = {"what": "dr_reshard_push: rank 0 of 2 repacks its shard into two arenas of this GPU in one kernel "
                                              "(4 B read + 2 x 2 B written per element); multi-GPU rate unmeasured in this run",
                                      "elements": int(xplan.info.elems_moved), "n_dst": 2, "bytes": int(xb),
                                      "ranges_of_this_rank": len(xplan.ranges()), "gbs_avg": xb / xavg / 1e6, "ms_avg": xavg,
                                      "ms_best": min(xms), "arenas_agree_on_window": same}
            del arena2
            plans[0].reshard(master, arena)  # put the whole arena back
        xplan.close()
        torch.cuda.empty_cache()

    # The timed region is short (a burst from a cool part).  Under a long run of launches the board reaches its power
    # limit and the SM clock drops; what one forward launch takes then is reported beside the burst figure.
    if halves == 1 and world == 1 and not args.profile and bytes_fwd > (1 << 30):
        n_long = max(50, int(1500 / fwd_avg))
        for _ in range(n_long // 2):
            plans[0].reshard(master, arena)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(n_long // 2):
            plans[0].reshard(master, arena)
        b.record()
        torch.cuda.synchronize()
        ms_long = a.elapsed_time(b) / (n_long // 2)
        line["forward"]["sustained"] = {"what": f"mean of the second half of {n_long} forward launches back to back "
                                                "(board at its power limit)", "ms": ms_long,
                                        "gbs": bytes_fwd / ms_long / 1e6, "frac_of_measured_peak": bytes_fwd / ms_long / 1e6 / peak}
        time.sleep(1.0)  # let the board leave its power limit before the next section

    # ---- host-link sections ---------------------------------------------------------------------
    if not args.no_staging:
        try:
            line.update(staging_sections(args, cfg, plans[0], master, arena, seed, base, dev, world, line, max_over_ranks))
        except Exception as exc:  # e.g. the box cannot pin this much host memory: keep the device-side line
            line.setdefault("staging", {})["error"] = f"{type(exc).__name__}: {exc}"[:300]
            line.setdefault("e2e", {"value": None, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0})

    # the other four workloads, device-resident transform only (a few seconds each), so that one run reports all five
    if world == 1 and not args.no_others and not (args.layers or args.vocab):
        del master, arena
        torch.cuda.empty_cache()
        others = []
        for i in range(5):
            if i == args.cfg:
                continue
            try:
                others.append(quick_transform(i, dev, peak))
            except Exception as exc:
                others.append({"cfg": i, "error": f"{type(exc).__name__}: {exc}"[:200]})
                torch.cuda.empty_cache()
        line["other_workloads"] = others

    if rank == 0 and not args.no_cpu and world == 1:
        gbs, elems, spent, desc = oracle_sample(cfg, args.cpu_seconds)
        line["cpu_baseline"] = {"value": gbs, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": desc,
                                "seconds": spent}
        g2, threads, e2, s2 = oracle_sample_all_cores(cfg)
        line["cpu_baseline_all_cores"] = {"value": g2, "unit": "GB/s", "cores": threads, "kind": "oracle",
                                          "sample": f"the same oracle, one thread per rollout tensor, {e2} elements",
                                          "seconds": s2}
    for p in plans:
        p.close()
    ctx.close()
    if rank == 0:
        print(json.dumps(line))


def staging_sections(args, cfg, plan, master, arena, seed, base, dev, world, line, max_over_ranks):
    """Chunked stage-out / stage-in of (master, Adam m, Adam v) to pinned host memory under the workload's
    budget, the switch latencies, the measured host link, the same engine through its pinned ring into
    pageable memory, and the end-to-end transform with host buffers."""
    import numpy as np
    import torch

    import paper_2607_22614_b200 as dr
    import synth

    out = {}
    info = plan.info
    n = master.numel()
    budget = cfg["budget"] or 2 * GiB
    chunk = budget // 2

    # measured pinned-copy bandwidth of the link, at 1 GiB and at this workload's chunk size
    pin = torch.empty(max(chunk, GiB), dtype=torch.uint8, pin_memory=True)
    scratch = torch.empty(max(chunk, GiB), dtype=torch.uint8, device=dev)

    def link(nbytes, d2h):
        best = 1e30
        for _ in range(8):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            if d2h:
                pin[:nbytes].copy_(scratch[:nbytes], non_blocking=True)
            else:
                scratch[:nbytes].copy_(pin[:nbytes], non_blocking=True)
            b.record()
            torch.cuda.synchronize()
            best = min(best, a.elapsed_time(b))
        return nbytes / best / 1e6

    link_d2h, link_h2d = link(GiB, True), link(GiB, False)
    link_d2h_c, link_h2d_c = link(chunk, True), link(chunk, False)

    # both directions at once (what a relay through the ring can reach): four 1 GiB copies each way on two streams
    pin2 = torch.empty(GiB, dtype=torch.uint8, pin_memory=True)
    scratch2 = torch.empty(GiB, dtype=torch.uint8, device=dev)
    s_out, s_in = torch.cuda.Stream(), torch.cuda.Stream()
    duplex = []
    for _ in range(3):
        torch.cuda.synchronize()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        with torch.cuda.stream(s_out):
            ev[0].record()
            for _ in range(4):
                pin[:GiB].copy_(scratch[:GiB], non_blocking=True)
            ev[1].record()
        with torch.cuda.stream(s_in):
            ev[2].record()
            for _ in range(4):
                scratch2.copy_(pin2, non_blocking=True)
            ev[3].record()
        torch.cuda.synchronize()
        duplex.append((4 * GiB / ev[0].elapsed_time(ev[1]) / 1e6, 4 * GiB / ev[2].elapsed_time(ev[3]) / 1e6))
    duplex_d2h, duplex_h2d = max(duplex, key=lambda x: min(x))
    del pin, scratch, pin2, scratch2
    torch.cuda.empty_cache()

    # which state buffers fit: device memory for m and v, host memory for the image
    names = list(cfg["stage"]) or ["master"]
    free_b, _ = torch.cuda.mem_get_info()
    host_room = int(mem_available_bytes() * 0.62 / world)
    bufs, ids = [master], [synth.BUF_MASTER]
    for nm, bid in (("m", synth.BUF_ADAM_M), ("v", synth.BUF_ADAM_V)):
        if nm in names and free_b > 4 * n * 1.1 and (len(bufs) + 1) * 4 * n <= host_room:
            t = torch.empty(n, dtype=torch.int32, device=dev)
            synth.cuda_fill_f32(t, seed, bid, start=base)
            bufs.append(t)
            ids.append(bid)
            free_b -= 4 * n
    if "master" not in names and len(bufs) > 1:
        bufs, ids = bufs[1:], ids[1:]
    total = 4 * n * len(bufs)
    if total > host_room:
        return {"staging": {"skipped": f"host memory: need {total} bytes, room {host_room}"}}
    sizes = [4 * n] * len(bufs)
    torch.cuda.synchronize()

    t0 = time.perf_counter()
    image = torch.empty(total, dtype=torch.uint8, pin_memory=True)  # the pinned host resting place
    pin_s = time.perf_counter() - t0

    # the link once more, but into fresh 1 GiB windows spread over the big pinned image instead of one small buffer
    # that stays hot in the IOMMU's translation cache: the rate a copy into the image can really reach on this machine
    link_d2h_image = None
    if total >= 8 * GiB:
        src1 = master.view(torch.uint8)[:GiB]
        ts = []
        for k in range(8):
            lo = (total - GiB) * k // 7 // 4096 * 4096
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            image[lo:lo + GiB].copy_(src1, non_blocking=True)
            b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        link_d2h_image = GiB / (sum(ts) / len(ts)) / 1e6

    def desc(ptrs, host, **kw):
        return dr.stage_desc(ptrs, sizes[:len(ptrs)], budget=budget, host_arena=host.data_ptr(),
                             host_arena_bytes=host.numel(), **kw)

    ptrs = [b.data_ptr() for b in bufs]
    # T -> R switch: repack enqueued first, stage-out pumps while it runs
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    ev[0].record()
    plan.reshard(master, arena)
    ev[1].record()
    st_out = plan.stage_out(desc(ptrs, image))
    torch.cuda.synchronize()
    t_switch = (time.perf_counter() - t0) * 1e3
    repack_overlapped_ms = ev[0].elapsed_time(ev[1])
    outs = [st_out.link_gbs] + [plan.stage_out(desc(ptrs, image)).link_gbs for _ in range(2)]
    # spot-check the host image against the generator (a few windows per buffer)
    img = image.numpy().view(np.uint32)
    rng = np.random.default_rng(0)
    image_ok = True
    for k, bid in enumerate(ids):
        for off in [0, n - 4096] + [int(x) for x in rng.integers(0, n - 4096, size=6)]:
            image_ok &= bool(np.array_equal(img[k * n + off:k * n + off + 4096], synth.fill_f32(seed, bid, base + off, 4096)))

    # R -> T switch: stage-in with the weights first; the inverse map can run as soon as they are resident
    for b in bufs:
        b.zero_()
    torch.cuda.synchronize()
    order = list(range(len(bufs)))
    st_in = plan.stage_in(desc(ptrs, image, order=order))
    torch.cuda.synchronize()
    restored_ok = all(synth.cuda_mismatch_f32(b, seed, bid, start=base) == 0 for b, bid in zip(bufs, ids))
    ins = [st_in.link_gbs] + [plan.stage_in(desc(ptrs, image, order=order)).link_gbs for _ in range(2)]

    # The same switch with the deferred call (dr_stage_begin): the host thread is free at once, the weights are waited
    # for on the caller's stream through their ready event, and the inverse map (rollout arena -> fp32 working copy,
    # independent of the reload) is enqueued right behind the begin; optimizer state keeps arriving meanwhile.
    deferred = None
    free_b, _ = torch.cuda.mem_get_info()
    if ids[0] == synth.BUF_MASTER and len(bufs) > 1 and free_b > 4 * n * 1.05:
        work = torch.empty(n, dtype=torch.int32, device=dev)
        for b in bufs:
            b.zero_()
        e0, e_inv = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        e0.record()
        job = plan.stage_begin(desc(ptrs, image, order=order), dr.DR_STAGE_DIR_IN)
        t_begin = (time.perf_counter() - t0) * 1e3
        plan.reshard_inverse(arena, work)
        e_inv.record()
        job.wait_buffer(0)
        e_inv.synchronize()
        t_critical = (time.perf_counter() - t0) * 1e3
        st_def = job.end()
        t_all = (time.perf_counter() - t0) * 1e3
        torch.cuda.synchronize()
        ok_def = all(synth.cuda_mismatch_f32(b, seed, bid, start=base) == 0 for b, bid in zip(bufs, ids))
        deferred = {"what": "dr_stage_begin(stage-in, weights first) + dr_reshard_inverse on the caller's stream + dr_stage_wait_buffer(weights) + dr_stage_end",
                    "begin_returns_ms": t_begin, "inverse_map_done_ms": e0.elapsed_time(e_inv),
                    "weights_resident_and_inverse_map_done_ms": t_critical, "weights_resident_ms": st_def.ready_ms[0],
                    "all_state_resident_ms": t_all, "stage_in_gbs": st_def.link_gbs,
                    "restored_state_matches_generator": bool(ok_def)}
        del work
        torch.cuda.empty_cache()

    out["staging"] = {
        "bytes": int(total), "buffers": [("master", "m", "v")[i] for i in ids], "budget_bytes": int(budget),
        "chunk_bytes": int(chunk), "chunks": int(st_out.n_chunks), "sink": "pinned host image, chunked direct copies, "
        "at most `budget` bytes in flight", "pin_seconds": pin_s,
        "stage_out_gbs": max(outs), "stage_in_gbs": max(ins), "stage_out_gbs_runs": outs, "stage_in_gbs_runs": ins,
        "link_d2h_gbs_1GiB": link_d2h, "link_h2d_gbs_1GiB": link_h2d, "link_d2h_gbs_chunk": link_d2h_c,
        "link_h2d_gbs_chunk": link_h2d_c, "stage_out_frac_of_link": max(outs) / link_d2h,
        "stage_in_frac_of_link": max(ins) / link_h2d, "link_d2h_gbs_into_image_windows": link_d2h_image,
        "stage_out_frac_of_link_into_image": (max(outs) / link_d2h_image) if link_d2h_image else None,
        "host_image_matches_generator": image_ok,
        "restored_state_matches_generator": bool(restored_ok),
    }
    out["switch_ms"] = {
        "train_to_rollout": {"repack_alone": line["forward"]["ms_avg"], "repack_while_staging_out": repack_overlapped_ms,
                             "until_state_staged_out": t_switch},
        "rollout_to_train": {"weights_resident": st_in.ready_ms[0] if ids[0] == synth.BUF_MASTER else None,
                             "inverse_map": line.get("inverse", {}).get("ms_avg"),
                             "all_state_resident_deferred": st_in.elapsed_ms,
                             "with_the_deferred_call": deferred},
    }

    # Re-shard across a changed training world size (Sec. 3.3; the paper's 6 -> 4 training GPUs): the device buffers
    # stand for the flat state; every old rank r of 6 stages its shard of master, m, v out to its place in the flat
    # host image (ranks one after the other on this GPU), then a new rank 1 of 4 stages its own, differently cut,
    # range back in, weights first.  Windows of the image are scribbled on first so that the check means something.
    if len(bufs) == 3 and cfg["gathered"]:
        W_OLD, W_NEW = 6, 4
        spots = []
        for r in range(W_OLD):
            rc, lo, hi, _ = dr.dr_shard_range(n, W_OLD, r)
            for k in range(3):
                for off in (lo, max(lo, hi - 4096)):
                    img[k * n + off:k * n + off + 4096] = 0xDEADBEEF
                    spots.append((k, off))
        outs6 = []
        for r in range(W_OLD):
            rc, lo, hi, _ = dr.dr_shard_range(n, W_OLD, r)
            d6 = dr.stage_desc([p + 4 * lo for p in ptrs], [4 * (hi - lo)] * 3, budget=budget, host_arena=image.data_ptr(),
                               host_arena_bytes=image.numel(), host_offsets=[4 * (k * n + lo) for k in range(3)])
            outs6.append(plan.stage_out(d6))
        ok6 = all(np.array_equal(img[k * n + off:k * n + off + 4096], synth.fill_f32(seed, ids[k], base + off, 4096))
                  for k, off in spots)
        for b in bufs:
            b.zero_()
        rc, lo, hi, s4 = dr.dr_shard_range(n, W_NEW, 1)
        d4 = dr.stage_desc(ptrs, [4 * (hi - lo)] * 3, budget=budget, host_arena=image.data_ptr(),
                           host_arena_bytes=image.numel(), host_offsets=[4 * (k * n + lo) for k in range(3)], order=[0, 1, 2])
        r4 = [plan.stage_in(d4) for _ in range(2)]
        ok4 = all(synth.cuda_mismatch_f32(b[:hi - lo], seed, bid, start=base + lo) == 0 for b, bid in zip(bufs, ids))
        best = max(r4, key=lambda x: x.link_gbs)
        out["restage"] = {"what": f"{W_OLD} old ranks stage their shards of master, m, v out to one flat host image; new rank 1 "
                                  f"of {W_NEW} stages its range back in, weights first",
                          "stage_out_bytes_per_old_rank": int(outs6[1].bytes),
                          "stage_out_gbs_per_old_rank": [x.link_gbs for x in outs6],
                          "stage_out_frac_of_link": max(x.link_gbs for x in outs6) / link_d2h,
                          "stage_out_ms_all_old_ranks": sum(x.elapsed_ms for x in outs6),
                          "image_matches_generator": bool(ok6),
                          "bytes": int(best.bytes), "stage_in_gbs": best.link_gbs, "frac_of_link": best.link_gbs / link_h2d,
                          "weights_resident_ms": best.ready_ms[0], "all_state_resident_ms": best.elapsed_ms,
                          "matches_generator": bool(ok4)}
        plan.stage_in(desc(ptrs, image, order=order))

    # Relay (Sec. 3.3, old rank -> new rank through bounded host buffers): one state buffer goes device -> pinned ring
    # -> another device buffer, both directions of the link busy at once; the target is the last state buffer,
    # which is regenerated afterwards.
    if len(bufs) >= 2:
        relay = {}
        for label, b_b, c_b in (("two_slots", budget, budget // 2), ("eight_slots", budget, budget // 8),
                                ("ring_64MiB_16x4MiB", 64 * MiB, 4 * MiB), ("no_chunk_size_given", budget, 0)):
            dd = dr.stage_desc(ptrs[:1], sizes[:1], budget=b_b, chunk=c_b, relay_dev=[ptrs[-1]])
            runs = [plan.stage_out(dd) for _ in range(2)]
            best = max(runs, key=lambda x: x.link_gbs)
            relay[label] = {"budget_bytes": b_b, "chunk_bytes": c_b, "gbs": best.link_gbs, "ms": best.elapsed_ms,
                            "frac_of_duplex_link": best.link_gbs / min(duplex_d2h, duplex_h2d),
                            "pinned_high_water_bytes": int(best.pinned_high_water_bytes)}
        torch.cuda.synchronize()
        relay["target_matches_source"] = bool(torch.equal(bufs[0], bufs[-1]))
        synth.cuda_fill_f32(bufs[-1], seed, ids[-1], start=base)
        torch.cuda.synchronize()
        out["relay"] = {"what": "dr_stage_out with a relay target: device buffer -> pinned ring -> second device buffer, "
                                f"{sizes[0]} bytes", "bytes": sizes[0],
                        "link_duplex_d2h_gbs": duplex_d2h, "link_duplex_h2d_gbs": duplex_h2d, **relay,
                        "gbs": max(relay[k]["gbs"] for k in ("two_slots", "eight_slots", "ring_64MiB_16x4MiB", "no_chunk_size_given"))}

    # the same engine with a pageable resting place: chunks go through the pinned ring and worker threads
    if mem_available_bytes() > 4 * n * 1.5:
        pageable = torch.empty(4 * n, dtype=torch.uint8)
        pageable.fill_(0)  # commit the pages before timing
        w = min(n, 1 << 20)

        def ring(budget_b, chunk_b):
            dd = dr.stage_desc(ptrs[:1], sizes[:1], budget=budget_b, chunk=chunk_b, host_arena=pageable.data_ptr(),
                               host_arena_bytes=pageable.numel())
            ro = [plan.stage_out(dd) for _ in range(2)]
            good = bool(np.array_equal(pageable.numpy().view(np.uint32)[:w], img[:w]))
            bufs[0].zero_()
            ri = [plan.stage_in(dd) for _ in range(2)]
            good &= synth.cuda_mismatch_f32(bufs[0], seed, ids[0], start=base) == 0
            o, i = max(x.link_gbs for x in ro), max(x.link_gbs for x in ri)
            return {"budget_bytes": int(budget_b), "chunk_bytes": int(chunk_b), "slots": int(budget_b // chunk_b) if chunk_b else None,
                    "pinned_high_water_bytes": int(ro[0].pinned_high_water_bytes), "stage_out_gbs": o, "stage_in_gbs": i,
                    "stage_out_frac_of_link": o / link_d2h, "stage_in_frac_of_link": i / link_h2d, "bytes_match": good}

        eight = ring(budget, budget // 8 // 4096 * 4096)          # the workload's budget as eight slots
        two = ring(budget, budget // 2 // 4096 * 4096)            # ... and as two
        # a ring small enough to stay in the host's last-level cache (it uses 64 MiB of the budget): the chunks are
        # copied out right behind the DMA that delivered them, and filled right before the DMA that reads them
        small = ring(64 << 20, 8 << 20) if 4 * n >= (1 << 30) else None
        small16 = ring(64 << 20, 4 << 20) if 4 * n >= (1 << 30) else None
        # no chunk size given: the engine takes its small ring by itself (what a caller who only states a budget gets)
        auto = ring(budget, 0)
        rings = [x for x in (eight, two, small, small16, auto) if x]

        def geometry_name(x):
            if not x["chunk_bytes"]:
                return "no chunk size given (the engine's own small ring)"
            return f'{x["slots"]} x {x["chunk_bytes"] // MiB} MiB'

        best_out = max(rings, key=lambda x: x["stage_out_gbs"])
        best_in = max(rings, key=lambda x: x["stage_in_gbs"])
        # CPU baseline of this path: the engine's multi-threaded host copy on its own, and the same copy while the
        # link moves data in the same direction beside it (what the ring path has to share the host's memory with)
        hb = min(4 * n, GiB)
        p1 = torch.empty(hb, dtype=torch.uint8, pin_memory=True)
        p2 = torch.empty(hb, dtype=torch.uint8, pin_memory=True)
        p1.fill_(1)
        scratch = torch.empty(hb, dtype=torch.uint8, device=dev)
        pg = pageable[:hb]

        def host_copy(dst, src, reps=3):
            best = 1e30
            for _ in range(reps):
                t0 = time.perf_counter()
                rc = dr.dr_host_copy(dst.data_ptr(), src.data_ptr(), hb, 0)
                best = min(best, time.perf_counter() - t0)
                if rc:
                    raise dr.DrError(rc, "dr_host_copy")
            return hb / best / 1e9

        def beside_dma(dst, src, d2h):
            stop, copied = threading.Event(), [0, 0.0]

            def worker():
                t0 = time.perf_counter()
                while not stop.is_set():
                    dr.dr_host_copy(dst.data_ptr(), src.data_ptr(), hb, 0)
                    copied[0] += hb
                copied[1] = time.perf_counter() - t0

            th = threading.Thread(target=worker)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            th.start()
            time.sleep(0.05)
            e0.record()
            reps = 24
            for _ in range(reps):
                if d2h:
                    p2.copy_(scratch, non_blocking=True)
                else:
                    scratch.copy_(p2, non_blocking=True)
            e1.record()
            torch.cuda.synchronize()
            stop.set()
            th.join()
            return copied[0] / copied[1] / 1e9, reps * hb / e0.elapsed_time(e1) / 1e6

        alone_out, alone_in = host_copy(pg, p1), host_copy(p1, pg)
        c_out, dma_out = beside_dma(pg, p1, True)
        c_in, dma_in = beside_dma(p1, pg, False)
        del p1, p2, scratch
        out["staging"]["through_ring_to_pageable"] = {
            "bytes": int(4 * n), "eight_slots": eight, "two_slots": two, "ring_64MiB_8x8MiB": small, "ring_64MiB_16x4MiB": small16,
            "no_chunk_size_given": auto,
            "stage_out_gbs": best_out["stage_out_gbs"], "stage_in_gbs": best_in["stage_in_gbs"],
            "stage_out_frac_of_link": best_out["stage_out_frac_of_link"], "stage_in_frac_of_link": best_in["stage_in_frac_of_link"],
            "best_geometry": {"stage_out": geometry_name(best_out), "stage_in": geometry_name(best_in)},
            "bytes_match": bool(all(x["bytes_match"] for x in rings)),
            "cpu_baseline_host_copy": {
                "what": "dr_host_copy, the engine's multi-threaded copy (non-temporal stores), 1 GiB, this box's host cores",
                "threads": engine_copy_threads(),
                "pinned_to_pageable_alone_gbs": alone_out, "pageable_to_pinned_alone_gbs": alone_in,
                "pinned_to_pageable_beside_d2h_gbs": c_out, "d2h_beside_host_copy_gbs": dma_out,
                "pageable_to_pinned_beside_h2d_gbs": c_in, "h2d_beside_host_copy_gbs": dma_in,
                "note": "every byte staged through the ring crosses host memory three times (link write, copy read, "
                        "copy write); the beside-the-link rates are what the host sustains for that mix"}}
        del pageable
    for b in bufs[1:]:
        del b
    bufs = None
    torch.cuda.empty_cache()

    # ---- end to end with host buffers: H2D of the master, repack, D2H of the rollout arena, all through the C ABI
    e2e_steps = 3
    if image.numel() >= info.src_bytes + info.dst_bytes:
        h_src, h_dst = image[:info.src_bytes], image[info.src_bytes:info.src_bytes + info.dst_bytes]
    else:
        del img, image
        image = torch.empty(info.src_bytes + info.dst_bytes, dtype=torch.uint8, pin_memory=True)
        h_src, h_dst = image[:info.src_bytes], image[info.src_bytes:]
        plan.stage_out(dr.stage_desc([master.data_ptr()], [info.src_bytes], budget=budget, host_arena=h_src.data_ptr(),
                                     host_arena_bytes=info.src_bytes))  # untimed: put the inputs on the host
    if ids[0] != synth.BUF_MASTER:
        plan.stage_out(dr.stage_desc([master.data_ptr()], [info.src_bytes], budget=budget, host_arena=h_src.data_ptr(),
                                     host_arena_bytes=info.src_bytes))
    master.zero_()
    done = torch.cuda.Event()
    done.record()
    times = []
    for i in range(e2e_steps + 1):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        plan.stage_in(dr.stage_desc([master.data_ptr()], [info.src_bytes], budget=budget, host_arena=h_src.data_ptr(),
                                    host_arena_bytes=info.src_bytes))
        plan.reshard(master, arena)
        done.record()
        plan.stage_out(dr.stage_desc([arena.data_ptr()], [info.dst_bytes], budget=budget, host_arena=h_dst.data_ptr(),
                                     host_arena_bytes=info.dst_bytes, wait_event=done.cuda_event))
        torch.cuda.synchronize()
        if i:
            times.append(time.perf_counter() - t0)
    t_seq = max_over_ranks(sum(times) / len(times))
    # the same switch as one streamed call: H2D chunks, per-chunk repack and D2H of finished arena ranges overlap
    window = torch.empty(budget, dtype=torch.uint8, device=dev)
    sd = dr.stream_desc(h_src.data_ptr(), info.src_bytes, arena.data_ptr(), info.dst_bytes, window.data_ptr(), budget,
                        chunk_bytes=0, host_dst=h_dst.data_ptr(), host_dst_bytes=info.dst_bytes)
    h_dst.zero_()
    times, kernels = [], 0
    for i in range(e2e_steps + 1):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        st = plan.reshard_stream(sd)
        if i:
            times.append(time.perf_counter() - t0)
        kernels = int(st.kernels)
    t = max_over_ranks(sum(times) / len(times))
    # spot check of the host result: the arena on the device is the already verified dr_reshard output
    probe = slice(info.dst_bytes // 2, info.dst_bytes // 2 + (1 << 20))
    host_ok = bool(np.array_equal(h_dst[probe].numpy(), arena[probe].cpu().numpy()))
    out["e2e"] = {"value": world * info.bytes_moved_fwd / t / 1e9, "unit": "GB/s", "ms_per_step": t * 1e3,
                  "steps": e2e_steps, "h2d_bytes_per_step": int(info.src_bytes), "d2h_bytes_per_step": int(info.dst_bytes),
                  "path": "dr_reshard_stream: pinned host master -> chunked H2D -> per-chunk repack -> D2H of finished arena "
                          "ranges to pinned host, three overlapped streams", "kernels_per_step": kernels,
                  "window_bytes": int(budget), "chunk_bytes": int(min(budget // 2 // 4096 * 4096, 32 * MiB)),
                  "chunk_choice": "the call's own (no chunk size given)", "host_result_matches_device": host_ok,
                  "duplex_ideal_ms": max(info.src_bytes / link_h2d, info.dst_bytes / link_d2h) / 1e6,
                  # what the link gives when both directions are busy (measured above): the copy back runs at the duplex
                  # D2H rate, the copy in at the duplex H2D rate beside it and at the full rate for the rest
                  "duplex_link_model_ms": duplex_model_ms(info.src_bytes, info.dst_bytes, link_h2d, duplex_h2d, duplex_d2h),
                  "sequential": {"value": world * info.bytes_moved_fwd / t_seq / 1e9, "ms_per_step": t_seq * 1e3,
                                 "path": "dr_stage_in(master) -> dr_reshard -> dr_stage_out(arena), one after the other",
                                 "link_bound_ideal_ms": (info.src_bytes / link_h2d + info.dst_bytes / link_d2h) / 1e6}}
    return out


if __name__ == "__main__":
    main()
