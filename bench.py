#!/usr/bin/env python
"""Benchmark: effective HBM GB/s of executing a synthesized redistribution on one B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c5] [--impl ours|reference]

A *step* is one pass of the workload.  The default is ``c5`` -- the largest configuration: bf16
[32768, 32768] (2 GiB) on a 4x4x4 mesh of 64 virtual devices -- and a step runs its two
redistributions, {d0:(x,y), d1:z} -> {d0:(y,x), d1:z} (an allpermute) and {d0:(x,y), d1:z} ->
{d0:z, d1:(y,x)} (alltoall + allpermute fused into one kernel): two launches of 2 GiB read + 2 GiB
written each.  Metric: effective bytes (every global element read once plus every destination byte
written once) per second, in GB/s.  Inputs are synthetic, seeded and resident in HBM before the
timed region; buffer sets rotate, and every launch moves far more than the 126 MB L2 holds.  The
timed region calls ``redist_execute`` once per redistribution on one stream (kernels use
programmatic dependent launch, so consecutive launches overlap their ramp-up with the previous
kernel's tail); ``--graph`` times CUDA-graph replays instead.  ``e2e`` is the same step through
``redist_execute_host`` with pinned host tiles, host<->device copies inside the timed region.

The same JSON line carries a ``configs`` block: every benchmark configuration (c1, c2, c3a, c3b, c3c,
c5a, c5b and a fixed subset of the c4 sweep) timed in its own event-bracketed region, with GB/s,
microseconds per launch (back to back and for one launch alone), fraction of the measured copy
bandwidth, launches and scratch per virtual device.

With ``--gpus N`` every rank runs an independent replica: the method has no inter-GPU step here
(virtual devices share one GPU), so there is no collective on the data path; only the timing is
reduced (max over ranks).  Started without a launcher (``WORLD_SIZE`` unset) the script re-executes
itself under ``torch.distributed.run`` with N ranks on 127.0.0.1.

``--impl reference`` times the CPU oracle (``oracle/``) on the host cores for the same metric.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "redistribution effective HBM GB/s (read+write)"
UNIT = "GB/s"
N_SETS = 4


def legs_of(workload: str):
    """The (source, target) problems one step executes, in order."""
    from paper_2112_01075_b200 import workloads as wl
    b = wl.bench_workloads()
    if workload in ("c1", "c2"):
        return [b[workload], b[workload + "_back"]]
    if workload == "c3":
        return [b["c3a"], b["c3b"], b["c3c"]]
    if workload == "c5":
        return [b["c5a"], b["c5b"]]
    return [b[workload]]


def effective_bytes(w) -> int:
    """globalsize*e read + N*localsize(dst)*e written."""
    n_tiles = 1
    for s, ax in zip(w.dst.global_shape, w.dst.axes):
        for a in ax:
            n_tiles *= w.mesh_shape[a]
    local_dst = w.global_elems // n_tiles
    return w.global_elems * w.elem_bytes + w.n_devices * local_dst * w.elem_bytes


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU while the timed region runs (read only)."""

    def __init__(self, index: int, period: float = 0.01):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop_ev = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.nv = None

    def _sample(self):
        nv = self.nv
        self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
        try:
            r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
        except Exception:
            r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
        names = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap",
                 0x80: "hw_power_brake", 0x2: "applications_clocks_setting", 0x100: "display_clock_setting",
                 0x10: "sync_boost"}
        for bit, name in names.items():
            if r & bit:
                self.reasons.add(name)

    def run(self):
        if not self.ok:
            return
        while not self._stop_ev.is_set():
            try:
                self._sample()
            except Exception:
                break
            time.sleep(self.period)

    def stop(self):
        self._stop_ev.set()
        self.join(timeout=2)
        med = statistics.median(self.samples) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def reduce_max(dist, value: float, device: str = "cuda") -> float:
    """Max over ranks of a per-rank duration (ranks run independent replicas)."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(world: int, bytes_per_rank_step: int, max_ms_per_step: float) -> float:
    """Whole-job GB/s: the bytes all ranks processed divided by the slowest rank's time."""
    return world * bytes_per_rank_step / (max_ms_per_step * 1e-3) / 1e9


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def ncu_traffic(workload: str):
    """DRAM bytes per launch of the dominant kernel from the committed ncu summary, if any."""
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.json")) as f:
            return json.load(f).get(workload)
    except Exception:
        return None


# ---------------------------------------------------------------------------------------- ours

def sets_for(eff_bytes: int) -> int:
    """Buffer sets that rotate: a launch that moves at least 1 GB streams far more than the L2 holds
    and two sets suffice; smaller workloads get four."""
    return 2 if eff_bytes >= (1 << 30) else N_SETS


class DeviceLeg:
    """One redistribution with rotating sets of device tiles."""

    def __init__(self, w, flags, torch, api, gen, sets=None, alias_replicas=True):
        self.w = w
        self.plan = api.Plan(w.mesh_shape, w.src, w.dst, w.elem_bytes, flags)
        p = self.plan
        self.n = p.n_devices
        self.eff_bytes = effective_bytes(w)
        sets = sets or sets_for(self.eff_bytes)
        db = p.local_elems(1) * w.elem_bytes
        G = torch.randint(0, 256, tuple(w.src.global_shape) + (w.elem_bytes,), dtype=torch.uint8, device="cuda",
                          generator=gen)
        self.src, self.dst = [], []
        _, offs = api.redist_base_offsets(w.mesh_shape, w.src)
        for _ in range(sets):
            tiles = api.shard_global(G, w.mesh_shape, w.src)
            # every set owns its memory; devices that replicate a tile share one buffer per set
            # (replicas hold identical bytes, and the boundary allows source pointers to alias)
            owned = {}
            for d, o in enumerate(offs):
                key = o if alias_replicas else d
                if key not in owned:
                    owned[key] = tiles[d].clone()
            del tiles
            self.src.append([owned[o if alias_replicas else d] for d, o in enumerate(offs)])
            self.dst.append([torch.empty(db, dtype=torch.uint8, device="cuda") for _ in range(self.n)])
        del G
        self.scratch = p.alloc_scratch()
        self.launches = p.num_launches
        sp = self.scratch.data_ptr() if self.scratch is not None else 0
        sn = self.scratch.numel() if self.scratch is not None else 0
        self.calls = [p.bind([t.data_ptr() for t in s], [t.data_ptr() for t in d], sp, sn)
                      for s, d in zip(self.src, self.dst)]

    def run(self, i, stream_ptr):
        self.calls[i % len(self.calls)](stream_ptr)


def capture_graphs(torch, legs):
    """One CUDA graph per buffer set; each holds one step (every leg's redist_execute once)."""
    sets = len(legs[0].calls)
    side = torch.cuda.Stream()
    graphs = []
    for i in range(sets):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            for leg in legs:
                leg.run(i, torch.cuda.current_stream().cuda_stream)
        graphs.append(g)
    return graphs


def time_legs(torch, legs, steps, warmup, per_launch=False, graphs=None):
    """Run `steps` timed steps (after `warmup`), each step = every leg once, bracketed by CUDA
    events on the launching stream.  Returns (total_ms, per-leg launch durations in ms or None)."""
    stream = torch.cuda.current_stream()
    sp = stream.cuda_stream

    def one(i):
        if graphs is not None:
            graphs[i % len(graphs)].replay()
        else:
            for leg in legs:
                leg.run(i, sp)

    for i in range(warmup):
        one(i)
    torch.cuda.synchronize()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if not per_launch:
        t0.record(stream)
        for i in range(steps):
            one(warmup + i)
        t1.record(stream)
        torch.cuda.synchronize()
        return t0.elapsed_time(t1), None
    ev = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
          for _ in legs]
    t0.record(stream)
    for i in range(steps):
        for k, leg in enumerate(legs):
            ev[k][i][0].record(stream)
            leg.run(warmup + i, sp)
            ev[k][i][1].record(stream)
    t1.record(stream)
    torch.cuda.synchronize()
    return t0.elapsed_time(t1), [[a.elapsed_time(b) for a, b in ev[k]] for k in range(len(legs))]


def kernel_name(api, li) -> str:
    kname = {"naive_gather": "allgather", "naive_slice": "dynslice", "copy": "allpermute"}.get(
        api.KERNELS[li.kernel], api.KERNELS[li.kernel])
    return f"redist_{kname}{ {4: '_bulk', 5: '_gather', 6: '_ragged_bulk', 7: '_zip', 8: '_box'}.get(li.variant, '') }_kernel"


def spawn_ranks(n: int):
    """Started without a launcher: run this script again under torch.distributed.run, one rank per GPU."""
    import socket
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    os.execv(sys.executable, cmd)


def run_standin(args):
    """The launch plumbing of an N-rank run with a CPU stand-in for the timed body (gloo, no CUDA):
    used by the tests of the multi-process path.  Every rank 'processes' a fixed number of bytes in a
    rank-dependent time; the line is built by the same reduce / aggregate code as the real run."""
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
    mine_ms = 10.0 + 5.0 * rank
    worst = reduce_max(dist if world > 1 else None, mine_ms, device="cpu")
    step_bytes = 512 << 20
    line = {"metric": METRIC, "value": round(aggregate_value(world, step_bytes, worst / args.steps), 3),
            "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": worst / args.steps, "higher_is_better": True, "scaling": "weak",
            "config": {"workload": "stand-in"}, "standin": True}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_ours(args):
    import torch
    from paper_2112_01075_b200 import api

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the redistribution runs in CUDA kernels only")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    api.load()
    gen = torch.Generator(device="cuda")
    gen.manual_seed(2112010752 + rank)
    ws = legs_of(args.workload)
    flags = {"adjacent": api.FUSE_ADJACENT, "none": api.FUSE_NONE, "all": api.FUSE_ALL, "naive": api.NAIVE}[args.fuse]
    if args.cost_permute:
        flags |= api.COST_PERMUTE
    legs = [DeviceLeg(w, flags, torch, api, gen, sets=args.sets or None) for w in ws]
    n_sets = len(legs[0].calls)
    step_bytes = sum(l.eff_bytes for l in legs)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    graphs = capture_graphs(torch, legs) if args.graph else None
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    total_ms, _ = time_legs(torch, legs, args.steps, args.warmup, graphs=graphs)
    window = "warm-up and timed region"
    if sampler.ok and len(sampler.samples) < 5:
        # a very short timed region gives the 10 ms sampler nothing to see: keep the same load running
        # (untimed) for a third of a second so that the clock record is taken under this workload
        t_end = time.perf_counter() + 0.35
        extra = 0
        while time.perf_counter() < t_end:
            time_legs(torch, legs, 20, 0, graphs=graphs)
            extra += 20
        window = f"warm-up, timed region and {extra} further untimed steps of the same workload"
    clocks = sampler.stop()
    clocks["window"] = window
    barrier()
    total_ms = reduce_max(dist, total_ms)
    ms_per_step = total_ms / args.steps
    value = aggregate_value(world, step_bytes, ms_per_step)

    # outside the headline region: the same steps the other way (CUDA-graph replay if the headline
    # used plain launches, and vice versa), and once more with an event pair around every launch
    # (per-leg numbers; the events themselves cost a few microseconds and break launch overlap)
    n_side = max(3, min(args.steps, 200))
    other_ms = None
    if not args.lean:
        other_graphs = None if args.graph else capture_graphs(torch, legs)
        other_ms, _ = time_legs(torch, legs, n_side, 3, graphs=other_graphs)
        del other_graphs
    _, per = time_legs(torch, legs, n_side, 3, per_launch=True)

    # Roofline of the dominant kernel (the leg that takes longest).  When every launch of the step runs the
    # same kernel on the same number of bytes, its average duration is the timed region divided by the
    # number of launches; otherwise the event pair around each of its launches decides.
    infos = [l.plan.launch_info(0) for l in legs]
    n_launch = sum(l.launches for l in legs)
    same = all(l.launches == 1 for l in legs) and \
        len({(kernel_name(api, i), i.bytes_read + i.bytes_written) for i in infos}) == 1
    sums = [sum(p) for p in per]
    k = max(range(len(legs)), key=lambda q: sums[q])
    dom, li = legs[k], infos[k]
    alg = li.bytes_read + li.bytes_written
    avg_ms = (total_ms / (args.steps * n_launch)) if same else statistics.mean(per[k]) / dom.launches
    peak, how = measured_peak()
    achieved = alg / (avg_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s",
                "frac": round(achieved / peak, 4), "traffic": ncu_traffic(dom.w.name),
                "kernel": kernel_name(api, li), "workload_leg": dom.w.name,
                "algorithmic_bytes_per_launch": alg,
                "avg_launch_us": round(avg_ms * 1e3, 2),
                "avg_from": "timed region / launches" if same else
                            f"event pair around each of its {len(per[k])} launches (a region of the same steps right after the headline region)",
                "timed_region_us_per_launch_all_kernels": round(total_ms / (args.steps * n_launch) * 1e3, 2),
                "peak_source": how + " copy bandwidth", "frac_of_8TBs_nominal": round(achieved / 8000.0, 4)}

    line = {
        "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms_per_step, 5), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": describe_workload(args.workload, ws)},
        "run": {"fuse": args.fuse, "tune": args.tune,
                "launch": "CUDA graph replay of captured redist_execute calls (one graph per buffer set)"
                if args.graph else "redist_execute called once per redistribution on the stream",
                "cache": f"{n_sets} rotating buffer sets; one launch moves {legs[0].eff_bytes >> 20} MiB "
                         f"(L2: 126 MB)",
                "parallelism": "replicas only" if world > 1 else "single GPU, virtual devices",
                "timed_region_ms": round(total_ms, 3)},
        "gpu_launches": args.steps * sum(l.launches for l in legs),
        "clocks": clocks, "roofline": roofline,
        "scratch_bytes_per_virtual_device": max(l.plan.scratch_bytes_per_device for l in legs),
        "memory_bound_bytes_per_virtual_device": max(max(l.plan.local_elems(0), l.plan.local_elems(1)) *
                                                     l.w.elem_bytes for l in legs),
        "legs": [{"name": l.w.name, "steps": l.plan.step_kinds(), "kernels": l.plan.launch_kernels(),
                  "gbs": round(l.eff_bytes / (statistics.mean(per[q]) * 1e-3) / 1e9, 1),
                  "us": round(statistics.mean(per[q]) * 1e3, 2)} for q, l in enumerate(legs)],
    }
    if other_ms is not None:
        line["stream_launch" if args.graph else "graph_replay"] = {
            "value": round(world * step_bytes / (other_ms / n_side * 1e-3) / 1e9, 1), "unit": UNIT,
            "ms_per_step": round(other_ms / n_side, 5), "steps": n_side,
            "note": "same steps, " + ("plain redist_execute calls" if args.graph else
                                      "replayed from CUDA graphs of captured redist_execute calls, one step per "
                                      "graph (no dependent-launch overlap from one graph launch to the next)")}
    del legs, graphs
    torch.cuda.empty_cache()
    e2e_steps = max(3, min(args.steps, 10))
    if rank == 0 and not args.no_e2e:
        line["e2e"] = run_e2e(torch, api, ws, flags, e2e_steps, world, dist)
    elif dist is not None and not args.no_e2e:
        run_e2e(torch, api, ws, flags, e2e_steps, world, dist)
    torch.cuda.empty_cache()
    if rank == 0 and world == 1 and not args.no_cpu:
        line["cpu_baseline"] = cpu_baseline(ws)
    if rank == 0 and world == 1 and args.fuse == "adjacent" and not args.lean:
        # comparison points on the same workload (short runs, outside the headline region): the
        # sequence run collective by collective through scratch, and the naive gather-then-slice method
        for key, fl in (("unfused", api.FUSE_NONE), ("naive_gpu_baseline", api.NAIVE)):
            cmp_legs = [DeviceLeg(w, fl, torch, api, gen, sets=args.sets or None) for w in ws]
            reps = 20
            ms, _ = time_legs(torch, cmp_legs, reps, 3)
            line[key] = {"value": round(step_bytes / (ms / reps * 1e-3) / 1e9, 1), "unit": UNIT,
                         "launches_per_step": sum(l.launches for l in cmp_legs),
                         "scratch_bytes_per_virtual_device": max(l.plan.scratch_bytes_per_device for l in cmp_legs)}
            del cmp_legs
            torch.cuda.empty_cache()
    if rank == 0 and world == 1 and args.fuse == "adjacent" and not args.lean and not args.no_configs:
        line["configs"] = run_configs(torch, api, gen)
    if rank == 0 and world == 1 and args.others:
        line["others"] = run_others(torch, api, gen, args)
    if rank == 0 and world == 1 and not args.lean:
        line["spread_model"] = spread_model(api, ws, flags, peak)
    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


CONFIG_ENTRIES = [("c1", ["c1", "c1_back"]), ("c2", ["c2", "c2_back"]), ("c3a", ["c3a"]), ("c3b", ["c3b"]),
                  ("c3c", ["c3c"]), ("c5a", ["c5a"]), ("c5b", ["c5b"])]
C4_SUBSET = list(range(0, 100, 8))      # the fixed subset of the 100 seeded pairs: every eighth


def run_configs(torch, api, gen, reps: int = 30):
    """Every benchmark configuration in its own event-bracketed region of `reps` steps (default mode):
    back-to-back launches on one stream (`gbs`, `us_per_launch`) and one launch alone between two
    events (`isolated_us`), with the fraction of the measured copy bandwidth, the number of kernel
    launches per step and the scratch per virtual device.  c1 moves 512 KiB per step and stays in L2:
    it measures launch latency.  c4 is a fixed subset of the sweep (every eighth pair)."""
    from paper_2112_01075_b200 import workloads as wl
    peak, _ = measured_peak()
    b = wl.bench_workloads()
    out = {}
    for name, parts in CONFIG_ENTRIES:
        legs = [DeviceLeg(b[p], api.FUSE_ADJACENT, torch, api, gen) for p in parts]
        eff = sum(l.eff_bytes for l in legs)
        n_launch = sum(l.launches for l in legs)
        r = max(reps, 20)
        _, per = time_legs(torch, legs, r, 3, per_launch=True)
        iso = statistics.median([sum(per[q][i] for q in range(len(legs))) for i in range(r)]) / n_launch
        if name == "c1":
            r = 2000        # a few microseconds per step: a region long enough that the idle stream's first launch does not count
        ms, _ = time_legs(torch, legs, r, 5)
        gbs = eff / (ms / r * 1e-3) / 1e9
        out[name] = {"gbs": round(gbs, 1), "us_per_launch": round(ms / r / n_launch * 1e3, 2),
                     "frac": round(gbs / peak, 4), "frac_of_8TBs_nominal": round(gbs / 8000.0, 4),
                     "isolated_us": round(iso * 1e3, 2),
                     "isolated_gbs": round(eff / n_launch / (iso * 1e-3) / 1e9, 1),
                     "launches_per_step": n_launch, "bytes_per_launch": eff // n_launch, "reps": r,
                     "steps": [l.plan.step_kinds() for l in legs],
                     "scratch_bytes_per_virtual_device": max(l.plan.scratch_bytes_per_device for l in legs),
                     "memory_bound_bytes_per_virtual_device": max(
                         max(l.plan.local_elems(0), l.plan.local_elems(1)) * l.w.elem_bytes for l in legs)}
        if name in ("c1", "c2"):
            # host time of one bound call (redist_bound_execute through ctypes): launches queued without waiting
            sp = torch.cuda.current_stream().cuda_stream
            torch.cuda.synchronize()
            calls = 500
            t0 = time.perf_counter()
            for i in range(calls):
                for l in legs:
                    l.run(i, sp)
            host = (time.perf_counter() - t0) / (calls * len(legs))
            torch.cuda.synchronize()
            out[name]["host_us_per_bound_call"] = round(host * 1e6, 2)
        del legs
        torch.cuda.empty_cache()
    rows = sweep_rows(torch, api, [wl.config4()[i] for i in C4_SUBSET], api.FUSE_ADJACENT, wl.CONFIG4_FILL_SEED)
    g = [r["gbs"] for r in rows]
    out["c4"] = {"pairs": [r["name"] for r in rows], "geomean_gbs": round(geomean(g), 1), "min_gbs": min(g),
                 "max_gbs": max(g), "frac_geomean": round(geomean(g) / peak, 4), "frac_min": round(min(g) / peak, 4),
                 "launches_max": max(r["launches"] for r in rows),
                 "scratch_bytes_per_virtual_device_max": max(r["scratch_per_device"] for r in rows),
                 "note": "every eighth of the 100 seeded pairs, each planned, executed and timed on its own "
                         "(global array 4 GiB; 5 timed repetitions per pair after 2 warm-up launches)"}
    return out


def spread_model(api, ws, flags, hbm_gbs, link_gbs=770.0):
    """NOT a measurement: what redist_plan_gpu_split says would stay inside a GPU and what would cross to
    a peer if the virtual devices of this workload sat on 2, 4 or 8 GPUs (leading mesh axes choose the
    GPU), and the time that bounds a step from below -- the slower of local bytes at the measured HBM
    rate and, for the busiest GPU, bytes out or in at 770 GB/s (measured peer copy per direction)."""
    out = {}
    for g in (2, 4, 8):
        local = cross = 0
        t_us = 0.0
        ok = True
        for w in ws:
            plan = api.Plan(w.mesh_shape, w.src, w.dst, w.elem_bytes, flags)
            for q in range(plan.num_launches):
                try:
                    m = plan.gpu_split(g, q)
                except api.RedistError:
                    ok = False
                    break
                li = plan.launch_info(q)
                loc = sum(m[i][i] for i in range(g))
                out_b = max(sum(m[i][j] for j in range(g) if j != i) for i in range(g))
                in_b = max(sum(m[i][j] for i in range(g) if i != j) for j in range(g))
                local += loc
                cross += sum(map(sum, m)) - loc
                # per GPU: its share of the reads and local writes at HBM speed, its link traffic at link speed
                t_us += max((li.bytes_read + loc) / g / (hbm_gbs * 1e3), max(out_b, in_b) / (link_gbs * 1e3))
        if ok:
            out[f"{g}_gpus"] = {"local_bytes_written": local, "cross_bytes_written": cross,
                                "lower_bound_us_per_step": round(t_us, 1)}
    out["note"] = "model from redist_plan_gpu_split, not run on several GPUs"
    return out


def geomean(v):
    import math
    return math.exp(sum(math.log(x) for x in v) / len(v))


def describe_workload(name, ws):
    w = ws[0]
    dt = {2: "bf16", 4: "f32/u32"}.get(w.elem_bytes, f"{w.elem_bytes}B")
    return (f"{name}: {dt} {list(w.src.global_shape)}, mesh {dict(zip(w.axis_names, w.mesh_shape))} "
            f"({w.n_devices} virtual devices), " +
            " then ".join(f"{x.src.notation(x.mesh_shape, x.axis_names)} -> {x.dst.notation(x.mesh_shape, x.axis_names)}"
                          for x in ws))


def run_e2e(torch, api, ws, flags, steps, world, dist):
    """The same step through redist_execute_host: pinned host tiles in, pinned host tiles out."""
    legs = []
    h2d = d2h = 0
    for w in ws:
        p = api.Plan(w.mesh_shape, w.src, w.dst, w.elem_bytes, flags)
        sb, db = p.local_elems(0) * w.elem_bytes, p.local_elems(1) * w.elem_bytes
        G = torch.randint(0, 256, tuple(w.src.global_shape) + (w.elem_bytes,), dtype=torch.uint8)
        hs = [t.reshape(-1).pin_memory() for t in api.shard_global(G, w.mesh_shape, w.src)]
        hd = [torch.empty(db, dtype=torch.uint8).pin_memory() for _ in range(p.n_devices)]
        dsrc = torch.empty(p.staging_bytes(0), dtype=torch.uint8, device="cuda")
        ddst = torch.empty(p.staging_bytes(1), dtype=torch.uint8, device="cuda")
        legs.append((p, hs, hd, dsrc, ddst, p.alloc_scratch(), effective_bytes(w)))
        h2d += sb * p.n_devices
        d2h += db * p.n_devices
    # independent redistributions go to different streams (one per leg), so the device-to-host copy
    # of one overlaps the host-to-device copy of the next: PCIe is full duplex
    main = torch.cuda.current_stream()
    streams = [torch.cuda.Stream() for _ in legs]

    def one():
        for (p, hs, hd, dsrc, ddst, scr, _), st in zip(legs, streams):
            p.execute_host(hs, hd, dsrc, ddst, scr, st)

    for _ in range(2):
        one()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record(main)
    for st in streams:
        st.wait_event(t0)
    for _ in range(steps):
        one()
    for st in streams:
        main.wait_stream(st)
    t1.record(main)
    torch.cuda.synchronize()
    ms = t0.elapsed_time(t1)
    ms = reduce_max(dist, ms)
    per_step = ms / steps
    return {"value": round(world * sum(l[6] for l in legs) / (per_step * 1e-3) / 1e9, 2), "unit": UNIT,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": round(per_step, 3), "steps": steps,
            "api": "redist_execute_host (pinned host tiles, one cudaMemcpyAsync per tile each way; one stream per "
                   "redistribution of the step)"}


def run_others(torch, api, gen, args):
    """Short measurements of the other configurations and of the comparison modes (not the headline)."""
    out = {}
    names = ["c1", "c3a", "c3b", "c3c", "c5a", "c5b"]
    for name in names:
        for fuse, flags in (("adjacent", api.FUSE_ADJACENT), ("none", api.FUSE_NONE), ("naive", api.NAIVE)):
            ws = legs_of(name)
            if fuse != "adjacent" and name in ("c1",):
                continue
            try:
                legs = [DeviceLeg(w, flags, torch, api, gen) for w in ws]
                total, per = time_legs(torch, legs, 10, 3, per_launch=True)
                eff = sum(l.eff_bytes for l in legs)
                med = statistics.median([sum(per[q][i] for q in range(len(legs))) for i in range(10)])
                out[f"{name}/{fuse}"] = {"gbs": round(eff / (med * 1e-3) / 1e9, 1), "us": round(med * 1e3, 2),
                                         "launches": sum(l.launches for l in legs),
                                         "scratch_per_device": max(l.plan.scratch_bytes_per_device for l in legs)}
                del legs
                torch.cuda.empty_cache()
            except Exception as ex:   # report, never hide
                out[f"{name}/{fuse}"] = {"error": str(ex)[:200]}
    for fuse, flags in (("none", api.FUSE_NONE), ("naive", api.NAIVE)):
        legs = [DeviceLeg(w, flags, torch, api, gen) for w in legs_of("c2")]
        total, per = time_legs(torch, legs, 20, 3)
        eff = sum(l.eff_bytes for l in legs)
        out[f"c2/{fuse}"] = {"gbs": round(eff / (total / 20 * 1e-3) / 1e9, 1), "us": round(total / 20 * 1e3, 2),
                             "launches": sum(l.launches for l in legs),
                             "scratch_per_device": max(l.plan.scratch_bytes_per_device for l in legs)}
    return out


def sweep_rows(torch, api, pairs, flags, fill_seed):
    """Plan, execute and time every problem of `pairs` on its own.  Global arrays are far larger than
    the L2, so no buffer rotation is needed; replicated source tiles share one buffer per distinct tile."""
    gen = torch.Generator(device="cuda")
    gen.manual_seed(fill_seed)
    G = None
    stream = torch.cuda.current_stream()
    rows = []
    for w in pairs:
        if G is None or tuple(G.shape[:-1]) != tuple(w.src.global_shape):
            G = None
            G = torch.randint(0, 256, tuple(w.src.global_shape) + (w.elem_bytes,), dtype=torch.uint8, device="cuda",
                              generator=gen)
        plan = api.Plan(w.mesh_shape, w.src, w.dst, w.elem_bytes, flags)
        _, offs = api.redist_base_offsets(w.mesh_shape, w.src)
        tiles = api.shard_global(G, w.mesh_shape, w.src)
        owned = {}
        for d, o in enumerate(offs):
            if o not in owned:
                owned[o] = tiles[d].clone()
        src = [owned[o] for o in offs]
        del tiles
        db = plan.local_elems(1) * w.elem_bytes
        dst = [torch.empty(db, dtype=torch.uint8, device="cuda") for _ in range(plan.n_devices)]
        scratch = plan.alloc_scratch()
        call = plan.bind([t.data_ptr() for t in src], [t.data_ptr() for t in dst],
                         scratch.data_ptr() if scratch is not None else 0,
                         scratch.numel() if scratch is not None else 0)
        for _ in range(2):
            call(stream.cuda_stream)
        reps = 5 if w.global_elems > 2**28 else 20
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record(stream)
        for _ in range(reps):
            call(stream.cuda_stream)
        t1.record(stream)
        torch.cuda.synchronize()
        ms = t0.elapsed_time(t1) / reps
        eff = effective_bytes(w)
        li = [plan.launch_info(q) for q in range(plan.num_launches)]
        rows.append({"name": w.name, "src": w.src.notation(w.mesh_shape, w.axis_names),
                     "dst": w.dst.notation(w.mesh_shape, w.axis_names), "steps": plan.step_kinds(),
                     "launches": plan.num_launches, "run_bytes": min(i.run_bytes for i in li),
                     "variants": [i.variant for i in li],
                     "fanout": max(i.fanout for i in li), "eff_bytes": eff, "us": round(ms * 1e3, 1),
                     "gbs": round(eff / (ms * 1e-3) / 1e9, 1),
                     # what the launches actually move (every intermediate is written and read again when the
                     # sequence runs collective by collective), per second: the efficiency of the kernels
                     "traffic_gbs": round(sum(i.bytes_read + i.bytes_written for i in li) / (ms * 1e-3) / 1e9, 1),
                     "launch_runs": [i.run_bytes for i in li], "kernels": plan.launch_kernels(),
                     "scratch_per_device": plan.scratch_bytes_per_device, "plan_cost_elems": plan.cost})
        del src, dst, owned, scratch, call, plan
        torch.cuda.empty_cache()
    return rows


def run_sweep(args):
    """Config 4: the 100 seeded random (source, target) pairs on f32 [64,128,256,512], mesh 2x4x2 -- or the
    paper's P1-P4 (`adv`), or random problems shaped like the paper's evaluation sample (`eval`)."""
    import torch
    from paper_2112_01075_b200 import api, workloads as wl

    torch.cuda.set_device(0)
    if args.workload == "c4":
        pairs, label = wl.config4(max(100, args.pairs)), "c4: f32 [64,128,256,512], mesh {x:2,y:4,z:2}, %d seeded random pairs"
    elif args.workload == "adv":
        pairs, label = wl.adversarial_problems(), "adv: the %d problems of the paper's table of largest slow-downs"
    elif args.workload == "probes":
        pairs, label = wl.structured_probes(), \
            "probes: %d transposes, slices and allgathers with every mesh axis on one dimension, 8-64 devices, odd widths"
        args.pairs = max(args.pairs, len(pairs))
    else:
        pairs, label = wl.evaluation_like_problems(args.pairs), \
            "eval: %d random problems shaped like the paper's evaluation sample (3 mesh axes, <= 6-D, 64-800 MB)"
    flags = {"adjacent": api.FUSE_ADJACENT, "none": api.FUSE_NONE, "all": api.FUSE_ALL, "naive": api.NAIVE}[args.fuse]
    if args.cost_permute:
        flags |= api.COST_PERMUTE
    if args.only:
        pairs = [w for w in pairs if w.name in args.only.split(",")]
    if args.elem_bytes:
        import dataclasses
        pairs = [dataclasses.replace(w, elem_bytes=args.elem_bytes) for w in pairs]
        label += ", elements of %d bytes instead of 4" % args.elem_bytes
    rows = sweep_rows(torch, api, pairs[: args.pairs], flags, wl.CONFIG4_FILL_SEED)
    g = [r["gbs"] for r in rows]
    peak, how = measured_peak()
    line = {"metric": METRIC, "workload": label % len(rows),
            "fuse": args.fuse, "cost_permute": bool(args.cost_permute),
            "plan_cost_elems_total": sum(r["plan_cost_elems"] for r in rows), "geomean_gbs": round(geomean(g), 1),
            "min_gbs": min(g), "max_gbs": max(g), "median_gbs": statistics.median(g),
            "total_gbs": round(sum(r["eff_bytes"] for r in rows) / sum(r["us"] * 1e-6 for r in rows) / 1e9, 1),
            "traffic_geomean_gbs": round(geomean([r["traffic_gbs"] for r in rows]), 1),
            "traffic_min_gbs": min(r["traffic_gbs"] for r in rows),
            "peak": peak, "peak_source": how, "pairs_below_70pct_of_peak": sum(x < 0.7 * peak for x in g)}
    if args.dump:
        with open(args.dump, "w") as f:
            json.dump({"summary": line, "pairs": rows}, f, indent=1)
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------ CPU oracle arms

def oracle_step_fn(ws, shrink=1):
    """Build host inputs once; return (callable running one step on the oracle, effective bytes, note)."""
    import oracle
    from paper_2112_01075_b200 import workloads as wl
    cases = []
    eff = 0
    for w in ws:
        if shrink > 1:
            # bounded sample: the same mesh and types on a global array with dimension `big` divided
            shape = list(w.src.global_shape)
            big = max(range(len(shape)), key=lambda k: shape[k])
            shape[big] //= shrink
            w = w.scaled(shape, f"_1/{shrink}")
        src = (w.src.global_shape, w.src.axes)
        dst = (w.dst.global_shape, w.dst.axes)
        G = wl.global_array_bytes(w.src.global_shape, w.elem_bytes, "random_bits", w.seed)
        tiles = oracle.reslice(w.mesh_shape, src, G)
        cases.append((w.mesh_shape, src, dst, tiles))
        eff += effective_bytes(w)

    def step():
        for mesh, src, dst, tiles in cases:
            oracle.redistribute(mesh, src, dst, tiles, check=False)

    return step, eff


def cpu_baseline(ws):
    """The oracle as it stands on the host cores: a bounded sample (about 10-30 s of CPU work)."""
    import oracle
    step, eff = oracle_step_fn(ws)
    cores = oracle.max_threads()
    res = {}
    for threads in (1, cores):
        oracle.set_threads(threads)
        step()
        t_end = time.perf_counter() + 6.0
        times = []
        while len(times) < 3 or (time.perf_counter() < t_end and len(times) < 50):
            t0 = time.perf_counter()
            step()
            times.append(time.perf_counter() - t0)
        res[threads] = (min(times), statistics.median(times), len(times))
    oracle.set_threads(1)
    best = res[cores]
    return {"value": round(eff / best[1] / 1e9, 3), "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"the whole workload, median of {best[2]} passes of the C oracle with {cores} threads "
                      f"(materialise the global array, re-slice per device)",
            "single_thread_gbs": round(eff / res[1][1] / 1e9, 3),
            "ms_per_step": round(best[1] * 1e3, 2), "ms_per_step_single_thread": round(res[1][1] * 1e3, 2)}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    ws = legs_of(args.workload)
    cores = oracle.max_threads()
    oracle.set_threads(cores)
    step, eff = oracle_step_fn(ws)
    t0 = time.perf_counter()
    step()
    one = time.perf_counter() - t0
    shrink = 1
    while one / shrink * (args.steps + args.warmup) > 120.0 and shrink < 256:
        shrink *= 2
    if shrink > 1:
        step, eff = oracle_step_fn(ws, shrink)
    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / args.steps
    value = round(eff / dt / 1e9, 3)
    sample = ("the whole workload per step" if shrink == 1 else
              f"1/{shrink} of the workload per step (largest dimension divided by {shrink})")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(dt * 1e3, 3),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
            "config": {"workload": describe_workload(args.workload, ws)},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c5",
                    choices=["c1", "c2", "c3", "c3a", "c3b", "c3c", "c4", "c5", "c5a", "c5b", "adv", "eval", "probes"])
    ap.add_argument("--pairs", type=int, default=100, help="sweeps: how many problems to run")
    ap.add_argument("--only", default="", help="sweeps: comma-separated problem names to run")
    ap.add_argument("--elem-bytes", type=int, default=0, choices=[0, 1, 2, 4, 8, 16],
                    help="sweeps: run the same shapes with elements of this many bytes (0: the workload's own, 4)")
    ap.add_argument("--dump", default="", help="sweeps: write the per-problem table to this JSON file")
    ap.add_argument("--fuse", default="adjacent", choices=["adjacent", "none", "all", "naive"])
    ap.add_argument("--cost-permute", action="store_true",
                    help="plan with REDIST_COST_PERMUTE (the final permutation counted when choosing the sequence)")
    ap.add_argument("--others", action="store_true", help="also measure every configuration unfused and naive")
    ap.add_argument("--graph", action="store_true", help="time CUDA-graph replays instead of plain stream launches")
    ap.add_argument("--no-graph", action="store_true", help=argparse.SUPPRESS)   # accepted, the default
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="leave out the per-configuration block")
    ap.add_argument("--lean", action="store_true",
                    help="headline region and per-launch events only (no graph replay, comparison modes or "
                         "per-configuration block): the small command for profiler captures")
    ap.add_argument("--sets", type=int, default=0, help="rotating buffer sets (0: chosen from the workload size)")
    ap.add_argument("--tune", default="", help="tuning values for the plans, e.g. pdl=0,item_kb=16 (redist_tuning_set)")
    ap.add_argument("--standin", action="store_true",
                    help="CPU stand-in for the timed body (gloo, no CUDA): tests the N-rank launch plumbing")
    args = ap.parse_args()
    args.warmup = max(3, args.warmup) if args.impl == "ours" else args.warmup
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.workload not in ("c4", "adv", "eval"):
        spawn_ranks(args.gpus)      # does not return
    if args.tune and args.impl == "ours" and not args.standin:
        from paper_2112_01075_b200 import api
        for kv in args.tune.split(","):
            k, v = kv.split("=")
            api.tuning_set(k.strip(), int(v))
    if args.standin:
        run_standin(args)
    elif args.workload in ("c4", "adv", "eval", "probes"):
        if args.impl == "reference":
            raise SystemExit("the sweeps (c4, adv, eval) are GPU-side measurements; use another workload for --impl reference")
        run_sweep(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
