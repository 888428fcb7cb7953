#!/usr/bin/env python
"""Throughput of the LIEC-SGD compression step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c4|c2|c3|sweep-sign-28|...]
    python bench.py --impl reference ...        # the CPU oracle on a bounded sample of the same workload

One "step" is one full compressed iteration (uplink compress, server aggregate, downlink
compress + global error, worker update) over one batch of synthetic gradients that is
already resident in HBM.  The step does not shard across GPUs (every stage is either
element-wise or a per-segment reduction and there is no exchange step), so with --gpus N
every rank runs an independent replica on its own GPU: "replicas only", weak scaling,
no data-path collective.  Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "LIEC step throughput"
UNIT = "elements*workers/s"
NOMINAL_HBM_GBS = 8000.0


# ------------------------------------------------------------------------------------ workloads

def resolve_workload(name: str):
    """Returns dict(name, N, layout, dist, scale, comp, k, lr, gdt)."""
    from liec_synth import WORKLOADS, flat_layout, scaled_layout, topk_counts
    base, _, div = name.partition("/")
    base, _, variant = base.partition("-")
    seeded = variant == "randkseed"   # random-k with the subsets drawn on the GPU from (seed, step) every iteration
    if seeded:
        variant = "randk"
    if base in WORKLOADS and variant in ("", "randk", "topk", "sign"):
        w = WORKLOADS[base]
        lay = w.layout()
        if div:   # "c4/8": same tensor list with every size divided by 8 (profiling-sized case)
            lay = scaled_layout(lay, int(div))
        # "c3-randk", "c4-topk", "c3-sign": the same tensor list, workers and gradients with another
        # operator both ways (k = 1 % per tensor where the workload names no fraction)
        comp = variant or w.compressor
        frac = w.topk_frac if w.topk_frac[0] else (1, 100)
        k = topk_counts(lay, *frac) if comp in ("topk", "randk") else None
        return dict(name=name, N=w.num_workers, layout=lay, dist=w.dist, scale=w.scale, comp=comp,
                    k=k, lr=w.lr, gdt=w.grad_dtype, seeded=seeded)
    if name.startswith("sweep-"):
        # sweep-sign-26, sweep-topk1000-28 (k = n/1000), sweep-topk100-24 (k = n/100),
        # sweep-randk100-26 (random-k, k = n/100): N=8, flat, N(0,1)
        _, comp, logd = name.split("-")
        lay = flat_layout(1 << int(logd))
        if comp == "sign":
            return dict(name=name, N=8, layout=lay, dist="normal", scale=1.0, comp="sign", k=None, lr=0.1, gdt="f32")
        kind = "randk" if comp.startswith("randk") else "topk"
        den = int(comp[len(kind):])
        return dict(name=name, N=8, layout=lay, dist="normal", scale=1.0, comp=kind,
                    k=topk_counts(lay, 1, den), lr=0.1, gdt="f32")
    raise SystemExit(f"unknown workload {name!r}")


def min_bytes_per_step(w) -> float:
    """Compulsory HBM bytes of one step: every array once per pass that a global dependency forces."""
    N, d, T = w["N"], w["layout"].dim, w["layout"].num_segments
    g = 2 if w["gdt"] == "bf16" else 4
    if w["comp"] == "sign":
        return N * d * (2 * g + 8 + 1 / 8) + d * (8 + N / 8 + 1 / 4) + 4 * T * (N + 1)
    K = int(w["k"].sum())
    if w["comp"] == "randk":   # no dense pass over g on the uplink: the subsets are read, the kept entries gathered
        return N * d * (g + 8) + 8 * d + 8 * K * (2 * N + 2) + 4 * K * (N + 1)
    return N * d * (2 * g + 8) + 8 * d + 8 * K * (2 * N + 2)


def update_kernel_bytes(w) -> float:
    """Algorithmic bytes of one worker-update launch: read g, read x, write x for N*d elements,
    plus one read of the downlink message."""
    N, d = w["N"], w["layout"].dim
    g = 2 if w["gdt"] == "bf16" else 4
    down = d / 8 if w["comp"] == "sign" else 8 * int(w["k"].sum())
    own = 4 * N * int(w["k"].sum()) if w["comp"] == "randk" else 0   # each worker's own index list
    return N * d * (g + 8) + down + own


# DRAM bytes (dram__bytes_read + dram__bytes_write, ncu) of one worker-update launch, per named
# workload.  c4: captured on c4/8 (4.924 GB for 497.8 M element-workers) and scaled by N*d, because
# this streaming kernel's traffic grows in proportion; c3 and c2: captured at full size (the tail
# of the parameter writes is still in the L2 when the kernel ends, hence slightly fewer bytes than
# the algorithmic count).  Any other workload or variant: not captured.
UPDATE_TRAFFIC_BYTES = {"c4": (2.989412e9 + 1.934865e9) / 497759232 * 32 * 124439808, "c3": 3274712064 + 1583202304,
                        "c2": 749630720 + 322008320}


# ------------------------------------------------------------------------------------ clocks

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.samples = []
        self.proc = None
        self.gpu_index = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append((time.monotonic(), line.strip()))

    def mark_begin(self):
        self.t0 = time.monotonic()

    def mark_end(self):
        self.t1 = time.monotonic()

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        t0, t1 = getattr(self, "t0", 0.0), getattr(self, "t1", float("inf"))
        inside = [line for (ts, line) in self.samples if t0 <= ts <= t1 + 0.05]
        for s in inside:
            parts = [q.strip() for q in s.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------ CPU oracle leg

def _segment_sample(w, budget, part=0, parts=1):
    """A bounded sample of the workload for the CPU oracle: all N workers on a subset of the
    segments (the step is segment-local, so this is the full computation for those segments).
    With parts > 1 the segments are dealt out in size order, so that the parts are disjoint and
    alike; a flat vector is cut into disjoint slices, each treated as a vector of its own."""
    from liec_synth import flat_layout
    lay, N = w["layout"], w["N"]
    if lay.num_segments == 1:
        n = int(min(lay.dim // parts, budget // N))
        return flat_layout(n), None, f"a slice of {n} elements of the flat vector, all {N} workers"
    order = sorted(range(lay.num_segments), key=lambda t: -lay.sizes[t])
    if parts == 1:   # a spread: every ceil(T/16)-th segment in size order, then whatever still fits
        stride = max(1, lay.num_segments // 16)
        order = order[::stride] + order
    else:
        order = order[part::parts]
    chosen, total = [], 0
    for t in order:
        if t in chosen or (total + lay.sizes[t]) * N > budget:
            continue
        chosen.append(t)
        total += lay.sizes[t]
    if not chosen:   # nothing fits the budget: the smallest segment of this part
        chosen = [min(order, key=lambda t: lay.sizes[t])]
    chosen.sort()
    sub = lay.subset(chosen, name=f"{lay.name}[{len(chosen)} segments]")
    return sub, chosen, f"{len(chosen)} of {lay.num_segments} segments ({sub.dim} elements), all {N} workers"


def _oracle_inputs(w, sub, chosen, seed):
    import numpy as np
    import torch
    import oracle
    from liec_synth import make_gradients, random_subsets
    N, d = w["N"], sub.dim
    k = None
    if w["comp"] in ("topk", "randk"):
        k = w["k"][chosen] if chosen is not None else np.asarray([max(1, int(w["k"][0] * d // w["layout"].dim))], np.int64)
    sets = random_subsets(sub.seg_offsets, k, N + 1, 0, seed) if w["comp"] == "randk" else None

    def grads(step):
        G = make_gradients(w["dist"], w["scale"], N, d, step, base_seed=seed)
        return oracle.widen_bf16(G.view(torch.int16).numpy().view(np.uint16)) if G.dtype == torch.bfloat16 else G.numpy()
    return k, sets, grads


def _oracle_step_seconds(w, sub, k, sets, Gf, X, e):
    import oracle
    comp = {"sign": oracle.SIGN, "topk": oracle.TOPK, "randk": oracle.RANDK}[w["comp"]]
    N = w["N"]
    t0 = time.perf_counter()
    oracle.step(X, e, Gf, w["lr"], sub.seg_offsets, comp, comp, k=k,
                up_sets=None if sets is None else sets[:N], down_set=None if sets is None else sets[N])
    return time.perf_counter() - t0


def time_oracle(w, steps: int, warmup: int):
    """The oracle as it stands (single-threaded C) on one core."""
    import numpy as np
    budget = 3e8 if w["comp"] == "sign" else 2.5e7   # element*workers per oracle step
    sub, chosen, desc = _segment_sample(w, budget)
    N, d = w["N"], sub.dim
    k, sets, grads = _oracle_inputs(w, sub, chosen, 99)
    X = np.zeros((N, d), np.float32)
    e = np.zeros(d, np.float32)
    times = []
    for s in range(warmup + steps):
        dt = _oracle_step_seconds(w, sub, k, sets, grads(s), X, e)
        if s >= warmup:
            times.append(dt)
    mean = sum(times) / len(times)
    return {"value": N * d / mean, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc,
            "host_cores": len(os.sched_getaffinity(0)), "seconds_per_sample_step": mean}


def _all_cores_worker(wname, part, parts, budget, barrier, out):
    """One single-threaded oracle process: prepares its own disjoint sample, waits for the others,
    runs one oracle step, reports (element*workers, start, end)."""
    try:
        import numpy as np
        import torch
        torch.set_num_threads(1)
        w = resolve_workload(wname)
        sub, chosen, _ = _segment_sample(w, budget, part, parts)
        k, sets, grads = _oracle_inputs(w, sub, chosen, 199 + part)
        Gf = grads(0)
        X = np.zeros((w["N"], sub.dim), np.float32)
        e = np.zeros(sub.dim, np.float32)
        import oracle
        oracle.lib()
        barrier.wait(timeout=600)
        t0 = time.time()
        _oracle_step_seconds(w, sub, k, sets, Gf, X, e)
        out.put((w["N"] * sub.dim, t0, time.time()))
    except Exception as exc:   # a worker that fails must not leave the others at the barrier
        try:
            barrier.abort()
        except Exception:
            pass
        out.put(("error", repr(exc), 0.0))


def time_oracle_all_cores(w):
    """The same single-threaded oracle, one process per host core, each on a disjoint sample of the
    workload; throughput = all element*workers processed / wall-clock from the common start to the
    last process's end.  The oracle's source is not touched (it has no threads of its own)."""
    import multiprocessing as mp
    import oracle
    oracle.build()
    cores = len(os.sched_getaffinity(0))
    T = w["layout"].num_segments
    parts = cores if T == 1 else max(1, min(cores, T // 2))
    total = (3e8 if w["comp"] == "sign" else 2.5e7) * 4
    budget = max(total / parts, 2e6)
    ctx = mp.get_context("spawn")
    barrier, out = ctx.Barrier(parts), ctx.Queue()
    procs = [ctx.Process(target=_all_cores_worker, args=(w["name"], q, parts, budget, barrier, out)) for q in range(parts)]
    for pr in procs:
        pr.start()
    results, deadline = [], time.time() + 900
    while len(results) < parts and time.time() < deadline:
        try:
            results.append(out.get(timeout=2))
        except Exception:   # queue empty: a process that died before it could report ends the wait
            if any(pr.exitcode not in (None, 0) for pr in procs):
                break
    for pr in procs:
        pr.join(timeout=5)
        if pr.is_alive():
            pr.terminate()
    if len(results) < parts:
        return {"unavailable": f"only {len(results)} of {parts} oracle processes reported"}
    bad = [r for r in results if r[0] == "error"]
    if bad:
        return {"unavailable": f"{len(bad)} of {parts} oracle processes failed: {bad[0][1]}"}
    units = sum(r[0] for r in results)
    wall = max(r[2] for r in results) - min(r[1] for r in results)
    return {"value": units / wall, "unit": UNIT, "cores": parts, "host_cores": cores, "kind": "oracle, one process per core",
            "sample": f"{parts} disjoint samples of about {budget:.3g} element*workers each ({units} in all)",
            "wall_seconds": wall}


# ------------------------------------------------------------------------------------ ranks

def max_over_ranks(values, device=None):
    """Element-wise maximum of a list of floats over all ranks (identity when not distributed)."""
    import torch
    if not (torch.distributed.is_available() and torch.distributed.is_initialized()):
        return list(values)
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return t.tolist()


def whole_job_throughput(units_per_rank: float, world: int, ms_step_max: float) -> float:
    """Replicas only: every rank processes units_per_rank per step; the job is as slow as its slowest rank."""
    return units_per_rank * world / (ms_step_max * 1e-3)


# ------------------------------------------------------------------------------------ GPU leg

def num_batches(w) -> int:
    """Distinct gradient batches kept resident in HBM and taken in turn by the steps: as many as fit
    in about 40 GB, between 4 and 16."""
    g = 2 if w["gdt"] == "bf16" else 4
    return int(min(16, max(4, 40e9 // (w["N"] * w["layout"].dim * g))))


def run_gpu(args, w, rank, world, local_rank, steps=None, extras=True):
    """Times `steps` iterations of workload w.  extras: also the CUDA-graph replay, the averaging
    iteration and the host-fed end-to-end leg (the headline workload); otherwise the step alone."""
    import torch
    from liec_synth import make_gradients
    from paper_2402_11857_b200 import liec

    steps = steps or args.steps
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    lay = w["layout"]
    N, d = w["N"], lay.dim
    comp = {"sign": liec.COMP_SCALED_SIGN, "topk": liec.COMP_TOPK, "randk": liec.COMP_RANDK}[w["comp"]]
    gdt = liec.BF16 if w["gdt"] == "bf16" else liec.F32
    X = torch.zeros(N, d, device=dev)
    e = torch.zeros(d, device=dev)
    ctx = liec.Context(X, e, lay.seg_offsets, comp, comp, w["k"], gdt)
    NUM_BATCHES = args.batches or num_batches(w)
    # the gradient of worker i at step t is drawn from seed (i, t): NUM_BATCHES consecutive steps'
    # draws are resident and the steps cycle through them (every step sees other values than the one
    # before, which matters for top-k: its uplink starts from the previous step's thresholds)
    batches = [make_gradients(w["dist"], w["scale"], N, d, step=b, base_seed=1000 + rank, device=dev)
               for b in range(NUM_BATCHES)]
    G = batches[0]
    seeded = bool(w.get("seeded"))
    if w["comp"] == "randk" and not seeded:   # the subsets are inputs: drawn once on the host, resident like the gradients
        import numpy as np
        from liec_synth import random_subsets
        sets = random_subsets(lay.seg_offsets, w["k"], N + 1, 0, 1000 + rank)
        up_sets = torch.from_numpy(np.ascontiguousarray(sets[:N]).view(np.int32)).to(dev)
        down_set = torch.from_numpy(np.ascontiguousarray(sets[N]).view(np.int32)).to(dev)
        ctx.liec_set_subsets(up_sets, down_set)
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            torch.distributed.barrier()

    stage_names = ["uplink_compress", "server_aggregate", "downlink_compress", "worker_update"]

    counter = [0]   # steps taken so far: selects the batch

    def one_step(events=None):
        g = batches[counter[0] % NUM_BATCHES]
        counter[0] += 1
        if events is None:
            if seeded:
                ctx.liec_draw_subsets(1000 + rank, counter[0])
            ctx.liec_step(g, w["lr"])
            return
        events[0].record()
        if seeded:   # (the draw is timed as part of the uplink stage)
            ctx.liec_draw_subsets(1000 + rank, counter[0])
        ctx.liec_uplink_compress(g); events[1].record()
        ctx.liec_server_aggregate(); events[2].record()
        ctx.liec_downlink_compress(); events[3].record()
        ctx.liec_worker_update(g, w["lr"]); events[4].record()

    sampler = ClockSampler(local_rank)
    sampler.start()          # nvidia-smi needs a moment to start: launch it before the warm-up
    for _ in range(args.warmup):
        one_step()
    torch.cuda.synchronize()
    barrier()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(steps)]
    launches0 = ctx.liec_launch_count()
    torch.cuda.synchronize()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.mark_begin()
    start.record()
    for s in range(steps):
        one_step(evs[s])
    stop.record()
    torch.cuda.synchronize()
    sampler.mark_end()
    total_ms = start.elapsed_time(stop)
    launches = ctx.liec_launch_count() - launches0
    barrier()
    clocks = sampler.stop()
    assert ctx.liec_device_status() == 0, "device status word is non-zero"

    stage_ms = [statistics.mean(evs[s][q].elapsed_time(evs[s][q + 1]) for s in range(steps)) for q in range(4)]

    # top-k: which route the selections take on these per-step gradients (untimed extra steps; the
    # count needs a synchronisation and a copy of the selection state)
    routes = None
    if w["comp"] == "topk":
        acc = {"uplink_single_pass": 0, "uplink_direct": 0, "uplink_refined": 0, "downlink_refined": 0, "slow": 0}
        extra = min(2 * NUM_BATCHES, 16)
        for _ in range(extra):
            one_step()
            up, down = ctx.liec_topk_route_counts(True), ctx.liec_topk_route_counts(False)
            acc["uplink_single_pass"] += up["single_pass"]; acc["uplink_refined"] += up["refined"]
            acc["uplink_direct"] += up["direct"]
            acc["downlink_refined"] += down["refined"]; acc["slow"] += up["slow"] + down["slow"]
        routes = {"uplink_problems": up["problems"], "downlink_problems": down["problems"], "steps_counted": extra,
                  "uplink_single_tile_fraction": acc["uplink_direct"] / (extra * up["problems"]),
                  "uplink_single_pass_fraction": acc["uplink_single_pass"] / (extra * up["problems"]),
                  "note": "single tile: segments of at most 8192 elements, selected by one CTA; single pass: "
                          "finished on the one dense pass seeded by the previous step's threshold; the rest "
                          "took the two-pass route",
                  "uplink_refined_per_step": acc["uplink_refined"] / extra,
                  "downlink_refined_per_step": acc["downlink_refined"] / extra, "slow_per_step": acc["slow"] / extra}
    # the same iteration with the fused telemetry switched on (squared norms of e, v and g left by the
    # server pass and the worker update), the accessor that reduces them, and, for comparison, the
    # separate passes that give the same numbers on demand (liec_sumsq over e and over the gradients)
    telemetry = None
    if args.telemetry:
        tsteps = max(3, min(steps, 10))
        ctx.liec_set_telemetry(True)
        for _ in range(2):
            one_step()
        t0, t1, t2, t3 = (torch.cuda.Event(enable_timing=True) for _ in range(4))
        torch.cuda.synchronize()
        t0.record()
        for _ in range(tsteps):
            one_step()
        t1.record()
        tel = ctx.liec_get_telemetry()
        t2.record()
        out_e = torch.empty(1, lay.num_segments, dtype=torch.float64, device=dev)
        out_g = torch.empty(N, lay.num_segments, dtype=torch.float64, device=dev)
        ctx.liec_sumsq(liec.SUMSQ_ERROR, out_e)
        ctx.liec_sumsq(liec.SUMSQ_GRADS, out_g, grads=batches[(counter[0] - 1) % NUM_BATCHES])
        t3.record()
        torch.cuda.synchronize()
        assert torch.equal(out_g, tel["g_sumsq"]), "fused and separate squared norms of g differ"
        ctx.liec_set_telemetry(False)
        on_ms = t0.elapsed_time(t1) / tsteps
        telemetry = {"ms_per_step_on": on_ms, "ms_per_step_off": total_ms / steps, "steps": tsteps,
                     "overhead_pct": 100 * (on_ms / (total_ms / steps) - 1), "accessor_ms": t1.elapsed_time(t2),
                     "separate_passes_ms": t2.elapsed_time(t3),
                     "note": "on: the server pass also leaves ||e_t||^2 and ||v_t||^2, the worker update ||g^i_t||^2 per "
                             "tile; accessor: liec_get_telemetry; separate passes: liec_sumsq over e and over the gradients"}
    if not extras:
        ms_step = total_ms / steps
        if world > 1:
            vals = max_over_ranks([ms_step] + stage_ms, device=dev)
            ms_step, stage_ms = vals[0], vals[1:]
        return dict(ms_step=ms_step, stage_ms=dict(zip(stage_names, stage_ms)), launches=launches, clocks=clocks,
                    e2e=None, average_ms=None, graph_ms=None, routes=routes, steps=steps, telemetry=telemetry)

    # the same step replayed from a CUDA graph (one capture of liec_step, K replays): shows what the
    # launch gaps cost on small workloads; reported beside the headline, not instead of it
    graph_ms = None
    if args.cuda_graph:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            ctx.liec_step(G, w["lr"], stream=side)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):     # one replay = NUM_BATCHES steps, one per resident batch
            for g in batches:
                ctx.liec_step(g, w["lr"])
        for _ in range(2):
            graph.replay()
        torch.cuda.synchronize()
        replays = max(1, steps // NUM_BATCHES)
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        for _ in range(replays):
            graph.replay()
        g1.record()
        torch.cuda.synchronize()
        graph_ms = g0.elapsed_time(g1) / (replays * NUM_BATCHES)
        assert ctx.liec_device_status() == 0

    # the model-averaging iteration (every 32nd / 100th step in the paper's runs): timed on its own,
    # not part of the headline step
    a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ctx.liec_average_step(G, w["lr"])
    torch.cuda.synchronize()
    a0.record()
    for _ in range(5):
        ctx.liec_average_step(G, w["lr"])
    a1.record()
    torch.cuda.synchronize()
    average_ms = a0.elapsed_time(a1) / 5

    # end to end through the host-buffer entry point: H2D of the gradients and D2H of the
    # downlink message inside the timed region
    e2e = None
    if not args.no_e2e:
        e2e_steps = max(1, min(steps, args.e2e_steps))
        Gh = torch.empty(G.shape, dtype=G.dtype, pin_memory=True)
        Gh.copy_(G)
        msg_bytes = liec.down_message_bytes(ctx.cfg)
        msg = torch.empty(max(msg_bytes, 4), dtype=torch.uint8, pin_memory=True)
        ctx.liec_step_host(Gh, G, w["lr"], msg)   # warm-up
        torch.cuda.synchronize()
        barrier()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record()
        for _ in range(e2e_steps):
            ctx.liec_step_host(Gh, G, w["lr"], msg)
        s1.record()
        torch.cuda.synchronize()
        e2e_ms = s0.elapsed_time(s1) / e2e_steps
        e2e = {"ms_per_step": e2e_ms, "steps": e2e_steps, "h2d": Gh.numel() * Gh.element_size(), "d2h": msg_bytes}

    ms_step = total_ms / steps
    if world > 1:
        vals = max_over_ranks([ms_step, e2e["ms_per_step"] if e2e else 0.0] + stage_ms, device=dev)
        ms_step, e2e_max, stage_ms = vals[0], vals[1], vals[2:]
        if e2e:
            e2e["ms_per_step"] = e2e_max
    return dict(ms_step=ms_step, stage_ms=dict(zip(stage_names, stage_ms)), launches=launches, clocks=clocks, e2e=e2e,
                average_ms=average_ms, graph_ms=graph_ms, routes=routes, steps=steps, telemetry=telemetry)


def describe(w, gpus):
    lay = w["layout"]
    return {"workload": f"{w['name']}: N={w['N']} workers, d={lay.dim} in {lay.num_segments} segments ({lay.name}), "
                        f"{w['comp']} both ways, gradients {w['dist']} {w['gdt']}",
            "num_workers": w["N"], "dim": lay.dim, "segments": lay.num_segments, "compressor": w["comp"],
            "gradient_batches": f"{num_batches(w)} resident batches drawn per (worker, step), taken in turn",
            "l2_policy": "inputs larger than L2 (gradients and parameters are streamed from HBM every step)",
            "parallelism": "replicas only" if gpus > 1 else "single GPU"}


def peak_bandwidth():
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        return json.load(open(peaks_path))["hbm_gbs"], "measured copy bandwidth (MEASURED_PEAKS.json)"
    return 6650.0, "fallback 6.65 TB/s"


def throughput_fields(w, r, world):
    """Step-level and dominant-kernel figures of one measured workload."""
    N, d = w["N"], w["layout"].dim
    peak, peak_src = peak_bandwidth()
    bmin = min_bytes_per_step(w)
    step_gbs = bmin / (r["ms_step"] * 1e-3) / 1e9
    upd_ms = r["stage_ms"]["worker_update"]
    upd_gbs = update_kernel_bytes(w) / (upd_ms * 1e-3) / 1e9
    out = {
        "value": whole_job_throughput(N * d, world, r["ms_step"]), "unit": UNIT, "steps": r["steps"],
        "ms_per_step": r["ms_step"],
        "hbm_gbs": step_gbs, "pct_of_8tbs_nominal": 100 * step_gbs / NOMINAL_HBM_GBS,
        "pct_of_measured_copy_peak": 100 * step_gbs / peak, "min_bytes_per_step": bmin,
        "stage_ms": r["stage_ms"],
        "roofline": {"bound": "hbm", "kernel": "worker_update_kernel", "achieved": upd_gbs, "peak": peak,
                     "unit": "GB/s", "frac": upd_gbs / peak,
                     "traffic": UPDATE_TRAFFIC_BYTES.get(w["name"]), "peak_source": peak_src,
                     "algorithmic_bytes_per_launch": update_kernel_bytes(w), "launch_ms": upd_ms},
        "gpu_launches": r["launches"], "clocks": r["clocks"],
    }
    if r["routes"] is not None:
        out["topk_routes"] = r["routes"]
    if r.get("telemetry") is not None:
        out["telemetry"] = r["telemetry"]
    return out


# Measured beside the headline when no --workload is given: the top-k target configuration and the
# 2^28 points of the bandwidth sweep (fewer steps: they only add context).
SECONDARY = (("topk_path", "c3", None), ("sweep_sign_2p28", "sweep-sign-28", 10), ("sweep_topk100_2p28", "sweep-topk100-28", 10))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=None,
                    help="one workload only (c1..c4, c4/8, c3-randk, sweep-sign-28, ...); default: c4 as the headline "
                         "plus c3 and two sweep points under their own keys")
    ap.add_argument("--batches", type=int, default=0,
                    help="resident gradient batches the steps cycle through (default: as many as fit in 40 GB, 4 to 16)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-telemetry", dest="telemetry", action="store_false", default=True,
                    help="skip the extra steps that time the iteration with the fused telemetry switched on")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cuda-graph", dest="cuda_graph", action="store_true", default=True,
                    help="also time the step replayed from a CUDA graph (default; reported beside the headline)")
    ap.add_argument("--no-cuda-graph", dest="cuda_graph", action="store_false")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    w = resolve_workload(args.workload or "c4")
    lay = w["layout"]
    N, d = w["N"], lay.dim
    config = describe(w, args.gpus)

    if args.impl == "reference":
        if rank != 0:
            return
        steps = max(1, min(args.steps, 3))
        cb = time_oracle(w, steps, min(args.warmup, 1))
        line = {"impl": "reference", "metric": METRIC, "value": cb["value"], "unit": UNIT, "n_gpus": args.gpus,
                "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": cb["seconds_per_sample_step"] * 1e3,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
                "data": "synthetic", "config": config, "cpu_baseline": cb,
                "e2e": {"value": cb["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
        print(json.dumps(line))
        return

    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    if world > 1:
        torch.distributed.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    r = run_gpu(args, w, rank, world, local_rank)
    secondary = {}
    if args.workload is None:
        for key, name, nsteps in SECONDARY:
            torch.cuda.empty_cache()
            w2 = resolve_workload(name)
            r2 = run_gpu(args, w2, rank, world, local_rank, steps=min(args.steps, nsteps) if nsteps else None, extras=False)
            secondary[key] = (w2, r2)
    if rank != 0:
        torch.distributed.destroy_process_group()
        return

    units = N * d * world
    line = {"metric": METRIC, "n_gpus": world, "warmup": args.warmup, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": config}
    line.update(throughput_fields(w, r, world))
    line["average_step"] = {"ms": r["average_ms"],
                            "gbs": (N * d * ((2 if w["gdt"] == "bf16" else 4) + 8) + 8 * d) / (r["average_ms"] * 1e-3) / 1e9,
                            "note": "model-averaging iteration of Algorithm 1, timed separately (5 runs)"}
    if r["graph_ms"] is not None:
        line["cuda_graph"] = {"ms_per_step": r["graph_ms"], "value": units / (r["graph_ms"] * 1e-3), "unit": UNIT}
    if r["e2e"]:
        line["e2e"] = {"value": units / (r["e2e"]["ms_per_step"] * 1e-3), "unit": UNIT,
                       "h2d_bytes_per_step": r["e2e"]["h2d"], "d2h_bytes_per_step": r["e2e"]["d2h"],
                       "ms_per_step": r["e2e"]["ms_per_step"], "steps": r["e2e"]["steps"]}
    for key, (w2, r2) in secondary.items():
        entry = {"config": describe(w2, args.gpus)}
        entry.update(throughput_fields(w2, r2, world))
        line[key] = entry
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = time_oracle(w, 1, 0)
        line["cpu_baseline"]["all_cores"] = time_oracle_all_cores(w)
    print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
