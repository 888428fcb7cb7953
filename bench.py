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
                    k=k, lr=w.lr, gdt=w.grad_dtype)
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
# workload.  c4: captured on c4/8 (4.925 GB for 497.8 M element-workers) and scaled by N*d, because
# this streaming kernel's traffic grows in proportion; c3 and c2: captured at full size (the tail
# of the parameter writes is still in the L2 when the kernel ends, hence slightly fewer bytes than
# the algorithmic count).  Any other workload or variant: not captured.
UPDATE_TRAFFIC_BYTES = {"c4": 4.924888e9 / 497759232 * 32 * 124439808, "c3": 3274704384 + 1587624448,
                        "c2": 749634816 + 323100160}


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

def oracle_sample(w):
    """A bounded sample of the workload for the CPU oracle: all N workers on a subset of the
    segments (the step is segment-local, so this is the full computation for those segments)."""
    lay = w["layout"]
    budget = 3e8 if w["comp"] == "sign" else 2.5e7   # element*workers per oracle step
    order = sorted(range(lay.num_segments), key=lambda t: -lay.sizes[t])
    chosen, total = [], 0
    # take a spread: every ceil(T/16)-th segment in size order until the budget is met
    stride = max(1, lay.num_segments // 16)
    for t in order[::stride] + order:
        if t in chosen:
            continue
        if (total + lay.sizes[t]) * w["N"] > budget and chosen:
            continue
        if lay.sizes[t] * w["N"] > budget and not chosen and lay.num_segments > 1:
            continue
        chosen.append(t)
        total += lay.sizes[t]
    if lay.num_segments == 1:
        # flat vector: use a prefix
        from liec_synth import flat_layout
        n = int(min(lay.dim, budget // w["N"]))
        return flat_layout(n), None, f"prefix of {n} elements of the flat vector, all {w['N']} workers"
    chosen.sort()
    sub = lay.subset(chosen, name=f"{lay.name}[{len(chosen)} segments]")
    return sub, chosen, f"{len(chosen)} of {lay.num_segments} segments ({sub.dim} elements), all {w['N']} workers"


def time_oracle(w, steps: int, warmup: int):
    import numpy as np
    import torch
    import oracle
    from liec_synth import make_gradients, topk_counts
    sub, chosen, desc = oracle_sample(w)
    N, d = w["N"], sub.dim
    from liec_synth import random_subsets
    comp = {"sign": oracle.SIGN, "topk": oracle.TOPK, "randk": oracle.RANDK}[w["comp"]]
    k = None
    if w["comp"] in ("topk", "randk"):
        k = w["k"][chosen] if chosen is not None else np.asarray([max(1, int(w["k"][0] * d // w["layout"].dim))], np.int64)
    X = np.zeros((N, d), np.float32)
    e = np.zeros(d, np.float32)
    sets = random_subsets(sub.seg_offsets, k, N + 1, 0, 99) if w["comp"] == "randk" else None
    times = []
    for s in range(warmup + steps):
        G = make_gradients(w["dist"], w["scale"], N, d, s, base_seed=99)
        Gf = oracle.widen_bf16(G.view(torch.int16).numpy().view(np.uint16)) if G.dtype == torch.bfloat16 else G.numpy()
        t0 = time.perf_counter()
        oracle.step(X, e, Gf, w["lr"], sub.seg_offsets, comp, comp, k=k,
                    up_sets=None if sets is None else sets[:N], down_set=None if sets is None else sets[N])
        dt = time.perf_counter() - t0
        if s >= warmup:
            times.append(dt)
    mean = sum(times) / len(times)
    return {"value": N * d / mean, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc,
            "seconds_per_sample_step": mean}


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

def run_gpu(args, w, rank, world, local_rank):
    import torch
    from liec_synth import make_gradients
    from paper_2402_11857_b200 import liec

    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    lay = w["layout"]
    N, d = w["N"], lay.dim
    comp = {"sign": liec.COMP_SCALED_SIGN, "topk": liec.COMP_TOPK, "randk": liec.COMP_RANDK}[w["comp"]]
    gdt = liec.BF16 if w["gdt"] == "bf16" else liec.F32
    X = torch.zeros(N, d, device=dev)
    e = torch.zeros(d, device=dev)
    ctx = liec.Context(X, e, lay.seg_offsets, comp, comp, w["k"], gdt)
    G = make_gradients(w["dist"], w["scale"], N, d, step=0, base_seed=1000 + rank, device=dev)
    if w["comp"] == "randk":   # the subsets are inputs: drawn once on the host, resident like the gradients
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

    def one_step(events=None):
        if events is None:
            ctx.liec_step(G, w["lr"])
            return
        events[0].record()
        ctx.liec_uplink_compress(G); events[1].record()
        ctx.liec_server_aggregate(); events[2].record()
        ctx.liec_downlink_compress(); events[3].record()
        ctx.liec_worker_update(G, w["lr"]); events[4].record()

    sampler = ClockSampler(local_rank)
    sampler.start()          # nvidia-smi needs a moment to start: launch it before the warm-up
    for _ in range(args.warmup):
        one_step()
    torch.cuda.synchronize()
    barrier()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(args.steps)]
    launches0 = ctx.liec_launch_count()
    torch.cuda.synchronize()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.mark_begin()
    start.record()
    for s in range(args.steps):
        one_step(evs[s])
    stop.record()
    torch.cuda.synchronize()
    sampler.mark_end()
    total_ms = start.elapsed_time(stop)
    launches = ctx.liec_launch_count() - launches0
    barrier()
    clocks = sampler.stop()
    assert ctx.liec_device_status() == 0, "device status word is non-zero"

    stage_ms = [statistics.mean(evs[s][q].elapsed_time(evs[s][q + 1]) for s in range(args.steps)) for q in range(4)]

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
        with torch.cuda.graph(graph):
            ctx.liec_step(G, w["lr"])
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        for _ in range(args.steps):
            graph.replay()
        g1.record()
        torch.cuda.synchronize()
        graph_ms = g0.elapsed_time(g1) / args.steps
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
        e2e_steps = max(1, min(args.steps, args.e2e_steps))
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

    ms_step = total_ms / args.steps
    if world > 1:
        vals = max_over_ranks([ms_step, e2e["ms_per_step"] if e2e else 0.0] + stage_ms, device=dev)
        ms_step, e2e_max, stage_ms = vals[0], vals[1], vals[2:]
        if e2e:
            e2e["ms_per_step"] = e2e_max
    return dict(ms_step=ms_step, stage_ms=dict(zip(stage_names, stage_ms)), launches=launches, clocks=clocks, e2e=e2e,
                average_ms=average_ms, graph_ms=graph_ms)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c4")
    ap.add_argument("--no-e2e", action="store_true")
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
    w = resolve_workload(args.workload)
    lay = w["layout"]
    N, d = w["N"], lay.dim
    config = {"workload": f"{w['name']}: N={N} workers, d={d} in {lay.num_segments} segments ({lay.name}), "
                          f"{w['comp']} both ways, gradients {w['dist']} {w['gdt']}",
              "num_workers": N, "dim": d, "segments": lay.num_segments, "compressor": w["comp"],
              "l2_policy": "inputs larger than L2 (gradients and parameters are streamed from HBM every step)",
              "parallelism": "replicas only" if args.gpus > 1 else "single GPU"}

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
    if rank != 0:
        torch.distributed.destroy_process_group()
        return

    units = N * d * world
    value = whole_job_throughput(N * d, world, r["ms_step"])
    bmin = min_bytes_per_step(w)
    step_gbs = bmin / (r["ms_step"] * 1e-3) / 1e9
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        peak, peak_src = json.load(open(peaks_path))["hbm_gbs"], "measured copy bandwidth (MEASURED_PEAKS.json)"
    else:
        peak, peak_src = 6650.0, "fallback 6.65 TB/s"
    upd_ms = r["stage_ms"]["worker_update"]
    upd_gbs = update_kernel_bytes(w) / (upd_ms * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": r["ms_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic", "config": config,
        "hbm_gbs": step_gbs, "pct_of_8tbs_nominal": 100 * step_gbs / NOMINAL_HBM_GBS,
        "pct_of_measured_copy_peak": 100 * step_gbs / peak, "min_bytes_per_step": bmin,
        "stage_ms": r["stage_ms"],
        "roofline": {"bound": "hbm", "kernel": "worker_update_kernel", "achieved": upd_gbs, "peak": peak,
                     "unit": "GB/s", "frac": upd_gbs / peak,
                     "traffic": UPDATE_TRAFFIC_BYTES.get(w["name"]), "peak_source": peak_src,
                     "algorithmic_bytes_per_launch": update_kernel_bytes(w), "launch_ms": upd_ms},
        "gpu_launches": r["launches"], "clocks": r["clocks"],
        "average_step": {"ms": r["average_ms"],
                         "gbs": (N * d * ((2 if w["gdt"] == "bf16" else 4) + 8) + 8 * d) / (r["average_ms"] * 1e-3) / 1e9,
                         "note": "model-averaging iteration of Algorithm 1, timed separately (5 runs)"},
    }
    if r["graph_ms"] is not None:
        line["cuda_graph"] = {"ms_per_step": r["graph_ms"], "value": units / (r["graph_ms"] * 1e-3), "unit": UNIT}
    if r["e2e"]:
        line["e2e"] = {"value": units / (r["e2e"]["ms_per_step"] * 1e-3), "unit": UNIT,
                       "h2d_bytes_per_step": r["e2e"]["h2d"], "d2h_bytes_per_step": r["e2e"]["d2h"],
                       "ms_per_step": r["e2e"]["ms_per_step"], "steps": r["e2e"]["steps"]}
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = time_oracle(w, 1, 0)
    print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
