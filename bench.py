#!/usr/bin/env python
"""Benchmark of the pdADMM-G iteration: ADMM iterations per second over all layers.

    python bench.py --gpus N --steps K --warmup W [--workload c1..c5|all] [--impl reference]

One step is one iteration of Algorithm 1 over every layer (p, W, b, z, q, u updates).  With N > 1 the
script runs under torchrun, one process per GPU; the nodes of the workload are divided among the
ranks (W and b replicated, the sums over nodes all-reduced by NCCL), or with --replicas every rank
runs an independent copy; the timed region is bracketed by barriers and the reported time is the
maximum over ranks.  Rank 0 prints one JSON line: its top-level fields are the headline
workload (c2), and on one GPU `workloads` holds one record for each of the five workloads.
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

import numpy as np

METRIC = "ADMM iterations/sec (all layers)"
UNIT = "iterations/s"
FP32_FMA_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12     # SMs x fp32 lanes x 2 flop x max SM clock


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def measured_traffic(workload: str, kernel_class: str):
    """DRAM bytes per launch of a kernel class from the committed ncu capture of this workload, or None if there
    is no capture or the kernel sources have changed since it was taken."""
    import glob
    import hashlib
    path = os.path.join(ROOT, "profiles", f"{workload}_kernel_traffic.json")
    if not os.path.exists(path):
        return None
    rec = json.load(open(path))
    h = hashlib.sha256()
    for f in sorted(glob.glob(os.path.join(ROOT, "paper_2105_09837_b200", "csrc", "*"))):
        h.update(open(f, "rb").read())
    if h.hexdigest() != rec.get("csrc_sha256"):
        return None
    return rec.get("traffic_bytes_per_launch", {}).get(kernel_class)


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "20",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
            t0 = time.time()
            while not self.rows and time.time() - t0 < 3.0:      # wait until the sampler delivers
                time.sleep(0.01)
            self.first = len(self.rows)
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def __exit__(self, *a):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
            self.thread.join(timeout=5)

    def summary(self):
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                smax.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(smax), "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------------------- oracle timing

def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        return max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
    except Exception:
        return os.cpu_count() or 1


def oracle_whole_iterations(inp, warmup, steps, budget_s):
    """Times whole iterations of the fp64 oracle, as it stands, from the feasible start (untimed set-up:
    adjacency, augmentation, start of Algorithm 1).  `warmup` untimed iterations, then up to `steps` timed ones,
    stopping early once `budget_s` seconds of timed work are spent.  Returns (list of seconds, description)."""
    import oracle.pdadmm_oracle as o
    w = inp.workload
    prm = o.Params(w.rho, w.nu, w.quant_levels)
    A = o.renormalized_adjacency(w.n_nodes, inp.edge_src, inp.edge_dst)
    X = o.augment(inp.features.T.astype(np.float64), A, w.n_blocks)
    s = o.init_state(X, [x.astype(np.float64) for x in inp.init_W], inp.labels, inp.train_mask, prm)
    times = []
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        s = o.iterate(s, prm)
        dt = time.perf_counter() - t0
        if i >= warmup:
            times.append(dt)
            if sum(times) > budget_s:
                break
    desc = (f"{len(times)} whole oracle iterations of workload {w.name} (all {w.n_layers} layers, every update of "
            f"Algorithm 1) after {warmup} untimed ones")
    return times, desc


def oracle_node_sample(inp, n_sample):
    """For workloads whose oracle iteration does not fit the time or the host memory: one whole oracle iteration on
    the sub-problem of the first n_sample nodes (all layers at full width; every per-layer update is linear in the
    node count), scaled by N / n_sample.  The sparse augmentation is done on the full graph and is not timed.
    Returns (seconds per full-size iteration, description)."""
    import oracle.pdadmm_oracle as o
    w = inp.workload
    prm = o.Params(w.rho, w.nu, w.quant_levels)
    A = o.renormalized_adjacency(w.n_nodes, inp.edge_src, inp.edge_dst)
    X = o.augment(inp.features.T.astype(np.float64), A, w.n_blocks)[:, :n_sample]
    s = o.init_state(X, [x.astype(np.float64) for x in inp.init_W], inp.labels[:n_sample], inp.train_mask[:n_sample], prm)
    s = o.iterate(s, prm)                      # untimed: leaves the feasible start, where every gradient is zero
    t0 = time.perf_counter()
    o.iterate(s, prm)
    dt = time.perf_counter() - t0
    desc = (f"one whole oracle iteration of workload {w.name} on its first {n_sample} of {w.n_nodes} nodes "
            f"(all {w.n_layers} layers at full width), time scaled by {w.n_nodes / n_sample:.1f}")
    return dt * w.n_nodes / n_sample, desc


def cpu_baseline_for(inp, budget_s=25.0):
    """The oracle on the host cores for one workload, bounded to about `budget_s` seconds of timed work."""
    w = inp.workload
    flop = 8.0 * w.n_nodes * w.hidden * w.hidden * max(w.n_layers - 2, 0) + 4.0 * w.n_nodes * w.hidden * w.n0
    if flop < 2e12:                                       # whole iterations fit: c1, c2, c3
        times, desc = oracle_whole_iterations(inp, 1, 3, budget_s)
        sec = sum(times) / len(times)
    else:
        n_sample = max(256, int(w.n_nodes * 3e11 / flop))
        sec, desc = oracle_node_sample(inp, n_sample)
    return {"value": 1.0 / sec, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle", "sample": desc}


# --------------------------------------------------------------------------------------- one workload on the device

def describe(w, quant_q=False):
    return (f"{w.name}: N={w.n_nodes} {w.graph.upper()} graph, d={w.feat_dim} x {w.n_blocks} hop blocks "
            f"(n0={w.n0}), {w.n_layers} layers x {w.hidden}, {w.n_classes} classes, "
            f"{'pdADMM-G' if not w.quant_levels else f'pdADMM-G-Q {w.quant_levels} levels'}"
            f"{' (p and q quantised)' if quant_q else ''}, rho=nu={w.rho}")


def run_workload(name, steps, warmup, flags, device, world, dist, simt, with_cpu, with_e2e=True, shard_nodes=False):
    """Times `steps` iterations of one workload (after `warmup`), a per-kernel pass, the end-to-end leg and the
    oracle sample.  Returns the record of that workload."""
    import torch
    from paper_2105_09837_b200 import binding as B
    from paper_2105_09837_b200 import replicas, synth
    w = synth.get(name)
    inp = synth.make_inputs(w)
    pk = peaks()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(device)

    # several GPUs: the nodes are divided among the ranks (every rank keeps p, z, q, u of its nodes and a copy of W, b;
    # the sums over nodes go through NCCL), so the job is ONE problem and more GPUs make it faster (strong scaling);
    # with --replicas every rank runs the whole problem on its own (weak scaling)
    shard, reducer = None, None
    if shard_nodes and world > 1:
        from paper_2105_09837_b200 import sharded
        reducer = sharded.TorchAllReduce(device)
        lo, cnt = sharded.node_range(dist.get_rank(), world, w.n_nodes)
        shard = (lo, cnt, reducer.fn)
    jobs = 1 if shard is not None else world
    ctx = B.from_inputs(inp, device=device, flags=flags, shard=shard)
    ctx.step(warmup)
    launches0 = ctx.launches()
    barrier()
    with ClockSampler(device) as clk:
        ctx.step(steps)
        ms = ctx.last_step_ms()
        barrier()
    launches = ctx.launches() - launches0
    ms = replicas.max_over_ranks(ms, dist, f"cuda:{device}")
    value = replicas.job_throughput(jobs, steps, ms)
    clocks = clk.summary()
    comm = ctx.comm_bytes() if shard is not None else 0
    obj = ctx.objective()
    spmm = None
    if w.n_blocks > 1 and shard is None:
        hop_ms, hop_bytes = ctx.time_augmentation(20)
        spmm = {"ms_per_hop": hop_ms, "gbs": hop_bytes / (hop_ms * 1e-3) / 1e9, "frac_of_hbm_peak": hop_bytes / (hop_ms * 1e-3) / 1e9 / pk["hbm_gbs"],
                "note": "algorithmic bytes nnz(8+4d)+8Nd; the gathered rows are served from L2 where the block fits"}

    # per-kernel device times (second pass with an event pair around every launch, one lane)
    ctx.profile(True)
    n_prof = min(steps, 5)
    ctx.step(n_prof)
    prof = ctx.profile_read()
    ctx.profile(False)
    ctx.destroy()
    # Denominators: the burst figure of the measured bf16 GEMM where the clocks stayed at their maximum, the sustained
    # one where the power cap was active during the timed region (fp16 MMAs run at the bf16 rate)
    capped = "sw_power_cap" in (clocks.get("reasons") or [])
    tensor_peak = pk["bf16_tflops_sustained"] if capped else pk["bf16_tflops"]
    tensor_peak_name = f"{pk['source']} bf16 GEMM, {'sustained (power cap active)' if capped else 'burst (clocks at maximum)'}"
    if simt:
        tensor_peak, tensor_peak_name = FP32_FMA_PEAK_TFLOPS, "148 SMs x 128 fp32 lanes x 2 flop x 1.965 GHz"
    kernels, t_roof = {}, 0.0
    for k, v in prof.items():
        if v["launches"] == 0:
            continue
        sec = v["ms"] * 1e-3
        # roofline time of the class: the larger of its algorithmic flop over the tensor peak and bytes over the copy peak
        roof_s = max(v["flops"] / (tensor_peak * 1e12), v["bytes"] / (pk["hbm_gbs"] * 1e9))
        t_roof += roof_s / n_prof
        kernels[k] = {"ms_per_iter": v["ms"] / n_prof, "launches_per_iter": v["launches"] / n_prof,
                      "gbs": v["bytes"] / sec / 1e9 if sec > 0 else None,
                      "tflops": v["flops"] / sec / 1e12 if sec > 0 else None,
                      "roof_ms_per_iter": roof_s * 1e3 / n_prof, "frac": roof_s / sec if sec > 0 else None}
    dom = max(kernels, key=lambda k: kernels[k]["ms_per_iter"])
    d = prof[dom]
    if d["flops"] > 0:
        achieved = d["flops"] / (d["ms"] * 1e-3) / 1e12
        roof = {"bound": "alu" if simt else "tensor", "achieved": achieved, "peak": tensor_peak, "unit": "TFLOP/s",
                "peak_source": tensor_peak_name}
    else:
        roof = {"bound": "hbm", "achieved": d["bytes"] / (d["ms"] * 1e-3) / 1e9, "peak": pk["hbm_gbs"],
                "unit": "GB/s", "peak_source": f"{pk['source']} copy bandwidth"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    if roof["bound"] == "tensor":
        # every useful product is issued as three fp16 MMAs (hi*hi, hi*lo, lo*hi): the tensor pipe's own load
        roof["frac_issued"] = 3.0 * roof["frac"]
        roof["note"] = "achieved counts useful fp32-equivalent flop; the kernel issues three fp16 MMAs per product"
    roof["kernel"] = dom
    roof["traffic"] = measured_traffic(name, dom)

    rec = {"workload": describe(w, bool(flags & B.FLAG_QUANT_Q)), "value": value, "unit": UNIT, "steps": steps, "warmup": warmup,
           "ms_per_step": ms / steps, "clocks": clocks, "gpu_launches": launches, "roofline": roof,
           "t_roof_ms": t_roof * 1e3, "frac_t_roof": t_roof * 1e3 / (ms / steps),
           "t_roof_note": "sum over kernel classes of max(algorithmic flop / tensor peak, algorithmic bytes / copy peak), "
                          "per iteration; frac_t_roof = t_roof / measured time per iteration",
           "kernels": kernels, "spmm": spmm, "objective": float(obj[5])}
    if shard is not None:
        rec["allreduce_bytes_per_step"] = comm / (warmup + steps)

    if with_e2e:
        # end to end through the public API from host buffers: init (H2D of graph, features, weights), K iterations,
        # objective and trained weights back to the host
        h2d = (inp.edge_src.nbytes + inp.edge_dst.nbytes + inp.features.nbytes + inp.labels.nbytes + inp.train_mask.nbytes
               + sum(x.nbytes for x in inp.init_W))

        def pinned(a):      # page-locked host buffers of the large inputs, as a caller that cares about the copy keeps them
            return torch.from_numpy(np.ascontiguousarray(a)).pin_memory().numpy()
        inp.features = pinned(inp.features)
        inp.init_W = [pinned(x) for x in inp.init_W]
        barrier()
        t0 = time.perf_counter()
        ctx2 = B.from_inputs(inp, device=device, flags=flags, shard=shard)
        ctx2.step(steps)
        ctx2.objective()
        d2h = 48
        for l in range(1, w.n_layers + 1):
            Wl, bl = ctx2.get_tensor(B.T_W, l), ctx2.get_tensor(B.T_B, l)
            d2h += Wl.nbytes + bl.nbytes
        torch.cuda.synchronize(device)
        e2e_s = time.perf_counter() - t0
        ctx2.destroy()
        e2e_s = replicas.max_over_ranks(e2e_s, dist, f"cuda:{device}")
        rec["e2e"] = {"value": replicas.job_throughput(jobs, steps, e2e_s * 1e3), "unit": UNIT,
                      "h2d_bytes_per_step": h2d / steps, "d2h_bytes_per_step": d2h / steps,
                      "note": "pdadmm_init from host buffers (features and weights page-locked) + K iterations + objective "
                              "and W,b read back; the one-off set-up is spread over only K iterations"}
    if with_cpu:
        rec["cpu_baseline"] = cpu_baseline_for(inp)
    return rec


# --------------------------------------------------------------------------------------- main

ALL = ["c1", "c2", "c3", "c4", "c5"]
HEADLINE = "c2"        # the configuration the metric is quoted on that fits one GPU with the oracle affordable beside it
STEP_CAP = {"c4": 10, "c5": 6}      # iterations of the two large workloads (0.13 s and 0.47 s each)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default=None,
                    help="c1..c5: that workload alone; 'all' or nothing: the headline workload in the top-level fields "
                         "and one record per workload under 'workloads' (single GPU)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--simt", action="store_true", help="run the dense products on CUDA cores")
    ap.add_argument("--one-lane", action="store_true", help="queue all layers on one stream (no concurrency across layers)")
    ap.add_argument("--quant-q", action="store_true",
                    help="pdADMM-G-Q workloads: keep q on the level set as well (variant of Sec. Quantization Extension)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--replicas", action="store_true",
                    help="several GPUs: one independent copy of the workload per GPU instead of one problem with its nodes "
                         "divided among the GPUs")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3

    from paper_2105_09837_b200 import replicas, synth
    rank, world, local_rank = replicas.env_rank_world()
    head = args.workload if args.workload in ALL else HEADLINE
    w = synth.get(head)
    sharded_run = args.gpus > 1 and not args.replicas
    config = {"workload": describe(w, args.quant_q),
              "parallelism": (f"nodes divided among {args.gpus} GPUs, W and b replicated, sums over nodes by NCCL all-reduce"
                              if sharded_run else f"{args.gpus} independent replica(s)"),
              "l2": "state (about %.1f GB per replica) is far larger than the 126 MB L2" %
                    (5 * 4e-9 * w.n_nodes * w.hidden * w.n_layers)}

    if args.impl == "reference":
        if rank != 0:
            return 0
        inp = synth.make_inputs(w)
        # whole oracle iterations: W untimed, then up to K timed ones within about four minutes
        times, desc = oracle_whole_iterations(inp, args.warmup, args.steps, 200.0)
        sec = sum(times) / len(times)
        value = 1.0 / sec
        line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
                "steps": len(times), "steps_requested": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
                "config": config,
                "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle", "sample": desc},
                "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
        print(json.dumps(line))
        return 0

    # ---- our arm
    import torch
    from paper_2105_09837_b200 import build as build_mod
    build_mod.build()
    from paper_2105_09837_b200 import binding as B

    dist = None
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    device = replicas.device_for(local_rank, world)
    flags = (B.FLAG_SIMT_GEMM if args.simt else 0) | (B.FLAG_QUANT_Q if args.quant_q else 0)
    flags |= B.FLAG_ONE_LANE if args.one_lane else 0

    with_cpu = rank == 0 and world == 1 and not args.no_cpu_baseline
    t_start = time.perf_counter()
    rec = run_workload(head, min(args.steps, STEP_CAP.get(head, args.steps)), args.warmup, flags, device, world, dist,
                       args.simt, with_cpu, shard_nodes=sharded_run)
    workloads = {head: rec}
    if args.workload in (None, "all") and world == 1:
        # the metric is quoted per workload: the other four, each with its own clocks, roofline, end-to-end leg and oracle sample
        for name in ALL:
            if name == head:
                continue
            try:
                q_flags = flags if synth.get(name).quant_levels else flags & ~B.FLAG_QUANT_Q
                workloads[name] = run_workload(name, min(args.steps, STEP_CAP.get(name, args.steps)), args.warmup, q_flags,
                                               device, world, dist, args.simt, with_cpu)
            except Exception as e:                                  # a workload that fails must not hide the others
                workloads[name] = {"error": f"{type(e).__name__}: {e}"}

    if rank == 0:
        line = {"metric": METRIC, "value": rec["value"], "unit": UNIT, "n_gpus": world, "steps": rec["steps"],
                "warmup": args.warmup, "ms_per_step": rec["ms_per_step"], "higher_is_better": True,
                "scaling": "strong" if sharded_run else "weak",
                "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": config,
                "clocks": rec["clocks"], "e2e": rec.get("e2e"), "gpu_launches": rec["gpu_launches"], "roofline": rec["roofline"],
                "cpu_baseline": rec.get("cpu_baseline"), "t_roof_ms": rec["t_roof_ms"], "frac_t_roof": rec["frac_t_roof"],
                "kernels": rec["kernels"], "objective": rec["objective"],
                "workloads": {k: v for k, v in sorted(workloads.items())},
                "wall_s": time.perf_counter() - t_start}
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
