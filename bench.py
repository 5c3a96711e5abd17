#!/usr/bin/env python
"""Benchmark of the pdADMM-G iteration: ADMM iterations per second over all layers.

    python bench.py --gpus N --steps K --warmup W [--workload c2] [--impl reference]

One step is one iteration of Algorithm 1 over every layer (p, W, b, z, q, u updates).  With N > 1 the
script runs under torchrun, one process per GPU; every rank runs an independent replica of the
workload (the path has no cross-GPU exchange), the timed region is bracketed by barriers and the
reported time is the maximum over ranks.  Rank 0 prints one JSON line.
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

def oracle_layer_sample(inp, n_threads_hint=None):
    """Times the fp64 oracle, as it stands, on a bounded sample of the workload: after one untimed full
    set-up (augmentation, feasible start), the per-layer updates of one iteration are run for layer 1,
    one middle layer and layer L; the middle layers are identical in shape, so the time of a full
    iteration is t_1 + (L-2) t_mid + t_L.  Returns (seconds per iteration, description, threads)."""
    import oracle.pdadmm_oracle as o
    w = inp.workload
    prm = o.Params(w.rho, w.nu, w.quant_levels)
    A = o.renormalized_adjacency(w.n_nodes, inp.edge_src, inp.edge_dst)
    X = o.augment(inp.features.T.astype(np.float64), A, w.n_blocks)
    s = o.init_state(X, [x.astype(np.float64) for x in inp.init_W], inp.labels, inp.train_mask, prm)
    L = s.L
    mid = L // 2 if L >= 3 else None
    picks = sorted(set([0, L - 1] + ([mid] if mid is not None else [])))
    # make the start non-trivial: perturb z so that gradients are not identically zero
    rng = np.random.default_rng(0)
    for l in picks:
        s.z[l] = s.z[l] + 0.01 * rng.standard_normal(s.z[l].shape)

    def layer_pass(l):
        t0 = time.perf_counter()
        p = s.p[l]
        if l >= 1:
            if prm.quant_levels:
                p = o.update_p_quantized(s.p[l], s.W[l], s.b[l], s.z[l], prm.nu, s.q[l - 1], s.u[l - 1], prm.rho,
                                         s.scale[l], prm.quant_levels)[0]
            else:
                p = o.update_p(s.p[l], s.W[l], s.b[l], s.z[l], prm.nu, s.q[l - 1], s.u[l - 1], prm.rho)[0]
        W, _ = o.update_W(p, s.W[l], s.b[l], s.z[l], prm.nu)
        b = o.update_b(p, W, s.b[l], s.z[l], prm.nu)
        a = W @ p + b[:, None]
        if l < L - 1:
            z = o.update_z_hidden(a, s.q[l], s.z[l])
            q = o.update_q(s.p[l + 1], s.u[l], z, prm.rho, prm.nu)
            o.update_u(s.u[l], s.p[l + 1], q, prm.rho)
        else:
            o.update_z_last(a, s.y, s.mask, prm.nu)
        return time.perf_counter() - t0

    t = {l: layer_pass(l) for l in picks}
    total = t[0] + (t[L - 1] if L > 1 else 0.0) + (max(L - 2, 0) * t[mid] if mid is not None else 0.0)
    try:
        from threadpoolctl import threadpool_info
        threads = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
    except Exception:
        threads = os.cpu_count() or 1
    desc = (f"one oracle iteration of workload {w.name}: layers {[l + 1 for l in picks]} timed, "
            f"the {max(L - 2, 0)} identical middle layers extrapolated from layer {(mid or 0) + 1}")
    return total, desc, threads


# --------------------------------------------------------------------------------------- main

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--simt", action="store_true", help="run the dense products on CUDA cores")
    ap.add_argument("--one-lane", action="store_true", help="queue all layers on one stream (no concurrency across layers)")
    ap.add_argument("--quant-q", action="store_true",
                    help="pdADMM-G-Q workloads: keep q on the level set as well (variant of Sec. Quantization Extension)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3

    from paper_2105_09837_b200 import replicas, synth
    rank, world, local_rank = replicas.env_rank_world()

    w = synth.get(args.workload)
    config = {"workload": f"{w.name}: N={w.n_nodes} {w.graph.upper()} graph, d={w.feat_dim} x {w.n_blocks} hop blocks "
                          f"(n0={w.n0}), {w.n_layers} layers x {w.hidden}, {w.n_classes} classes, "
                          f"{'pdADMM-G' if not w.quant_levels else f'pdADMM-G-Q {w.quant_levels} levels'}"
                          f"{' (p and q quantised)' if args.quant_q else ''}, rho=nu={w.rho}",
              "replicas": args.gpus,
              "l2": "state (about %.1f GB per replica) is far larger than the 126 MB L2" %
                    (5 * 4e-9 * w.n_nodes * w.hidden * w.n_layers)}

    if args.impl == "reference":
        if rank != 0:
            return 0
        inp = synth.make_inputs(w)
        times = []
        desc, threads = "", 1
        for i in range(args.warmup + args.steps):
            t, desc, threads = oracle_layer_sample(inp)
            if i >= args.warmup:
                times.append(t)
            if sum(times) > 240 and len(times) >= 1 and i >= args.warmup:
                break                              # keep the whole run within a few minutes
        sec = sum(times) / len(times)
        value = 1.0 / sec
        line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
                "steps": len(times), "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config,
                "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
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

    inp = synth.make_inputs(w)
    ctx = B.from_inputs(inp, device=device, flags=flags)
    ctx.step(args.warmup)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(device)

    # timed region: exactly K iterations, device time from CUDA events on the library's stream
    launches0 = ctx.launches()
    barrier()
    with ClockSampler(device) as clk:
        t0 = time.perf_counter()
        ctx.step(args.steps)
        ms = ctx.last_step_ms()
        barrier()
        wall = time.perf_counter() - t0
    launches = ctx.launches() - launches0
    ms = replicas.max_over_ranks(ms, dist, f"cuda:{device}")
    value = replicas.job_throughput(world, args.steps, ms)
    obj = ctx.objective()

    # per-kernel device times (second pass with an event pair around every launch)
    ctx.profile(True)
    n_prof = min(args.steps, 5)
    ctx.step(n_prof)
    prof = ctx.profile_read()
    ctx.profile(False)
    pk = peaks()
    kernels = {}
    for name, v in prof.items():
        if v["launches"] == 0:
            continue
        sec = v["ms"] * 1e-3
        kernels[name] = {"ms_per_iter": v["ms"] / n_prof, "launches_per_iter": v["launches"] / n_prof,
                         "gbs": v["bytes"] / sec / 1e9 if sec > 0 else None,
                         "tflops": v["flops"] / sec / 1e12 if sec > 0 else None}
    dom = max(kernels, key=lambda k: kernels[k]["ms_per_iter"])
    d = prof[dom]
    if d["flops"] > 0:
        achieved = d["flops"] / (d["ms"] * 1e-3) / 1e12
        if args.simt:
            roof = {"bound": "alu", "achieved": achieved, "peak": FP32_FMA_PEAK_TFLOPS, "unit": "TFLOP/s",
                    "peak_source": "148 SMs x 128 fp32 lanes x 2 flop x 1.965 GHz"}
        else:
            # the products run as fp16 MMAs with fp32 accumulation: same tensor rate as the measured bf16 GEMM
            roof = {"bound": "tensor", "achieved": achieved, "peak": pk["bf16_tflops_sustained"],
                    "unit": "TFLOP/s", "peak_source": f"{pk['source']} bf16 GEMM, sustained (fp16 MMAs run at the bf16 rate)"}
    else:
        roof = {"bound": "hbm", "achieved": d["bytes"] / (d["ms"] * 1e-3) / 1e9, "peak": pk["hbm_gbs"],
                "unit": "GB/s", "peak_source": f"{pk['source']} copy bandwidth"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    if roof["bound"] == "tensor":
        # every useful product is issued as three fp16 MMAs (hi*hi, hi*lo, lo*hi): the tensor pipe's own load
        roof["frac_issued"] = 3.0 * roof["frac"]
        roof["note"] = "achieved counts useful fp32-equivalent flop; the kernel issues three fp16 MMAs per product"
    roof["kernel"] = dom
    roof["traffic"] = measured_traffic(args.workload, dom)
    ctx.destroy()

    # end to end through the public API from host buffers: init (H2D of graph, features, weights), K iterations,
    # objective and trained weights back to the host
    h2d = (inp.edge_src.nbytes + inp.edge_dst.nbytes + inp.features.nbytes + inp.labels.nbytes + inp.train_mask.nbytes
           + sum(x.nbytes for x in inp.init_W))
    # the host buffers of the large inputs are page-locked, as a caller that cares about the copy would keep them
    def pinned(a):
        return torch.from_numpy(np.ascontiguousarray(a)).pin_memory().numpy()
    inp.features = pinned(inp.features)
    inp.init_W = [pinned(x) for x in inp.init_W]
    barrier()
    t0 = time.perf_counter()
    ctx2 = B.from_inputs(inp, device=device, flags=flags)
    ctx2.step(args.steps)
    out = [ctx2.objective()]
    d2h = 48
    for l in range(1, w.n_layers + 1):
        Wl, bl = ctx2.get_tensor(B.T_W, l), ctx2.get_tensor(B.T_B, l)
        d2h += Wl.nbytes + bl.nbytes
    torch.cuda.synchronize(device)
    e2e_s = time.perf_counter() - t0
    ctx2.destroy()
    e2e_s = replicas.max_over_ranks(e2e_s, dist, f"cuda:{device}")
    e2e = {"value": replicas.job_throughput(world, args.steps, e2e_s * 1e3), "unit": UNIT, "h2d_bytes_per_step": h2d / args.steps,
           "d2h_bytes_per_step": d2h / args.steps,
           "note": "pdadmm_init from host buffers (features and weights page-locked) + K iterations + objective and W,b read back"}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sec, desc, threads = oracle_layer_sample(inp)
        cpu = {"value": 1.0 / sec, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": config,
                "clocks": clk.summary(), "e2e": e2e, "gpu_launches": launches, "roofline": roof,
                "cpu_baseline": cpu, "kernels": kernels, "objective": float(obj[5]), "wall_s": wall}
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
