#!/usr/bin/env python
"""Benchmark of the CriticalKV compression step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one pass of the whole path (window attention, projection norm, two-stage selection, gather) over a
32-layer Llama-3.1-8B-shaped stack: 32 query heads / 8 KV heads, head_dim 128, d_model 4096, n = 32768 cached
entries per head, window 32, pool kernel 7, flattened adaptive budget of 20% of the entries per layer; bf16 inputs,
float32 scores.  Inputs are seeded synthetic tensors (gen/workloads.py).  With N > 1 (torchrun) every rank runs its
own stack (independent layers, no collective on the data path): weak scaling.

Prints one JSON line: whole-job KV entries scored+selected per second with inputs resident in HBM (`value`), the same
through host buffers with the copies inside the timed region (`e2e`), the roofline of the dominant kernel (the
projection-norm contraction, timed with CUDA events inside the timed region), and the CPU oracle timed on a bounded
sample (`cpu_baseline`).  `--impl reference` times the CPU oracle alone.
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

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "kv_entries_scored_selected_per_s"
UNIT = "entries/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def parse_args():
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=5)
    p.add_argument("--warmup", type=int, default=3)
    p.add_argument("--impl", default="ours", choices=["ours", "reference"])
    p.add_argument("--cfg", type=int, default=3, help="workload id in gen.CONFIGS (3 = the headline 32-layer stack)")
    p.add_argument("--layers", type=int, default=0, help="override the number of layers (debugging)")
    p.add_argument("--group-sum", action="store_true",
                   help="measure the grouped-query shortcut of step 2 (CKV_FLAG_WO_GROUP_SUM) instead of the headline path")
    p.add_argument("--l2", action="store_true", help="measure the L2-norm variant of step 2 (CKV_NORM_L2, Gram matrix)")
    p.add_argument("--cta-pairs", action="store_true",
                   help="projection norm with two CTAs per MMA (CKV_FLAG_CTA_PAIR_MMA) instead of the default kernel")
    p.add_argument("--no-cpu-baseline", action="store_true")
    p.add_argument("--no-e2e", action="store_true")
    return p.parse_args()


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            pk = json.load(f)
        return pk, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        rows = [ln for (t, ln) in self.lines if t0 <= t <= t1 + 0.2] or [ln for (_, ln) in self.lines]
        for ln in rows:
            parts = [x.strip() for x in ln.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0]))
                smax = float(parts[1])
            except ValueError:
                continue
            for name, val in zip(names, parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": smax, "reasons": sorted(reasons),
                "samples": len(sm)}


def oracle_sample(wl, layer=0, kv_heads=None):
    """One layer of the workload (all KV heads, or the first `kv_heads` of them with their query heads) through the
    CPU oracle, as it stands.  Returns (entries, seconds, threads)."""
    from gen import make_layer
    from oracle import criticalkv_oracle as oc
    L = make_layer(wl, layer)
    hk = wl.Hkv if kv_heads is None else max(1, min(int(kv_heads), wl.Hkv))
    hq = hk * wl.G
    budget = wl.budget if wl.budget_mode == "uniform" else wl.budget * hk // wl.Hkv
    t0 = time.perf_counter()
    oc.compress_layer(L.Qw[:hq], L.K[:hk], L.V[:hk], L.WO[:hq], kp=wl.kp, budget_mode=wl.budget_mode, budget=budget,
                      alpha=wl.alpha, eps=wl.eps, K_store=L.K_store[:hk], V_store=L.V_store[:hk])
    dt = time.perf_counter() - t0
    return hk * wl.n, dt, len(os.sched_getaffinity(0))


def run_reference(args, wl):
    """The CPU oracle as the reference arm.  Each step is one layer of the workload restricted to as many KV heads
    (with their query heads) as keeps the whole run to a couple of minutes; the first warm-up step sizes it."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    total_steps = args.warmup + args.steps
    entries, dt1, cores = oracle_sample(wl, 0, kv_heads=1)          # probe: seconds per KV head
    budget_s = 150.0
    heads = int(max(1, min(wl.Hkv, budget_s / max(total_steps, 1) / max(dt1, 1e-3))))
    times, done_entries = [], 0
    for s in range(total_steps):
        entries, dt, cores = oracle_sample(wl, layer=s % wl.layers, kv_heads=heads)
        if s >= args.warmup:
            times.append(dt)
            done_entries += entries
    total = sum(times)
    value = done_entries / total
    sample = (f"per step: layer (step mod {wl.layers}), first {heads} of {wl.Hkv} KV heads with their "
              f"{heads * wl.G} query heads, full n={wl.n}; numpy float64")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "note": "CPU oracle on a bounded sample of the workload per step"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    args = parse_args()
    from gen import config, make_layer
    wl = config(args.cfg)
    if args.layers:
        wl = wl.with_(layers=args.layers)
    if args.impl == "reference":
        run_reference(args, wl)
        return

    import torch
    import torch.distributed as dist
    from paper_2502_03805_b200 import binding as B
    from paper_2502_03805_b200 import session_for
    from paper_2502_03805_b200.dist_util import max_over_ranks, rank_layer_ids, whole_job_throughput

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the compression path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    B.load()

    nb = wl.layers
    # every rank owns its own stack: layer seeds are offset by the rank
    t_gen = time.time()
    layers = [make_layer(wl, l) for l in rank_layer_ids(rank, nb)]
    host = {}
    for name in ("Qw_store", "K_store", "V_store", "WO_store"):
        arr = np.stack([getattr(L, name) for L in layers])
        t = torch.from_numpy(arr)
        if wl.dtype == "bf16":
            t = t.view(torch.bfloat16)
        host[name] = t.pin_memory()
    del layers
    Qw, K, V, WO = (host[k].to(dev, non_blocking=True) for k in ("Qw_store", "K_store", "V_store", "WO_store"))
    torch.cuda.synchronize()
    t_gen = time.time() - t_gen

    flags = B.CKV_FLAG_WO_GROUP_SUM if args.group_sum else 0
    if args.cta_pairs:
        flags |= B.CKV_FLAG_CTA_PAIR_MMA
    s = session_for(wl, nb=nb, device=local, want_stage=False, flags=flags, norm=1 if args.l2 else 0)
    stream = torch.cuda.current_stream()
    gemm_ev = []

    def step(record=False):
        # the two halves of criticalkv_score are issued separately so that events can bracket the contraction
        B.criticalkv_score(s.handle, s.desc, Qw, K, None, None, s.attn, None, s.ws, stream=stream)
        if record:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
        B.criticalkv_score(s.handle, s.desc, None, None, V, WO, None, s.vnorm, s.ws, stream=stream)
        if record:
            e1.record(stream)
            gemm_ev.append((e0, e1))
        s.select(stream=stream)
        s.compact(K, V, stream=stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)
    launches0 = s.launches
    barrier()
    t0 = time.time()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    step_ev = [ev0]
    for _ in range(args.steps):
        step(record=True)
        e = torch.cuda.Event(enable_timing=True)
        e.record(stream)
        step_ev.append(e)
    ev1.record(stream)
    barrier()
    t1 = time.time()
    clocks = sampler.stop(t0, t1)
    launches = s.launches - launches0
    assert s.device_status() == 0, "device status word set during the timed region"
    ms_total = ev0.elapsed_time(ev1)
    gemm_ms = [a.elapsed_time(b) for a, b in gemm_ev]
    per_step = sorted(a.elapsed_time(b) for a, b in zip(step_ev[:-1], step_ev[1:]))
    path = s.last_path

    # ---- per-stage device times, taken after the timed region (three more steps with events between the stages) ----
    stage_ms = {"window_attention": [], "projection_norm": [], "select": [], "compact": []}
    for _ in range(3):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(5)]
        ev[0].record(stream)
        B.criticalkv_score(s.handle, s.desc, Qw, K, None, None, s.attn, None, s.ws, stream=stream)
        ev[1].record(stream)
        B.criticalkv_score(s.handle, s.desc, None, None, V, WO, None, s.vnorm, s.ws, stream=stream)
        ev[2].record(stream)
        s.select(stream=stream)
        ev[3].record(stream)
        s.compact(K, V, stream=stream)
        ev[4].record(stream)
        torch.cuda.synchronize()
        for i, k in enumerate(stage_ms):
            stage_ms[k].append(ev[i].elapsed_time(ev[i + 1]))
    stage_ms = {k: sorted(v)[1] for k, v in stage_ms.items()}

    # ---- the same step captured once in a CUDA graph and replayed (no host launches between the nine kernels) ----
    graph_ms = None
    if world == 1:
        side = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            graph.capture_begin()
            B.criticalkv_score(s.handle, s.desc, Qw, K, V, WO, s.attn, s.vnorm, s.ws, stream=side)
            s.select(stream=side)
            s.compact(K, V, stream=side)
            graph.capture_end()
            for _ in range(2):
                graph.replay()
            g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            g0.record(side)
            for _ in range(args.steps):
                graph.replay()
            g1.record(side)
        torch.cuda.synchronize()
        graph_ms = g0.elapsed_time(g1) / args.steps
        assert s.device_status() == 0

    # ---- end to end: host buffers, copies inside the timed region, layer by layer on two streams ----
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(args, wl, host, local, world, flags)

    ms_total = max_over_ranks(ms_total, dev)
    ms_per_step = ms_total / args.steps
    value = whole_job_throughput(nb * wl.Hkv * wl.n, world, ms_per_step * 1e-3)

    if rank == 0:
        peaks, how = load_peaks()
        heads = wl.Hkv if args.group_sum else wl.Hq
        flops = 2.0 * wl.n * wl.dh * wl.dm * heads * nb
        if args.l2:   # Gram matrix + two-part quadratic form
            flops = (2.0 * wl.dh * wl.dh * wl.dm + 2.0 * 2.0 * wl.n * wl.dh * wl.dh) * heads * nb
        gemm_avg = sum(gemm_ms) / len(gemm_ms)
        achieved = flops / (gemm_avg * 1e-3) / 1e12
        peak = float(peaks.get("bf16_tflops_sustained", FALLBACK_PEAKS["bf16_tflops_sustained"]))
        roofline = {"kernel": "projection norm (V W^O row L1 norm), step 2", "bound": "tensor",
                    "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                    "peak_source": f"{how} (sustained bf16, kernel timed inside a long step)",
                    "ms_per_launch": gemm_avg, "flops_per_launch": flops, "traffic": None,
                    "tensor_core_path": bool(path & 2), "cta_pairs": bool(path & 16)}
        if args.cfg == 3 and not args.group_sum and not args.l2 and (path & 2) and not (path & 16):
            # dram__bytes_read.sum + dram__bytes_write.sum of vnorm_umma_kernel<128> from the ncu capture summarised in
            # profiles/vnorm_umma_cfg3.md: 211.66 MB for 2 layers; every layer touches its own V, W_O and output once,
            # so the traffic of a launch is proportional to the layers it processes
            roofline["traffic"] = 211.66e6 / 2 * nb
            roofline["traffic_unit"] = "bytes per launch (ncu, 2-layer capture scaled by layers)"
            roofline["algorithmic_bytes"] = (2.0 * wl.Hkv * wl.n * wl.dh + 2.0 * wl.Hq * wl.dh * wl.dm +
                                             4.0 * wl.Hq * wl.n) * nb
        # the memory-bound stages against the measured copy bandwidth (algorithmic bytes: K once, attn out; the
        # retained rows of K and V read and written once)
        hbm = float(peaks.get("hbm_gbs", FALLBACK_PEAKS["hbm_gbs"]))
        es = 2 if wl.dtype == "bf16" else 4
        attn_bytes = (wl.Hkv * wl.n * wl.dh * es + wl.Hq * wl.w * wl.dh * es + 4.0 * wl.Hq * wl.n) * nb
        compact_bytes = (4.0 * wl.btot * wl.dh * es + 4.0 * wl.btot) * nb
        stages = {k: {"ms": v} for k, v in stage_ms.items()}
        for k, nbytes in (("window_attention", attn_bytes), ("compact", compact_bytes)):
            gbs = nbytes / (stage_ms[k] * 1e-3) / 1e9
            stages[k].update({"bound": "hbm", "achieved_gbs": gbs, "peak_gbs": hbm, "frac": gbs / hbm})
        cpu = None
        if not args.no_cpu_baseline:
            entries, dt, cores = oracle_sample(wl, 0)
            cpu = {"value": entries / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
                   "sample": f"layer 0 of {wl.layers} (all heads, full n={wl.n}), {dt:.1f} s; numpy float64"}
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_per_step, "ms_per_step_median": per_step[len(per_step) // 2],
                "ms_per_step_min": per_step[0], "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16" if wl.dtype == "bf16" else "f32", "data": "synthetic",
                "config": {"workload": wl.name, "layers": nb, "Hq": wl.Hq, "Hkv": wl.Hkv, "head_dim": wl.dh,
                           "d_model": wl.dm, "n": wl.n, "window": wl.w, "pool_kernel": wl.kp,
                           "budget": f"{wl.budget_mode} {wl.budget} per layer", "alpha": wl.alpha,
                           "projection": ("summed W_O slice per KV head" if args.group_sum else "per query head") +
                                         (", L2 norm via Gram matrix" if args.l2 else ", L1 norm"),
                           "l2": "inputs of one step (5.4 GB) exceed L2; layers are distinct buffers",
                           "ms_per_32_layer_compression": ms_per_step * 32.0 / nb},
                "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline,
                "stages": stages,
                "graph_replay": None if graph_ms is None else {
                    "ms_per_step": graph_ms, "value": nb * wl.Hkv * wl.n / (graph_ms * 1e-3), "unit": UNIT,
                    "how": "the step captured once in a CUDA graph, replayed back to back after the timed region"},
                "cpu_baseline": cpu, "input_generation_s": round(t_gen, 1)}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_e2e(args, wl, host, local, world, flags=0):
    """Same metric through criticalkv_compress_host: every step's inputs start in pinned host memory and its results
    (idx, offsets, compacted K and V) end there; the library streams the layers through two device staging buffers."""
    import torch
    import torch.distributed as dist
    from paper_2502_03805_b200 import binding as B
    from paper_2502_03805_b200.dist_util import max_over_ranks, whole_job_throughput
    dev = torch.device("cuda", local)
    nb = wl.layers
    tdt = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
    desc = B.make_desc(nb=nb, Hq=wl.Hq, Hkv=wl.Hkv, dh=wl.dh, dm=wl.dm, n=wl.n, w=wl.w, pool_k=wl.kp, dtype=wl.dtype,
                       budget_mode=wl.budget_mode, budget=wl.budget, alpha=wl.alpha, eps=wl.eps, flags=flags)
    handle = B.criticalkv_create(local)
    staging = torch.empty(B.criticalkv_host_staging_bytes(desc), dtype=torch.uint8, device=dev)
    out_host = {"idx": torch.empty((nb, wl.btot), dtype=torch.int32).pin_memory(),
                "offsets": torch.empty((nb, wl.Hkv + 1), dtype=torch.int32).pin_memory(),
                "K_out": torch.empty((nb, wl.btot, wl.dh), dtype=tdt).pin_memory(),
                "V_out": torch.empty((nb, wl.btot, wl.dh), dtype=tdt).pin_memory()}
    h2d = sum(v.numel() * v.element_size() for v in host.values())
    d2h = sum(v.numel() * v.element_size() for v in out_host.values())
    stream = torch.cuda.current_stream()

    def step():
        B.criticalkv_compress_host(handle, desc, host["Qw_store"], host["K_store"], host["V_store"], host["WO_store"],
                                   None, out_host["idx"], out_host["offsets"], out_host["K_out"], out_host["V_out"],
                                   staging, stream=stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(min(args.warmup, 2)):
        step()
    barrier()
    steps = max(1, min(args.steps, 3))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        step()
    e1.record(stream)      # the library ties its copy streams back to this stream before it returns
    barrier()
    dt = max_over_ranks(e0.elapsed_time(e1) * 1e-3, dev)
    assert B.criticalkv_device_status(handle) == 0
    B.criticalkv_destroy(handle)
    value = whole_job_throughput(nb * wl.Hkv * wl.n * steps, world, dt)
    return {"value": value, "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
            "ms_per_step": 1e3 * dt / steps, "steps": steps,
            "how": "criticalkv_compress_host: pinned host Qw, K, V, W_O in; idx, offsets, K_out, V_out back to pinned "
                   "host; layers streamed through two device staging buffers on two streams"}


if __name__ == "__main__":
    main()
