#!/usr/bin/env python
"""Benchmark of the CriticalKV compression step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--cfg C] [--modes uniform,adaptive]

One step = one pass of the whole path (window attention, projection norm, two-stage selection, gather) over a stack of
layers.  Default workload: the 32-layer Llama-3.1-8B-shaped stack (32 query heads / 8 KV heads, head_dim 128, d_model
4096, n = 32768 cached entries per head, window 32, pool kernel 7, flattened adaptive budget of 20% of the entries per
layer; bf16 inputs, float32 scores).  `--cfg 1|2|4` select the other synthetic workloads of gen/workloads.py
(single-layer 4K and 32K shapes, the 64-layer Qwen2.5-32B-shaped stack at n = 131072).  Inputs are seeded synthetic
tensors.  With N > 1 (torchrun) every rank runs its own stack (independent layers, no collective on the data path):
weak scaling; `--shard kv-heads` instead splits ONE stack by KV head over the ranks (strong scaling, one all-gather
per step for adaptive budgets).

Prints one JSON line per budget mode: whole-job KV entries scored+selected per second with inputs resident in HBM
(`value`), the same through host buffers with the copies inside the timed region (`e2e`), the roofline of the dominant
kernel (the projection-norm contraction, timed with CUDA events inside the timed region), every stage's fraction of
its roofline, a check of the timed outputs of one layer against the CPU oracle (`parity`), and the CPU oracle timed on
a bounded sample (`cpu_baseline`).  `--impl reference` times the CPU oracle alone.
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
TARGETS = {"window_attention": 0.60, "projection_norm": 0.50, "select": 0.60, "compact": 0.60}
E2E_HOST_LIMIT = 16 << 30     # bytes of pinned host inputs the end-to-end leg is willing to hold


def parse_args():
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=5)
    p.add_argument("--warmup", type=int, default=3)
    p.add_argument("--impl", default="ours", choices=["ours", "reference"])
    p.add_argument("--cfg", type=int, default=3, help="workload id in gen.CONFIGS (3 = the headline 32-layer stack)")
    p.add_argument("--layers", type=int, default=0, help="override the number of layers")
    p.add_argument("--modes", default="", help="comma-separated budget modes to measure on the same inputs "
                   "(uniform, adaptive); default: the workload's own.  adaptive uses B_total = Hkv * B")
    p.add_argument("--group-sum", action="store_true",
                   help="measure the grouped-query shortcut of step 2 (CKV_FLAG_WO_GROUP_SUM) instead of the headline path")
    p.add_argument("--l2", action="store_true", help="measure the L2-norm variant of step 2 (CKV_NORM_L2, Gram matrix)")
    p.add_argument("--select-multipass", action="store_true",
                   help="steps 3-4 as separate kernels (CKV_FLAG_SELECT_MULTIPASS) instead of the single kernel")
    p.add_argument("--shard", default="", choices=["", "kv-heads"],
                   help="kv-heads: one stack split by KV head over the ranks (strong scaling)")
    p.add_argument("--no-cpu-baseline", action="store_true")
    p.add_argument("--no-e2e", action="store_true")
    p.add_argument("--no-parity", action="store_true")
    return p.parse_args()


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            pk = json.load(f)
        return pk, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def load_traffic(kernel_file):
    """DRAM traffic of the dominant kernel from a tracked ncu record (bytes per layer, and where it came from)."""
    path = os.path.join(ROOT, "profiles", kernel_file)
    if not os.path.exists(path):
        return None
    with open(path) as f:
        rec = json.load(f)
    per_layer = (rec["dram_bytes_read"] + rec["dram_bytes_write"]) / rec["shape"]["layers"]
    return {"bytes_per_layer": per_layer, "shape": rec["shape"], "command": rec["command"]}


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


# ---------------------------------------------------------------------------------------------------------------------
# CPU oracle legs
# ---------------------------------------------------------------------------------------------------------------------
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


def parity_check(wl, L, layer, outs, rows_per_head=4096, norm="l1"):
    """The timed outputs of one layer against the CPU oracle (outside the timed region): the attention row of every
    query head of one KV group, `rows_per_head` sampled projection norms of every query head, the oracle's selection
    rule applied to the GPU's own float32 scores (must reproduce idx / offsets bit for bit), and the gather against a
    NumPy gather at the GPU's indices."""
    from oracle import criticalkv_oracle as oc
    rng = np.random.default_rng(1000 + layer)
    attn, vnorm, idx, off = outs["attn"], outs["vnorm"], outs["idx"], outs["offsets"]
    g = int(rng.integers(wl.Hkv))
    attn_err = 0.0
    for h in range(g * wl.G, (g + 1) * wl.G):
        P = oc.max_pool(oc.window_mean(oc.window_softmax(L.Qw[h], L.K[g], wl.scale)), wl.kp)
        attn_err = max(attn_err, float(np.max(np.abs(attn[h] - P) / np.maximum(np.abs(P), 1e-30 * np.max(P)))))
    rows = np.sort(rng.choice(wl.n, min(rows_per_head, wl.n), replace=False))
    vnorm_err = 0.0
    group_sum = vnorm.shape[0] == wl.Hkv and wl.Hkv != wl.Hq
    if not group_sum:
        for h in range(wl.Hq):
            nu = oc.projection_norm(L.V[h // wl.G][None], L.WO[h][None], rows=rows, norm=norm)[0]
            vnorm_err = max(vnorm_err, float(np.max(np.abs(vnorm[h, rows] - nu) / np.maximum(nu, 1e-30))))
    ref = oc.select(attn, vnorm, G=wl.G, budget_mode=wl.budget_mode, budget=wl.budget, alpha=wl.alpha, eps=wl.eps,
                    group_sum=group_sum)
    tot = int(ref["offsets"][-1])
    select_exact = bool(np.array_equal(off, ref["offsets"]) and np.array_equal(idx[:tot], ref["idx"]))
    gather_exact = True
    for gg in range(wl.Hkv):
        s, e = int(off[gg]), int(off[gg + 1])
        sel = idx[s:e]
        gather_exact &= bool(np.array_equal(outs["K_out"][s:e], L.K_store[gg][sel]) and
                             np.array_equal(outs["V_out"][s:e], L.V_store[gg][sel]))
    ok = attn_err < 2e-3 and vnorm_err < 2e-3 and select_exact and gather_exact
    return {"ok": bool(ok), "layer": layer, "attn_rel_err_max": attn_err, "attn_heads_checked": wl.G,
            "vnorm_rel_err_max": None if group_sum else vnorm_err,
            "vnorm_rows_per_head": None if group_sum else int(rows.size), "score_tolerance": 2e-3,
            "selection_rule_on_gpu_scores_bit_exact": select_exact, "gather_bit_exact": bool(gather_exact),
            "how": "CPU oracle on one layer of the timed launch, after the timed region"}


# ---------------------------------------------------------------------------------------------------------------------
# GPU arm
# ---------------------------------------------------------------------------------------------------------------------
def algorithmic_work(wl, nb, group_sum, l2):
    """Bytes / flops the method itself needs per step (one read of every input, one write of every output)."""
    es = 2 if wl.dtype == "bf16" else 4
    heads = wl.Hkv if group_sum else wl.Hq
    flops2 = 2.0 * wl.n * wl.dh * wl.dm * heads * nb
    if l2:   # Gram matrix + two-part quadratic form
        flops2 = (2.0 * wl.dh * wl.dh * wl.dm + 2.0 * 2.0 * wl.n * wl.dh * wl.dh) * heads * nb
    return {
        "attn_bytes": (wl.Hkv * wl.n * wl.dh * es + wl.Hq * wl.w * wl.dh * es + 4.0 * wl.Hq * wl.n) * nb,
        "attn_flops": 2.0 * wl.n * wl.dh * wl.Hq * wl.w * nb,
        "vnorm_flops": flops2,
        "vnorm_bytes": (wl.Hkv * wl.n * wl.dh * es + wl.Hq * wl.dh * wl.dm * es + 4.0 * heads * wl.n) * nb,
        "select_bytes": (4.0 * wl.Hq * wl.n + 4.0 * heads * wl.n + 4.0 * wl.btot + 4.0 * (wl.Hkv + 1)) * nb,
        "compact_bytes": (4.0 * wl.btot * wl.dh * es + 4.0 * wl.btot) * nb,
    }


def main():
    args = parse_args()
    from gen import config
    wl = config(args.cfg)
    if args.layers:
        wl = wl.with_(layers=args.layers)
    if args.impl == "reference":
        run_reference(args, wl)
        return
    modes = [m for m in args.modes.split(",") if m] or [wl.budget_mode]
    for m in modes:
        if m not in ("uniform", "adaptive"):
            raise SystemExit(f"unknown budget mode {m}")

    import torch
    import torch.distributed as dist
    from paper_2502_03805_b200 import binding as B

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

    inputs = load_inputs(args, wl, rank, world, dev)
    for m in modes:
        if m == wl.budget_mode:
            wl_m = wl
        elif m == "adaptive":
            wl_m = wl.with_(budget_mode="adaptive", budget=wl.budget * wl.Hkv)
        else:
            wl_m = wl.with_(budget_mode="uniform", budget=wl.budget // wl.Hkv)
        run_mode(args, wl_m, inputs, rank, world, local, dev)
    if world > 1:
        dist.destroy_process_group()


def load_inputs(args, wl, rank, world, dev):
    """Generates the stack layer by layer and uploads it; keeps pinned host copies only when the end-to-end leg will
    run, and the oracle's view of one layer for the parity check."""
    import torch
    from gen import make_layer
    from paper_2502_03805_b200.dist_util import rank_layer_ids, shard_kv_heads
    nb = wl.layers
    shard = args.shard == "kv-heads" and world > 1
    g0, g1 = shard_kv_heads(wl.Hkv, world, rank) if shard else (0, wl.Hkv)
    h0, h1 = g0 * wl.G, g1 * wl.G
    tdt = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
    es = 2 if wl.dtype == "bf16" else 4
    shapes = {"Qw_store": (nb, h1 - h0, wl.w, wl.dh), "K_store": (nb, g1 - g0, wl.n, wl.dh),
              "V_store": (nb, g1 - g0, wl.n, wl.dh), "WO_store": (nb, h1 - h0, wl.dh, wl.dm)}
    host_bytes = sum(int(np.prod(s)) * es for s in shapes.values())
    keep_host = not args.no_e2e and not shard and host_bytes <= E2E_HOST_LIMIT
    t_gen = time.time()
    devt = {k: torch.empty(s, dtype=tdt, device=dev) for k, s in shapes.items()}
    host = {k: torch.empty(s, dtype=tdt).pin_memory() for k, s in shapes.items()} if keep_host else None
    # every rank of the replica mode owns its own stack (layer seeds offset by the rank); the sharded mode splits ONE
    # stack, so every rank draws the same layers and keeps its heads
    ids = list(range(nb)) if shard else rank_layer_ids(rank, nb)
    parity_layer = nb // 2
    parity_inputs = None
    for i, l in enumerate(ids):
        L = make_layer(wl, l)
        for name, (lo, hi) in (("Qw_store", (h0, h1)), ("K_store", (g0, g1)), ("V_store", (g0, g1)),
                               ("WO_store", (h0, h1))):
            t = torch.from_numpy(np.ascontiguousarray(getattr(L, name)[lo:hi]))
            if wl.dtype == "bf16":
                t = t.view(torch.bfloat16)
            if host is not None:
                host[name][i].copy_(t)
                devt[name][i].copy_(host[name][i], non_blocking=True)
            else:
                devt[name][i].copy_(t)
        if i == parity_layer and not args.no_parity and not shard and rank == 0:
            parity_inputs = L
        del L
    torch.cuda.synchronize()
    return {"dev": devt, "host": host, "host_bytes": host_bytes, "gen_s": time.time() - t_gen,
            "parity_layer": parity_layer, "parity_inputs": parity_inputs, "shard": shard, "heads": (g0, g1)}


def run_mode(args, wl, inputs, rank, world, local, dev):
    import torch
    import torch.distributed as dist
    from paper_2502_03805_b200 import binding as B
    from paper_2502_03805_b200 import session_for, to_host
    from paper_2502_03805_b200.dist_util import ShardedCompressor, max_over_ranks, whole_job_throughput

    nb = wl.layers
    Qw, K, V, WO = (inputs["dev"][k] for k in ("Qw_store", "K_store", "V_store", "WO_store"))
    flags = B.CKV_FLAG_WO_GROUP_SUM if args.group_sum else 0
    if args.select_multipass:
        flags |= B.CKV_FLAG_SELECT_MULTIPASS
    shard = inputs["shard"]
    if shard:
        sc = ShardedCompressor(nb=nb, Hq=wl.Hq, Hkv=wl.Hkv, dh=wl.dh, dm=wl.dm, n=wl.n, w=wl.w, pool_k=wl.kp,
                               dtype=wl.dtype, budget_mode=wl.budget_mode, budget=wl.budget, world=world, rank=rank,
                               alpha=wl.alpha, eps=wl.eps, device=local, flags=flags, norm=1 if args.l2 else 0)
        s = sc.session
    else:
        s = session_for(wl, nb=nb, device=local, want_stage=False, flags=flags, norm=1 if args.l2 else 0)
    stream = torch.cuda.current_stream()
    gemm_ev = []

    def step(record=False):
        if shard:
            sc.compress(Qw, K, V, WO, stream=stream)
            return
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

    # the outputs of the last timed step, copied before anything else runs on the buffers
    parity = None
    if inputs["parity_inputs"] is not None:
        pl = inputs["parity_layer"]
        outs = {"attn": to_host(s.attn[pl]), "vnorm": to_host(s.vnorm[pl]), "idx": to_host(s.idx[pl]),
                "offsets": to_host(s.offsets[pl]), "K_out": to_host(s.K_out[pl]), "V_out": to_host(s.V_out[pl])}

    # ---- per-stage device times, taken after the timed region (three more steps with events between the stages) ----
    stage_ms = None
    if not shard:
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

    # ---- end to end: host buffers, copies inside the timed region, layer by layer on two streams ----
    e2e = None
    if inputs["host"] is not None:
        e2e = run_e2e(args, wl, inputs["host"], local, world, flags)
    elif not args.no_e2e:
        e2e = {"value": None, "unit": UNIT, "h2d_bytes_per_step": int(inputs["host_bytes"]), "d2h_bytes_per_step": None,
               "how": ("not measured: the sharded mode has no host-staged entry point" if shard else
                       f"not measured: the inputs of one step ({inputs['host_bytes'] / 2**30:.1f} GiB) exceed the "
                       "pinned host memory this benchmark is willing to hold; the figure is bound by the host link "
                       "(about 53 GB/s measured on the default workload), not by the kernels")}

    ms_total = max_over_ranks(ms_total, dev)
    ms_per_step = ms_total / args.steps
    g0, g1 = inputs["heads"]
    units_rank = nb * (g1 - g0) * wl.n
    value = whole_job_throughput(units_rank, world, ms_per_step * 1e-3)

    if rank == 0:
        peaks, how = load_peaks()
        work = algorithmic_work(wl, nb, args.group_sum, args.l2)
        burst = float(peaks.get("bf16_tflops", FALLBACK_PEAKS["bf16_tflops"]))
        sustained = float(peaks.get("bf16_tflops_sustained", FALLBACK_PEAKS["bf16_tflops_sustained"]))
        hbm = float(peaks.get("hbm_gbs", FALLBACK_PEAKS["hbm_gbs"]))
        roofline = None
        if gemm_ms:
            gemm_avg = sum(gemm_ms) / len(gemm_ms)
            achieved = work["vnorm_flops"] / (gemm_avg * 1e-3) / 1e12
            # the fraction is taken against the burst figure (an upper bound); the kernel is timed inside a long step
            # at the power cap, where the library GEMM behind `bf16_tflops_sustained` runs too: that ratio is given
            # next to it
            kernel = ("projection norm (Gram matrix W^O W^O^T and quadratic form per row, L2), step 2" if args.l2 else
                      "projection norm (V W^O row L1 norm), step 2")
            roofline = {"kernel": kernel, "bound": "tensor",
                        "achieved": achieved, "peak": burst, "unit": "TFLOP/s", "frac": achieved / burst,
                        "peak_source": f"{how} (burst bf16 GEMM)", "target": TARGETS["projection_norm"],
                        "peak_sustained": sustained, "frac_of_sustained": achieved / sustained,
                        "ms_per_launch": gemm_avg, "flops_per_launch": work["vnorm_flops"], "traffic": None,
                        "tensor_core_path": bool(path & 2)}
            tr = load_traffic("vnorm_umma_cfg3_traffic.json")
            sh = tr["shape"] if tr else None
            if (tr and not args.group_sum and not args.l2 and (path & 2) and
                    all(sh[k] == v for k, v in (("Hq", wl.Hq), ("Hkv", wl.Hkv), ("head_dim", wl.dh),
                                                ("d_model", wl.dm), ("n", wl.n)))):
                roofline["traffic"] = tr["bytes_per_layer"] * nb
                roofline["traffic_unit"] = ("bytes per launch (ncu capture of " + str(sh["layers"]) +
                                            " layers scaled by layers: " + tr["command"] + ")")
                roofline["algorithmic_bytes"] = work["vnorm_bytes"]
        stages = None
        if stage_ms is not None:
            stages = {k: {"ms": v, "target": TARGETS[k]} for k, v in stage_ms.items()}
            for k, nbytes in (("window_attention", work["attn_bytes"]), ("select", work["select_bytes"]),
                              ("compact", work["compact_bytes"])):
                gbs = nbytes / (stage_ms[k] * 1e-3) / 1e9
                stages[k].update({"bound": "hbm", "algorithmic_bytes": nbytes, "achieved_gbs": gbs, "peak_gbs": hbm,
                                  "frac": gbs / hbm})
            tf = work["vnorm_flops"] / (stage_ms["projection_norm"] * 1e-3) / 1e12
            stages["projection_norm"].update({"bound": "tensor", "achieved_tflops": tf, "peak_tflops": burst,
                                              "frac": tf / burst, "frac_of_sustained": tf / sustained})
            # step 1 also runs its products on the tensor cores (G*w query rows per key): report that side as well
            atf = work["attn_flops"] / (stage_ms["window_attention"] * 1e-3) / 1e12
            stages["window_attention"].update({"flop_per_byte": work["attn_flops"] / work["attn_bytes"],
                                               "achieved_tflops": atf, "tensor_frac": atf / burst})
            stages["select"]["single_kernel"] = bool(path & 32)
        if inputs["parity_inputs"] is not None:
            parity = parity_check(wl, inputs["parity_inputs"], inputs["parity_layer"], outs,
                                  norm="l2" if args.l2 else "l1")
        cpu = None
        if not args.no_cpu_baseline:
            entries, dt, cores = oracle_sample(wl, 0)
            cpu = {"value": entries / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
                   "sample": f"layer 0 of {wl.layers} (all heads, full n={wl.n}), {dt:.1f} s; numpy float64"}
        mhz = clocks.get("sm_mhz")
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_per_step, "ms_per_step_median": per_step[len(per_step) // 2],
                "ms_per_step_min": per_step[0], "higher_is_better": True,
                "scaling": "strong" if shard else "weak",
                "vs_baseline": None, "dtype": "bf16" if wl.dtype == "bf16" else "f32", "data": "synthetic",
                "config": {"workload": wl.name, "layers": nb, "Hq": wl.Hq, "Hkv": wl.Hkv, "head_dim": wl.dh,
                           "d_model": wl.dm, "n": wl.n, "window": wl.w, "pool_kernel": wl.kp,
                           "budget": f"{wl.budget_mode} {wl.budget} per " +
                                     ("KV head" if wl.budget_mode == "uniform" else "layer"),
                           "alpha": wl.alpha,
                           "projection": ("summed W_O slice per KV head" if args.group_sum else "per query head") +
                                         (", L2 norm via Gram matrix" if args.l2 else ", L1 norm"),
                           "partition": ("one stack split by KV head over the ranks, all-gather of the group "
                                         "attention scores for adaptive budgets" if shard else
                                         "one independent stack per rank, no collective"),
                           "l2": f"inputs of one step ({inputs['host_bytes'] / 1e9:.1f} GB) " +
                                 ("exceed L2; layers are distinct buffers" if inputs["host_bytes"] > 256e6 else
                                  "fit in L2: single-layer latency, steps run back to back on warm caches"),
                           "ms_per_full_model_compression": ms_per_step},
                "clocks": clocks,
                "ms_per_step_times_sm_mhz": None if mhz is None else ms_per_step * mhz,
                "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline,
                "stages": stages, "parity": parity,
                "cpu_baseline": cpu, "input_generation_s": round(inputs["gen_s"], 1)}
        print(json.dumps(line), flush=True)
    s.close()


def run_e2e(args, wl, host, local, world, flags=0):
    """Same metric through criticalkv_compress_host: every step's inputs start in pinned host memory and its results
    (idx, offsets, compacted K and V) end there; the library streams the layers through two device staging buffers.
    The figure is bound by the host link, not by the kernels."""
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
            "ms_per_step": 1e3 * dt / steps, "steps": steps, "h2d_gb_per_s": h2d * steps / dt / 1e9,
            "how": "criticalkv_compress_host: pinned host Qw, K, V, W_O in; idx, offsets, K_out, V_out back to pinned "
                   "host; layers streamed through two device staging buffers on two streams; bound by the host link"}


if __name__ == "__main__":
    main()
