#!/usr/bin/env python
"""Benchmark of the CSP scoring-and-compaction pass.

A step is one pass of the whole path (score -> select -> compact, i.e. csp_prune_layer) over
every layer of one synthetic multimodal KV cache.  The reported metric is KV tokens pruned per
second per layer: (sum of sequence lengths) / (time of one layer's prune).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config I] [--impl reference]

With N > 1 (launched under torch.distributed.run) every rank prunes its own replica of the
workload; there is no exchange step on this path, so the job throughput is the sum.
"""
from __future__ import annotations

import argparse
import concurrent.futures
import json
import os
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import csp_synth as synth  # noqa: E402

METRIC = "kv_tokens_pruned_per_sec_per_layer"
UNIT = "tokens/s"


# ------------------------------------------------------------------------------------ helpers

def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.01):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons = [], set()
        self.sm_max = None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.sm_max = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.nv = None

    def _sample(self):
        nv = self.nv
        self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
        try:
            r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
        except Exception:
            r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
        names = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
                 0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown"}
        for bit, name in names.items():
            if r & bit:
                self.reasons.add(name)

    def run(self):
        if not self.ok:
            return
        while not self._stop_evt.is_set():
            try:
                self._sample()
            except Exception:
                break
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.sm_max, "reasons": []}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.sm_max,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def max_over_ranks(ms: float, dist, device) -> float:
    """Slowest rank's time: the job is done when every replica is."""
    if dist is None:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(world: int, tokens_per_layer: int, n_layers: int, ms_step: float) -> float:
    """Whole-job metric: every rank prunes its own replica (no exchange step), so the units add up."""
    return world * tokens_per_layer * n_layers / (ms_step * 1e-3)


# DRAM bytes (read + write) per launch of each kernel on configs[1], one layer per launch, from the ncu
# captures summarised under profiles/ (dram__bytes_read.sum + dram__bytes_write.sum).  Scales with the
# number of layers a launch covers.  None for workloads that were not captured.
NCU_DRAM_BYTES_PER_LAYER = {
    ("all_layers_one_call", 1): {"score": 1.1145e9 / 32, "select": 33.48e6 / 32, "compact": 1.0256e9 / 32},
    ("one_layer_per_call", 1): {"score": 33.88e6, "select": 1.08e6, "compact": 16.97e6},
    ("one_layer_per_call", 3): {"score": 95.1e6},
}


# the same for one launch of the decode kernel (bench.py --decode), all layers in one call
NCU_DECODE_DRAM_BYTES = {1: 543.55e6}


def algorithmic_bytes(cfg, n_out_total: int):
    """Per-layer algorithmic bytes of each kernel (every tensor touched exactly once)."""
    es = 2 if cfg.dtype == torch.bfloat16 else 4
    d, Hkv, Hq, W = cfg.head_dim, cfg.n_kv_heads, cfg.n_q_heads, cfg.window
    sum_l = int(cfg.seq_lens.sum())
    sum_n = int((cfg.seq_lens - cfg.recent).clip(min=0).sum())
    score = sum_l * Hkv * d * es + cfg.batch * Hq * W * d * es + sum_l + 2 * 4 * sum_n * Hkv
    select = 2 * 4 * sum_n * Hkv + sum_n * Hkv + 4 * n_out_total
    compact = 4 * n_out_total + 2 * 2 * n_out_total * d * es + 2 * n_out_total
    return {"score": score, "select": select, "compact": compact, "total": score + select + compact}


class LayerBuffers:
    """Inputs and outputs of one library call: one layer, or `n_fold` layers stacked on the batch axis."""

    def __init__(self, csp, cfg, p, layer, device, n_fold=1):
        if n_fold == 1:
            self.q, self.k, self.v = synth.make_layer(cfg, layer, device)
        else:
            parts = [synth.make_layer(cfg, layer + i, device) for i in range(n_fold)]
            self.q, self.k, self.v = (torch.cat([x[j] for x in parts], 0) for j in range(3))
            del parts
        B, H, cap, d = cfg.batch * n_fold, cfg.n_kv_heads, p.out_capacity, cfg.head_dim
        self.k_out = torch.empty((B, H, cap, d), dtype=cfg.dtype, device=device)
        self.v_out = torch.empty((B, H, cap, d), dtype=cfg.dtype, device=device)
        self.mod_out = torch.empty((B, H, cap), dtype=torch.uint8, device=device)
        self.n_out = torch.zeros((B, H), dtype=torch.int32, device=device)
        self.ss = torch.empty((B, H, cfg.max_len), dtype=torch.float32, device=device)
        self.sc = torch.empty((B, H, cfg.max_len), dtype=torch.float32, device=device)
        self.idx = torch.empty((B, H, cap), dtype=torch.int32, device=device)


# ------------------------------------------------------------------------------------ reference arm

def run_reference(args, rank, world):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload."""
    if rank != 0:
        return
    from oracle import csp_oracle as orc
    orc.build()
    cfg = synth.config(args.config)
    G = cfg.group
    n_units = min(args.ref_units, cfg.n_kv_heads)
    b = int(np.argmax(cfg.seq_lens)) if cfg.batch > 1 else 0
    L = int(cfg.seq_lens[b])
    q, k, v = synth.make_layer(cfg, 0, "cpu")
    qs = q[b:b + 1, :n_units * G].contiguous()
    ks, vs = k[b:b + 1, :n_units, :L].contiguous(), v[b:b + 1, :n_units, :L].contiguous()
    mod = cfg.modality()[b:b + 1, :L]
    op = orc.Params(1, n_units * G, n_units, cfg.head_dim, cfg.window, cfg.recent, L, cfg.out_capacity(),
                    dtype=orc.F32 if cfg.dtype == torch.float32 else orc.BF16)
    tb = None if cfg.total_budget is None else cfg.total_budget[b:b + 1]

    def step():
        orc.prune_layer(op, qs, ks, vs, mod, np.array([L], np.int32), cfg.budgets[b:b + 1], tb)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / max(args.steps, 1)
    # one sample = n_units of the H_kv heads of one sequence of one layer
    value = L * n_units / cfg.n_kv_heads / dt
    sample = f"{n_units} of {cfg.n_kv_heads} KV heads of sequence {b} (L={L}) of one layer per step"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"configs[{args.config}] {cfg.name}", "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------ CUDA arm

def kernels_per_call(p) -> int:
    """Kernels one csp_prune_layer call launches: score, select, compact, and, for a bf16 cache with more
    (sequence, head) units than SMs and several sequences, the kernel that orders them by length."""
    units, tiles = p.batch * p.n_kv_heads, (p.max_len + 127) // 128
    ordered = p.dtype == 1 and 2 <= p.batch <= 4096 and (units > 148 or units * min(tiles, 8) > 120)
    return 4 if ordered else 3


def run_decode(args, rank, world, local_rank):
    """`--decode`: the step after the pruning pass (Section 3.3): one new query per head attends, with the
    n-softmax normaliser, to the compacted caches that csp_prune_layer left.  All layers of the workload in one
    csp_decode_attn call (layer axis folded into the batch axis).  Prints its own JSON line; not the default."""
    from paper_2412_04652_b200 import binding as csp
    csp.lib()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    cfg = synth.config(args.config, budget_pct=args.budget_pct) if args.config == 4 else synth.config(args.config)
    n_layers, cap = cfg.n_layers, cfg.out_capacity()
    import copy
    pf = csp.Params(cfg.batch * n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.window, cfg.recent,
                    cfg.max_len, cap)
    lb = LayerBuffers(csp, cfg, pf, 0, dev, n_fold=n_layers)
    mod = torch.from_numpy(cfg.modality()).to(dev).repeat(n_layers, 1)
    lens = torch.from_numpy(cfg.seq_lens).to(dev).repeat(n_layers)
    bud = torch.from_numpy(cfg.budgets).to(dev).repeat(n_layers, 1)
    tot = None if cfg.total_budget is None else torch.from_numpy(cfg.total_budget).to(dev).repeat(n_layers)
    ws = csp.new_workspace(pf, dev)
    csp.prune_layer(pf, lb.q, lb.k, lb.v, mod, lens, bud, lb.k_out, lb.v_out, lb.mod_out, lb.n_out, ws, total_budget=tot)
    status = csp.device_status(ws)
    k_c, v_c, n_rows = lb.k_out, lb.v_out, lb.n_out
    del lb.k, lb.v
    pd = csp.Params(pf.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, 1, 0, cap, cap)
    g = torch.Generator(device=dev).manual_seed(1234)
    q1 = torch.randn(pf.batch, cfg.n_q_heads, cfg.head_dim, generator=g, device=dev).to(torch.bfloat16)
    out = torch.zeros(pf.batch, cfg.n_q_heads, cfg.head_dim, device=dev)
    wd = csp.new_decode_workspace(pd, dev)
    rows_total = int(n_rows.clamp(min=0).sum().item())
    stream = torch.cuda.Stream(dev)
    with torch.cuda.stream(stream):
        for _ in range(max(args.warmup, 3)):
            csp.decode_attn(pd, q1, k_c, v_c, n_rows, out, wd)
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            csp.decode_attn(pd, q1, k_c, v_c, n_rows, out, wd)
        graph.replay()
        stream.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        sampler = ClockSampler(local_rank)
        sampler.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.steps):
            graph.replay()
        e1.record(stream)
        stream.synchronize()
        clocks = sampler.stop()
    ms_step = max_over_ranks(e0.elapsed_time(e1), dist, dev) / args.steps
    status |= csp.device_status(wd)
    es = 2
    ab = rows_total * 2 * cfg.head_dim * es + q1.numel() * es + out.numel() * 4 + n_rows.numel() * 4
    peak, peak_kind = measured_peaks()
    achieved = ab / (ms_step * 1e-3) / 1e9
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import csp_oracle as orc
        orc.build()
        po = orc.Params(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, 1, 0, cap, cap, dtype=orc.BF16)
        B0 = cfg.batch
        qs, ks, vs, rs = q1[:B0].cpu(), k_c[:B0].cpu(), v_c[:B0].cpu(), n_rows[:B0].clamp(min=0).cpu().numpy()
        t0 = time.perf_counter()
        reps = 0
        while reps < 1 or (time.perf_counter() - t0 < 10.0 and reps < 5000):
            orc.decode_attn(po, qs, ks, vs, rs)
            reps += 1
        dt = (time.perf_counter() - t0) / reps
        cpu_baseline = {"value": float(rs.sum()) / dt, "unit": "kv_rows/s", "cores": orc.num_threads(),
                        "kind": "oracle", "sample": f"all heads of one layer, {reps} repetitions, {dt:.4f} s each"}
    if rank == 0:
        line = {"metric": "decode_attn_kv_rows_per_sec", "value": world * rows_total / (ms_step * 1e-3), "unit": "kv_rows/s",
                "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_step,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": f"decode over the pruned caches of configs[{args.config}] {cfg.name}",
                           "layers": n_layers, "kv_heads": cfg.n_kv_heads, "q_heads": cfg.n_q_heads,
                           "head_dim": cfg.head_dim, "row_capacity": cap, "kv_rows_per_step": rows_total,
                           "launch": "one csp_decode_attn call for all layers (layer axis folded into the batch axis)",
                           "l2": "inputs larger than L2" if ab > 2 * 126e6 else "inputs smaller than L2",
                           "replicas": "one independent replica per GPU, no collective"},
                "clocks": clocks, "e2e": None, "gpu_launches": args.steps * 2,
                "roofline": {"bound": "hbm", "kernel": "decode_attn", "achieved": achieved, "peak": peak, "unit": "GB/s",
                             "frac": achieved / peak, "traffic": NCU_DECODE_DRAM_BYTES.get(args.config),
                             "peak_kind": f"of {peak_kind}",
                             "algorithmic_bytes_per_launch": ab, "us_per_launch": ms_step * 1e3},
                "cpu_baseline": cpu_baseline, "device_status": status}
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--config", type=int, default=1)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--ref-units", type=int, default=8, help="KV heads per reference-arm step")
    ap.add_argument("--layers", type=int, default=0, help="distinct layer buffers (0 = all layers)")
    ap.add_argument("--launch", default="graph", choices=["graph", "stream"])
    ap.add_argument("--streams", type=int, default=32, help="concurrent layer chains inside the step graph")
    ap.add_argument("--per-layer-calls", dest="fold_layers", action="store_false",
                    help="one csp_prune_layer call per layer (concurrent chains in a CUDA graph) instead of the "
                         "default: one call for all layers, the layer axis of a [layers*B, H, L, d] cache "
                         "passed as the batch axis")
    ap.set_defaults(fold_layers=True)
    ap.add_argument("--e2e-lanes", type=int, default=2, help="host threads (each with a stream and a staging area) of the end-to-end measurement")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-baseline-units", type=int, default=1 << 30)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--decode", action="store_true",
                    help="time the step after the pruning pass instead: n-softmax decode attention over the pruned caches")
    ap.add_argument("--budget-pct", type=int, default=20, help="budget of configs[4]")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if args.steps == 300:
            args.steps, args.warmup = 5, 1
        run_reference(args, rank, world)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    if args.decode:
        run_decode(args, rank, world, local_rank)
        return
    from paper_2412_04652_b200 import binding as csp
    csp.lib()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    cfg = synth.config(args.config, budget_pct=args.budget_pct) if args.config == 4 else synth.config(args.config)
    n_layers = cfg.n_layers
    n_buf = n_layers if args.layers <= 0 else min(args.layers, n_layers)
    cap = cfg.out_capacity()
    p = csp.Params(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.window, cfg.recent, cfg.max_len,
                   cap, dtype=csp.F32 if cfg.dtype == torch.float32 else csp.BF16)
    mod = torch.from_numpy(cfg.modality()).to(dev)
    lens = torch.from_numpy(cfg.seq_lens).to(dev)
    bud = torch.from_numpy(cfg.budgets).to(dev)
    tot = None if cfg.total_budget is None else torch.from_numpy(cfg.total_budget).to(dev)
    sum_l = int(cfg.seq_lens.sum())

    # One entry per library call of a step: (params, buffers, labels, lengths, budgets, totals, layers covered)
    kv_bytes = 2 * n_layers * cfg.batch * cfg.n_kv_heads * cfg.max_len * cfg.head_dim * (2 if cfg.dtype == torch.bfloat16 else 4)
    if args.fold_layers and (args.layers > 0 or kv_bytes > 40e9):
        args.fold_layers = False                     # a subset of layer buffers only makes sense per layer
        if args.layers <= 0 and kv_bytes > 40e9:
            n_buf = 4                                 # cycle four distinct layers when the cache is huge
    if args.fold_layers:
        import copy
        pf = copy.copy(p)
        pf.batch = cfg.batch * n_layers
        calls = [(pf, LayerBuffers(csp, cfg, pf, 0, dev, n_fold=n_layers), mod.repeat(n_layers, 1),
                  lens.repeat(n_layers), bud.repeat(n_layers, 1), None if tot is None else tot.repeat(n_layers),
                  n_layers)]
        n_buf, n_chains = n_layers, 1
    else:
        layers = [LayerBuffers(csp, cfg, p, i, dev) for i in range(n_buf)]
        calls = [(p, layers[i % n_buf], mod, lens, bud, tot, 1) for i in range(n_layers)]
        n_chains = max(1, min(args.streams, n_layers)) if args.launch == "graph" else 1
    wss = [csp.new_workspace(calls[0][0], dev) for _ in range(n_chains)]   # one scratch area per concurrent chain
    first_lb = calls[0][1]

    def prune(call, w):
        cp, lb, cmod, clens, cbud, ctot, _ = call
        csp.prune_layer(cp, lb.q, lb.k, lb.v, cmod, clens, cbud, lb.k_out, lb.v_out, lb.mod_out, lb.n_out, w,
                        total_budget=ctot)

    def step():
        for call in calls:
            prune(call, wss[0])

    side = [torch.cuda.Stream(dev) for _ in range(n_chains - 1)]

    def step_chains(main_stream):
        # layers are independent: chain c prunes calls c, c + n_chains, ... on its own stream
        fork = torch.cuda.Event()
        fork.record(main_stream)
        for c in range(n_chains):
            st = main_stream if c == 0 else side[c - 1]
            if c:
                st.wait_event(fork)
            with torch.cuda.stream(st):
                for i in range(c, len(calls), n_chains):
                    prune(calls[i], wss[c])
            if c:
                join = torch.cuda.Event()
                join.record(st)
                main_stream.wait_event(join)

    stream = torch.cuda.Stream(dev)
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        for _ in range(max(args.warmup, 3)):
            step()
        stream.synchronize()
        graph = None
        if args.launch == "graph":
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                step_chains(stream)
            for _ in range(3):
                graph.replay()
            stream.synchronize()
        run_step = graph.replay if graph is not None else step

        status = 0
        for w in wss:
            status |= csp.device_status(w)
        n_out_total = int(first_lb.n_out.clamp(min=0).sum().item()) // calls[0][6]      # kept rows per layer

        # ---- timed region: K steps, device resident ----
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        sampler = ClockSampler(local_rank)
        sampler.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.steps):
            run_step()
        e1.record(stream)
        stream.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        clocks = sampler.stop()
        ms_total = max_over_ranks(e0.elapsed_time(e1), dist, dev)
        ms_step = ms_total / args.steps
        value = job_throughput(world, sum_l, n_layers, ms_step)

        # ---- per-kernel durations, live: one CUDA graph per kernel holding that kernel's launch for
        # every call of a step, replayed back to back and timed with events on the launching stream ----
        ws = wss[0]

        def score_all():
            for cp, lb, cmod, clens, cbud, ctot, _ in calls:
                csp.score(cp, lb.q, lb.k, cmod, clens, lb.ss, lb.sc, ws)

        def select_all():
            for cp, lb, cmod, clens, cbud, ctot, _ in calls:
                csp.select(cp, lb.ss, lb.sc, cmod, clens, cbud, lb.idx, lb.n_out, ws, total_budget=ctot)

        def compact_all():
            for cp, lb, cmod, clens, cbud, ctot, _ in calls:
                csp.compact(cp, lb.k, lb.v, cmod, lb.idx, lb.n_out, lb.k_out, lb.v_out, lb.mod_out)

        per = {}
        reps = max(3, min(50, args.steps))
        for name, fn in (("score", score_all), ("select", select_all), ("compact", compact_all)):
            fn()
            stream.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                fn()
            g.replay()
            stream.synchronize()
            k0, k1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            k0.record(stream)
            for _ in range(reps):
                g.replay()
            k1.record(stream)
            stream.synchronize()
            per[name] = k0.elapsed_time(k1) / (reps * len(calls))       # ms per launch
        status |= csp.device_status(ws)

    peak, peak_kind = measured_peaks()
    ab = algorithmic_bytes(cfg, n_out_total)
    layers_per_launch = calls[0][6]
    ab_launch = {k_: v_ * layers_per_launch for k_, v_ in ab.items()}
    dominant = max(per, key=per.get)
    achieved = ab_launch[dominant] / (per[dominant] * 1e-3) / 1e9
    traffic = NCU_DRAM_BYTES_PER_LAYER.get(("all_layers_one_call" if args.fold_layers else "one_layer_per_call",
                                            args.config), {}).get(dominant)
    roofline = {"bound": "hbm", "kernel": dominant, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "traffic": None if traffic is None else traffic * layers_per_launch,
                "peak_kind": f"of {peak_kind}",
                "algorithmic_bytes_per_launch": ab_launch[dominant], "us_per_launch": per[dominant] * 1e3}
    # The scoring kernel takes one exponential per (query head of the group, window row, key): with G >= 3 that
    # is more special-function work per K byte than the SMs can keep up with at the HBM peak, so the bound of
    # that kernel is the ex2 rate (16 per clock and SM at the maximum SM clock), each exponential counted once.
    if dominant == "score":
        sms = torch.cuda.get_device_properties(dev).multi_processor_count
        ex2_peak = 16.0 * sms * clocks["sm_max_mhz"] * 1e6 if clocks.get("sm_max_mhz") else None
        n_exp = float(cfg.group * cfg.window * cfg.n_kv_heads) * float(cfg.seq_lens.sum()) * layers_per_launch
        if ex2_peak and n_exp / ex2_peak > ab_launch["score"] / (peak * 1e9):
            ex2_rate = n_exp / (per["score"] * 1e-3)
            roofline = {"bound": "alu", "kernel": "score", "achieved": ex2_rate / 1e12, "peak": ex2_peak / 1e12,
                        "unit": "T ex2/s", "frac": ex2_rate / ex2_peak, "traffic": roofline["traffic"],
                        "peak_kind": "16 ex2 per clock and SM x SM count x maximum SM clock",
                        "exponentials_per_launch": n_exp, "us_per_launch": per["score"] * 1e3, "hbm": roofline}
    path = {"algorithmic_bytes_per_layer": ab["total"], "us_per_layer": ms_step * 1e3 / n_layers,
            "achieved_gbs": ab["total"] / (ms_step * 1e-3 / n_layers) / 1e9,
            "frac_of_hbm_peak": ab["total"] / (ms_step * 1e-3 / n_layers) / 1e9 / peak,
            "kernel_us_per_launch": {k_: v_ * 1e3 for k_, v_ in per.items()},
            "kernel_gbs": {k_: ab_launch[k_] / (per[k_] * 1e-3) / 1e9 for k_ in per}}

    # ---- end to end through the host-buffer entry point (pinned host memory, copies timed) ----
    e2e = None
    if args.e2e_steps > 0:
        n_host = min(n_buf, 4)
        pin = lambda t: t.cpu().contiguous().pin_memory()
        host = []
        if args.fold_layers:      # the host-buffer entry point is called per layer: slice the folded cache
            B0 = cfg.batch
            fl = calls[0][1]

            class _View:
                pass
            layers = []
            for i in range(n_host):
                lv = _View()
                for name in ("q", "k", "v", "k_out", "v_out", "mod_out", "n_out"):
                    setattr(lv, name, getattr(fl, name)[i * B0:(i + 1) * B0])
                layers.append(lv)
        for i in range(n_host):
            lb = layers[i]
            host.append(dict(q=pin(lb.q), k=pin(lb.k), v=pin(lb.v), k_out=pin(lb.k_out), v_out=pin(lb.v_out),
                             mod_out=pin(lb.mod_out), n_out=pin(lb.n_out)))
        h_mod, h_lens, h_bud = pin(mod), pin(lens), pin(bud)
        h_tot = None if tot is None else pin(tot)
        # Two host threads, each with its own stream and staging area, take alternate layers: the call is
        # synchronous, so this is what lets one layer's device-to-host copy run beside the next one's
        # host-to-device copy (PCIe is full duplex) and beside its kernels.
        n_lanes = max(1, args.e2e_lanes)
        stagings = [torch.empty(csp.host_staging_bytes(p), dtype=torch.uint8, device=dev) for _ in range(n_lanes)]
        lane_streams = [torch.cuda.Stream(device=dev) for _ in range(n_lanes)]

        def lane_work(lane):
            torch.cuda.set_device(dev)
            with torch.cuda.stream(lane_streams[lane]):
                for i in range(lane, n_layers, n_lanes):
                    hb = host[i % n_host]
                    csp.prune_layer_host(p, hb["q"], hb["k"], hb["v"], h_mod, h_lens, h_bud, hb["k_out"],
                                         hb["v_out"], hb["mod_out"], hb["n_out"], stagings[lane], total_budget=h_tot)

        pool = concurrent.futures.ThreadPoolExecutor(max_workers=n_lanes)

        def host_step():
            for f in [pool.submit(lane_work, lane) for lane in range(n_lanes)]:
                f.result()                      # every call has synchronised its stream before returning

        with torch.cuda.stream(stream):
            host_step()
            if dist is not None:
                dist.barrier()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(args.e2e_steps):
                host_step()
            e1.record(stream)                   # all lanes are idle again: the interval covers every copy and kernel
            stream.synchronize()
            ms_e2e = e0.elapsed_time(e1) / args.e2e_steps
        pool.shutdown()
        ms_e2e = max_over_ranks(ms_e2e, dist, dev)
        hb = host[0]
        h2d = n_layers * sum(hb[x].numel() * hb[x].element_size() for x in ("q", "k", "v")) + \
            n_layers * (h_mod.numel() + 4 * h_lens.numel() + 4 * h_bud.numel())
        d2h = n_layers * sum(hb[x].numel() * hb[x].element_size() for x in ("k_out", "v_out", "mod_out", "n_out"))
        e2e = {"value": job_throughput(world, sum_l, n_layers, ms_e2e), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e, "api": "csp_prune_layer_host",
               "host_threads": n_lanes}

    # ---- CPU baseline: the oracle on a bounded sample, rank 0 at N=1 only ----
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import csp_oracle as orc
        orc.build()
        G = cfg.group
        b = int(np.argmax(cfg.seq_lens)) if cfg.batch > 1 else 0
        L = int(cfg.seq_lens[b])
        n_units = min(args.cpu_baseline_units, cfg.n_kv_heads)
        lb = first_lb
        qs = lb.q[b:b + 1, :n_units * G].cpu().contiguous()
        ks, vs = lb.k[b:b + 1, :n_units, :L].cpu().contiguous(), lb.v[b:b + 1, :n_units, :L].cpu().contiguous()
        op = orc.Params(1, n_units * G, n_units, cfg.head_dim, cfg.window, cfg.recent, L, cap,
                        dtype=orc.F32 if cfg.dtype == torch.float32 else orc.BF16)
        t0 = time.perf_counter()
        reps_cpu = 0
        while reps_cpu < 1 or (time.perf_counter() - t0 < 12.0 and reps_cpu < 5000):
            orc.prune_layer(op, qs, ks, vs, cfg.modality()[b:b + 1, :L], np.array([L], np.int32),
                            cfg.budgets[b:b + 1], None if cfg.total_budget is None else cfg.total_budget[b:b + 1])
            reps_cpu += 1
        dt = (time.perf_counter() - t0) / reps_cpu
        cpu_baseline = {"value": L * n_units / cfg.n_kv_heads / dt, "unit": UNIT, "cores": orc.num_threads(),
                        "kind": "oracle",
                        "sample": f"{n_units} of {cfg.n_kv_heads} KV heads of sequence {b} (L={L}) of layer 0, "
                                  f"{reps_cpu} repetitions, {dt:.3f} s each"}

    if rank == 0:
        launch = ("one csp_prune_layer call for all layers (layer axis folded into the batch axis)" if args.fold_layers
                  else f"cuda graph of one step, {n_chains} concurrent layer chains" if graph is not None
                  else "one stream, one csp_prune_layer call per layer")
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if cfg.dtype == torch.bfloat16 else "f32",
                "data": "synthetic",
                "config": {"workload": f"configs[{args.config}] {cfg.name}", "layers": n_layers,
                           "distinct_layer_buffers": n_buf, "batch": cfg.batch, "kv_heads": cfg.n_kv_heads,
                           "q_heads": cfg.n_q_heads, "head_dim": cfg.head_dim, "sum_seq_len": sum_l,
                           "window": cfg.window, "recent": cfg.recent, "kept_rows_per_layer": n_out_total,
                           "launch": launch,
                           "l2": "inputs larger than L2: every layer has its own K/V buffers"
                                 if n_buf * ab["score"] > 2 * 126e6 else "inputs smaller than L2",
                           "replicas": "one independent replica per GPU, no collective"},
                "clocks": clocks, "e2e": e2e, "gpu_launches": args.steps * sum(kernels_per_call(c[0]) for c in calls),
                "roofline": roofline, "path": path, "cpu_baseline": cpu_baseline, "device_status": status}
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
