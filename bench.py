#!/usr/bin/env python
"""Benchmark of the CSP scoring-and-compaction pass.

A step is one pass of the whole path (score -> select -> compact, i.e. csp_prune_layer) over
every layer of one synthetic multimodal KV cache.  The reported metric is KV tokens pruned per
second per layer: (sum of sequence lengths) / (time of one layer's prune).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config I] [--impl reference]
    python bench.py --all-configs          one JSON line per workload 1-4 (4: every budget of its sweep)
    python bench.py --decode               the step after the pass: n-softmax decode attention
    python bench.py --incremental          a re-prune from the sums that decode steps carried, against the rescan
    python bench.py --diagnostic           per-layer JS divergence between intra- and inter-modality window weights

With N > 1 (launched under torch.distributed.run) every rank prunes its own replica of the
workload; there is no exchange step on this path, so the job throughput is the sum.
"""
from __future__ import annotations

import argparse
import concurrent.futures
import copy
import json
import os
import re
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
REL_TOL, ABS_FRAC = 2e-3, 1e-6          # score tolerance of the parity summary (the one the tests use)


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

    def __init__(self, index: int, period_s: float = 0.005):
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


def ncu_traffic(kernel: str, workload: str, launch: str):
    """DRAM bytes (read + write) of one launch of `kernel`, from the ncu summary committed under profiles/ for
    exactly this workload and launch mode: its line 'dram_bytes_per_launch: <bytes>'.  None when there is no
    such summary (nothing is carried over from another kernel variant, workload or launch mode)."""
    import glob
    for path in sorted(glob.glob(os.path.join(ROOT, "profiles", f"{kernel}*_{workload}_{launch}.md"))):
        m = re.search(r"^dram_bytes_per_launch:\s*([0-9.eE+]+)", open(path).read(), re.M)
        if m:
            return float(m.group(1)), os.path.relpath(path, ROOT)
    return None, None


def algorithmic_bytes(cfg, lens, n_out_total: int, labels_per_head: bool = False):
    """Per-layer algorithmic bytes of each kernel (every tensor touched exactly once).  `lens`: the cache
    lengths this pass prunes."""
    es = 2 if cfg.dtype == torch.bfloat16 else 4
    d, Hkv, Hq, W = cfg.head_dim, cfg.n_kv_heads, cfg.n_q_heads, cfg.window
    sum_l = int(np.asarray(lens, np.int64).sum())
    sum_n = int((np.asarray(lens, np.int64) - cfg.recent).clip(min=0).sum())
    labels = sum_l * (Hkv if labels_per_head else 1)
    score = sum_l * Hkv * d * es + len(lens) * Hq * W * d * es + labels + 2 * 4 * sum_n * Hkv
    select = 2 * 4 * sum_n * Hkv + sum_n * Hkv + 4 * n_out_total
    compact = 4 * n_out_total + 2 * 2 * n_out_total * d * es + 2 * n_out_total
    return {"score": score, "select": select, "compact": compact, "select_compact": select + compact,
            "total": score + select + compact}


class LayerBuffers:
    """Inputs and outputs of one library call: one layer, or `n_fold` layers stacked on the batch axis."""

    def __init__(self, cfg, cap, layer, device, n_fold=1, qkv=None, max_len=None):
        if qkv is not None:
            self.q, self.k, self.v = qkv
        elif n_fold == 1:
            self.q, self.k, self.v = synth.make_layer(cfg, layer, device)
        else:
            parts = [synth.make_layer(cfg, layer + i, device) for i in range(n_fold)]
            self.q, self.k, self.v = (torch.cat([x[j] for x in parts], 0) for j in range(3))
            del parts
        B, H, d = self.k.shape[0], cfg.n_kv_heads, cfg.head_dim
        Lm = max_len if max_len is not None else cfg.max_len
        self.k_out = torch.empty((B, H, cap, d), dtype=cfg.dtype, device=device)
        self.v_out = torch.empty((B, H, cap, d), dtype=cfg.dtype, device=device)
        self.mod_out = torch.empty((B, H, cap), dtype=torch.uint8, device=device)
        self.n_out = torch.zeros((B, H), dtype=torch.int32, device=device)
        self.ss = torch.empty((B, H, Lm), dtype=torch.float32, device=device)
        self.sc = torch.empty((B, H, Lm), dtype=torch.float32, device=device)
        self.idx = torch.empty((B, H, cap), dtype=torch.int32, device=device)

    def layer_view(self, i, B0):
        """The i-th layer of a folded buffer as a buffer of its own (views, no copies)."""
        lv = copy.copy(self)
        for name in ("q", "k", "v", "k_out", "v_out", "mod_out", "n_out", "ss", "sc", "idx"):
            setattr(lv, name, getattr(self, name)[i * B0:(i + 1) * B0])
        return lv


class Call:
    """One csp_prune_layer call of a step."""

    def __init__(self, p, lb, mod, lens, bud, tot, layers, lse=None):
        self.p, self.lb, self.mod, self.lens, self.bud, self.tot, self.layers = p, lb, mod, lens, bud, tot, layers
        self.lse = lse        # log of the window rows' exponential sums, if an upstream attention kernel supplies it


def oracle_params(orc, cfg, batch, max_len, cap):
    return orc.Params(batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.window, cfg.recent, max_len, cap,
                      dtype=orc.F32 if cfg.dtype == torch.float32 else orc.BF16)


def oracle_layer_inputs(cfg, call, B0):
    """Host copies of the first layer of a call: what one oracle step reads."""
    lb = call.lb
    mod = call.mod[:B0].cpu().numpy()
    tot = None if call.tot is None else call.tot[:B0].cpu().numpy()
    return dict(q=lb.q[:B0].cpu().contiguous(), k=lb.k[:B0].cpu().contiguous(), v=lb.v[:B0].cpu().contiguous(),
                mod=mod, lens=call.lens[:B0].cpu().numpy(), bud=call.bud[:B0].cpu().numpy(), tot=tot)


# ------------------------------------------------------------------------------------ reference arm

def run_reference(args, rank, world):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload: one full layer per step
    (every sequence and KV head: at least as many independent units as the oracle has threads, which is
    what its OpenMP loop spreads over the cores)."""
    if rank != 0:
        return
    from oracle import csp_oracle as orc
    orc.build()
    cfg = synth.config(args.config, budget_pct=args.budget_pct) if args.config == 4 else synth.config(args.config)
    q, k, v = synth.make_layer(cfg, 0, "cpu")
    cap = cfg.out_capacity()
    op = oracle_params(orc, cfg, cfg.batch, cfg.max_len, cap)
    mod = cfg.modality()

    def step():
        orc.prune_layer(op, q, k, v, mod, cfg.seq_lens, cfg.budgets, cfg.total_budget)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / max(args.steps, 1)
    sum_l = int(cfg.seq_lens.sum())
    value = sum_l / dt
    sample = (f"one full layer per step: {cfg.batch} sequence(s) x {cfg.n_kv_heads} KV heads = "
              f"{cfg.batch * cfg.n_kv_heads} units, {sum_l} tokens; the per-layer metric needs no extrapolation, "
              f"a whole cache of {cfg.n_layers} layers would take {cfg.n_layers} x this (extrapolated)")
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

def fused_select_compact(p, sms) -> bool:
    """Whether csp_select_compact runs as one persistent kernel for dense, contiguous outputs in a second buffer (what
    this file passes): at least one unit per SM and caches of 1 K - 4 K positions, or two per SM up to 8 K when at least a
    twelfth of the rows can be kept."""
    units = p.batch * p.n_kv_heads
    return p.out_capacity > 0 and ((units >= sms and 1024 < p.max_len <= 4096) or
                                   (units >= 2 * sms and 4096 < p.max_len <= 8192 and p.out_capacity * 12 >= p.max_len))


def kernels_per_call(p, sms) -> int:
    """Kernels one csp_prune_layer call launches: score, select and compact (one kernel where they are fused), and,
    for a bf16 cache with more (sequence, head) units than SMs and several sequences, the kernel that orders them by
    length."""
    units, tiles = p.batch * p.n_kv_heads, (p.max_len + 127) // 128
    ordered = p.dtype == 1 and 2 <= p.batch <= 4096 and (units > sms or units * min(tiles, 8) > sms * 13 // 16)
    return (4 if ordered else 3) - (1 if fused_select_compact(p, sms) else 0)


class PathBench:
    """Everything timed for one workload on one GPU: the step (a CUDA graph of all calls), each kernel alone,
    a sustained replay, the host-buffer entry point, and the oracle on one layer."""

    def __init__(self, csp, args, dev, local_rank, dist):
        self.csp, self.args, self.dev, self.local_rank, self.dist = csp, args, dev, local_rank, dist
        self.sms = torch.cuda.get_device_properties(dev).multi_processor_count
        self.stream = torch.cuda.Stream(dev)

    # ---- launching
    def prune(self, c: Call, w):
        lb = c.lb
        self.csp.prune_layer(c.p, lb.q, lb.k, lb.v, c.mod, c.lens, c.bud, lb.k_out, lb.v_out, lb.mod_out, lb.n_out, w,
                             total_budget=c.tot, lse=c.lse)

    def capture(self, calls, n_chains, wss):
        """A CUDA graph of one step: chain c prunes calls c, c + n_chains, ... on its own stream."""
        stream, dev = self.stream, self.dev
        side = [torch.cuda.Stream(dev) for _ in range(n_chains - 1)]
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            fork = torch.cuda.Event()
            fork.record(stream)
            for c in range(n_chains):
                st = stream if c == 0 else side[c - 1]
                if c:
                    st.wait_event(fork)
                with torch.cuda.stream(st):
                    for i in range(c, len(calls), n_chains):
                        self.prune(calls[i], wss[c])
                if c:
                    join = torch.cuda.Event()
                    join.record(st)
                    stream.wait_event(join)
        return graph

    def time_replays(self, graph, steps, sample_clocks=True):
        stream = self.stream
        if self.dist is not None:
            self.dist.barrier()
        torch.cuda.synchronize()
        sampler = ClockSampler(self.local_rank) if sample_clocks else None
        if sampler:
            sampler.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            graph.replay()
        e1.record(stream)
        stream.synchronize()
        if self.dist is not None:
            self.dist.barrier()
        torch.cuda.synchronize()
        clocks = sampler.stop() if sampler else None
        return max_over_ranks(e0.elapsed_time(e1), self.dist, self.dev) / steps, clocks

    def time_graph_of(self, fn, reps):
        """ms per replay of a graph holding only what fn() launches, events on the launching stream."""
        stream = self.stream
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
        return k0.elapsed_time(k1) / reps

    def ex2_rates(self):
        """Exponentials per second of this GPU, measured once: on the special-function unit and through the FMA pipe."""
        if getattr(self, "_ex2", None) is None:
            csp, stream = self.csp, self.stream
            sink = torch.zeros(2 * self.sms * 1024, device=self.dev)
            res = {}
            with torch.cuda.stream(stream):
                for name, fma in (("special_function_unit", 0), ("fma_pipe_two_wide", 1), ("half_precision_pairs", 2)):
                    csp.probe_ex2_rate(fma, 256, sink)
                    stream.synchronize()
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record(stream)
                    n = csp.probe_ex2_rate(fma, 4096, sink)
                    e1.record(stream)
                    stream.synchronize()
                    res[name] = n / (e0.elapsed_time(e1) * 1e-3)
            self._ex2 = res
        return self._ex2

    # ---- one workload
    def measure(self, cfg, calls, n_chains, tokens_per_layer, n_layers, workload_name, launch_name, launch_tag,
                labels_per_head=False, want_extras=True, lens_per_layer=None):
        csp, args, dev, stream = self.csp, self.args, self.dev, self.stream
        world = 1 if self.dist is None else self.dist.get_world_size()
        wss = [csp.new_workspace(calls[0].p, dev) for _ in range(n_chains)]   # one scratch area per concurrent chain
        out = {}
        # the inputs and the zeroed workspaces were produced on torch's default stream; the calls below run on a
        # stream of their own that does not wait for it
        torch.cuda.synchronize()
        with torch.cuda.stream(stream):
            for _ in range(max(args.warmup, 3)):
                for c in calls:
                    self.prune(c, wss[0])
            stream.synchronize()
            graph = self.capture(calls, n_chains, wss)
            for _ in range(3):
                graph.replay()
            stream.synchronize()
            status = 0
            for w in wss:
                status |= csp.device_status(w)
            first = calls[0]
            n_out_total = int(first.lb.n_out.clamp(min=0).sum().item()) // first.layers      # kept rows per layer
            ms_step, clocks = self.time_replays(graph, args.steps)

            # ---- per-kernel durations, live: one CUDA graph per kernel holding that kernel's launch for
            # every call of a step, replayed back to back and timed with events on the launching stream
            ws = wss[0]

            def score_all():
                for c in calls:
                    csp.score(c.p, c.lb.q, c.lb.k, c.mod, c.lens, c.lb.ss, c.lb.sc, ws, lse=c.lse)

            def select_all():
                for c in calls:
                    csp.select(c.p, c.lb.ss, c.lb.sc, c.mod, c.lens, c.bud, c.lb.idx, c.lb.n_out, ws, total_budget=c.tot)

            def compact_all():
                for c in calls:
                    csp.compact(c.p, c.lb.k, c.lb.v, c.mod, c.lb.idx, c.lb.n_out, c.lb.k_out, c.lb.v_out, c.lb.mod_out)

            def select_compact_all():
                for c in calls:
                    csp.select_compact(c.p, c.lb.ss, c.lb.sc, c.lb.k, c.lb.v, c.mod, c.lens, c.bud, c.lb.k_out, c.lb.v_out,
                                       c.lb.mod_out, c.lb.n_out, ws, total_budget=c.tot, keep_idx=c.lb.idx)

            per = {}
            reps = max(3, min(50, args.steps))
            stages = [("score", score_all), ("select", select_all), ("compact", compact_all)]
            if any(fused_select_compact(c.p, self.sms) for c in calls):
                stages.append(("select_compact", select_compact_all))     # what the step runs instead of the two
            for name, fn in stages:
                per[name] = self.time_graph_of(fn, reps) / len(calls)                # ms per launch
            status |= csp.device_status(ws)

            # ---- sustained: the same graph replayed for about args.sustain_s seconds; the SM clock is sampled
            # throughout, and time x clock shows how much of a difference to the short run is the clock's.  Last,
            # so that the per-kernel durations above are taken at the clocks of the short run
            sustained = None
            if want_extras and args.sustain_s > 0:
                n_rep = max(args.steps, int(args.sustain_s * 1e3 / max(ms_step, 1e-3)) + 1)
                ms_sus, clk_sus = self.time_replays(graph, n_rep)
                sustained = {"seconds": ms_sus * n_rep * 1e-3, "steps": n_rep, "ms_per_step": ms_sus,
                             "value": job_throughput(world, tokens_per_layer, n_layers, ms_sus), "clocks": clk_sus,
                             "ms_x_ghz": None if not clk_sus or not clk_sus.get("sm_mhz") else ms_sus * clk_sus["sm_mhz"] * 1e-3,
                             "short_run_ms_x_ghz": None if not clocks or not clocks.get("sm_mhz") else ms_step * clocks["sm_mhz"] * 1e-3}

        peak, peak_kind = measured_peaks()
        lens = lens_per_layer if lens_per_layer is not None else cfg.seq_lens
        ab = algorithmic_bytes(cfg, lens, n_out_total, labels_per_head)
        lpl = first.layers
        ab_launch = {k_: v_ * lpl for k_, v_ in ab.items()}
        dominant = max(per, key=per.get)
        achieved = ab_launch[dominant] / (per[dominant] * 1e-3) / 1e9
        traffic, traffic_src = ncu_traffic(dominant, workload_name, launch_tag)
        roofline = {"bound": "hbm", "kernel": dominant, "achieved": achieved, "peak": peak, "unit": "GB/s",
                    "frac": achieved / peak, "traffic": traffic, "traffic_source": traffic_src,
                    "peak_kind": f"of {peak_kind}",
                    "algorithmic_bytes_per_launch": ab_launch[dominant], "us_per_launch": per[dominant] * 1e3}
        # The scoring kernel takes the exponential of every (query head of the group, window row, key) logit twice:
        # once for the row sums of Eq. 7, once for the weights.  With G >= 3 that is more special-function work per
        # K byte than the SMs can do at the HBM peak, so the bound of that kernel is the exponential rate of the
        # SMs: 16 ex2 per clock and SM on the special-function unit (the documented rate of sm_100) at the
        # maximum SM clock.
        if dominant == "score" and clocks and clocks.get("sm_max_mhz"):
            derived = 16.0 * self.sms * clocks["sm_max_mhz"] * 1e6
            probe = self.ex2_rates()
            ex2_peak = probe["special_function_unit"] if probe else derived
            passes = 1.0 if calls[0].lse is not None else 2.0       # a supplied LSE removes the pass for the row sums
            n_exp = passes * float(cfg.group * cfg.window * cfg.n_kv_heads) * float(np.asarray(lens, np.int64).sum()) * lpl
            if n_exp / ex2_peak > ab_launch["score"] / (peak * 1e9):
                ex2_rate = n_exp / (per["score"] * 1e-3)
                roofline = {"bound": "alu", "kernel": "score", "achieved": ex2_rate / 1e12, "peak": ex2_peak / 1e12,
                            "unit": "T ex2/s", "frac": ex2_rate / ex2_peak, "traffic": traffic,
                            "traffic_source": traffic_src,
                            "peak_kind": ("measured: csp_probe_ex2_rate, ex2.approx.ftz.f32 in registers only" if probe else
                                          "derived: 16 ex2 per clock and SM x SM count x maximum SM clock"),
                            "peak_derived": derived / 1e12, "probe": probe,
                            "exponentials_per_launch": n_exp,
                            "exponentials_counted": ("G W per key: the weights (row sums supplied)" if passes == 1.0 else
                                                     "2 G W per key: one for the row sums, one for the weights"),
                            "us_per_launch": per["score"] * 1e3, "hbm": roofline}
        path = {"algorithmic_bytes_per_layer": ab["total"], "us_per_layer": ms_step * 1e3 / n_layers,
                "achieved_gbs": ab["total"] / (ms_step * 1e-3 / n_layers) / 1e9,
                "frac_of_hbm_peak": ab["total"] / (ms_step * 1e-3 / n_layers) / 1e9 / peak,
                "frac_of_nominal_8tbs": ab["total"] / (ms_step * 1e-3 / n_layers) / 1e9 / 8000.0,
                "kernel_us_per_launch": {k_: v_ * 1e3 for k_, v_ in per.items()},
                "kernel_gbs": {k_: ab_launch[k_] / (per[k_] * 1e-3) / 1e9 for k_ in per}}
        out.update(ms_step=ms_step, clocks=clocks, sustained=sustained, roofline=roofline, path=path, status=status,
                   n_out_total=n_out_total, ab=ab, launches=sum(kernels_per_call(c.p, self.sms) for c in calls),
                   value=job_throughput(world, tokens_per_layer, n_layers, ms_step), launch=launch_name)
        return out

    # ---- end to end through the host-buffer entry point (pinned host memory, copies timed)
    def e2e(self, cfg, p, layer_bufs, mod, lens, bud, tot, n_layers, tokens_per_layer, steps):
        csp, dev, stream, args = self.csp, self.dev, self.stream, self.args
        world = 1 if self.dist is None else self.dist.get_world_size()
        pin = lambda t: t.cpu().contiguous().pin_memory()
        host = [dict(q=pin(lb.q), k=pin(lb.k), v=pin(lb.v), k_out=pin(lb.k_out), v_out=pin(lb.v_out),
                     mod_out=pin(lb.mod_out), n_out=pin(lb.n_out)) for lb in layer_bufs]
        n_host = len(host)
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
            if self.dist is not None:
                self.dist.barrier()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(steps):
                host_step()
            e1.record(stream)                   # all lanes are idle again: the interval covers every copy and kernel
            stream.synchronize()
            ms_e2e = e0.elapsed_time(e1) / steps
        pool.shutdown()
        ms_e2e = max_over_ranks(ms_e2e, self.dist, dev)
        hb = host[0]
        nbytes = lambda t: t.numel() * t.element_size()
        # K, Q, labels, lengths and budgets are copied in full; of V only the kept rows cross the bus: the
        # compaction kernel reads them straight from the pinned host buffer
        row_bytes = cfg.head_dim * hb["v"].element_size()
        kept_rows = int(hb["n_out"].clamp(min=0).sum().item())
        h2d = n_layers * (nbytes(hb["q"]) + nbytes(hb["k"]) + kept_rows * row_bytes + nbytes(h_mod) + nbytes(h_lens) +
                          nbytes(h_bud) + (0 if h_tot is None else nbytes(h_tot)))
        d2h = n_layers * sum(nbytes(hb[x]) for x in ("k_out", "v_out", "mod_out", "n_out"))
        return {"value": job_throughput(world, tokens_per_layer, n_layers, ms_e2e), "unit": UNIT,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e,
                "api": "csp_prune_layer_host", "host_threads": n_lanes,
                "v_rows": "kept rows only, read from the pinned host buffer by the compaction kernel"}

    # ---- CPU baseline and parity summary: the oracle on one full layer of the bytes the GPU pruned
    def cpu_baseline(self, cfg, call, B0, max_len, cap, tokens_per_layer, seconds=10.0):
        from oracle import csp_oracle as orc
        orc.build()
        x = oracle_layer_inputs(cfg, call, B0)
        op = oracle_params(orc, cfg, B0, max_len, cap)
        t0 = time.perf_counter()
        reps = 0
        ref = None
        while reps < 1 or (time.perf_counter() - t0 < seconds and reps < 5000):
            ref = orc.prune_layer(op, x["q"], x["k"], x["v"], x["mod"], x["lens"], x["bud"], x["tot"])
            reps += 1
        dt = (time.perf_counter() - t0) / reps
        units = B0 * cfg.n_kv_heads
        base = {"value": tokens_per_layer / dt, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle",
                "sample": f"one full layer ({units} units, {tokens_per_layer} tokens), {reps} repetitions, {dt:.3f} s each; "
                          f"per-layer metric, so a whole cache of {cfg.n_layers} layers would take {cfg.n_layers} x this (extrapolated)"}
        # parity summary of that layer (the tests hold the assertions; this is a record beside the timing)
        lb = call.lb
        g_ss, g_sc = lb.ss[:B0].cpu().numpy(), lb.sc[:B0].cpu().numpy()
        g_idx, g_n = lb.idx[:B0].cpu().numpy(), lb.n_out[:B0].cpu().numpy()
        worst, same_sets, differing = 0.0, 0, 0
        for b in range(B0):
            N = int(x["lens"][b]) - cfg.recent
            for h in range(cfg.n_kv_heads):
                for got, want in ((g_ss, ref["score_self"]), (g_sc, ref["score_cross"])):
                    w = want[b, h, :max(N, 0)].astype(np.float64)
                    if w.size:
                        tol = REL_TOL * np.abs(w) + ABS_FRAC * np.abs(w).max()
                        worst = max(worst, float((np.abs(got[b, h, :N] - w) / np.maximum(tol, 1e-300)).max()))
                n = int(ref["n_out"][b, h])
                if int(g_n[b, h]) == n and (n <= 0 or (g_idx[b, h, :n] == ref["keep_idx"][b, h, :n]).all()):
                    same_sets += 1
                else:
                    differing += len(set(g_idx[b, h, :max(int(g_n[b, h]), 0)].tolist()) ^ set(ref["keep_idx"][b, h, :max(n, 0)].tolist()))
        parity = {"units": units, "score_error_over_tolerance_max": worst, "scores_within_tolerance": worst <= 1.0,
                  "units_with_identical_index_list": same_sets, "positions_differing_in_the_rest": differing,
                  "tolerance": f"|gpu-oracle| <= {REL_TOL} |oracle| + {ABS_FRAC} max|oracle| per unit"}
        return base, parity


def make_calls(csp, cfg, dev, fold, n_buf, n_layers, with_lse=False):
    """The library calls of one step.  fold: one call for all layers (layer axis on the batch axis); else one
    call per layer over n_buf distinct layer buffers (views into one folded allocation)."""
    cap = cfg.out_capacity()
    p = csp.Params(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.window, cfg.recent, cfg.max_len,
                   cap, dtype=csp.F32 if cfg.dtype == torch.float32 else csp.BF16)
    mod = torch.from_numpy(cfg.modality()).to(dev)
    lens = torch.from_numpy(cfg.seq_lens).to(dev)
    bud = torch.from_numpy(cfg.budgets).to(dev)
    tot = None if cfg.total_budget is None else torch.from_numpy(cfg.total_budget).to(dev)
    folded = LayerBuffers(cfg, cap, 0, dev, n_fold=n_buf)
    pf = copy.copy(p)
    pf.batch = cfg.batch * n_buf
    fold_call = Call(pf, folded, mod.repeat(n_buf, 1), lens.repeat(n_buf), bud.repeat(n_buf, 1),
                     None if tot is None else tot.repeat(n_buf), n_buf)
    views = [folded.layer_view(i, cfg.batch) for i in range(n_buf)]
    lse_views = [None] * n_buf
    if with_lse:
        fold_call.lse = window_lse(cfg, folded.q, folded.k, lens.repeat(n_buf))
        lse_views = [fold_call.lse[i * cfg.batch:(i + 1) * cfg.batch] for i in range(n_buf)]
    layer_calls = [Call(p, views[i % n_buf], mod, lens, bud, tot, 1, lse_views[i % n_buf]) for i in range(n_layers)]
    return p, fold_call, layer_calls, (mod, lens, bud, tot)


def window_lse(cfg, q, k, lens):
    """Natural log of sum_t e^{o_t} of every window row over the keys it sees: what the attention kernel that
    produced the window's outputs already holds.  Input preparation (plain torch, untimed), not part of the path."""
    B, Hq, W, d = q.shape
    G = cfg.group
    out = torch.empty(B, Hq, W, dtype=torch.float32, device=q.device)
    lens_h = lens.cpu().numpy()
    for b in range(B):
        L = int(lens_h[b])
        kk = k[b, :, :L].float()                                        # [Hkv, L, d]
        qq = q[b].float().view(cfg.n_kv_heads, G * W, d)                # heads of a group share their KV head
        o = torch.bmm(qq, kk.transpose(1, 2)) / float(np.sqrt(d))       # [Hkv, G W, L]
        pos = (L - W + torch.arange(W, device=q.device)).repeat(G)      # position of each window row
        hidden = torch.arange(L, device=q.device)[None, :] > pos[:, None]
        o.masked_fill_(hidden[None], float("-inf"))
        out[b] = torch.logsumexp(o, dim=2).view(Hq, W)
    return out


def append_round(csp, cfg, dev, prev_calls, n_buf, gen, totals, budgets):
    """Inputs of the next re-prune round (Algorithm 1's iteration): every head's compacted cache plus 64 appended
    text tokens with fresh K, V and window queries; labels now differ per head."""
    B, H, d, W, R = cfg.batch, cfg.n_kv_heads, cfg.head_dim, cfg.window, cfg.recent
    n_prev = [c.lb.n_out.clamp(min=0).cpu().numpy() for c in prev_calls[:n_buf]]      # [B, H] per buffer
    # budgets per key modality with disjoint supports: every head of a sequence, in every layer, keeps the same
    # number of rows, so one length per sequence describes all heads
    assert all((n == n_prev[0][:, :1]).all() for n in n_prev), "heads of a sequence kept different numbers of rows"
    lens2 = torch.from_numpy(n_prev[0][:, 0].astype(np.int64) + 64).to(dev)
    Lm = int(lens2.max().item())
    cap = int((budgets.sum(axis=1) + R).max())
    p2 = csp.Params(B, cfg.n_q_heads, H, d, W, R, Lm, cap)
    calls = []
    for i in range(n_buf):
        prev = prev_calls[i].lb
        k2 = torch.zeros(B, H, Lm, d, dtype=cfg.dtype, device=dev)
        v2 = torch.zeros_like(k2)
        mod2 = torch.zeros(B, H, Lm, dtype=torch.uint8, device=dev)
        new_k = torch.randn(B, H, 64, d, device=dev, generator=gen).to(cfg.dtype)
        new_v = torch.randn(B, H, 64, d, device=dev, generator=gen).to(cfg.dtype)
        for b in range(B):
            n = int(n_prev[i][b, 0])
            k2[b, :, :n], v2[b, :, :n], mod2[b, :, :n] = prev.k_out[b, :, :n], prev.v_out[b, :, :n], prev.mod_out[b, :, :n]
            k2[b, :, n:n + 64], v2[b, :, n:n + 64] = new_k[b], new_v[b]     # appended decode tokens are text (label 0)
        q2 = torch.randn(B, cfg.n_q_heads, W, d, device=dev, generator=gen).to(cfg.dtype)
        lb = LayerBuffers(cfg, cap, 0, dev, qkv=(q2, k2, v2), max_len=Lm)
        calls.append(Call(p2, lb, mod2, lens2.to(torch.int32), torch.from_numpy(budgets).to(dev),
                          torch.from_numpy(totals.astype(np.int32)).to(dev), 1))
    return p2, calls, lens2.cpu().numpy()


def bench_line(cfg, args, world, config_index, m, e2e, cpu_baseline, parity, n_layers, n_buf, tokens_per_layer, extra=None):
    line = {"metric": METRIC, "value": m["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": m["ms_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if cfg.dtype == torch.bfloat16 else "f32",
            "data": "synthetic",
            "config": {"workload": f"configs[{config_index}] {cfg.name}" +
                                   (f", first {n_layers} of {cfg.n_layers} layers only" if n_layers != cfg.n_layers else ""),
                       "layers": n_layers,
                       "distinct_layer_buffers": n_buf, "batch": cfg.batch, "kv_heads": cfg.n_kv_heads,
                       "q_heads": cfg.n_q_heads, "head_dim": cfg.head_dim, "sum_seq_len": tokens_per_layer,
                       "window": cfg.window, "recent": cfg.recent, "kept_rows_per_layer": m["n_out_total"],
                       "launch": m["launch"],
                       "l2": "inputs larger than L2: every layer has its own K/V buffers"
                             if n_buf * m["ab"]["score"] > 2 * 126e6 else "inputs smaller than L2",
                       "replicas": "one independent replica per GPU, no collective"},
            "clocks": m["clocks"], "e2e": e2e, "gpu_launches": args.steps * m["launches"],
            "roofline": m["roofline"], "path": m["path"], "sustained": m["sustained"],
            "cpu_baseline": cpu_baseline, "parity": parity, "device_status": m["status"]}
    if extra:
        line.update(extra)
    return line


def run_config(pb: PathBench, csp, args, config_index, rank, world, dev, budget_pct=None, default_line=True):
    """All measurements of one workload; returns the JSON line(s) as dicts (rank 0 prints)."""
    cfg = synth.config(config_index, budget_pct=budget_pct or args.budget_pct) if config_index == 4 else synth.config(config_index)
    n_layers = cfg.n_layers if args.layers <= 0 else min(args.layers, cfg.n_layers)   # --layers: a cache cut to its first layers
    sum_l = int(cfg.seq_lens.sum())
    es = 2 if cfg.dtype == torch.bfloat16 else 4
    kv_bytes = 2 * n_layers * cfg.batch * cfg.n_kv_heads * cfg.max_len * cfg.head_dim * es
    huge = kv_bytes > 40e9                       # cycle four distinct layers when the whole cache is too large
    n_buf = 4 if huge else n_layers
    fold = args.fold_layers and n_buf == n_layers
    p, fold_call, layer_calls, (mod, lens, bud, tot) = make_calls(csp, cfg, dev, fold, n_buf, n_layers, args.with_lse)
    wl = f"configs{config_index}" + (f"_{budget_pct or args.budget_pct}pct" if config_index == 4 else "") + \
        ("_lse" if args.with_lse else "")
    n_chains = max(1, min(args.streams, n_layers))
    per_layer_name = f"cuda graph of one step, {n_chains} concurrent chains of one csp_prune_layer call per layer"
    fold_name = "one csp_prune_layer call for all layers (layer axis folded into the batch axis)"
    lines = []
    want_cpu = rank == 0 and world == 1 and not args.no_cpu_baseline
    if fold:
        m = pb.measure(cfg, [fold_call], 1, sum_l, n_layers, wl, fold_name, "all_layers_one_call")
        # Section 8(d)'s literal t_layer next to it: one call per layer, the independent layers as concurrent chains
        alt = pb.measure(cfg, layer_calls, n_chains, sum_l, n_layers, wl, per_layer_name, "one_layer_per_call", want_extras=False)
        extra = {"per_layer_calls": {"launch": alt["launch"], "ms_per_step": alt["ms_step"], "value": alt["value"],
                                     "us_per_layer": alt["path"]["us_per_layer"], "frac_of_hbm_peak": alt["path"]["frac_of_hbm_peak"],
                                     "kernel_us_per_launch": alt["path"]["kernel_us_per_launch"], "clocks": alt["clocks"]}}
        # leave the outputs of the folded call in the buffers (parity summary reads them)
        with torch.cuda.stream(pb.stream):
            pb.prune(fold_call, csp.new_workspace(fold_call.p, dev))
            pb.stream.synchronize()
    else:
        m = pb.measure(cfg, layer_calls, n_chains, sum_l, n_layers, wl, per_layer_name, "one_layer_per_call")
        extra = {}
    # the optional outputs (scores, index list) of the first layer, for the parity summary
    first = layer_calls[0]
    with torch.cuda.stream(pb.stream):
        ws1 = csp.new_workspace(first.p, dev)
        csp.prune_layer(first.p, first.lb.q, first.lb.k, first.lb.v, first.mod, first.lens, first.bud, first.lb.k_out,
                        first.lb.v_out, first.lb.mod_out, first.lb.n_out, ws1, total_budget=first.tot,
                        score_self=first.lb.ss, score_cross=first.lb.sc, keep_idx=first.lb.idx, lse=first.lse)
        pb.stream.synchronize()
    e2e = None
    if args.e2e_steps > 0 and not args.with_lse:
        e2e = pb.e2e(cfg, p, [c.lb for c in layer_calls[:min(n_buf, 4 if not huge else 2)]], mod, lens, bud, tot, n_layers,
                     sum_l, args.e2e_steps)
    cpu_baseline = parity = None
    if want_cpu:
        cpu_baseline, parity = pb.cpu_baseline(cfg, first, cfg.batch, cfg.max_len, p.out_capacity, sum_l,
                                               seconds=args.cpu_seconds)
    lines.append(bench_line(cfg, args, world, config_index, m, e2e, cpu_baseline, parity, n_layers, n_buf, sum_l, extra))
    if args.with_lse:
        lines[-1]["config"]["workload"] += ", log-sum-exp of the window rows supplied by the caller (no pass for the row sums)"

    # ---- the serving shape's re-prune rounds: 64 decode tokens appended to every head's compacted cache, four times
    if config_index == 4 and args.rounds > 0 and not default_line:
        gen = torch.Generator(device=dev).manual_seed(100 + (budget_pct or args.budget_pct))
        totals = cfg.total_budget.astype(np.int64)
        budgets = np.array([synth.budgets_from_total(int(t), cfg.recent) for t in totals], np.int32)
        prev = layer_calls
        round_ms, round_tokens = [m["ms_step"]], [sum_l]
        for rnd in range(1, args.rounds + 1):
            p2, bufs, lens2 = append_round(csp, cfg, dev, prev, n_buf, gen, totals, budgets)
            calls2 = [bufs[i % n_buf] for i in range(n_layers)]
            tok2 = int(lens2.sum())
            m2 = pb.measure(cfg, calls2, n_chains, tok2, n_layers, wl + f"_round{rnd}", per_layer_name, "one_layer_per_call",
                            labels_per_head=True, want_extras=False, lens_per_layer=lens2)
            cb2 = par2 = None
            if want_cpu and rnd == 1:
                c0 = calls2[0]
                with torch.cuda.stream(pb.stream):
                    wsr = csp.new_workspace(c0.p, dev)
                    csp.prune_layer(c0.p, c0.lb.q, c0.lb.k, c0.lb.v, c0.mod, c0.lens, c0.bud, c0.lb.k_out, c0.lb.v_out,
                                    c0.lb.mod_out, c0.lb.n_out, wsr, total_budget=c0.tot, score_self=c0.lb.ss,
                                    score_cross=c0.lb.sc, keep_idx=c0.lb.idx)
                    pb.stream.synchronize()
                cb2, par2 = pb.cpu_baseline(cfg, c0, cfg.batch, p2.max_len, p2.out_capacity, tok2, seconds=min(args.cpu_seconds, 4.0))
            lines.append(bench_line(cfg, args, world, config_index, m2, None, cb2, par2, n_layers, n_buf, tok2,
                                    {"round": rnd}))
            lines[-1]["config"]["workload"] += f", re-prune round {rnd} (compacted cache + 64 appended tokens)"
            round_ms.append(m2["ms_step"])
            round_tokens.append(tok2)
            prev = calls2
            del bufs
        lines[0]["round"] = 0
        lines[0]["rounds_total"] = {"ms_round0": round_ms[0], "ms_rounds_1_to_4": float(sum(round_ms[1:])),
                                    "ms_all_rounds": float(sum(round_ms)),
                                    "tokens_per_layer_by_round": round_tokens,
                                    "value_all_rounds": world * n_layers * float(sum(round_tokens)) / (sum(round_ms) * 1e-3)}
    return lines


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
    pf = csp.Params(cfg.batch * n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.window, cfg.recent,
                    cfg.max_len, cap)
    lb = LayerBuffers(cfg, cap, 0, dev, n_fold=n_layers)
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
        traffic, traffic_src = ncu_traffic("decode_attn", f"configs{args.config}", "all_layers_one_call")
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
                             "frac": achieved / peak, "traffic": traffic, "traffic_source": traffic_src,
                             "peak_kind": f"of {peak_kind}",
                             "algorithmic_bytes_per_launch": ab, "us_per_launch": ms_step * 1e3},
                "cpu_baseline": cpu_baseline, "device_status": status}
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def run_diagnostic(args, rank, world, local_rank):
    """`--diagnostic`: the measurement behind the method (Section 1: the gap between intra- and inter-modality attention
    weights) on the synthetic caches: csp_weight_histogram once per layer, the Jensen-Shannon divergence of every
    layer's pooled intra / inter histograms (64 half-octave bins of log2(weight)), and what the call costs.  Prints its
    own JSON line; not the default.  The values describe the synthetic generator, not a model."""
    from paper_2412_04652_b200 import binding as csp
    csp.lib()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    cfg = synth.config(args.config, budget_pct=args.budget_pct) if args.config == 4 else synth.config(args.config)
    n_layers = min(cfg.n_layers, 8 if args.config == 4 else cfg.n_layers)
    p = csp.Params(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.window, cfg.recent, cfg.max_len,
                   cfg.out_capacity())
    mod = torch.from_numpy(cfg.modality()).to(dev)
    lens = torch.from_numpy(cfg.seq_lens).to(dev)
    ws = csp.new_workspace(p, dev)
    hist = torch.zeros(cfg.batch, cfg.n_kv_heads, 2, csp.HIST_BINS, dtype=torch.int32, device=dev)
    js_all = torch.zeros(1, device=dev)
    pb = PathBench(csp, args, dev, local_rank, None)
    js, totals, ms = [], np.zeros((2, csp.HIST_BINS), np.int64), []
    with torch.cuda.stream(pb.stream):
        for layer in range(n_layers):
            q, k, v = synth.make_layer(cfg, layer, dev)
            call = lambda: csp.weight_histogram(p, q, k, mod, lens, hist, ws, js_all=js_all)
            ms.append(pb.time_graph_of(call, 5))
            js.append(float(js_all.item()))
            totals += hist.sum(dim=(0, 1)).cpu().numpy().astype(np.int64)
            del q, k, v
        status = csp.device_status(ws)
    weights_per_layer = int(totals.sum()) // n_layers
    if rank == 0:
        line = {"metric": "window_attention_weights_binned_per_sec", "value": weights_per_layer / (float(np.mean(ms)) * 1e-3),
                "unit": "weights/s", "n_gpus": world, "steps": 5, "warmup": 1, "ms_per_step": float(np.mean(ms)),
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": f"configs[{args.config}] {cfg.name}: csp_weight_histogram, one call per layer, {n_layers} layers",
                           "bins": f"{csp.HIST_BINS} half-octave bins of log2(weight) from 2^{int(csp.HIST_LO)}",
                           "weights_per_layer": weights_per_layer},
                "js_divergence_per_layer_nats": js, "js_max_possible": float(np.log(2.0)),
                "intra_histogram": totals[0].tolist(), "inter_histogram": totals[1].tolist(),
                "device_status": status, "gpu_launches": n_layers * 5 * 3, "e2e": None, "cpu_baseline": None}
        print(json.dumps(line), flush=True)


def run_incremental(args, rank, world, local_rank):
    """`--incremental`: a re-prune round of the serving shape (configs[4]) two ways.  Every head's compacted cache
    has grown by 64 decoded tokens and is pruned back to its budget, either by csp_prune_layer (the window's 32
    queries rescan the whole cache) or from the intra / inter sums that the last 32 decode steps carried along
    (csp_decode_step), which leaves csp_select_compact.  Four distinct layers folded into one call each;
    decode calls are timed at the final cache length.  Prints its own JSON line; not the default."""
    from paper_2412_04652_b200 import binding as csp
    csp.lib()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    cfg = synth.config(4, budget_pct=args.budget_pct)
    n_fold, W, R, d, H, Hq = 4, cfg.window, cfg.recent, cfg.head_dim, cfg.n_kv_heads, cfg.n_q_heads
    B = cfg.batch * n_fold
    cap0 = cfg.out_capacity()
    cap2 = cap0 + 64
    p0 = csp.Params(B, Hq, H, d, W, R, cfg.max_len, cap2)
    parts = [synth.make_layer(cfg, i, dev) for i in range(n_fold)]
    q0, k0, v0 = (torch.cat([x[j] for x in parts], 0) for j in range(3))
    del parts
    mod0 = torch.from_numpy(cfg.modality()).to(dev).repeat(n_fold, 1)
    lens0 = torch.from_numpy(cfg.seq_lens).to(dev).repeat(n_fold)
    bud0 = torch.from_numpy(cfg.budgets).to(dev).repeat(n_fold, 1)
    tot0 = torch.from_numpy(cfg.total_budget).to(dev).repeat(n_fold)
    k_c = torch.zeros(B, H, cap2, d, dtype=cfg.dtype, device=dev)
    v_c = torch.zeros_like(k_c)
    mod_c = torch.zeros(B, H, cap2, dtype=torch.uint8, device=dev)
    n0 = torch.zeros(B, H, dtype=torch.int32, device=dev)
    ws0 = csp.new_workspace(p0, dev)
    csp.prune_layer(p0, q0, k0, v0, mod0, lens0, bud0, k_c, v_c, mod_c, n0, ws0, total_budget=tot0)   # round 0
    status = csp.device_status(ws0)
    del q0, k0, v0, ws0
    torch.cuda.empty_cache()
    n_host = n0.cpu().numpy()
    assert (n_host == n_host[:, :1]).all() and (n_host > 0).all()
    gen = torch.Generator(device=dev).manual_seed(77)
    for b in range(B):                                           # 64 decoded text tokens behind the kept rows
        n = int(n_host[b, 0])
        k_c[b, :, n:n + 64] = torch.randn(H, 64, d, device=dev, generator=gen).to(cfg.dtype)
        v_c[b, :, n:n + 64] = torch.randn(H, 64, d, device=dev, generator=gen).to(cfg.dtype)
        mod_c[b, :, n:n + 64] = 0
    n_rows = (n0 + 64).contiguous()
    lens2 = n_rows[:, 0].contiguous()
    tokens_per_layer = int(lens2.sum().item()) // n_fold
    qs = torch.randn(W, B, Hq, d, device=dev, generator=gen).to(cfg.dtype)
    qlab = torch.zeros(B, dtype=torch.uint8, device=dev)
    pd = csp.Params(B, Hq, H, d, 1, 0, cap2, cap2)
    out = torch.zeros(B, Hq, d, device=dev)
    acc_s = torch.zeros(B, H, cap2, device=dev)
    acc_c = torch.zeros(B, H, cap2, device=dev)
    wd, wst = csp.new_decode_workspace(pd, dev), csp.new_decode_step_workspace(pd, dev)
    # the prune that follows: budgets per sequence as in round 0, cache length = kept rows + 64
    totals = cfg.total_budget.astype(np.int64)
    budgets = np.array([synth.budgets_from_total(int(t), R) for t in totals], np.int32)
    bud2 = torch.from_numpy(budgets).to(dev).repeat(n_fold, 1)
    tot2 = torch.from_numpy(totals.astype(np.int32)).to(dev).repeat(n_fold)
    p2 = csp.Params(B, Hq, H, d, W, R, cap2, cap0)
    k_o = torch.empty(B, H, cap0, d, dtype=cfg.dtype, device=dev)
    v_o = torch.empty_like(k_o)
    mod_o = torch.empty(B, H, cap0, dtype=torch.uint8, device=dev)
    n_o = torch.zeros(B, H, dtype=torch.int32, device=dev)
    idx = torch.empty(B, H, cap0, dtype=torch.int32, device=dev)
    ws2 = csp.new_workspace(p2, dev)
    q_win = qs.permute(1, 2, 0, 3).contiguous()
    pb = PathBench(csp, args, dev, local_rank, None)
    stream = pb.stream
    reps = max(3, min(50, args.steps))
    with torch.cuda.stream(stream):
        for i in range(W):                                       # the window's decode steps, so the sums are real
            csp.decode_step(pd, qs[i], k_c, v_c, n_rows, mod_c, qlab, i == 0, out, acc_s, acc_c, wst)
        stream.synchronize()
        t_dec = pb.time_graph_of(lambda: csp.decode_attn(pd, qs[0], k_c, v_c, n_rows, out, wd), reps)
        acc_s2, acc_c2 = acc_s.clone(), acc_c.clone()           # timing replays must not disturb the real sums
        t_step = pb.time_graph_of(lambda: csp.decode_step(pd, qs[1], k_c, v_c, n_rows, mod_c, qlab, False, out, acc_s2, acc_c2, wst), reps)
        t_full = pb.time_graph_of(lambda: csp.prune_layer(p2, q_win, k_c, v_c, mod_c, lens2, bud2, k_o, v_o, mod_o, n_o, ws2,
                                                          total_budget=tot2), reps)
        n_full = n_o.clone()

        def from_sums():
            csp.select_compact(p2, acc_s, acc_c, k_c, v_c, mod_c, lens2, bud2, k_o, v_o, mod_o, n_o, ws2, total_budget=tot2,
                               keep_idx=idx)
        t_inc = pb.time_graph_of(from_sums, reps)
        status |= csp.device_status(ws2) | csp.device_status(wd) | csp.device_status(wst)
        same_rows = bool(torch.equal(n_full, n_o))
    per_layer = lambda ms: ms / n_fold
    extra_per_step = per_layer(t_step - t_dec)
    inc_total = per_layer(t_inc) + W * max(extra_per_step, 0.0)
    es = 2
    rows_total = int(n_rows.clamp(min=0).sum().item())
    dec_bytes = rows_total * 2 * d * es
    peak, peak_kind = measured_peaks()
    if rank == 0:
        line = {"metric": METRIC, "value": world * tokens_per_layer / (inc_total * 1e-3), "unit": UNIT, "n_gpus": world,
                "steps": reps, "warmup": 3, "ms_per_step": inc_total * cfg.n_layers, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": f"configs[4] {cfg.name}, re-prune round 1 from the sums the decode steps carried",
                           "layers_timed": n_fold, "batch": cfg.batch, "kv_heads": H, "head_dim": d,
                           "sum_seq_len": tokens_per_layer, "window": W, "recent": R,
                           "launch": "four layers folded into one call of each kind; decode calls timed at the final cache length"},
                "per_layer_ms": {"decode_attn": per_layer(t_dec), "decode_step": per_layer(t_step),
                                 "extra_per_decode_step": extra_per_step,
                                 "select_plus_compact_from_sums": per_layer(t_inc),
                                 "reprune_incremental_total": inc_total,
                                 "reprune_full_rescan": per_layer(t_full)},
                "full_rescan": {"value": world * tokens_per_layer / (per_layer(t_full) * 1e-3), "unit": UNIT},
                "decode": {"achieved_gbs": dec_bytes / (t_dec * 1e-3) / 1e9, "with_sums_gbs": dec_bytes / (t_step * 1e-3) / 1e9,
                           "peak": peak, "peak_kind": f"of {peak_kind}"},
                "same_row_counts_both_ways": same_rows, "device_status": status,
                # decode attention + merge, decode step + merge, the rescan's kernels, selection + compaction from the sums
                "gpu_launches": reps * (2 + 2 + kernels_per_call(p2, pb.sms) + (1 if fused_select_compact(p2, pb.sms) else 2)),
                "e2e": None,
                "cpu_baseline": None}
        print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--config", type=int, default=1)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--layers", type=int, default=0,
                    help="prune only the first N layers of the workload (0 = all): a smaller case of the same kernels, "
                         "for profiler captures; the workload name in the line says so")
    ap.add_argument("--streams", type=int, default=32, help="concurrent layer chains inside the step graph")
    ap.add_argument("--per-layer-calls", dest="fold_layers", action="store_false",
                    help="time only one csp_prune_layer call per layer (concurrent chains in a CUDA graph); by default "
                         "the headline is one call for all layers, the layer axis of a [layers*B, H, L, d] cache "
                         "passed as the batch axis, and the per-layer figure is reported beside it")
    ap.set_defaults(fold_layers=True)
    ap.add_argument("--e2e-lanes", type=int, default=2, help="host threads (each with a stream and a staging area) of the end-to-end measurement")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--sustain-s", type=float, default=2.0, help="seconds of back-to-back replays for the sustained figure (0: skip)")
    ap.add_argument("--cpu-seconds", type=float, default=10.0, help="bound on the oracle's share of the run")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--decode", action="store_true",
                    help="time the step after the pruning pass instead: n-softmax decode attention over the pruned caches")
    ap.add_argument("--diagnostic", action="store_true",
                    help="per-layer Jensen-Shannon divergence between intra- and inter-modality attention weights of the window")
    ap.add_argument("--incremental", action="store_true",
                    help="a re-prune round of configs[4] from the sums carried by csp_decode_step, against the full rescan")
    ap.add_argument("--with-lse", action="store_true",
                    help="supply the log-sum-exp of the window rows (as an upstream attention kernel would): csp_score then "
                         "skips the pass that computes the row sums; a separate, labelled line")
    ap.add_argument("--budget-pct", type=int, default=20, help="budget of configs[4]")
    ap.add_argument("--rounds", type=int, default=4, help="re-prune rounds of configs[4] under --all-configs")
    ap.add_argument("--all-configs", action="store_true",
                    help="one JSON line per workload 1-4; for 4, every budget of {5,10,20,40} %% with round 0, "
                         "rounds 1-4 and their total (not the default: takes several minutes)")
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
    if args.incremental:
        run_incremental(args, rank, world, local_rank)
        return
    if args.diagnostic:
        run_diagnostic(args, rank, world, local_rank)
        return
    from paper_2412_04652_b200 import binding as csp
    csp.lib()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    pb = PathBench(csp, args, dev, local_rank, dist)
    if args.all_configs:
        if args.steps == 300:
            args.steps = 50
        args.e2e_steps = min(args.e2e_steps, 1)
        todo = [(1, None), (2, None), (3, None)] + [(4, pct) for pct in (5, 10, 20, 40)]
        for ci, pct in todo:
            for line in run_config(pb, csp, args, ci, rank, world, dev, budget_pct=pct, default_line=False):
                if rank == 0:
                    print(json.dumps(line), flush=True)
            torch.cuda.empty_cache()
    else:
        for line in run_config(pb, csp, args, args.config, rank, world, dev):
            if rank == 0:
                print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
