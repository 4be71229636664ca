#!/usr/bin/env python
"""Benchmark of the SemantiCache hot path on B200.

One *step* = one pass of the whole path over one synthetic batch: sc_chunk once, sc_compress for
every layer, then ``decode_steps`` decode steps of sc_decode_attn over every layer's cores; inside
a decode step the layers form a dependent chain (layer l+1's query is layer l's output), as in a
model's decode loop.
Reported ``value`` = decoded tokens per second over the whole step (compress included); the
decode-only rate, the compress time per 32K context and the achieved HBM bandwidth of both
stages are added as extra keys.  Everything is launched through the C-ABI library; the launch
sequence is captured into CUDA graphs so Python is not on the timed path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config I] [--impl ours|reference]

After the headline run (N = 1) short passes cover the other four workloads, the noise sweep and the
chunk-length x reduction grid with exact attention over the raw cache beside it (``configs``).

``--impl reference`` times the CPU oracle (plain C, fp64) on a bounded sample of the same
workload on the host cores.
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

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2603_14303_b200 import synth  # noqa: E402

METRIC = "compressed_kv_decode_tokens_per_s"
UNIT = "tokens/s"


def recorded_traffic(workload: str, stage: str):
    """DRAM bytes (read + write) per launch from an ncu capture, or None.

    The record (written by ``python -m paper_2603_14303_b200.ncu_traffic`` from an ncu CSV) names the
    workload and carries a hash of the kernel's source file as it was when the counters were taken; a
    kernel that has changed since gives None rather than a stale figure.  Not a measurement of this run."""
    from paper_2603_14303_b200 import ncu_traffic
    return ncu_traffic.lookup(workload, stage)



def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def measured_tensor_peak():
    """Dense bf16 TFLOP/s: the sustained figure (kernels here are timed inside loops of many launches)."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["bf16_tflops_sustained"]), "measured (sustained)"
    return 1400.0, "fallback (sustained)"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while timed regions run."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def summary(self, t0: float = 0.0, t1: float = float("inf")):
        """Median SM clock and the throttle reasons seen between host times t0 and t1."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        sm, smax, reasons = [], [], set()
        for ts, ln in list(self.lines):
            if ts < t0 or ts > t1 + 0.1:
                continue
            p = [x.strip() for x in ln.split(",")]
            if len(p) < 7:
                continue
            try:
                sm.append(float(p[0])); smax.append(float(p[1]))
            except ValueError:
                continue
            for nm, v in zip(self.NAMES, p[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}

    def stop(self, t0: float = 0.0, t1: float = float("inf")):
        if self.proc is not None:
            self.proc.terminate()
            self.thread.join(timeout=2)
        return self.summary(t0, t1)


# ------------------------------------------------------------------------------------- ours

# How the L per-layer sc_decode_attn calls of one decode step are launched:
#   chain        layer l+1's query is layer l's output, as in a model's decode loop; launched with
#                SC_FLAG_OVERLAP_CHAIN (the cores are prefetched while the previous layer still runs, the
#                query is read once it is complete)
#   serial       the same dependent chain in plain stream order
#   independent  every layer has its own seeded query and SC_FLAG_OVERLAP_PREV: an attention-only loop
#                whose launches do not depend on one another
DECODE_MODES = ("chain", "serial", "independent")


class Pipeline:
    """Device-resident state of one rank: inputs, plan, cores, and the captured launch graphs."""

    def __init__(self, w: synth.Workload, device, cap_frac: float = 0.5, raw_comparator: bool = False):
        from paper_2603_14303_b200 import binding
        self.b, self.w, self.dev = binding, w, device
        self.ids, self.run_id, self.run_lens = synth.token_ids(w)
        self.ids_dev = self.ids.to(device)
        self.K, self.V = [], []
        for layer in range(w.L):
            k, v = synth.layer_kv(w, layer, self.run_id, self.run_lens, device)
            self.K.append(k); self.V.append(v)
        self.cap = max(int(w.n * cap_frac), 1)
        dt = self.K[0].dtype
        i32 = dict(dtype=torch.int32, device=device)
        self.layers = [binding.CompressedLayer(torch.empty((w.B, w.Hkv, self.cap, w.d), dtype=dt, device=device),
                                               torch.empty((w.B, w.Hkv, self.cap, w.d), dtype=dt, device=device),
                                               torch.zeros((w.B, w.Hkv, self.cap), **i32),
                                               torch.zeros((w.B, w.Hkv), **i32)) for _ in range(w.L)]
        self.cws = [binding.compress_workspace(w.B, w.Hkv, w.n, device) for _ in range(w.L)]
        self.dws = [binding.decode_workspace(w.B, w.Hq, w.Hkv, w.d, self.cap, device) for _ in range(w.L)]
        # q[s, 0] feeds layer 0 of decode step s in every mode; q[s, l > 0] only the independent mode
        self.q = torch.stack([torch.stack([synth.queries(w, s, l, device) for l in range(w.L)])
                              for s in range(w.decode_steps)])            # [steps, L, B, Hq, d]
        self.out = torch.empty_like(self.q)
        self.plan = None
        self.status = torch.zeros((w.L, 1), **i32)
        self.cstatus = torch.zeros((w.L, 1), **i32)
        self.launches_compress = 0
        self.g_compress = None
        self.g_compress_per_layer = None
        self.lws = None
        self.one_launch = False
        self.g_decode, self.launches_decode = {}, {}
        # exact attention over the raw cache with the same kernel (count = NULL, every head n rows long)
        self.raw = None
        if raw_comparator:
            self.raw_len = torch.full((w.B, w.Hkv), w.n, **i32)
            self.raw_ws = [binding.decode_workspace(w.B, w.Hq, w.Hkv, w.d, w.n, device) for _ in range(w.L)]
            self.raw = True

    # the launch sequences (also what the graphs capture)
    def run_compress(self, one_launch: bool = False):
        """sc_chunk, then the compress stage: one sc_compress per layer, or every layer in one sc_compress_layers."""
        b, w = self.b, self.w
        if self.plan is None:
            self.plan = b.chunk(self.ids_dev, w.delims, w.max_chunk_len)
            self._chunk_ws = torch.empty(b.lib().sc_chunk_workspace_bytes(w.B, w.n), dtype=torch.uint8, device=self.dev)
        else:
            p = self.plan
            b.sc_chunk(self.ids_dev, w.delims, w.max_chunk_len, p.seg_off, p.seq_seg_off, p.n_seg, p.tile_seg,
                       p.seq_tile_cnt, self._chunk_ws, p.status)
        if one_launch:
            if self.lws is None:
                self.lws = b.compress_layers_workspace(w.L, w.B, w.Hkv, w.n, self.dev)
            b.sc_compress_layers(self.K, self.V, self.plan, w.tau, self.layers, self.lws, self.cstatus[0], 0)
            return
        for l in range(w.L):
            ly = self.layers[l]
            b.sc_compress(self.K[l], self.V[l], self.plan, w.tau, ly.core_k, ly.core_v, ly.count, ly.core_len, None,
                          self.cws[l], self.cstatus[l], 0)

    def run_decode(self, mode: str, steps: int | None = None, raw: bool = False):
        b, w = self.b, self.w
        flag = {"chain": b.SC_FLAG_OVERLAP_CHAIN, "serial": 0, "independent": b.SC_FLAG_OVERLAP_PREV}[mode]
        for s in range(steps or w.decode_steps):
            for l in range(w.L):
                q = self.q[s, l] if (l == 0 or mode == "independent") else self.out[s, l - 1]
                # the first launch of a decode step is an ordinary one: it orders the step behind all earlier work
                fl = flag if l > 0 else 0
                if raw:
                    b.sc_decode_attn(q, self.K[l], self.V[l], None, self.raw_len, self.out[s, l], self.raw_ws[l],
                                     0.0, self.status[l], fl)
                else:
                    b.decode_attn(q, self.layers[l], out=self.out[s, l], workspace=self.dws[l],
                                  status=self.status[l], flags=fl)

    def capture(self, modes=("chain",), short_steps: int | None = None, one_launch: bool = False):
        """Warm-up pass, then one graph for the compress stage and one per decode mode.  The first mode
        is captured with all decode steps; the others with ``short_steps`` (they are side measurements).
        ``one_launch``: the timed compress stage is sc_compress_layers; the per-layer form gets a graph of its own."""
        self.one_launch = one_launch
        self.run_compress()   # allocates the plan outside capture
        if one_launch:
            self.run_compress(True)
        torch.cuda.synchronize(self.dev)
        self.b.check_status(self.plan.status, "warm-up pass")
        if int(self.cstatus.abs().max().item()) != 0:
            raise RuntimeError("sc_compress reported a device-side error in the warm-up pass")
        c0 = self.b.launch_counter()
        self.g_compress = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.g_compress):
            self.run_compress(one_launch)
        self.launches_compress = self.b.launch_counter() - c0
        if one_launch:
            self.g_compress_per_layer = torch.cuda.CUDAGraph()
            with torch.cuda.graph(self.g_compress_per_layer):
                self.run_compress(False)
        self.steps_of = {}
        for i, mode in enumerate(modes):
            steps = self.w.decode_steps if (i == 0 or not short_steps) else min(short_steps, self.w.decode_steps)
            self.run_decode(mode, 1)
            torch.cuda.synchronize(self.dev)
            c0 = self.b.launch_counter()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                self.run_decode(mode, steps)
            self.g_decode[mode], self.launches_decode[mode], self.steps_of[mode] = g, self.b.launch_counter() - c0, steps
        if self.raw:
            steps = min(short_steps or self.w.decode_steps, self.w.decode_steps)
            self.run_decode("chain", 1, raw=True)
            torch.cuda.synchronize(self.dev)
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                self.run_decode("chain", steps, raw=True)
            self.g_decode["raw"], self.steps_of["raw"] = g, steps
        torch.cuda.synchronize(self.dev)
        if int(self.status.abs().max().item()) != 0:
            raise RuntimeError("sc_decode_attn reported a device-side error in the warm-up pass")

    def time_graph(self, g, reps: int):
        """Median device time (ms) of ``reps`` replays of a graph, one warm-up replay first."""
        g.replay()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
        for a, z in ev:
            a.record(); g.replay(); z.record()
        torch.cuda.synchronize(self.dev)
        return statistics.median(a.elapsed_time(z) for a, z in ev)

    def algorithmic_bytes(self):
        """(compress bytes per step, decode bytes per decode step over all layers, per-layer list, kept)."""
        w = self.w
        esz = self.K[0].element_size()
        lens = torch.stack([ly.core_len for ly in self.layers]).to(torch.int64).cpu()   # [L, B, Hkv]
        rows = lens.sum().item()
        kv_in = w.L * w.B * w.Hkv * w.n * w.d * esz * 2
        core_bytes = rows * (2 * w.d * esz + 4)
        qo = w.L * w.B * w.Hq * w.d * esz * 2
        per_layer = [(lens[l].sum().item() * (2 * w.d * esz + 4) + qo // w.L) for l in range(w.L)]
        return kv_in + core_bytes, core_bytes + qo, per_layer, rows / (w.L * w.B * w.Hkv * w.n)


def decode_mode_record(pipe: Pipeline, mode: str, ms: float, layer_bytes: float, peak: float):
    """Per-launch time and achieved bandwidth of one decode graph replay that took ``ms``."""
    w = pipe.w
    launches = pipe.steps_of[mode] * w.L
    us = ms * 1e3 / launches
    gbs = layer_bytes / (us * 1e-6) / 1e9
    return {"us_per_launch": us, "achieved_gbs": gbs, "frac": gbs / peak, "frac_of_nominal_8tbs": gbs / 8000.0,
            "decode_tokens_per_s": w.B * pipe.steps_of[mode] / (ms * 1e-3), "decode_steps_timed": pipe.steps_of[mode]}


def run_ours(args):
    from paper_2603_14303_b200 import dist as scdist
    distributed = args.gpus > 1
    rank, local, _ = scdist.env_rank()
    dev = torch.device(f"cuda:{local}")
    torch.cuda.set_device(dev)
    if distributed:
        scdist.init("nccl", dev)
    from paper_2603_14303_b200 import binding, build
    build.build()
    w = synth.config(args.config)
    if args.decode_steps:
        w = w.replace(decode_steps=args.decode_steps)
    if args.layers:
        w = w.replace(L=args.layers)
    if distributed:
        w = scdist.rank_workload(w, rank)           # every rank owns an independent batch (weak scaling)
    pipe = Pipeline(w, dev)
    main_mode = "serial" if args.no_overlap else "chain"
    side_modes = [m for m in DECODE_MODES if m != main_mode] if (args.gpus == 1 and not args.no_modes) else []
    one_launch = (not args.per_layer_compress) and w.L <= binding.SC_MAX_LAYERS_PER_CALL
    pipe.capture([main_mode] + side_modes, short_steps=max(8, min(32, w.decode_steps // 8)), one_launch=one_launch)
    cbytes, dbytes, per_layer, kept = pipe.algorithmic_bytes()
    g_decode = pipe.g_decode[main_mode]

    def barrier():
        scdist.barrier(dev)

    for _ in range(max(args.warmup, 3)):
        pipe.g_compress.replay()
        g_decode.replay()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    barrier()
    t_host0 = time.time()
    t_wall = time.perf_counter()
    for s in range(args.steps):
        ev[s][0].record()
        pipe.g_compress.replay()
        ev[s][1].record()
        g_decode.replay()
        ev[s][2].record()
    barrier()
    t_wall = time.perf_counter() - t_wall
    clocks = sampler.summary(t_host0, time.time()) if rank == 0 else None
    binding.check_status(pipe.plan.status, "timed region")
    if int(pipe.status.abs().max().item()) != 0 or int(pipe.cstatus.abs().max().item()) != 0:
        raise RuntimeError("sc_compress / sc_decode_attn reported a device-side error")
    ms_c = [e[0].elapsed_time(e[1]) for e in ev]
    ms_d = [e[1].elapsed_time(e[2]) for e in ev]
    total_ms = ev[0][0].elapsed_time(ev[-1][2])
    total_ms, sum_c, sum_d = scdist.max_over_ranks([total_ms, sum(ms_c), sum(ms_d)], dev)
    value = scdist.whole_job_rate(w.B * w.decode_steps * args.steps, args.gpus, total_ms)

    # end to end through the public API with HOST buffers (copies inside the timed region)
    e2e = run_e2e(pipe, args, barrier, g_decode) if not args.no_e2e else None
    if distributed and e2e is not None:
        e2e["value"] = scdist.whole_job_rate(w.B * w.decode_steps * e2e["_steps"], args.gpus,
                                             scdist.max_over_ranks([e2e["_ms"]], dev)[0])
    if e2e is not None:
        e2e = {k: v for k, v in e2e.items() if not k.startswith("_")}

    if rank != 0:
        return
    peak, peak_kind = measured_peaks()
    launches_per_decode = w.decode_steps * w.L    # sc_decode_attn calls per step
    dec_launch_us = sum_d / args.steps / launches_per_decode * 1e3
    layer_bytes = sum(per_layer) / len(per_layer)
    achieved = layer_bytes / (dec_launch_us * 1e-6) / 1e9
    comp_ms = sum_c / args.steps
    comp_gbs = cbytes / (comp_ms * 1e-3) / 1e9
    launch_text = {"chain": "cuda graphs; within a decode step layer l+1's query is layer l's output and the launches are "
                            "chained (SC_FLAG_OVERLAP_CHAIN: cores prefetched under the previous layer, query read after it)",
                   "serial": "cuda graphs; dependent per-layer launches in plain stream order"}[main_mode]
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": total_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "n_ctx": w.n, "layers": w.L, "kv_heads": w.Hkv, "q_heads": w.Hq,
                   "head_dim": w.d, "tau": w.tau, "decode_steps": w.decode_steps, "kept_fraction": round(kept, 4),
                   "l2": "inputs larger than L2 (every step streams all layers)", "launch": launch_text,
                   "compress_launch": "one sc_compress_layers for all layers" if one_launch else "one sc_compress per layer",
                   "parallelism": f"replicas x{args.gpus}" if distributed else "single gpu"},
        "decode_tokens_per_s": w.B * w.decode_steps * args.gpus / (sum_d / args.steps * 1e-3),
        "decode_bytes_per_step": dbytes,
        "decode_gbs": dbytes * w.decode_steps / (sum_d / args.steps * 1e-3) / 1e9,
        "compress_ms_per_32k_ctx": comp_ms * 32768 / (w.B * w.n),
        "compress_gbs": comp_gbs, "compress_frac_of_peak": comp_gbs / peak,
        "roofline": {"kernel": "sc_decode_attn (one layer per launch, " + main_mode + " launches)", "bound": "hbm",
                     "achieved": achieved, "peak": peak, "peak_kind": peak_kind, "unit": "GB/s", "frac": achieved / peak,
                     "frac_of_nominal_8tbs": achieved / 8000.0, "bytes_per_launch": layer_bytes,
                     "us_per_launch": dec_launch_us,
                     "traffic": args.traffic if args.traffic is not None else recorded_traffic(w.name, "decode"),
                     "traffic_source": "ncu capture recorded under profiles/ (not this run); null once the kernel source changed"},
        "roofline_compress": {"kernel": "sc_compress_layers (every layer in one launch, as at the end of a prefill)" if one_launch
                              else "sc_compress (one layer per launch)", "bound": "hbm", "achieved": comp_gbs,
                              "peak": peak, "peak_kind": peak_kind, "unit": "GB/s", "frac": comp_gbs / peak,
                              "frac_of_nominal_8tbs": comp_gbs / 8000.0, "bytes_per_launch": cbytes / (1 if one_launch else w.L),
                              "us_per_launch": comp_ms * 1e3 / (1 if one_launch else w.L), "us_per_layer": comp_ms * 1e3 / w.L,
                              "launches_per_step": 1 if one_launch else w.L,
                              "traffic": recorded_traffic(w.name, "compress_layers" if one_launch else "compress")},
        "gpu_launches": args.steps * (pipe.launches_compress + pipe.launches_decode[main_mode]),
        "gpu_launches_per_step": {"chunk+compress": pipe.launches_compress, "decode": pipe.launches_decode[main_mode]},
        "clocks": clocks, "e2e": e2e, "wall_s": t_wall,
    }
    if side_modes:
        # the same decode work under the other launch disciplines (decode graph alone, a few replays each)
        modes = {main_mode: {"us_per_launch": dec_launch_us, "achieved_gbs": achieved, "frac": achieved / peak,
                             "frac_of_nominal_8tbs": achieved / 8000.0,
                             "decode_tokens_per_s": line["decode_tokens_per_s"], "decode_steps_timed": w.decode_steps,
                             "timed": "inside the benchmark step"}}
        for m in side_modes:
            modes[m] = decode_mode_record(pipe, m, pipe.time_graph(pipe.g_decode[m], 5), layer_bytes, peak)
        line["decode_launch_modes"] = {
            "what": "chain = layer l+1's query is layer l's output, launches chained with SC_FLAG_OVERLAP_CHAIN (what a "
                    "model's decode loop can use); serial = the same chain in plain stream order; independent = every "
                    "layer has its own query, SC_FLAG_OVERLAP_PREV (an attention-only loop without the dependence)",
            **modes}
        line["decode_serial"] = modes["serial"]
        line["decode_independent_overlap"] = modes["independent"]
    if one_launch and args.gpus == 1:
        # the same stage as one sc_compress per layer (the per-layer call of the scope table), graph alone
        ms_p = pipe.time_graph(pipe.g_compress_per_layer, 5)
        gbs_p = cbytes / (ms_p * 1e-3) / 1e9
        line["roofline_compress_per_layer_calls"] = {
            "kernel": "sc_compress (one layer per launch)", "bound": "hbm", "achieved": gbs_p, "peak": peak, "peak_kind": peak_kind,
            "unit": "GB/s", "frac": gbs_p / peak, "frac_of_nominal_8tbs": gbs_p / 8000.0, "bytes_per_launch": cbytes / w.L,
            "us_per_launch": ms_p * 1e3 / w.L, "ms_per_32k_ctx": ms_p * 32768 / (w.B * w.n),
            "traffic": recorded_traffic(w.name, "compress")}
        if int(pipe.cstatus.abs().max().item()) != 0:
            raise RuntimeError("sc_compress reported a device-side error")
    if args.gpus == 1 and not args.no_append:
        line["append"] = measure_append(pipe)
    del pipe
    torch.cuda.empty_cache()
    if args.gpus == 1 and not args.no_sweep:
        t0 = time.time()
        line["configs"] = sweep_configs(args, dev, sampler, peak)
        line["configs"]["wall_s"] = time.time() - t0
        t0 = time.time()
        line["extras"] = measure_extras(dev, sampler, peak)
        line["extras"]["wall_s"] = time.time() - t0
    sampler.stop()
    if not args.no_cpu_baseline and args.gpus == 1:
        line["cpu_baseline"] = cpu_baseline(w, budget_s=args.cpu_budget)
    print(json.dumps(line))


# ------------------------------------------------------------ the five workloads and their sweeps


def measure_cell(w: synth.Workload, full_L: int, dev, sampler, peak, label: dict, raw: bool = False,
                 decode_steps: int = 8, cap_frac: float = 0.5):
    """Short pass of one workload cell on a reduced layer count: compress (median of 3 graph replays) and
    chained decode (median of 3 replays of ``decode_steps`` steps), optionally exact attention over the raw
    cache with the same kernel.  Rates are for the workload's full layer count ``full_L``."""
    t0 = time.time()
    w = w.replace(decode_steps=decode_steps)
    pipe = Pipeline(w, dev, cap_frac=cap_frac, raw_comparator=raw)
    pipe.capture(["chain"], short_steps=decode_steps)
    cbytes, dbytes, per_layer, kept = pipe.algorithmic_bytes()
    ms_c = pipe.time_graph(pipe.g_compress, 3)
    ms_d = pipe.time_graph(pipe.g_decode["chain"], 3)
    ms_l = time_calls(lambda: pipe.run_compress(True), 3)   # the same layers in one sc_compress_layers launch
    layer_bytes = sum(per_layer) / len(per_layer)
    us_launch = ms_d * 1e3 / (decode_steps * w.L)
    dgbs = layer_bytes / (us_launch * 1e-6) / 1e9
    cgbs = cbytes / (ms_c * 1e-3) / 1e9
    rec = dict(label)
    rec.update({
        "layers_run": w.L, "layers_full": full_L, "kept_fraction": round(kept, 4),
        "achieved_reduction": round(1.0 / kept, 3) if kept > 0 else None,
        "decode_tokens_per_s": w.B / (us_launch * 1e-6 * full_L), "decode_bytes_per_step": dbytes / w.L * full_L,
        "decode_us_per_launch": us_launch, "decode_gbs": dgbs, "decode_frac": dgbs / peak,
        "decode_frac_of_nominal_8tbs": dgbs / 8000.0, "compress_frac_of_nominal_8tbs": cgbs / 8000.0,
        "compress_ms_per_32k_ctx": ms_c / w.L * full_L * 32768 / (w.B * w.n), "compress_us_per_layer": ms_c * 1e3 / w.L,
        "compress_gbs": cgbs, "compress_frac": cgbs / peak,
        "compress_all_layers_one_launch": {"layers": w.L, "ms_per_32k_ctx": ms_l / w.L * full_L * 32768 / (w.B * w.n),
                                           "us_per_layer": ms_l * 1e3 / w.L, "frac": cbytes / (ms_l * 1e-3) / 1e9 / peak}})
    if raw:
        ms_r = pipe.time_graph(pipe.g_decode["raw"], 3)
        us_r = ms_r * 1e3 / (pipe.steps_of["raw"] * w.L)
        raw_bytes = w.B * w.Hkv * w.n * 2 * w.d * pipe.K[0].element_size() + 2 * w.B * w.Hq * w.d * pipe.K[0].element_size()
        rgbs = raw_bytes / (us_r * 1e-6) / 1e9
        rec["uncompressed_exact_attention"] = {
            "what": "the same decode kernel over the raw K/V (count = NULL, every head n rows)",
            "decode_tokens_per_s": w.B / (us_r * 1e-6 * full_L), "decode_bytes_per_step": raw_bytes * full_L,
            "decode_us_per_launch": us_r, "decode_gbs": rgbs, "decode_frac": rgbs / peak,
            "speedup_of_compressed": us_r / us_launch, "bytes_ratio": raw_bytes / layer_bytes}
    if int(pipe.status.abs().max().item()) != 0 or int(pipe.cstatus.abs().max().item()) != 0:
        raise RuntimeError(f"device-side error in sweep cell {label}")
    del pipe
    torch.cuda.empty_cache()
    rec["clocks"] = sampler.summary(t0, time.time())
    rec["cell_wall_s"] = round(time.time() - t0, 2)
    return rec


def time_calls(fn, reps: int = 10):
    """Median device time (ms) of fn() launched `reps` times after one warm-up call."""
    fn()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
    for a, z in ev:
        a.record(); fn(); z.record()
    torch.cuda.synchronize()
    return statistics.median(a.elapsed_time(z) for a, z in ev)


def measure_extras(dev, sampler, peak):
    """The rows beyond the three main calls, each on the Llama-3-8B 32K shape (a few layers): multi-query
    Proportional Attention, clustering without chunking, fixed-size chunks, compression to a budget."""
    from paper_2603_14303_b200 import binding as b
    out = {}
    tpeak, tkind = measured_tensor_peak()
    w = synth.config(1, L=4)
    pipe = Pipeline(w, dev)
    pipe.run_compress()
    torch.cuda.synchronize()
    lens = torch.stack([ly.core_len for ly in pipe.layers]).to(torch.int64)
    rows_per_layer = lens.sum().item() / w.L

    # -- sc_prefill_attn: m queries per head against the compressed cache, one launch per layer
    t0 = time.time()
    pre = {"what": "sc_prefill_attn: a block of m queries per head over the compressed cache, one launch per layer; "
                   "flops = 4 * (G*m) * core rows * d per KV head (scores + weighted sum)", "peak_tflops": tpeak,
           "peak_kind": tkind, "cells": []}
    for m in (8, 128, 512, 2048):
        q = torch.randn((w.L, w.B, w.Hq, m, w.d), device=dev).to(torch.bfloat16)
        o = torch.empty_like(q)
        st = torch.zeros(1, dtype=torch.int32, device=dev)

        def run():
            for l in range(w.L):
                b.sc_prefill_attn(q[l], pipe.layers[l].core_k, pipe.layers[l].core_v, pipe.layers[l].count,
                                  pipe.layers[l].core_len, o[l], 0.0, st)
        ms = time_calls(run) / w.L
        flops = 4.0 * w.G * m * rows_per_layer * w.d
        tf = flops / (ms * 1e-3) / 1e12
        pre["cells"].append({"m": m, "query_rows_per_kv_head": w.G * m, "us_per_layer": ms * 1e3, "tflops": tf,
                             "frac_of_tensor_peak": tf / tpeak, "query_tokens_per_s": w.B * m / (ms * 1e-3 * 32)})
        if int(st.item()) != 0:
            raise RuntimeError("sc_prefill_attn reported a device-side error")
        del q, o
    pre["roofline"] = {"bound": "tensor", "achieved": max(c["tflops"] for c in pre["cells"]), "peak": tpeak,
                       "unit": "TFLOP/s", "frac": max(c["frac_of_tensor_peak"] for c in pre["cells"]),
                       "traffic": recorded_traffic(w.name, "prefill")}
    pre["clocks"] = sampler.summary(t0, time.time())
    out["prefill_attn"] = pre

    # -- fixed-size chunks of 64 tokens (Table 4a's second arm): same kernels, other plan
    t0 = time.time()
    plan64 = b.chunk_fixed(pipe.ids_dev, 64)
    lay = pipe.layers

    def run_fixed():
        for l in range(w.L):
            b.sc_compress(pipe.K[l], pipe.V[l], plan64, w.tau, lay[l].core_k, lay[l].core_v, lay[l].count, lay[l].core_len,
                          None, pipe.cws[l], pipe.cstatus[l], 0)
    ms = time_calls(run_fixed) / w.L
    kept = torch.stack([ly.core_len for ly in lay]).sum().item() / (w.L * w.B * w.Hkv * w.n)
    cbytes = w.B * w.Hkv * w.n * w.d * 2 * 2 * (1 + kept) + 4 * kept * w.B * w.Hkv * w.n
    out["fixed_chunks_64"] = {"what": "sc_chunk with no delimiters and max_chunk_len 64, then sc_compress", "layers_run": w.L,
                              "kept_fraction": round(kept, 4), "compress_us_per_layer": ms * 1e3,
                              "compress_ms_per_32k_ctx": ms * 32 * 32768 / (w.B * w.n),
                              "compress_frac": cbytes / (ms * 1e-3) / 1e9 / peak, "clocks": sampler.summary(t0, time.time())}
    pipe.run_compress()      # back to the semantic plan's cores

    # -- clustering without chunking (Table 4a's third arm)
    t0 = time.time()
    gws = torch.empty(b.lib().sc_compress_global_workspace_bytes(w.B, w.Hkv, w.n), dtype=torch.uint8, device=dev)
    gl_layers = 2

    def run_global():
        for l in range(gl_layers):
            b.sc_compress_global(pipe.K[l], pipe.V[l], w.tau, lay[l].core_k, lay[l].core_v, lay[l].count, lay[l].core_len,
                                 gws, None, pipe.cstatus[l], 0)
    ms = time_calls(run_global, 5) / gl_layers
    kept = torch.stack([ly.core_len for ly in lay[:gl_layers]]).sum().item() / (gl_layers * w.B * w.Hkv * w.n)
    pair_flops = float(w.B * w.Hkv) * w.n * w.n * w.d       # n^2 / 2 pairs, 2 d flops each
    out["global_clustering"] = {"what": "sc_compress_global: Algorithm 1 over whole sequences; pairwise stage = n^2/2 * 2d flops per head",
                                "layers_run": gl_layers, "kept_fraction": round(kept, 4), "ms_per_layer": ms,
                                "ms_per_32k_ctx": ms * 32 * 32768 / (w.B * w.n), "pairwise_tflops_if_all_time": pair_flops / (ms * 1e-3) / 1e12,
                                "workspace_mb": gws.numel() / 1e6, "clocks": sampler.summary(t0, time.time())}
    del gws
    if int(pipe.cstatus.abs().max().item()) != 0:
        raise RuntimeError("device-side error in the ablation arms")
    del pipe
    torch.cuda.empty_cache()

    # -- compression to a budget: keys noisy enough that the kept fraction depends on the threshold
    t0 = time.time()
    wb = synth.config(1, L=4, sigma=0.6)
    pipe = Pipeline(wb, dev, cap_frac=1.0)
    pipe.run_compress()
    bws = [torch.zeros(b.lib().sc_compress_budget_workspace_bytes(wb.B, wb.Hkv, wb.n), dtype=torch.uint8, device=dev)
           for _ in range(wb.L)]
    tau = torch.zeros((wb.L, 1), dtype=torch.float32, device=dev)
    srch = torch.zeros((wb.L, 2), dtype=torch.int32, device=dev)
    lay = pipe.layers
    cells = []
    for target in (0.35, 0.5):
        def run_budget():
            for l in range(wb.L):
                b.sc_compress_budget(pipe.K[l], pipe.V[l], pipe.plan, target, 0.5, 0.9, 17, lay[l].core_k, lay[l].core_v,
                                     lay[l].count, lay[l].core_len, tau[l], srch[l], bws[l], None, pipe.cstatus[l], 0)
        ms = time_calls(run_budget, 5) / wb.L
        ms_plain = time_calls(lambda: [b.sc_compress(pipe.K[l], pipe.V[l], pipe.plan, 0.7, lay[l].core_k, lay[l].core_v,
                                                     lay[l].count, lay[l].core_len, None, pipe.cws[l], pipe.cstatus[l], 0)
                                       for l in range(wb.L)], 3) / wb.L
        run_budget()
        torch.cuda.synchronize()
        kept = torch.stack([ly.core_len for ly in lay]).sum().item() / (wb.L * wb.B * wb.Hkv * wb.n)
        cells.append({"target_kept": target, "achieved_kept": round(kept, 4), "tau_chosen": [round(float(x), 4) for x in tau.flatten().tolist()],
                      "counting_passes": srch[:, 1].tolist(), "us_per_layer": ms * 1e3, "ms_per_32k_ctx": ms * 32 * 32768 / (wb.B * wb.n),
                      "plain_compress_us_per_layer": ms_plain * 1e3})
    out["budget"] = {"what": "sc_compress_budget on keys with noise 0.6 (kept fraction varies over the grid), grid of 17 thresholds in [0.5, 0.9]",
                     "layers_run": wb.L, "cells": cells, "clocks": sampler.summary(t0, time.time())}
    if int(pipe.cstatus.abs().max().item()) != 0:
        raise RuntimeError("device-side error in the budget search")
    del pipe
    torch.cuda.empty_cache()
    return out


def sweep_configs(args, dev, sampler, peak):
    """Short passes over the other workloads and the sweeps two of them name (after the headline run).

    Every cell runs a reduced number of layers whose cores still exceed the L2 by a wide margin (the
    toy workload excepted: it is L2-resident by definition and its fractions are informational)."""
    out = {"what": "per cell: chained decode and compress (one sc_compress per layer; compress_all_layers_one_launch: the "
                   "same layers in one sc_compress_layers) on a reduced layer count (layers_run), rates scaled to "
                   "layers_full; fractions of the measured HBM copy peak", "peak_gbs": peak}
    c0, c2, c3, c4 = (synth.config(i) for i in (0, 2, 3, 4))
    out["cfg0"] = measure_cell(c0, c0.L, dev, sampler, peak, {"workload": c0.name, "note": "L2-resident toy"},
                               decode_steps=32)
    out["cfg2"] = measure_cell(c2.replace(L=4), c2.L, dev, sampler, peak, {"workload": c2.name})
    # cfg3: noise swept at tau = 0.9 (the norm reading of the noise), plus the literal reading where nothing merges
    cells = []
    for sigma in (0.05, 0.15, 0.3):
        cells.append(measure_cell(c3.replace(L=6, sigma=sigma, tau=0.9), c3.L, dev, sampler, peak,
                                  {"workload": c3.name, "sigma": sigma, "tau": 0.9, "noise_reading": "norm"}))
    cells.append(measure_cell(c3.replace(L=2, sigma=0.15, tau=0.9, noise_reading="literal"), c3.L, dev, sampler, peak,
                              {"workload": c3.name, "sigma": 0.15, "tau": 0.9, "noise_reading": "literal (no merge)"},
                              cap_frac=1.0))
    out["cfg3_sigma_sweep"] = cells
    # cfg4: mean chunk length x target reduction, with exact attention over the raw cache on the same inputs
    grid = []
    for mean_len in (8, 32, 128):
        for r in (2, 4, 8):
            wc = c4.replace(L=3, gap=("poisson", float(mean_len)), centroids=("ratio", float(r)))
            rec = measure_cell(wc, c4.L, dev, sampler, peak,
                               {"workload": c4.name, "mean_chunk_len": mean_len, "target_reduction": r}, raw=True,
                               cap_frac=1.0 if r == 2 else 0.5)
            best = (mean_len + 1) / 2.0     # one core per chunk plus its delimiter
            rec["reachable"] = r <= best
            if not rec["reachable"]:
                rec["note"] = f"unreachable: at best {best:.1f}x (one core per chunk plus the delimiter)"
            grid.append(rec)
    out["cfg4_grid"] = grid
    return out


def measure_append(pipe, m: int = 256, layers: int = 4):
    """sc_append behind the compressed prompt (outside the timed step; it changes the caches, so it runs
    last): m generated tokens into the first few layers.  Device time per call comes from one CUDA graph
    holding all m x layers calls (replayed once to warm up, once timed: the stream is appended twice more);
    calls launched one by one from Python are bound by the host and only show what finishing a chunk adds."""
    b, w, dev = pipe.b, pipe.w, pipe.dev
    layers = min(layers, w.L)
    i32 = dict(dtype=torch.int32, device=dev)
    status = torch.zeros(1, **i32)
    plain, closing, calls = [], [], []
    for layer in range(layers):
        ids, K, V = synth.generated_stream(w, m, layer)
        ids, K, V = ids.to(dev), K.to(dev), V.to(dev)
        lay = pipe.layers[layer]
        tail, alen = torch.zeros((w.B, w.Hkv), **i32), torch.zeros((w.B, w.Hkv), **i32)
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(m)]
        before = []
        for t in range(m):
            args_t = (K[:, :, t].contiguous(), V[:, :, t].contiguous(), ids[:, t].contiguous(), w.delims, w.max_chunk_len,
                      w.tau, lay.core_k, lay.core_v, lay.count, lay.core_len, tail, alen, status)
            calls.append(args_t)
            before.append(tail.clone())
            ev[t][0].record()
            b.sc_append(*args_t)
            ev[t][1].record()
        torch.cuda.synchronize()
        before.append(tail.clone())
        for t in range(8, m):   # the first calls warm up
            shrank = bool((before[t + 1] < before[t]).any())   # some sequence's open chunk was finished by this call
            (closing if shrank else plain).append(ev[t][0].elapsed_time(ev[t][1]) * 1e3)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for args_t in calls:
            b.sc_append(*args_t)
    g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    g.replay()
    e1.record()
    torch.cuda.synchronize()
    b.check_status(status, "sc_append")
    # every layer of a token in one launch (sc_append_layers): all of the workload's layers, the same stream
    med = lambda a: float(np.median(a)) if a else None
    Lall = w.L
    gids, gK, gV = synth.generated_stream(w, m, 0)
    gids, gK, gV = gids.to(dev), gK.to(dev), gV.to(dev)
    k_new = torch.zeros((w.B, w.Hkv, w.d), dtype=gK.dtype, device=dev)
    v_new = torch.zeros_like(k_new)
    tok = torch.zeros(w.B, **i32)
    tails = [torch.zeros((w.B, w.Hkv), **i32) for _ in range(Lall)]
    alens = [torch.zeros((w.B, w.Hkv), **i32) for _ in range(Lall)]
    pipe.run_compress()        # every layer starts from its compressed prompt again (rows behind core_len are free)
    torch.cuda.synchronize()
    table = b.append_table([(k_new, v_new, pipe.layers[l].core_k, pipe.layers[l].core_v, pipe.layers[l].count,
                             pipe.layers[l].core_len, tails[l], alens[l]) for l in range(Lall)])
    gb = torch.cuda.CUDAGraph()
    steps_b = min(m, 64)       # stays far below the free rows of every head
    with torch.cuda.graph(gb):
        for t in range(steps_b):
            k_new.copy_(gK[:, :, t]); v_new.copy_(gV[:, :, t]); tok.copy_(gids[:, t])
            b.sc_append_layers(table, k_new, tok, w.delims, w.max_chunk_len, w.tau, pipe.cap, status)
    gb.replay()
    torch.cuda.synchronize()
    e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2.record(); gb.replay(); e3.record()
    torch.cuda.synchronize()
    gc = torch.cuda.CUDAGraph()    # the three small copies alone, to take them out of the figure
    with torch.cuda.graph(gc):
        for t in range(steps_b):
            k_new.copy_(gK[:, :, t]); v_new.copy_(gV[:, :, t]); tok.copy_(gids[:, t])
    gc.replay()
    e4, e5 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e4.record(); gc.replay(); e5.record()
    torch.cuda.synchronize()
    b.check_status(status, "sc_append_layers")
    batched_us = (e2.elapsed_time(e3) - e4.elapsed_time(e5)) * 1e3 / steps_b
    return {"what": "sc_append: one call per layer and generated token; sc_append_layers: one call per generated token",
            "all_layers_one_launch": {"layers": Lall, "us_per_token_device": batched_us,
                                      "note": "CUDA graph of 64 tokens, the three staging copies per token timed alone and subtracted"},
            "tokens": m, "layers": layers, "us_per_call_device": e0.elapsed_time(e1) * 1e3 / len(calls),
            "calls_finishing_a_chunk_fraction": len(closing) / max(len(closing) + len(plain), 1),
            "host_bound_us_per_call_storing": med(plain), "host_bound_us_per_call_finishing_a_chunk": med(closing)}


def run_e2e(pipe, args, barrier, g_decode):
    """Same step with inputs in pinned HOST memory: H2D of ids/K/V/q and D2H of the outputs timed."""
    w, dev = pipe.w, pipe.dev
    steps = max(1, min(args.steps, args.e2e_steps))
    host_ids = pipe.ids.pin_memory()
    host_K = [k.cpu().pin_memory() for k in pipe.K]
    host_V = [v.cpu().pin_memory() for v in pipe.V]
    host_q = pipe.q.cpu().pin_memory()
    host_out = torch.empty(pipe.out.shape, dtype=pipe.out.dtype).pin_memory()
    host_len = torch.empty((w.L, w.B, w.Hkv), dtype=torch.int32).pin_memory()
    h2d = host_ids.numel() * 4 + sum(k.numel() * k.element_size() * 2 for k in host_K) + host_q.numel() * host_q.element_size()
    d2h = host_out.numel() * host_out.element_size() + host_len.numel() * 4

    # The copies run on a stream of their own: a layer is compressed as soon as its K and V have landed, and the
    # next step's copies may start once this step's compress launches have read their inputs (they overlap
    # this step's decode, which touches neither).
    b, main, cs = pipe.b, torch.cuda.current_stream(), torch.cuda.Stream()
    ev_ids, ev_done = torch.cuda.Event(), torch.cuda.Event()
    ev_layer = [torch.cuda.Event() for _ in range(w.L)]
    p = pipe.plan

    def step():
        cs.wait_event(ev_done)
        with torch.cuda.stream(cs):
            pipe.ids_dev.copy_(host_ids, non_blocking=True)
            ev_ids.record(cs)
            for l in range(w.L):
                pipe.K[l].copy_(host_K[l], non_blocking=True)
                pipe.V[l].copy_(host_V[l], non_blocking=True)
                ev_layer[l].record(cs)
        main.wait_event(ev_ids)
        b.sc_chunk(pipe.ids_dev, w.delims, w.max_chunk_len, p.seg_off, p.seq_seg_off, p.n_seg, p.tile_seg,
                   p.seq_tile_cnt, pipe._chunk_ws, p.status)
        for l in range(w.L):
            main.wait_event(ev_layer[l])
            ly = pipe.layers[l]
            b.sc_compress(pipe.K[l], pipe.V[l], p, w.tau, ly.core_k, ly.core_v, ly.count, ly.core_len, None,
                          pipe.cws[l], pipe.cstatus[l], 0)
        ev_done.record(main)
        pipe.q.copy_(host_q, non_blocking=True)
        g_decode.replay()
        host_out.copy_(pipe.out, non_blocking=True)
        for l in range(w.L):
            host_len[l].copy_(pipe.layers[l].core_len, non_blocking=True)

    step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    return {"value": w.B * w.decode_steps * steps * args.gpus / (ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "steps": steps, "ms_per_step": ms / steps, "_ms": ms, "_steps": steps,
            "overlap": "copy stream: a layer is compressed when its K/V have landed; the next step's copies overlap this step's decode"}


# -------------------------------------------------------------------------- oracle (cpu) arm


def oracle_sample(w: synth.Workload, n_decode: int = 2, layers=(0,)):
    """Time the oracle on some layers of the workload: compress each once, then n_decode decode steps on it.

    Returns (seconds for chunk+compress of one layer, seconds per one-layer decode step), means over the layers."""
    import oracle
    ids, run_id, run_lens = synth.token_ids(w)
    t_c = t_d = 0.0
    for l in layers:
        K, V = synth.layer_kv(w, l, run_id, run_lens)
        Kb, Vb = synth.to_numpy_bits(K), synth.to_numpy_bits(V)
        t0 = time.perf_counter()
        r = oracle.compress(ids.numpy(), w.delims, Kb, Vb, w.tau, w.max_chunk_len, cap=w.n)
        t_c += time.perf_counter() - t0
        for s in range(n_decode):
            q = synth.to_numpy_bits(synth.queries(w, s, l))
            t0 = time.perf_counter()
            oracle.attn(q, r["core_k"], r["core_v"], r["count"], r["core_len"])
            t_d += time.perf_counter() - t0
    return t_c / len(layers), t_d / (n_decode * len(layers))


def cpu_baseline(w: synth.Workload, budget_s: float = 20.0):
    """The oracle, as it stands, on a bounded sample of the workload: about budget_s / 2 seconds of timed CPU work
    (a quick probe sizes the sample: as many layers and decode steps as fit), scaled linearly to the full step."""
    import oracle
    # shrink the batch so the sample stays bounded; the per-sequence cost is what gets scaled
    ws = w.replace(B=1) if w.B > 1 else w
    p_c, p_d = oracle_sample(ws, n_decode=1)
    n_layers = int(min(ws.L, 8, max(1, 0.25 * budget_s / max(p_c, 1e-6))))   # generating a layer's inputs is not free
    n_decode = int(min(ws.decode_steps, max(2, 0.5 * budget_s / max(n_layers * p_d, 1e-6))))
    t_c, t_d = oracle_sample(ws, n_decode=n_decode, layers=tuple(range(n_layers)))
    step_s = w.B * (w.L * t_c + w.decode_steps * w.L * t_d)
    threads = oracle.num_threads()
    # the oracle's loops run in parallel over (sequence, KV head) for chunk/GSC/merge and over (sequence, query
    # head) for attention: no more threads than that have work on the one-sequence sample
    busy_c, busy_a = min(threads, ws.B * ws.Hkv), min(threads, ws.B * ws.Hq)
    return {"value": w.B * w.decode_steps / step_s, "unit": UNIT, "cores": max(busy_c, busy_a), "kind": "oracle",
            "threads_available": threads, "cores_with_work": {"chunk_gsc_merge": busy_c, "attention": busy_a},
            "sample": f"layers 0..{n_layers - 1} of {w.L}, sequence 0 of {w.B}: chunk+GSC+merge of each layer "
                      f"({t_c:.2f} s per layer) and {n_decode} of {w.decode_steps} decode steps on each "
                      f"({t_d * 1e3:.1f} ms per layer and step): {n_layers * (t_c + n_decode * t_d):.1f} s of timed CPU "
                      "work, scaled linearly to the full step",
            "compress_s_per_layer": t_c, "decode_s_per_layer_step": t_d}


def run_reference(args):
    rank = int(os.environ.get("RANK", 0))
    if rank != 0:
        return
    import oracle
    oracle.build()
    w = synth.config(args.config)
    if args.decode_steps:
        w = w.replace(decode_steps=args.decode_steps)
    ws = w.replace(B=1) if w.B > 1 else w
    times = []
    for i in range(args.warmup + args.steps):
        t_c, t_d = oracle_sample(ws, n_decode=1)
        if i >= args.warmup:
            times.append(w.B * (w.L * t_c + w.decode_steps * w.L * t_d))
    step_s = sum(times) / len(times)
    value = w.B * w.decode_steps / step_s
    sample = (f"each step times layer 0 of {w.L}, sequence 0 of {w.B} (chunk+GSC+merge, then 1 of {w.decode_steps} "
              "decode steps) and scales linearly to the full step")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": step_s * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "n_ctx": w.n, "layers": w.L, "kv_heads": w.Hkv, "q_heads": w.Hq,
                   "head_dim": w.d, "tau": w.tau, "decode_steps": w.decode_steps},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": min(oracle.num_threads(), ws.B * ws.Hq), "kind": "oracle",
                         "threads_available": oracle.num_threads(), "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=1, help="workload 0..4 (1 = Llama-3-8B, 32K context, batch 1)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--decode-steps", type=int, default=0, help="override the workload's decode steps per step")
    ap.add_argument("--layers", type=int, default=0, help="override the number of layers (small profiling cases)")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-overlap", action="store_true", help="time the step with plain stream-ordered decode launches")
    ap.add_argument("--no-modes", action="store_true", help="skip the side measurements of the other decode launch modes")
    ap.add_argument("--no-append", action="store_true", help="skip the sc_append side measurement")
    ap.add_argument("--per-layer-compress", action="store_true",
                    help="time the step with one sc_compress per layer instead of one sc_compress_layers for all")
    ap.add_argument("--no-sweep", action="store_true", help="skip the short passes over the other workloads and sweeps")
    ap.add_argument("--extras-only", action="store_true",
                    help="run only the measurements of sc_prefill_attn, the ablation arms and the budget search (a small case for profiling)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-budget", type=float, default=20.0)
    ap.add_argument("--traffic", type=float, default=None,
                    help="DRAM bytes per decode launch from an ncu capture (see profiles/)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.extras_only:
        from paper_2603_14303_b200 import build
        build.build()
        dev = torch.device("cuda:0")
        torch.cuda.set_device(dev)
        sampler = ClockSampler(0)
        sampler.start()
        extras = measure_extras(dev, sampler, measured_peaks()[0])
        sampler.stop()
        print(json.dumps({"extras": extras}))
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
