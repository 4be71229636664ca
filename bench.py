#!/usr/bin/env python
"""Benchmark of the SemantiCache hot path on B200.

One *step* = one pass of the whole path over one synthetic batch: sc_chunk once, sc_compress for
every layer, then ``decode_steps`` decode steps of sc_decode_attn over every layer's cores.
Reported ``value`` = decoded tokens per second over the whole step (compress included); the
decode-only rate, the compress time per 32K context and the achieved HBM bandwidth of both
stages are added as extra keys.  Everything is launched through the C-ABI library; the launch
sequence is captured into CUDA graphs so Python is not on the timed path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config I] [--impl ours|reference]

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

# DRAM bytes (read + write) per launch from the ncu captures summarised under profiles/, by workload:
# sc_decode_attn (decode_mma_kernel_cfg1_8layers.md) and sc_compress (compress_fused_kernel_cfg1_8layers.md).
# Only valid while those kernels are the ones that were captured; other workloads report null.
NCU_TRAFFIC = {"cfg1-llama3-8b-32k": {"decode": 34.31e6, "compress": 153.7e6}}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

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
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        self.thread.join(timeout=2)
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            p = [x.strip() for x in ln.split(",")]
            if len(p) < 7:
                continue
            try:
                sm.append(float(p[0])); smax.append(float(p[1]))
            except ValueError:
                continue
            for nm, v in zip(names, p[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------- ours


class Pipeline:
    """Device-resident state of one rank: inputs, plan, cores, and the captured launch graphs."""

    def __init__(self, w: synth.Workload, device, cap_frac: float = 0.5):
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
        # one workspace per layer (both stages): consecutive layer launches overlap and must not share scratch
        self.cws = [binding.compress_workspace(w.B, w.Hkv, w.n, device) for _ in range(w.L)]
        self.dws = [binding.decode_workspace(w.B, w.Hq, w.Hkv, w.d, self.cap, device) for _ in range(w.L)]
        self.q = torch.stack([torch.stack([synth.queries(w, s, l, device) for l in range(w.L)])
                              for s in range(w.decode_steps)])            # [steps, L, B, Hq, d]
        self.out = torch.empty_like(self.q)
        self.plan = None
        self.decode_flags = 0
        self.compress_flags = 0
        self.status = torch.zeros((w.L, 1), **i32)
        self.cstatus = torch.zeros((w.L, 1), **i32)
        self.launches_compress = self.launches_decode = 0
        self.g_compress = self.g_decode = None

    # the launch sequences (also what the graphs capture)
    def run_compress(self):
        b, w = self.b, self.w
        if self.plan is None:
            self.plan = b.chunk(self.ids_dev, w.delims, w.max_chunk_len)
            self._chunk_ws = torch.empty(b.lib().sc_chunk_workspace_bytes(w.B, w.n), dtype=torch.uint8, device=self.dev)
        else:
            p = self.plan
            b.sc_chunk(self.ids_dev, w.delims, w.max_chunk_len, p.seg_off, p.seq_seg_off, p.n_seg, p.tile_seg,
                       p.seq_tile_cnt, self._chunk_ws, p.status)
        for l in range(w.L):
            # layer 0 follows sc_chunk and needs its plan; the other layers share nothing they write with
            # their predecessor (own K/V, cores, workspace, status) and may overlap its tail
            ly = self.layers[l]
            b.sc_compress(self.K[l], self.V[l], self.plan, w.tau, ly.core_k, ly.core_v, ly.count, ly.core_len, None,
                          self.cws[l], self.cstatus[l], self.compress_flags if l > 0 else 0)

    def run_decode(self):
        b, w = self.b, self.w
        for s in range(w.decode_steps):
            for l in range(w.L):
                # layer 0 of each step is an ordinary launch (ordered after all earlier work); the other
                # layers share no buffer with their predecessor and may overlap it
                b.decode_attn(self.q[s, l], self.layers[l], out=self.out[s, l], workspace=self.dws[l],
                              status=self.status[l], flags=self.decode_flags if l > 0 else 0)

    def capture(self):
        self.run_compress()   # allocates the plan outside capture
        self.run_decode()
        torch.cuda.synchronize(self.dev)
        self.b.check_status(self.plan.status, "warm-up pass")
        if int(self.cstatus.abs().max().item()) != 0:
            raise RuntimeError("sc_compress reported a device-side error in the warm-up pass")
        self.g_compress, self.g_decode = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
        c0 = self.b.launch_counter()
        with torch.cuda.graph(self.g_compress):
            self.run_compress()
        c1 = self.b.launch_counter()
        with torch.cuda.graph(self.g_decode):
            self.run_decode()
        self.launches_compress, self.launches_decode = c1 - c0, self.b.launch_counter() - c1
        torch.cuda.synchronize(self.dev)

    def algorithmic_bytes(self):
        """(compress bytes per step, decode bytes per decode step over all layers, per-layer list)."""
        w = self.w
        esz = self.K[0].element_size()
        lens = torch.stack([ly.core_len for ly in self.layers]).to(torch.int64).cpu()   # [L, B, Hkv]
        rows = lens.sum().item()
        kv_in = w.L * w.B * w.Hkv * w.n * w.d * esz * 2
        core_bytes = rows * (2 * w.d * esz + 4)
        qo = w.L * w.B * w.Hq * w.d * esz * 2
        per_layer = [(lens[l].sum().item() * (2 * w.d * esz + 4) + qo // w.L) for l in range(w.L)]
        return kv_in + core_bytes, core_bytes + qo, per_layer, rows / (w.L * w.B * w.Hkv * w.n)


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
    # the per-layer decode calls of a step are independent (own q, out, workspace): let them overlap
    pipe.decode_flags = 0 if args.no_overlap else binding.SC_FLAG_OVERLAP_PREV
    # sc_compress also takes the flag, but overlapping consecutive layers gains 2 % on cfg1 and loses a factor
    # of two on cfg3 (4 KV heads, 128K tokens): its layers are launched the ordinary way
    pipe.compress_flags = 0
    pipe.capture()
    cbytes, dbytes, per_layer, kept = pipe.algorithmic_bytes()

    def barrier():
        scdist.barrier(dev)

    def one_step():
        pipe.g_compress.replay()
        pipe.g_decode.replay()

    for _ in range(max(args.warmup, 3)):
        one_step()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    barrier()
    t_wall = time.perf_counter()
    for s in range(args.steps):
        ev[s][0].record()
        pipe.g_compress.replay()
        ev[s][1].record()
        pipe.g_decode.replay()
        ev[s][2].record()
    barrier()
    t_wall = time.perf_counter() - t_wall
    clocks = sampler.stop() if rank == 0 else None
    binding.check_status(pipe.plan.status, "timed region")
    if int(pipe.status.abs().max().item()) != 0 or int(pipe.cstatus.abs().max().item()) != 0:
        raise RuntimeError("sc_compress / sc_decode_attn reported a device-side error")
    ms_c = [e[0].elapsed_time(e[1]) for e in ev]
    ms_d = [e[1].elapsed_time(e[2]) for e in ev]
    total_ms = ev[0][0].elapsed_time(ev[-1][2])
    total_ms, sum_c, sum_d = scdist.max_over_ranks([total_ms, sum(ms_c), sum(ms_d)], dev)
    value = scdist.whole_job_rate(w.B * w.decode_steps * args.steps, args.gpus, total_ms)

    # end to end through the public API with HOST buffers (copies inside the timed region)
    e2e = run_e2e(pipe, args, barrier) if not args.no_e2e else None
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
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": total_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "n_ctx": w.n, "layers": w.L, "kv_heads": w.Hkv, "q_heads": w.Hq,
                   "head_dim": w.d, "tau": w.tau, "decode_steps": w.decode_steps, "kept_fraction": round(kept, 4),
                   "l2": "inputs larger than L2 (every step streams all layers)", "launch": "cuda graphs" + ("" if args.no_overlap else "; the independent per-layer decode launches of a step overlap (programmatic stream serialization, no wait)"),
                   "parallelism": f"replicas x{args.gpus}" if distributed else "single gpu"},
        "decode_tokens_per_s": w.B * w.decode_steps * args.gpus / (sum_d / args.steps * 1e-3),
        "decode_bytes_per_step": dbytes,
        "decode_gbs": dbytes * w.decode_steps / (sum_d / args.steps * 1e-3) / 1e9,
        "compress_ms_per_32k_ctx": comp_ms * 32768 / (w.B * w.n),
        "compress_gbs": comp_gbs, "compress_frac_of_peak": comp_gbs / peak,
        "roofline": {"kernel": "sc_decode_attn (one layer per launch)", "bound": "hbm", "achieved": achieved,
                     "peak": peak, "peak_kind": peak_kind, "unit": "GB/s", "frac": achieved / peak,
                     "frac_of_nominal_8tbs": achieved / 8000.0, "bytes_per_launch": layer_bytes,
                     "us_per_launch": dec_launch_us,
                     "traffic": args.traffic if args.traffic is not None else
                     NCU_TRAFFIC.get(w.name, {}).get("decode")},
        "roofline_compress": {"kernel": "sc_compress (one layer per launch)", "bound": "hbm", "achieved": comp_gbs,
                              "peak": peak, "peak_kind": peak_kind, "unit": "GB/s", "frac": comp_gbs / peak,
                              "frac_of_nominal_8tbs": comp_gbs / 8000.0, "bytes_per_launch": cbytes / w.L,
                              "us_per_launch": comp_ms * 1e3 / w.L,
                              "traffic": NCU_TRAFFIC.get(w.name, {}).get("compress")},
        "gpu_launches": args.steps * (pipe.launches_compress + pipe.launches_decode),
        "gpu_launches_per_step": {"chunk+compress": pipe.launches_compress, "decode": pipe.launches_decode},
        "clocks": clocks, "e2e": e2e, "wall_s": t_wall,
    }
    if args.gpus == 1:
        line["append"] = measure_append(pipe)
    if not args.no_cpu_baseline and args.gpus == 1:
        line["cpu_baseline"] = cpu_baseline(w, budget_s=args.cpu_budget)
    print(json.dumps(line))


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
    med = lambda a: float(np.median(a)) if a else None
    return {"what": "sc_append: one call per layer and generated token",
            "tokens": m, "layers": layers, "us_per_call_device": e0.elapsed_time(e1) * 1e3 / len(calls),
            "calls_finishing_a_chunk_fraction": len(closing) / max(len(closing) + len(plain), 1),
            "host_bound_us_per_call_storing": med(plain), "host_bound_us_per_call_finishing_a_chunk": med(closing)}


def run_e2e(pipe, args, barrier):
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
        pipe.g_decode.replay()
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


def oracle_sample(w: synth.Workload, n_decode: int = 2):
    """Time the oracle on layer 0 of the workload: compress once, n_decode decode steps.

    Returns (seconds for chunk+compress of one layer, seconds per one-layer decode step)."""
    import oracle
    ids, run_id, run_lens = synth.token_ids(w)
    K, V = synth.layer_kv(w, 0, run_id, run_lens)
    Kb, Vb = synth.to_numpy_bits(K), synth.to_numpy_bits(V)
    t0 = time.perf_counter()
    r = oracle.compress(ids.numpy(), w.delims, Kb, Vb, w.tau, w.max_chunk_len, cap=w.n)
    t_c = time.perf_counter() - t0
    t_d = 0.0
    for s in range(n_decode):
        q = synth.to_numpy_bits(synth.queries(w, s, 0))
        t0 = time.perf_counter()
        oracle.attn(q, r["core_k"], r["core_v"], r["count"], r["core_len"])
        t_d += time.perf_counter() - t0
    return t_c, t_d / n_decode


def cpu_baseline(w: synth.Workload, budget_s: float = 20.0):
    import oracle
    # shrink the batch so the sample stays bounded; the per-sequence cost is what gets scaled
    ws = w.replace(B=1) if w.B > 1 else w
    t_c, t_d = oracle_sample(ws, n_decode=2)
    del budget_s
    step_s = w.B * (w.L * t_c + w.decode_steps * w.L * t_d)
    return {"value": w.B * w.decode_steps / step_s, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"layer 0 of {w.L}, sequence 0 of {w.B}: chunk+GSC+merge once ({t_c:.2f} s) and 2 of "
                      f"{w.decode_steps} decode steps ({t_d * 1e3:.1f} ms each), scaled linearly to the full step",
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
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
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
    ap.add_argument("--no-overlap", action="store_true", help="plain launches (no programmatic dependent launch)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-budget", type=float, default=20.0)
    ap.add_argument("--traffic", type=float, default=None,
                    help="DRAM bytes per decode launch from an ncu capture (see profiles/)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
