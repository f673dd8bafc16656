#!/usr/bin/env python
"""Benchmark of the token-pruned prefill on the Llama-2-7B shape.

One "step" = one whole prefill (every layer, every pruning point, first-token logits) of one
3376-token synthetic prompt with cumulative keep 100/70/50/30 % entering layers 0/8/16/24.
Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle on a bounded sample of the
same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

N_PROMPT = 3376
METRIC = "prefill tokens/s (TTFT), 7B-shape 3376-token prompt, token-pruned"
UNIT = "tokens/s"
WORKLOAD = ("llama2-7b-shape prefill (32 layers, d=4096, 32x128 heads, ffn 11008, vocab 32000), batch 1, "
            "3376-token prompt, keep 100/70/50/30% entering layers 0/8/16/24")


# DRAM traffic of the dominant kernel comes from the committed ncu capture: the data file beside its
# summary holds the mean of dram__bytes_read.sum + dram__bytes_write.sum over the four GEMM launches of one
# layer and the hash of the kernel sources it was taken on.  It is reported only while those sources are
# unchanged.
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "gemm_bf16_tcgen05_2layer_3376.traffic.json")
GEMM_SOURCES = ("gemm_tcgen05.cu", "gemm_tcgen05_pair.cu", "gemm_epilogue.cuh", "tc_common.cuh", "tc_pair.cuh")


def _gemm_source_sha16():
    import hashlib
    h = hashlib.sha256()
    for name in GEMM_SOURCES:
        with open(os.path.join(ROOT, "paper_2407_14057_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def _gemm_traffic():
    """DRAM bytes per GEMM launch from the committed ncu capture, or None once the kernels' sources changed."""
    try:
        with open(TRAFFIC_FILE) as f:
            rec = json.load(f)
        return float(rec["dram_bytes_per_launch"]) if rec["source_sha16"] == _gemm_source_sha16() else None
    except (OSError, KeyError, ValueError):
        return None


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        self.t.join(timeout=2)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except Exception:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------ CPU oracle leg
def _rows_per_layer(n_layers, schedule, n):
    """(rows in attention, rows in MLP) of every layer under a schedule of (layer_entered, bp)."""
    pts = dict(schedule)
    rows, out = n, []
    for l in range(n_layers):
        n_attn = rows
        if (l + 1) in pts:
            rows = max(1, min(rows, (n * pts[l + 1] + 9999) // 10000))
        out.append((n_attn, rows))
    return out


def _algorithmic_flops(shape, schedule, n):
    d, F = shape.d_model, shape.d_ffn
    tot = 0.0
    for n_attn, n_mlp in _rows_per_layer(shape.n_layers, schedule, n):
        tot += n_attn * (2.0 * 3 * d * d + 2.0 * d * d) + 2.0 * d * n_attn * (n_attn + 1.0) + n_mlp * 6.0 * d * F
    return tot + 2.0 * d * shape.vocab


class OracleSample:
    """The CPU oracle on a bounded sample of the workload: a shallow stack of the 7B widths that
    visits the same row counts (4 layers, cuts entering layers 1/2/3: 3376/2364/1688/1013 rows; or
    2 layers, 3376 -> 1013 rows, when many steps are asked for).  The whole-prompt time is taken as
    the sample's time scaled by the ratio of algorithmic FLOPs (32-layer workload / sample)."""

    def __init__(self, n_prompt: int, small: bool):
        import torch  # noqa: F401
        sys.path.insert(0, os.path.join(ROOT, "oracle"))
        import lazyllm_oracle as O
        from paper_2407_14057_b200 import synth
        self.O = O
        self.n = n_prompt
        if small:
            self.shape, self.schedule = synth.LLAMA7B.with_layers(2), ((1, 3000),)
        else:
            self.shape, self.schedule = synth.LLAMA7B.with_layers(4), ((1, 7000), (2, 5000), (3, 3000))
        W = synth.make_weights(self.shape, 0, bf16=True)
        self.W = {k: v.float().numpy() for k, v in W.items() if k != "layers"}
        self.W["layers"] = [{k: v.float().numpy() for k, v in lw.items()} for lw in W["layers"]]
        self.ids = synth.make_prompt(self.shape.vocab, n_prompt, 1).numpy()
        self.scale = (_algorithmic_flops(synth.LLAMA7B, synth.SCHEDULE_7B, n_prompt)
                      / _algorithmic_flops(self.shape, self.schedule, n_prompt))
        self.cores = _host_cores()
        rows = "/".join(str(r) for r, _ in _rows_per_layer(self.shape.n_layers, self.schedule, n_prompt))
        self.sample = (f"{self.shape.n_layers} of 32 layers at 7B widths, one layer per visited segment "
                       f"({rows} rows), fp64 numpy oracle; whole-prompt time = sample time x "
                       f"{self.scale:.2f} (ratio of algorithmic FLOPs)")

    def step_seconds(self) -> float:
        t0 = time.perf_counter()
        self.O.prefill(self.shape, self.W, self.ids, self.schedule, keep_records=False)
        return (time.perf_counter() - t0) * self.scale


class _LayerView:
    """Per-layer weights handed to the oracle one layer at a time (fp32 numpy copies of the bf16
    tensors, made when the layer is asked for), so that the 13.5 GB model is never widened at once."""

    def __init__(self, layers):
        self.layers = layers

    def __len__(self):
        return len(self.layers)

    def __getitem__(self, l):
        return {k: v.float().cpu().numpy() for k, v in self.layers[l].items()}


def oracle_whole_prompt_seconds(shape, schedule, W, ids):
    """Wall-clock of the CPU oracle's `prefill` on the WHOLE workload (all layers, the full prompt), as it
    stands.  W: the torch weights (any device); ids: torch int32 [N]."""
    sys.path.insert(0, os.path.join(ROOT, "oracle"))
    import lazyllm_oracle as O
    Wn = {k: v.float().cpu().numpy() for k, v in W.items() if k != "layers"}
    Wn["layers"] = _LayerView(W["layers"])
    t0 = time.perf_counter()
    O.prefill(shape, Wn, ids.cpu().numpy(), schedule, keep_records=False)
    return time.perf_counter() - t0


def _host_cores():
    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else os.cpu_count()
    try:
        from threadpoolctl import threadpool_info
        nt = [p.get("num_threads") for p in threadpool_info() if p.get("user_api") == "blas"]
        if nt:
            cores = min(cores, max(nt))
    except Exception:
        pass
    return cores


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2407_14057_b200 import synth
    config = {"workload": WORKLOAD, "batch": 1, "seq_len": args.prompt, "parallelism": "single",
              "l2": "inputs (13.5 GB of weights) larger than L2"}
    if args.steps + args.warmup <= 2:
        # few enough steps for the whole workload: every step is one full 32-layer oracle prefill
        shape, schedule = synth.LLAMA7B, synth.SCHEDULE_7B
        W = synth.make_weights(shape, 2, bf16=True)
        ids = synth.make_prompt(shape.vocab, args.prompt, 100)
        times = [oracle_whole_prompt_seconds(shape, schedule, W, ids) for _ in range(args.warmup + args.steps)]
        times = times[args.warmup:]
        step_ms = whole_ms = 1e3 * sum(times) / len(times)
        sample, cores = "the whole workload: all 32 layers, the full prompt (no extrapolation)", _host_cores()
    else:
        # a step is the bounded sample (a shallow stack of the 7B widths visiting the same row counts);
        # ms_per_step is what a step really took, the whole-prompt figure is that time x the FLOP ratio
        smp = OracleSample(args.prompt, small=(args.steps + args.warmup) > 13)
        times = []
        for i in range(args.warmup + args.steps):
            dt = smp.step_seconds()
            if i >= args.warmup:
                times.append(dt)
        whole_ms = 1e3 * sum(times) / len(times)
        step_ms = whole_ms / smp.scale
        sample, cores = smp.sample, smp.cores
    value = args.prompt / (whole_ms / 1e3)
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_ms,
           "ms_per_whole_prompt": whole_ms, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": config,
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out), flush=True)


# ------------------------------------------------------------------------------------------ replicas
def max_over_ranks(ms: float, world: int, device: str) -> float:
    """Replicas only: no collective touches the data path; the one reduction is this MAX of the
    per-rank step times, so that the whole job is charged with its slowest replica."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(tokens_per_replica: int, world: int, ms: float) -> float:
    """Aggregate throughput of `world` independent replicas that each process their own prompt."""
    return world * tokens_per_replica / (ms * 1e-3)


# ------------------------------------------------------------------------------------------ GPU leg
def run_gpu(args):
    import torch
    import torch.distributed as dist
    from paper_2407_14057_b200 import binding as B
    from paper_2407_14057_b200 import build, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    B.lib()
    peaks = _peaks()

    shape = synth.LLAMA7B
    if args.layers:
        shape = shape.with_layers(args.layers)
    schedule = synth.SCHEDULE_7B if shape.n_layers == 32 else synth.scaled_schedule(shape.n_layers)
    n = args.prompt
    # Replicas only: every rank holds all weights and its own prompt; there is no collective.
    W = synth.make_weights(shape, 2, bf16=True, device="cuda")
    ids_host = synth.make_prompt(shape.vocab, n, 100 + rank).pin_memory()
    ids = ids_host.cuda()
    logits = torch.empty((1, shape.vocab), dtype=torch.float32, device="cuda")
    logits_host = torch.empty((1, shape.vocab), dtype=torch.float32).pin_memory()
    eng = B.LazyPrefill(shape, W, schedule, torch.bfloat16, 1, n)
    full = B.LazyPrefill(shape, W, (), torch.bfloat16, 1, n)
    cu = [0, n]

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(engine, steps, warmup, timing=False, kinds=None):
        for _ in range(warmup):
            engine.lazy_prefill_run(ids, cu, logits)
        engine.lazy_sync_status()
        engine.lazy_set_kernel_timing(timing, kinds)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        per_kind = None
        events = []
        e0.record()
        for _ in range(steps):
            engine.lazy_prefill_run(ids, cu, logits)
            if timing:   # event pairs belong to one run: collect them before the next one reuses them
                kt = engine.lazy_get_kernel_times()
                events.extend(engine.lazy_get_kernel_events())
                if per_kind is None:
                    per_kind = {k: dict(v) for k, v in kt.items()}
                else:
                    for k, v in kt.items():
                        for f in ("ms", "launches", "flops", "bytes"):
                            per_kind[k][f] += v[f]
        e1.record()
        barrier()
        engine.lazy_sync_status()
        engine.lazy_set_kernel_timing(False)
        ms = max_over_ranks(e0.elapsed_time(e1) / steps, world, "cuda")
        return (ms, per_kind, events) if timing else (ms, per_kind)

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ms_pruned, _ = timed(eng, args.steps, args.warmup)
    clocks = sampler.stop() if rank == 0 else None
    launches = eng.lazy_get_stats().kernel_launches * args.steps
    ms_full, _ = timed(full, max(2, args.steps // 2), 2)
    # per-kernel device times: a separate pass with every launch bracketed by events on the same stream
    ksteps = max(2, min(5, args.steps))
    _, kinds, _ = timed(eng, ksteps, 1, timing=True)
    # the dominant kernel alone: event pairs around the 128 GEMM launches only, so that the events of
    # the ~350 small kernels do not stretch the step the GEMMs are timed in
    GEMM_KINDS = ["gemm_qkv", "gemm_o", "gemm_gate_up", "gemm_down"]
    _, gkinds, gevents = timed(eng, ksteps, 1, timing=True, kinds=GEMM_KINDS + ["attention"])

    # end to end through the public call with host buffers: pinned ids in, logits out, every step
    def e2e_step():
        ids.copy_(ids_host, non_blocking=True)
        eng.lazy_prefill_run(ids, cu, logits)
        logits_host.copy_(logits, non_blocking=True)
        torch.cuda.current_stream().synchronize()
    for _ in range(2):
        e2e_step()
    barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        e2e_step()
    barrier()
    e2e_ms = (time.perf_counter() - t0) * 1e3 / args.steps
    e2e_ms = max_over_ranks(e2e_ms, world, "cuda")
    eng.lazy_sync_status()

    # the same two schedules with the projections on e4m3 operands (reported beside the 16-bit line, which stays
    # the headline: the metric's dtype is bf16).  The 16-bit weights are replaced by the de-quantised e4m3
    # values first, so this leg runs last.
    fp8 = None
    if not args.no_fp8 and shape.n_layers == 32:
        q8 = synth.quantize_projections_e4m3(W)
        for e_ in (eng, full):
            e_.lazy_set_fp8_weights(q8)
        ms8, _ = timed(eng, args.steps, 2)
        ms8_full, _ = timed(full, max(2, args.steps // 2), 2)
        _, k8, _ = timed(eng, ksteps, 1, timing=True, kinds=GEMM_KINDS)
        g8_ms = sum(k8[k]["ms"] for k in GEMM_KINDS) / ksteps
        g8_fl = sum(k8[k]["flops"] for k in GEMM_KINDS) / ksteps
        fp8 = {"what": "QKV / output / gate-up / down projections on e4m3 codes (per-row activation scales, per-matrix "
                       "weight scales, tcgen05 kind::f8f6f4), everything else bf16",
               "ttft_ms_pruned": ms8, "ttft_ms_full_keep": ms8_full, "tokens_per_s": world * n / (ms8 * 1e-3),
               "gemm_ms_per_step": g8_ms, "gemm_tflops": g8_fl / (g8_ms * 1e-3) / 1e12,
               "frac_of_fp8_peak": g8_fl / (g8_ms * 1e-3) / 1e12 / (2.0 * peaks["bf16_tflops_sustained"]),
               "fp8_peak_kind": "2 x the measured sustained bf16 figure (nominal ratio)"}
        for e_ in (eng, full):
            e_.lazy_set_fp8_weights(None)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    gemm = GEMM_KINDS
    g_ms = sum(gkinds[k]["ms"] for k in gemm) / ksteps
    g_fl = sum(gkinds[k]["flops"] for k in gemm) / ksteps
    g_launch = sum(gkinds[k]["launches"] for k in gemm) / ksteps
    achieved = g_fl / (g_ms * 1e-3) / 1e12
    peak = peaks["bf16_tflops_sustained"]
    breakdown = {}
    for k, v in kinds.items():
        if v["launches"] == 0:
            continue
        ms = v["ms"] / ksteps
        ent = {"ms": round(ms, 4), "launches": int(v["launches"] / ksteps)}
        if v["flops"] > 0:
            ent["tflops"] = round(v["flops"] / ksteps / (ms * 1e-3) / 1e12, 1)
        if v["bytes"] > 0:
            ent["gbs"] = round(v["bytes"] / ksteps / (ms * 1e-3) / 1e9, 1)
        breakdown[k] = ent
    # the tensor-core kinds by surviving row count: rows follow from a launch's work (flops per row are fixed
    # per kind; attention: 2 d n (n + 1))
    d_, F_ = shape.d_model, shape.d_ffn
    per_row = {"gemm_qkv": 6.0 * d_ * d_, "gemm_o": 2.0 * d_ * d_, "gemm_gate_up": 4.0 * d_ * F_,
               "gemm_down": 2.0 * d_ * F_}
    by_rows = {}
    for kind, ms_, fl_, _ in gevents:
        rows_ = int(round(fl_ / per_row[kind])) if kind in per_row else int(round(((1 + 2 * fl_ / d_) ** 0.5 - 1) / 2))
        ent = by_rows.setdefault(kind, {}).setdefault(rows_, [0.0, 0.0, 0])
        ent[0] += ms_
        ent[1] += fl_
        ent[2] += 1
    for kind, m in by_rows.items():
        breakdown.setdefault(kind, {})["by_rows"] = {
            str(r): {"us_per_launch": round(v[0] / v[2] * 1e3, 1), "tflops": round(v[1] / (v[0] * 1e-3) / 1e12, 1),
                     "launches": v[2] // ksteps} for r, v in sorted(m.items(), reverse=True)}
    value = whole_job_value(n, world, ms_pruned)
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_pruned, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": WORKLOAD if (shape.n_layers == 32 and n == N_PROMPT) else
                   f"REDUCED (profiling only): {shape.n_layers} layers, {n}-token prompt, schedule {schedule}",
                   "batch": 1, "seq_len": n, "parallelism": "replicas" if world > 1 else "single",
                   "l2": "inputs (13.5 GB of weights) larger than L2"},
        "ttft_ms_pruned": ms_pruned, "ttft_ms_full_keep": ms_full, "pruned_speedup": ms_full / ms_pruned,
        "tokens_per_s_full_keep": world * n / (ms_full * 1e-3),
        "clocks": clocks,
        "e2e": {"value": world * n / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": n * 4, "d2h_bytes_per_step": shape.vocab * 4},
        "gpu_launches": int(launches),
        "roofline": {"bound": "tensor", "kernel": "gemm_bf16_tcgen05_kernel + gemm_bf16_tcgen05_pair_kernel (QKV, O, gate/up+SwiGLU, down)",
                     "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                     "peak_kind": f"sustained bf16, {peaks['source']}", "launches_per_step": g_launch,
                     "ms_per_step": g_ms, "algorithmic_flops_per_launch": g_fl / max(g_launch, 1),
                     "traffic": _gemm_traffic()},
        "kernels": breakdown,
    }
    if fp8:
        out["fp8_projections"] = fp8
    if not args.no_cpu and world == 1:
        # the oracle, as it stands, on the machine's host cores.  By default on the whole workload (one run of
        # all layers over the full prompt: a measurement, a couple of minutes); --cpu-sample times the
        # bounded sample instead (about 15 s) and scales it by the ratio of algorithmic FLOPs.  The sampled
        # estimate is printed beside the measurement either way.
        smp = OracleSample(n, small=False)
        est = smp.step_seconds()
        cb = {"unit": UNIT, "cores": smp.cores, "kind": "oracle", "sampled_estimate_seconds": est,
              "sampled_estimate": smp.sample}
        if args.cpu_sample or shape.n_layers != 32:
            cb.update({"value": n / est, "sample": smp.sample, "whole_prompt_seconds": est})
        else:
            del smp
            dt = oracle_whole_prompt_seconds(shape, schedule, W, ids_host)
            cb.update({"value": n / dt, "whole_prompt_seconds": dt,
                       "sample": "the whole workload, once: all 32 layers, the full prompt (no extrapolation)"})
        out["cpu_baseline"] = cb
    print(json.dumps(out), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_sweep(args):
    """Timing side of the single-pruning-layer study (Section 4.4): one cut, swept over its location
    and the fraction kept, plus the "static pruning" point (one early cut) and the progressive
    schedule.  Prints one JSON object; accuracy needs the datasets and is out of scope."""
    import torch
    from paper_2407_14057_b200 import binding as B
    from paper_2407_14057_b200 import build, synth
    torch.cuda.set_device(0)
    build.build()
    B.lib()
    shape, n = synth.LLAMA7B, args.prompt
    W = synth.make_weights(shape, 2, bf16=True, device="cuda")
    ids = synth.make_prompt(shape.vocab, n, 100).cuda()
    logits = torch.empty((1, shape.vocab), dtype=torch.float32, device="cuda")

    def ttft(schedule):
        eng = B.LazyPrefill(shape, W, schedule, torch.bfloat16, 1, n)
        for _ in range(3):
            eng.lazy_prefill_run(ids, [0, n], logits)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            eng.lazy_prefill_run(ids, [0, n], logits)
        e1.record()
        torch.cuda.synchronize()
        eng.lazy_sync_status()
        st = eng.lazy_get_stats()
        rows = [st.rows_computed[l] for l in range(shape.n_layers)]
        eng.close()
        return e0.elapsed_time(e1) / args.steps, 100.0 * sum(rows) / (n * shape.n_layers)

    base, _ = ttft(())
    out = {"workload": f"llama2-7b shape, {n}-token prompt, bf16, 1 GPU", "ttft_ms_full_keep": round(base, 3),
           "single_cut": [], "schedules": {}}
    for layer in (4, 8, 12, 16, 20, 24, 28):
        for keep in (9000, 7000, 5000, 3000, 1000):
            ms, pct = ttft(((layer, keep),))
            out["single_cut"].append({"layer_entered": layer, "keep_pct": keep // 100, "ttft_ms": round(ms, 3),
                                      "speedup": round(base / ms, 3), "token_layers_computed_pct": round(pct, 2)})
    for name, sched in (("progressive 100/70/50/30 @ 0/8/16/24", synth.SCHEDULE_7B),
                        ("static: one cut entering layer 2, keep 50%", ((2, 5000),))):
        ms, pct = ttft(sched)
        out["schedules"][name] = {"ttft_ms": round(ms, 3), "speedup": round(base / ms, 3),
                                  "token_layers_computed_pct": round(pct, 2)}
    print(json.dumps(out), flush=True)


def _event_ms(fn, iters, warmup):
    """Mean device time of fn(i) over `iters` calls after `warmup` calls (CUDA events on the current stream)."""
    import torch
    for i in range(warmup):
        fn(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(iters):
        fn(warmup + i)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def run_other_workload(args):
    """The configurations beside the bench line (prompt + greedy decode, packed batch of 8, the single-layer
    pruning op) and the stand-alone kernels (weight-streaming GEMV, tensor-core GEMM per shape), timed
    through the public binding.  Every number in profiles/other_workloads_7b.md comes from these modes."""
    import torch
    from paper_2407_14057_b200 import binding as B
    from paper_2407_14057_b200 import build, synth
    torch.cuda.set_device(0)
    build.build()
    B.lib()
    peaks = _peaks()
    shape, sched = synth.LLAMA7B, synth.SCHEDULE_7B
    out = {"workload": args.workload, "dtype": "bf16", "data": "synthetic", "peaks": peaks}
    sampler = ClockSampler(0)
    sampler.start()

    if args.workload == "decode":
        n, steps = 4096, 32
        W = synth.make_weights(shape, 2, bf16=True, device="cuda")
        ids = synth.make_prompt(shape.vocab, n, 101).cuda()
        lg = torch.empty((1, shape.vocab), dtype=torch.float32, device="cuda")
        nxt = torch.empty(1, dtype=torch.int32, device="cuda")
        for name, sc in (("pruned", sched), ("full_keep", ())):
            eng = B.LazyPrefill(shape, W, sc, torch.bfloat16, 1, n, max_new_tokens=steps)
            ttft = _event_ms(lambda i: eng.lazy_prefill_run(ids, [0, n], lg), 5, 3)
            eng.lazy_sync_status()
            tok = torch.argmax(lg, dim=1).to(torch.int32)
            times, inflight = [], []
            for _ in range(steps):       # a step reads counters back, so it is timed by the host clock around a sync
                torch.cuda.synchronize()
                t0 = time.perf_counter()
                eng.lazy_decode_step(tok, lg, nxt)
                torch.cuda.synchronize()
                times.append(round((time.perf_counter() - t0) * 1e3, 3))
                st = eng.lazy_get_stats()
                inflight.append([st.rows_computed[l] for l in (0, 8, 16, 24)])
                tok = nxt.clone()
            eng.lazy_sync_status()
            steady = sorted(times[-8:])[len(times[-8:]) // 2]
            out[name] = {"prefill_ttft_ms": round(ttft, 3), "decode_step_ms": times,
                         "rows_in_flight_layers_0_8_16_24": inflight, "all_steps_ms": round(sum(times), 2),
                         "steady_state_step_ms": steady, "launches_last_step": int(st.kernel_launches),
                         "weight_streaming_floor_ms": round(12.95e9 / (peaks["hbm_gbs"] * 1e9) * 1e3, 3),
                         "frac_of_floor": round(12.95e9 / (peaks["hbm_gbs"] * 1e9) * 1e3 / steady, 3)}
            eng.close()
            del eng
            torch.cuda.empty_cache()

    elif args.workload == "batch8":
        W = synth.make_weights(shape, 2, bf16=True, device="cuda")
        lengths = synth.make_varlen_lengths(8, 1024, 4096, seed=4)
        ids, cu = synth.make_varlen_batch(shape.vocab, lengths, seed=5)
        ids, tot = ids.cuda(), sum(lengths)
        lg = torch.empty((8, shape.vocab), dtype=torch.float32, device="cuda")
        out.update({"lengths": lengths, "tokens": tot})
        for name, sc in (("pruned", sched), ("full_keep", ())):
            eng = B.LazyPrefill(shape, W, sc, torch.bfloat16, 8, tot)
            ms = _event_ms(lambda i: eng.lazy_prefill_run(ids, cu, lg), 3, 2)
            eng.lazy_sync_status()
            out[name] = {"ms": round(ms, 2), "tokens_per_s": round(tot / ms * 1e3)}
            eng.close()
            del eng
            torch.cuda.empty_cache()

    elif args.workload == "prune-op":
        n, d, H, dh = 4096, shape.d_model, shape.n_heads, shape.head_dim
        x = synth.make_hidden(n, d, 1, bf16=True, device="cuda")
        pos = torch.arange(n, dtype=torch.int32, device="cuda")
        lw = synth.make_weights(shape.with_layers(1), 1, bf16=True, device="cuda")["layers"][0]
        res = B.lazy_prune_op(x, pos, lw["w_qkv"], lw["w_o"], lw["g_attn"], H, dh, 6000, n)
        ws = res["workspace"]
        ms = _event_ms(lambda i: B.lazy_prune_op(x, pos, lw["w_qkv"], lw["w_o"], lw["g_attn"], H, dh, 6000, n,
                                                 workspace=ws, outputs=res), 20, 5)
        B.lazy_device_status()
        n_keep, rb = res["n_keep"], d * 2
        # the HBM-bound steps alone; sources rotate over copies larger than L2 together
        srcs = [torch.randn((n, d), device="cuda").bfloat16() for _ in range(8)]
        idx = res["keep_idx"][:n_keep].contiguous()
        g_out = torch.empty((n_keep, d), dtype=torch.bfloat16, device="cuda")
        g_ms = _event_ms(lambda i: B.lazy_k_gather_rows(srcs[i % 8], idx, out=g_out), 40, 8)
        # the same kernel on enough rows for the launch to outlast the host's per-call cost (a 40 MB gather is over
        # before the next call has been issued): a random permutation of 32768 rows, sources rotating
        big_n = 32768
        big_src = [torch.randn((big_n, d), device="cuda").bfloat16() for _ in range(3)]
        big_idx = torch.randperm(big_n, device="cuda").to(torch.int32)
        big_out = torch.empty((big_n, d), dtype=torch.bfloat16, device="cuda")
        gb_ms = _event_ms(lambda i: B.lazy_k_gather_rows(big_src[i % 3], big_idx, out=big_out), 20, 5)
        del big_src, big_out
        torch.cuda.empty_cache()
        sc = synth.make_scores(n, "lognormal", 5).cuda()
        cu_in = torch.tensor([0, n], dtype=torch.int32).cuda()
        cu_keep = torch.tensor([0, n_keep], dtype=torch.int32).cuda()
        s_out = (torch.empty(n_keep, dtype=torch.int32, device="cuda"),
                 torch.empty(n - n_keep, dtype=torch.int32, device="cuda"))
        s_ms = _event_ms(lambda i: B.lazy_k_select(sc, cu_in, cu_keep, n, n_keep, s_out), 40, 8)
        qs = [torch.randn((n, d), device="cuda").bfloat16() for _ in range(8)]
        nf = B.lib().lazy_k_score_scratch_floats(1, n, H)
        k_out = (torch.empty(nf, dtype=torch.float32, device="cuda"), torch.empty(n, dtype=torch.float32, device="cuda"))
        k_ms = _event_ms(lambda i: B.lazy_k_score(qs[i % 8], d, srcs[i % 8], d, cu_in, n, H, dh, out=k_out), 40, 8)
        B.lazy_device_status()
        gbs = 2.0 * n_keep * rb / (g_ms * 1e-3) / 1e9
        out.update({"rows": n, "kept": n_keep, "whole_op_ms": round(ms, 4),
                    "gather_rows": {"us": round(g_ms * 1e3, 2), "gbs": round(gbs, 1),
                                    "frac_of_hbm_peak": round(gbs / peaks["hbm_gbs"], 3)},
                    "gather_rows_32768": {"us": round(gb_ms * 1e3, 2),
                                          "gbs": round(2.0 * big_n * rb / (gb_ms * 1e-3) / 1e9, 1),
                                          "frac_of_hbm_peak": round(2.0 * big_n * rb / (gb_ms * 1e-3) / 1e9
                                                                    / peaks["hbm_gbs"], 3)},
                    "select": {"us": round(s_ms * 1e3, 2), "bytes": 8 * n},
                    "score_standalone": {"us": round(k_ms * 1e3, 2),
                                         "gbs": round(n * rb / (k_ms * 1e-3) / 1e9, 1)}})

    elif args.workload == "gemv":
        rows = []
        for M in (1, 4):
            for name, N, K, sw in (("qkv", 12288, 4096, False), ("o", 4096, 4096, False),
                                   ("gate_up", 11008, 4096, True), ("down", 4096, 11008, False)):
                A = torch.randn(M, K, device="cuda").bfloat16()
                Ws = [(torch.randn(N, K, device="cuda") * 0.02).bfloat16() for _ in range(8)]
                Us = [(torch.randn(N, K, device="cuda") * 0.02).bfloat16() for _ in range(8)] if sw else None
                Cm = torch.empty(M, N, device="cuda", dtype=torch.bfloat16)
                if sw:
                    ms = _event_ms(lambda i: B.lazy_k_gemm_swiglu(A, Ws[i % 8], Us[i % 8], out=Cm), 40, 8)
                else:
                    ms = _event_ms(lambda i: B.lazy_k_gemm(A, Ws[i % 8], None, out=Cm), 40, 8)
                gbs = N * K * 2 * (2 if sw else 1) / (ms * 1e-3) / 1e9
                rows.append({"M": M, "product": name, "N": N, "K": K, "us": round(ms * 1e3, 2), "gbs": round(gbs),
                             "frac_of_hbm_peak": round(gbs / peaks["hbm_gbs"], 3)})
                del Ws, Us
                torch.cuda.empty_cache()
        B.lazy_device_status()
        out["gemv"] = rows
        out["note"] = ("context-free calls launch the weight-streaming kernel the ordinary way; inside a decode step it "
                       "is a programmatic dependent that requests its first weights while the kernel before it drains")

    elif args.workload == "gemm":
        ws = B.lazy_k_gemm_scratch()
        row_list = [int(r) for r in args.rows.split(",")] if args.rows else [1013, 1688, 2364, 3376]
        rows = []
        for M in row_list:
            for name, N, K, sw in (("qkv", 12288, 4096, False), ("o", 4096, 4096, False),
                                   ("gate_up", 11008, 4096, True), ("down", 4096, 11008, False)):
                A = torch.randn(M, K, device="cuda").bfloat16()
                Ws = [(torch.randn(N, K, device="cuda") * 0.02).bfloat16() for _ in range(3)]
                Us = [(torch.randn(N, K, device="cuda") * 0.02).bfloat16() for _ in range(3)] if sw else None
                R = None if sw else torch.randn(M, N, device="cuda").bfloat16()
                Cm = torch.empty(M, N, device="cuda", dtype=torch.bfloat16)
                ent = {"M": M, "product": name, "N": N, "K": K}
                for label, impl in (("auto", 0), ("one_cta", 2), ("pair", 3)):
                    if sw:
                        ms = _event_ms(lambda i: B.lazy_k_gemm_swiglu(A, Ws[i % 3], Us[i % 3], impl=impl, out=Cm,
                                                                      scratch=ws), args.steps, 5)
                    else:
                        ms = _event_ms(lambda i: B.lazy_k_gemm(A, Ws[i % 3], R, impl=impl, out=Cm, scratch=ws),
                                       args.steps, 5)
                    fl = 2.0 * M * N * K * (2 if sw else 1)
                    ent[label] = {"us": round(ms * 1e3, 1), "tflops": round(fl / (ms * 1e-3) / 1e12)}
                rows.append(ent)
                del Ws, Us
                torch.cuda.empty_cache()
        B.lazy_device_status()
        out["gemm"] = rows
        out["note"] = "isolated back-to-back launches, weights rotating over three copies; impl: auto = chosen by shape"

    elif args.workload == "gemm-sustained":
        # Every projection shape of the bench line looped for about a second, so that the card settles at its
        # power cap as it does inside the step, with the SM clock sampled during each loop; beside it the
        # library's plain GEMM (torch.matmul, no epilogue) on the same operands, as the per-shape reference that
        # the single roofline denominator (an 8192^3 product) cannot give.
        ws = B.lazy_k_gemm_scratch()
        row_list = [int(r) for r in args.rows.split(",")] if args.rows else [1013, 1688, 2364, 3376]

        def sustained(fn, flops):
            per = _event_ms(fn, 10, 5)
            iters = max(20, int(1000.0 / per))
            cs = ClockSampler(0)
            cs.start()
            ms = _event_ms(fn, iters, 0)
            clk = cs.stop()
            return {"us": round(ms * 1e3, 1), "tflops": round(flops / (ms * 1e-3) / 1e12), "sm_mhz": clk["sm_mhz"]}

        rows = []
        for M in row_list:
            for name, N, K, sw in (("qkv", 12288, 4096, False), ("o", 4096, 4096, False),
                                   ("gate_up", 11008, 4096, True), ("down", 4096, 11008, False)):
                A = torch.randn(M, K, device="cuda").bfloat16()
                Ws = [(torch.randn(N, K, device="cuda") * 0.02).bfloat16() for _ in range(3)]
                Us = [(torch.randn(N, K, device="cuda") * 0.02).bfloat16() for _ in range(3)] if sw else None
                W2 = [torch.cat([Ws[i], Us[i]], 0) for i in range(3)] if sw else Ws
                R = None if sw else torch.randn(M, N, device="cuda").bfloat16()
                Cm = torch.empty(M, N, device="cuda", dtype=torch.bfloat16)
                C2 = torch.empty(M, N * (2 if sw else 1), device="cuda", dtype=torch.bfloat16)
                fl = 2.0 * M * N * K * (2 if sw else 1)
                if sw:
                    ours = sustained(lambda i: B.lazy_k_gemm_swiglu(A, Ws[i % 3], Us[i % 3], out=Cm, scratch=ws), fl)
                else:
                    ours = sustained(lambda i: B.lazy_k_gemm(A, Ws[i % 3], R, out=Cm, scratch=ws), fl)
                lib_ref = sustained(lambda i: torch.matmul(A, W2[i % 3].t(), out=C2), fl)
                rows.append({"M": M, "product": name, "N": N, "K": K, "ours": ours, "library_plain_gemm": lib_ref})
                del Ws, Us, W2
                torch.cuda.empty_cache()
        B.lazy_device_status()
        out["gemm_sustained"] = rows
        out["note"] = ("about one second of back-to-back launches per entry (power-capped clocks, sampled); the library "
                       "entry is a plain product without residual / SwiGLU / rotary epilogue")

    out["clocks"] = sampler.stop()
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=0, help="reduced depth (profiling captures only)")
    ap.add_argument("--prompt", type=int, default=N_PROMPT)
    ap.add_argument("--no-cpu", action="store_true", help="skip the oracle timing leg")
    ap.add_argument("--no-fp8", action="store_true", help="skip the extra leg with e4m3 projections")
    ap.add_argument("--fp8", action="store_true", help=argparse.SUPPRESS)   # the leg runs by default
    ap.add_argument("--cpu-sample", action="store_true",
                    help="time the oracle on the bounded sample only (about 15 s) instead of the whole workload")
    ap.add_argument("--workload", default="prefill", choices=["prefill", "decode", "batch8", "prune-op", "gemv", "gemm", "gemm-sustained"],
                    help="prefill = the bench line; the others time the remaining configurations and single "
                         "kernels through the public binding and print one JSON object each")
    ap.add_argument("--rows", default="", help="--workload gemm: comma-separated row counts (default: the bench's)")
    ap.add_argument("--sweep", action="store_true",
                    help="single-cut location x keep-fraction TTFT surface instead of the bench line")
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
    elif args.workload != "prefill":
        run_other_workload(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
