#!/usr/bin/env python
"""Benchmark of the MixKV per-layer KV-cache compression step on B200.

A step is one pass of the whole hot path (score -> mix -> select -> gather) over all layers of
one synthetic prefill: one mixkv_compress_layers call.  The metric
is KV tokens compressed per second: tokens of the batch / time of one step (every layer
compresses the same tokens), whole job over all GPUs.  Each GPU runs an independent replica
(the step has no cross-GPU exchange), so scaling is weak.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C3] [--impl reference]

The default workload is C3 (long-video prefill, L = 32768): the metric's target is quoted for
L >= 8192, and C3 is the largest single-sequence configuration; C1 / C2 / C4 / C5 are parity-test
cases and can be timed with --workload.

One JSON line is printed by rank 0.  `--impl reference` times the CPU oracle instead (a
deliberately plain program; a baseline, not a target).
"""
from __future__ import annotations

import argparse
import ctypes as C
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "kv_tokens_compressed_per_s"
UNIT = "tokens/s"
L2_BYTES = 126e6


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="C3")
    ap.add_argument("--variant", default="calibrated")
    ap.add_argument("--impl", default="mixkv", choices=["mixkv", "reference"])
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (debug)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-per-layer", action="store_true")
    ap.add_argument("--min-seconds", type=float, default=1.0,
                    help="repeat the block of --steps steps until this much has been timed")
    ap.add_argument("--max-blocks", type=int, default=200)
    return ap.parse_args()


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def measured_traffic(workload, kernel, layers):
    """DRAM bytes per launch of `kernel` from the committed ncu capture, scaled to `layers`
    layers; None when there is no capture for this workload or the kernel source has changed
    since the counters were taken."""
    import hashlib
    path = os.path.join(ROOT, "profiles", f"dram_traffic_{workload}.json")
    if not os.path.exists(path):
        return None
    with open(path) as f:
        rec = json.load(f)
    try:
        with open(os.path.join(ROOT, rec["kernel_source"]), "rb") as f:
            if hashlib.sha256(f.read()).hexdigest() != rec["sha256"]:
                return None
        return rec[kernel]["dram_bytes_per_layer"] * layers
    except (KeyError, OSError):
        return None


def workload_config(wl, variant, extra=None):
    cfg = {"workload": f"{wl.name}: {wl.layers} layers, H={wl.kv_heads}, G={wl.gqa_ratio}, d=128, "
                       f"batch {wl.batch}, L={list(wl.seq_lens) if wl.batch > 1 else wl.seq_lens[0]}, "
                       f"W={wl.window}, pool {wl.pool_kernel}, B={wl.budget}"
                       f"{' adaptive' if wl.budget_mode else ''}, {variant} keys",
           "layers": wl.layers, "tokens_per_step": wl.total_tokens}
    if extra:
        cfg.update(extra)
    return cfg


def algorithmic_bytes(wl):
    """Bytes the method must move per layer (compulsory reads of K, V, Q once, the gather's
    read + write of the kept rows, the index list)."""
    d, H, G, W = wl.head_dim, wl.kv_heads, wl.gqa_ratio, wl.window
    kvq = sum(H * (2 * L * d * 2 + G * W * d * 2) for L in wl.seq_lens)
    rows = sum(H * min(wl.budget, L) for L in wl.seq_lens)
    gather = 2 * 2 * rows * d * 2
    idx = 4 * sum(H * min(wl.budget - W, L - W) for L in wl.seq_lens)
    k_bytes = sum(H * L * d * 2 for L in wl.seq_lens)
    q_bytes = sum(H * G * W * d * 2 for L in wl.seq_lens)
    # compulsory bytes of each pass: pass 1 streams K (and reads Q); pass 2 streams V (and reads
    # Q).  The second read of K in pass 2 is not compulsory and is not counted.
    return {"layer": kvq + gather + idx, "pass1": k_bytes + q_bytes, "pass2": k_bytes + q_bytes}


# ------------------------------------------------------------------------- reference arm
def run_reference(args):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload."""
    import oracle
    from paper_2510_20707_b200 import synth

    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = synth.CONFIGS[args.workload]
    po = oracle.Params(kv_heads=wl.kv_heads, gqa_ratio=wl.gqa_ratio, window=wl.window,
                       pool_kernel=wl.pool_kernel, budget=wl.budget, budget_mode=wl.budget_mode,
                       ada_floor=wl.ada_floor)
    cu = None if wl.batch == 1 else wl.cu_seqlens
    x = synth.make_layer(wl, 0, args.variant)
    t0 = time.perf_counter()
    oracle.compress_layer(x["K"], x["V"], x["Q"], po, cu=cu)   # builds + warms the library
    t_layer = time.perf_counter() - t0
    # bounded sample per step: the first `hs` KV heads of ONE layer, sized so that the whole run
    # stays near two minutes; scaled back to all heads and all layers
    H = wl.kv_heads
    budget_s = 120.0
    hs = int(max(1, min(H, budget_s / max((args.warmup + args.steps) * t_layer / H, 1e-9))))
    G = wl.gqa_ratio
    xs = {"K": np.ascontiguousarray(x["K"][:hs]), "V": np.ascontiguousarray(x["V"][:hs]),
          "Q": np.ascontiguousarray(x["Q"][:, :hs * G])}
    pos = oracle.Params(kv_heads=hs, gqa_ratio=G, window=wl.window, pool_kernel=wl.pool_kernel,
                        budget=wl.budget, budget_mode=wl.budget_mode, ada_floor=wl.ada_floor)
    times = []
    for s in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        oracle.compress_layer(xs["K"], xs["V"], xs["Q"], pos, cu=cu)
        if s >= args.warmup:
            times.append(time.perf_counter() - t0)
    sample_s = statistics.mean(times)       # what one timed step of this arm really ran
    scale = (H / hs) * wl.layers            # a full step is all heads of all layers
    step_s = sample_s * scale
    value = wl.total_tokens / step_s
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": sample_s * 1e3, "sample_to_full_step_scale": scale,
            "full_step_ms_scaled": step_s * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(wl, args.variant),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(),
                             "kind": "oracle",
                             "sample": f"each timed step is {hs} of {H} KV heads of layer 0 "
                                       f"(ms_per_step is that sample's time); value scales it by "
                                       f"{scale:g} to {H} heads x {wl.layers} layers"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------ helpers
def max_over_ranks(ms, world, device):
    """The step time of the whole job is the slowest rank's (replicas run side by side)."""
    import torch
    import torch.distributed as dist

    t = torch.tensor([ms], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(tokens_per_replica, world, ms_per_step):
    """KV tokens compressed per second over all replicas (weak scaling: every rank compresses
    its own copy of the workload)."""
    return world * tokens_per_replica / (ms_per_step * 1e-3)



class ClockSampler:
    """nvidia-smi clocks / throttle reasons sampled every 200 ms while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "50", "-i", str(self.index)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in out.strip().splitlines():
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "samples": len(sm),
                "reasons": sorted(reasons)}


def cpu_baseline(wl, variant, budget_s=12.0):
    """The oracle, untuned, on the host cores: whole layers until about budget_s seconds."""
    import oracle
    from paper_2510_20707_b200 import synth

    po = oracle.Params(kv_heads=wl.kv_heads, gqa_ratio=wl.gqa_ratio, window=wl.window,
                       pool_kernel=wl.pool_kernel, budget=wl.budget, budget_mode=wl.budget_mode,
                       ada_floor=wl.ada_floor)
    cu = None if wl.batch == 1 else wl.cu_seqlens
    oracle.lib()
    n, t_total = 0, 0.0
    while n < wl.layers and (t_total < budget_s or n < 1):
        x = synth.make_layer(wl, n, variant)      # each layer's own tensors (drawn outside the timing)
        t0 = time.perf_counter()
        oracle.compress_layer(x["K"], x["V"], x["Q"], po, cu=cu)
        t_total += time.perf_counter() - t0
        n += 1
    per_layer = t_total / n
    return {"value": wl.total_tokens / (per_layer * wl.layers), "unit": UNIT,
            "cores": oracle.threads(), "kind": "oracle",
            "sample": f"layers 0..{n - 1} of {wl.layers} (their own tensors), {t_total:.1f} s of "
                      f"oracle time, scaled to all layers",
            "ms_per_layer": per_layer * 1e3}


# ------------------------------------------------------------------------------ main arm
def run_mixkv(args):
    import torch
    import torch.distributed as dist

    from paper_2510_20707_b200 import binding, build, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    binding.load_library()

    wl = synth.CONFIGS[args.workload]
    if args.layers:
        from dataclasses import replace
        wl = replace(wl, layers=args.layers)
    pg = binding.Params(kv_heads=wl.kv_heads, gqa_ratio=wl.gqa_ratio, window=wl.window,
                        pool_kernel=wl.pool_kernel, budget=wl.budget, budget_mode=wl.budget_mode,
                        ada_floor=wl.ada_floor)
    cu_list = None if wl.batch == 1 else [int(c) for c in wl.cu_seqlens]
    H, Ltot, NL = wl.kv_heads, wl.total_tokens, wl.layers
    stage_names = binding.stage_names_for(pg, NL, wl.batch, max(wl.seq_lens))
    n_stage = len(stage_names)

    # ---- inputs: K, V [layers, H, Ltot, d] and Q [layers, batch, H*G, W, d] in pinned host
    # memory; enough device copies ("sets") that the bytes streamed between two uses of a
    # buffer exceed L2 several times
    host = {k: torch.empty((NL,) + shp, dtype=torch.bfloat16).pin_memory()
            for k, shp in (("K", (H, Ltot, 128)), ("V", (H, Ltot, 128)),
                           ("Q", (wl.batch, H * wl.gqa_ratio, wl.window, 128)))}
    for layer in range(NL):
        x = synth.make_layer(wl, layer, args.variant)
        for k, v in x.items():
            host[k][layer].copy_(torch.from_numpy(v.view(np.int16)).view(torch.bfloat16))
    set_bytes = sum(t.numel() * 2 for t in host.values())
    n_sets = max(1, int(np.ceil(4 * L2_BYTES / set_bytes)))
    dev_in = [{k: t.to(dev) for k, t in host.items()} for _ in range(n_sets)]
    ws_bytes = binding.workspace_size_layers(pg, NL, wl.batch, Ltot, max(wl.seq_lens))
    workspace = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    rows_cap = wl.batch * H * wl.budget

    def new_out():
        return {"K_out": torch.empty((NL, rows_cap, 128), dtype=torch.bfloat16, device=dev),
                "V_out": torch.empty((NL, rows_cap, 128), dtype=torch.bfloat16, device=dev),
                "out_row_offsets": torch.empty((NL, wl.batch * H + 1), dtype=torch.int32, device=dev),
                "status": torch.zeros(1, dtype=torch.int32, device=dev)}

    out = new_out()
    stream = torch.cuda.current_stream()

    def step(s, trace=None):
        """One step = the whole hot path over all layers: ONE mixkv_compress_layers call."""
        b = dev_in[s % n_sets]
        binding.compress_layers(b["K"], b["V"], b["Q"], pg, cu_seqlens=cu_list,
                                workspace=workspace, stream=stream, out=out, want_aux=False,
                                trace_events=trace)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def check_status():
        st_ = int(out["status"].item())
        if st_ != 0:
            raise SystemExit(f"device status {st_} reported by a kernel")

    def timed(run, n_warm, n_steps):
        for s in range(n_warm):
            run(s)
        barrier()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        t0.record(stream)
        for s in range(n_steps):
            run(n_warm + s)
        t1.record(stream)
        barrier()
        return max_over_ranks(t0.elapsed_time(t1), world, dev) / n_steps

    # ---- timed region: K steps, device-resident inputs, CUDA events on the launching stream
    for s in range(args.warmup):
        step(s)
    barrier()
    check_status()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    # A block is exactly --steps steps between two barriers.  Blocks are repeated until about
    # --min-seconds of steps have been timed, so that the figure is the sustained one (clocks
    # and power settle over hundreds of milliseconds); the line carries the median block, the
    # best block and what the clocks did meanwhile.
    blocks = [timed(step, 0, args.steps)]
    n_blocks = int(min(args.max_blocks, max(1, np.ceil(args.min_seconds * 1e3 / (blocks[0] * args.steps)))))
    n_blocks = int(max_over_ranks(float(n_blocks), world, dev))
    for _ in range(n_blocks - 1):
        blocks.append(timed(step, 0, args.steps))
    clocks = sampler.stop() if rank == 0 else None
    check_status()
    ms_per_step = statistics.median(blocks)
    value = whole_job_value(wl.total_tokens, world, ms_per_step)

    # ---- per-kernel CUDA-event times: every kernel of a step bracketed by events on the
    # launching stream
    n_tr = max(1, min(args.steps, 10))
    tr_ev = [[torch.cuda.Event(enable_timing=True) for _ in range(n_stage + 1)] for _ in range(n_tr)]
    for st_ in tr_ev:
        for e in st_:
            e.record(stream)          # forces creation of the underlying CUDA event
    torch.cuda.synchronize()
    tr_c = [(C.c_void_p * (n_stage + 1))(*[e.cuda_event for e in st_]) for st_ in tr_ev]
    for s in range(n_tr):
        step(s, trace=tr_c[s])
    torch.cuda.synchronize()
    check_status()
    stage_ms = {name: statistics.mean(st_[i].elapsed_time(st_[i + 1]) for st_ in tr_ev)
                for i, name in enumerate(stage_names)}

    # ---- the same layers through the one-layer entry point, one call per layer (context)
    per_layer_ms = None
    if not args.no_per_layer:
        ws1 = torch.empty(binding.workspace_size(pg, wl.batch, Ltot, max(wl.seq_lens)),
                          dtype=torch.uint8, device=dev)
        o1 = {"K_out": out["K_out"][0], "V_out": out["V_out"][0],
              "out_row_offsets": out["out_row_offsets"][0], "status": out["status"]}

        def step_per_layer(s):
            b = dev_in[s % n_sets]
            for layer in range(NL):
                binding.compress_layer(b["K"][layer], b["V"][layer], b["Q"][layer], pg,
                                       cu_seqlens=cu_list, workspace=ws1, stream=stream, out=o1,
                                       want_aux=False)

        per_layer_ms = timed(step_per_layer, 1, max(3, min(args.steps, 5)))
        check_status()

    # ---- end to end: host buffers in, compact cache out, copies inside the timed region
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(args, wl, pg, cu_list, host, dev, world, barrier, binding)

    if world > 1:
        dist.barrier()
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    peak, peak_kind = peaks()
    ab = algorithmic_bytes(wl)
    dom = max(("pass1", "pass2"), key=lambda k: stage_ms[k])
    dom_ms = stage_ms[dom]
    achieved = NL * ab[dom] / (dom_ms * 1e-3) / 1e9
    layer_ms = ms_per_step / NL
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16 in, f32 accumulate",
        "data": "synthetic",
        "config": workload_config(wl, args.variant, {
            "l2": f"{n_sets} set(s) of inputs, {n_sets * set_bytes / 2**20:.0f} MiB cycled "
                  f"(> 126 MB L2) between two uses of a buffer",
            "launch": "one mixkv_compress_layers call per step (all layers in one set of kernels)",
            "parallelism": "replicas only" if world > 1 else "single GPU"}),
        "timing": {"blocks": len(blocks), "steps_per_block": args.steps,
                   "ms_per_step_median_block": ms_per_step, "ms_per_step_best_block": min(blocks),
                   "ms_per_step_first_block": blocks[0],
                   # context only: the median block rescaled from the median sampled SM clock to the
                   # maximum one (the HBM-bound share of a step does not follow the SM clock)
                   "ms_per_step_scaled_to_max_sm_clock": (
                       ms_per_step * clocks["sm_mhz"] / clocks["sm_max_mhz"]
                       if clocks and clocks.get("sm_mhz") and clocks.get("sm_max_mhz") else None),
                   "regime": ("sustained: sw_power_cap seen during the timed blocks"
                              if clocks and "sw_power_cap" in clocks.get("reasons", [])
                              else "no throttle reason seen during the timed blocks")},
        "per_layer_latency_us": layer_ms * 1e3,
        "token_layers_per_s": world * wl.total_tokens * NL / (ms_per_step * 1e-3),
        "stage_ms": stage_ms,
        "layer_roofline": {"bound": "hbm", "achieved": ab["layer"] / (layer_ms * 1e-3) / 1e9,
                           "peak": peak, "unit": "GB/s",
                           "frac": ab["layer"] / (layer_ms * 1e-3) / 1e9 / peak,
                           "frac_of_8TBs_nominal": ab["layer"] / (layer_ms * 1e-3) / 8e12,
                           "algorithmic_bytes_per_layer": ab["layer"]},
        "roofline": {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak,
                     "unit": "GB/s", "frac": achieved / peak,
                     "traffic": measured_traffic(wl.name, dom, NL),
                     "peak_source": f"{peak_kind} copy bandwidth",
                     "algorithmic_bytes_per_launch": NL * ab[dom],
                     "kernel_ms": dom_ms},
        "clocks": clocks,
        "gpu_launches": n_stage * args.steps * len(blocks),
    }
    # the head-wise redundancy the kernels measured on these inputs (Eq. 4), first layer: the
    # weight that Eq. 5 gives the diversity score of each head
    sc0 = binding.scores(dev_in[0]["K"][0], dev_in[0]["V"][0], dev_in[0]["Q"][0], pg,
                         cu_seqlens=cu_list, want_parts=True)
    torch.cuda.synchronize()
    line["config"]["rbar_first_layer"] = [round(float(x), 3) for x in sc0["rbar"].flatten().tolist()]
    if per_layer_ms is not None:
        one_us = per_layer_ms / NL * 1e3
        line["one_layer_per_call"] = {
            "ms_per_step": per_layer_ms, "per_layer_latency_us": one_us,
            "roofline": {"bound": "hbm", "achieved": ab["layer"] / (one_us * 1e-6) / 1e9,
                         "peak": peak, "unit": "GB/s",
                         "frac": ab["layer"] / (one_us * 1e-6) / 1e9 / peak,
                         "frac_of_8TBs_nominal": ab["layer"] / (one_us * 1e-6) / 8e12},
            "note": "same step as one mixkv_compress_layer call per layer, issued from Python"}
    if e2e is not None:
        line["e2e"] = e2e
    if not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(wl, args.variant)
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_e2e(args, wl, pg, cu_list, host, dev, world, barrier, binding):
    """Same metric through the public call with HOST buffers: the layers are cut into groups;
    each group's K, V, Q are copied from pinned host memory, compressed with one
    mixkv_compress_layers call, and its compact cache is copied back, all inside the timed
    region.  Two streams alternate groups so copies overlap compute."""
    import torch
    import torch.distributed as dist

    H, NL = wl.kv_heads, wl.layers
    rows_cap = wl.batch * H * wl.budget
    grp = max(1, min(NL, 4))
    groups = [(g0, min(g0 + grp, NL)) for g0 in range(0, NL, grp)]
    streams = [torch.cuda.Stream(device=dev) for _ in range(2)]
    ws_bytes = binding.workspace_size_layers(pg, grp, wl.batch, wl.total_tokens, max(wl.seq_lens))
    slots = []
    for i in range(2):
        slots.append({
            "in": {k: torch.empty((grp,) + tuple(t.shape[1:]), dtype=t.dtype, device=dev)
                   for k, t in host.items()},
            "ws": torch.empty(ws_bytes, dtype=torch.uint8, device=dev),
            "out": {"K_out": torch.empty((grp, rows_cap, 128), dtype=torch.bfloat16, device=dev),
                    "V_out": torch.empty((grp, rows_cap, 128), dtype=torch.bfloat16, device=dev),
                    "out_row_offsets": torch.empty((grp, wl.batch * H + 1), dtype=torch.int32,
                                                   device=dev),
                    "status": torch.zeros(1, dtype=torch.int32, device=dev)}})
    host_out = {"K_out": torch.empty((NL, rows_cap, 128), dtype=torch.bfloat16).pin_memory(),
                "V_out": torch.empty((NL, rows_cap, 128), dtype=torch.bfloat16).pin_memory(),
                "out_row_offsets": torch.empty((NL, wl.batch * H + 1), dtype=torch.int32).pin_memory()}
    h2d = sum(t.numel() * t.element_size() for t in host.values())
    d2h = sum(t.numel() * t.element_size() for t in host_out.values())

    def step():
        for gi, (g0, g1) in enumerate(groups):
            sl, st = slots[gi % 2], streams[gi % 2]
            n = g1 - g0
            with torch.cuda.stream(st):
                for k, t in host.items():
                    sl["in"][k][:n].copy_(t[g0:g1], non_blocking=True)
                o = {k: (v if k == "status" else v[:n]) for k, v in sl["out"].items()}
                binding.compress_layers(sl["in"]["K"][:n], sl["in"]["V"][:n], sl["in"]["Q"][:n], pg,
                                        cu_seqlens=cu_list, workspace=sl["ws"], stream=st, out=o,
                                        want_aux=False)
                for k, t in host_out.items():
                    t[g0:g1].copy_(sl["out"][k][:n], non_blocking=True)

    steps = max(3, min(args.steps, 10))
    for _ in range(3):
        step()
    barrier()
    t0 = time.perf_counter()
    beg = [torch.cuda.Event(enable_timing=True) for _ in streams]
    end = [torch.cuda.Event(enable_timing=True) for _ in streams]
    for e, s in zip(beg, streams):
        e.record(s)
    for _ in range(steps):
        step()
    for e, s in zip(end, streams):
        e.record(s)
    torch.cuda.synchronize()
    wall_ms = (time.perf_counter() - t0) * 1e3
    bad = [int(sl["out"]["status"].item()) for sl in slots if int(sl["out"]["status"].item()) != 0]
    if bad:
        raise SystemExit(f"device status {bad[0]} reported by a kernel (e2e)")
    dev_ms = max(b.elapsed_time(e) for b in beg for e in end)
    t = torch.tensor([dev_ms], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms = float(t.item()) / steps
    return {"value": world * wl.total_tokens / (ms * 1e-3), "unit": UNIT,
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": ms,
            "steps": steps, "wall_ms_per_step": wall_ms / steps,
            "note": f"pinned host K/V/Q -> device in groups of {grp} layers, "
                    "mixkv_compress_layers per group, compact cache -> pinned host"}


def run_widened(args):
    """Builder-run lines for the rows widened after the hot path (not the driver's metric):
    --workload SIM     the dense redundancy-analysis map (block 16) of the keys of a C3 layer, a
                       tensor-core contraction: roofline bound "tensor" against the measured bf16
                       peak, algorithmic flops = 2 L^2 d per head;
    --workload DECODE  one decode token over the C3b compact cache (28 layers x 4 heads x 512
                       rows): bytes of cache read per second against the measured copy peak."""
    import torch

    from paper_2510_20707_b200 import binding, build, synth

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(0)
    build.build()
    binding.load_library()
    with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
        pk = json.load(f)
    stream = torch.cuda.current_stream()

    def timed(fn, n):
        for _ in range(max(3, args.warmup)):
            fn()
        torch.cuda.synchronize()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record(stream)
        for _ in range(n):
            fn()
        t1.record(stream)
        torch.cuda.synchronize()
        return t0.elapsed_time(t1) / n

    if args.workload == "SIM":
        wl = synth.CONFIGS["C3"]
        H, L, block = wl.kv_heads, wl.total_tokens, 16
        # keys of four layers in turn: 134 MB of input, larger than L2
        Xs = [torch.from_numpy(synth.make_layer(wl, l, args.variant)["K"].view(np.int16)).cuda()
              .view(torch.bfloat16) for l in range(4)]
        it = [0]

        def fn():
            binding.similarity_map(Xs[it[0] % 4], block)
            it[0] += 1

        ms = timed(fn, max(4, min(args.steps, 20)))
        flops = 2.0 * L * L * 128 * H
        ach = flops / (ms * 1e-3) / 1e12
        line = {"metric": "similarity_rows_per_s", "value": H * L / (ms * 1e-3), "unit": "rows/s",
                "n_gpus": 1, "ms_per_step": ms, "higher_is_better": True, "dtype": "bf16 hi/lo in, f32 accumulate",
                "data": "synthetic",
                "config": {"workload": f"SIM: block-{block} cosine map of the keys of a C3 layer, "
                                       f"H={H}, L={L}, d=128, {args.variant} keys; inputs of 4 layers cycled"},
                "roofline": {"bound": "tensor", "achieved": ach, "peak": pk["bf16_tflops"],
                             "unit": "TFLOP/s", "frac": ach / pk["bf16_tflops"], "traffic": None,
                             "peak_source": "measured cuBLAS bf16 (burst)",
                             "algorithmic_flops_per_launch": flops,
                             "executed_flops_per_launch": flops * 1.5,
                             "note": "executed = upper triangle (x 1/2) of three bf16 products "
                                     "(hi.hi, hi.lo, lo.hi: x 3)"}}
    else:
        NL, H, G, B = 28, 4, 7, 512
        rows = H * B
        K = torch.randn((NL, rows, 128), device="cuda", dtype=torch.bfloat16)
        V = torch.randn_like(K)
        offs = (torch.arange(H + 1, dtype=torch.int32) * B).repeat(NL, 1).contiguous().cuda()
        q = torch.randn((NL, 1, H * G, 128), device="cuda", dtype=torch.bfloat16)
        big = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

        def fn():
            big.zero_()          # flushes L2 between two reads of the 29 MB cache
            binding.decode_attention(K, V, offs, q, H, G, B)

        n = max(4, min(args.steps, 20))
        ms_both = timed(fn, n)
        ms_flush = timed(lambda: big.zero_(), n)
        ms = ms_both - ms_flush
        nbytes = 2.0 * NL * rows * 256
        ach = nbytes / (ms * 1e-3) / 1e9
        line = {"metric": "decode_tokens_per_s", "value": 1.0 / (ms * 1e-3), "unit": "tokens/s",
                "n_gpus": 1, "ms_per_step": ms, "higher_is_better": True, "dtype": "bf16 in, f32 accumulate",
                "data": "synthetic",
                "config": {"workload": f"DECODE: one token over a compact cache of {NL} layers x {H} KV "
                                       f"heads x {B} rows, G={G}, d=128; L2 flushed between calls "
                                       f"(flush time {ms_flush * 1e3:.1f} us subtracted)"},
                "roofline": {"bound": "hbm", "achieved": ach, "peak": pk["hbm_gbs"], "unit": "GB/s",
                             "frac": ach / pk["hbm_gbs"], "traffic": None,
                             "peak_source": "measured copy bandwidth",
                             "algorithmic_bytes_per_launch": nbytes}}
    print(json.dumps(line), flush=True)


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.workload in ("SIM", "DECODE"):
        run_widened(args)
    else:
        run_mixkv(args)


if __name__ == "__main__":
    main()
