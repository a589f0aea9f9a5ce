#!/usr/bin/env python
"""Benchmark of the HeadCast attention path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 480p|720p|1080p|tiny] [--impl reference]

A *step* is one block-denoise-step of the steady state: one ``headcast_attend`` call, preceded every 4th step by
the per-block ``headcast_append`` (4 denoise steps reuse the cache).  The one-time phases of the path (warm-up
appends, dense attention, classification, split) are timed once and reported in ``phases``.  Rank 0 prints ONE
JSON line.  ``--impl reference`` times the float64 CPU oracle on a bounded sample instead.

The path does not shard (one attention layer on one GPU): with ``--gpus N`` every rank runs an independent
replica and the slowest rank's time is reported.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2607_20125_b200 import synth  # noqa: E402

METRIC = "headcast_attn_ms_per_block_step"
STEPS_PER_BLOCK = 4
# dram__bytes_read.sum + dram__bytes_write.sum of one attention-kernel launch, from the ncu captures summarised
# under profiles/ (None where not captured at that size)
NCU_TRAFFIC_BYTES = {"480p": 279.0e6, "720p": 606.0e6, "1080p": None, "tiny": None}


def workload_of(name: str):
    return synth.tiny() if name == "tiny" else synth.wan(name)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"tflops": d["bf16_tflops"], "tflops_sustained": d.get("bf16_tflops_sustained"), "hbm_gbs": d["hbm_gbs"],
                "source": "measured"}
    return {"tflops": 1590.0, "tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": "nvmlClocksEventReasonHwSlowdown", "hw_thermal_slowdown": "nvmlClocksEventReasonHwThermalSlowdown",
                 "sw_thermal_slowdown": "nvmlClocksEventReasonSwThermalSlowdown", "sw_power_cap": "nvmlClocksEventReasonSwPowerCap"}
        bits = {k: getattr(nv, v, None) or getattr(nv, v.replace("Event", "Throttle"), 0) for k, v in names.items()}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.handle)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle)
                self.reasons.update(k for k, b in bits.items() if b and (r & b))
            except Exception:
                pass
            time.sleep(0.004)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def max_over_ranks(value: float, dist, torch, device) -> float:
    """The slowest rank's value (every rank gets it); the identity on a single process."""
    if dist is None:
        return float(value)
    t = torch.tensor([value], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def to_dev(bits, torch):
    return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).cuda()


def timed(torch, fn, flush, reps):
    """Mean CUDA-event time of fn() over reps calls, L2 flushed (outside the events) before each."""
    total = 0.0
    for _ in range(reps):
        flush()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        b.synchronize()
        total += a.elapsed_time(b)
    return total / reps


_ORACLE_STATE = {}


def _oracle_state(w):
    """Cache model, geometry, queries and sampled rows of the oracle arm (built once per process)."""
    if w.name not in _ORACLE_STATE:
        from oracle import headcast_oracle as orc
        geom = orc.Geometry.make(w.grid_h, w.grid_w, w.frames_per_block, w.cell_h, w.cell_w)
        cache = orc.CacheModel(w.n_blocks, w.n_heads)
        for b in range(w.n_blocks):
            cache.append(*synth.make_kv(w, b))
        cache.split(w.labels)
        q = synth.make_q(w, w.n_blocks - 1, 0)
        rows = np.random.default_rng(0).permutation(w.block_tokens)  # seeded order over all query rows
        t0 = time.perf_counter()
        orc.attend(q, cache, geom, rows=rows[:256])
        per_row = (time.perf_counter() - t0) / 256
        _ORACLE_STATE[w.name] = (orc, geom, cache, q, rows, per_row)
    return _ORACLE_STATE[w.name]


def cpu_baseline(w, target_s=12.0):
    """The oracle, as it stands, on a bounded sample of the same workload: head-specific attention for a few query
    rows of every head, extrapolated linearly to the whole block (rows are independent)."""
    orc, geom, cache, q, rows, per_row = _oracle_state(w)
    n = int(max(256, min(rows.size, target_s / max(per_row, 1e-9))))
    t0 = time.perf_counter()
    orc.attend(q, cache, geom, rows=rows[:n])
    dt = time.perf_counter() - t0
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count()
    return {"value": dt / n * w.block_tokens * 1e3, "unit": "ms", "cores": int(cores), "kind": "oracle",
            "sample": f"{n} of {w.block_tokens} query rows of every head, one attend; {dt:.1f} s measured, extrapolated linearly"}


def run_reference(args, w):
    """--impl reference: the CPU oracle as the reference arm (bounded sample per step)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    per_step = []
    base = None
    for i in range(args.warmup + args.steps):
        base = cpu_baseline(w, target_s=max(2.0, min(12.0, 150.0 / (args.warmup + args.steps))))
        if i >= args.warmup:
            per_step.append(base["value"])
    value = float(np.mean(per_step))
    base["value"] = value
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "ms", "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": value, "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "heads": w.n_heads, "head_dim": w.head_dim, "grid": [w.grid_h, w.grid_w],
                       "block_tokens": w.block_tokens, "kv_tokens": w.n_blocks * w.block_tokens},
            "cpu_baseline": base, "e2e": {"value": value, "unit": "ms", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def run_rollout(args):
    """Streaming rollout at the 720P token grid (benchmark config 5): per layer a 2-block dense warm-up, the third
    block appended and classified at its first denoise step, the split with 3 cached blocks, then `--blocks` generated
    blocks x 4 denoise steps, each block appended to (and rolled through) the per-archetype buffers of every layer.
    The dense arm repeats the generated blocks with headcast_full_attend on the monolithic caches kept alongside.
    Inputs are seeded N(0,1) bf16 drawn on the device and shared by the layers; every layer gets its own seeded
    2/3/4/3 head mix through headcast_set_labels (labels from classification need planted patterns, which the
    parity tests cover; here classification is only timed)."""
    import torch
    from paper_2607_20125_b200.binding import HeadCast
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    base = synth.wan("720p")
    L, H, D = base.block_tokens, base.n_heads, base.head_dim
    g = torch.Generator(device="cuda")
    g.manual_seed(synth.BASE_SEED)
    pool = 4
    kv = [(torch.randn((L, H, D), device="cuda", generator=g).bfloat16(), torch.randn((L, H, D), device="cuda", generator=g).bfloat16())
          for _ in range(pool)]
    qs = [torch.randn((L, H, D), device="cuda", generator=g).bfloat16() for _ in range(STEPS_PER_BLOCK)]
    out = torch.empty_like(qs[0])
    layers = [HeadCast.from_workload(synth.wan("720p", layer=l), keep_monolithic=True) for l in range(args.layers)]
    mixes = (synth.reported_mixes("720p", args.layers) if args.mix == "reported"
             else [synth.wan("720p", layer=l).labels for l in range(args.layers)])
    if args.ablation != "full":
        mixes = [synth.ablation_labels(m)[args.ablation] for m in mixes]
    ev = lambda: torch.cuda.Event(enable_timing=True)
    t = {}
    a, b = ev(), ev()
    a.record()
    for hc in layers:  # warm-up: two blocks, dense attention for their 4 steps each
        for blk in range(2):
            hc.append(*kv[blk])
            for s_ in range(STEPS_PER_BLOCK):
                hc.full_attend(qs[s_], out)
    b.record(); b.synchronize()
    t["warmup_ms"] = a.elapsed_time(b)
    a, b = ev(), ev()
    a.record()
    for hc, mix in zip(layers, mixes):
        hc.append(*kv[2])
        hc.classify(qs[0])
        hc.set_labels(mix)
        hc.split_cache()
    b.record(); b.synchronize()
    t["classify_split_ms"] = a.elapsed_time(b)
    launches0 = sum(hc.launch_count() for hc in layers)
    a, b = ev(), ev()
    a.record()
    for blk in range(args.blocks):
        for hc in layers:
            hc.append(*kv[(3 + blk) % pool])
            for s_ in range(STEPS_PER_BLOCK):
                hc.attend(qs[s_], out)
    b.record(); b.synchronize()
    t["headcast_ms"] = a.elapsed_time(b)
    launches = sum(hc.launch_count() for hc in layers) - launches0
    flops = sum(hc.attend_flops(False) for hc in layers)
    if args.graphs:
        # The same steady-state blocks replayed from CUDA graphs: one graph per layer and ring position (the slot a new
        # block lands in cycles with period n_blocks - 1, and after that many appends the host-side ring is back where
        # it started, so capture leaves the contexts consistent).  Capture records the launches, it does not run them.
        period = base.n_blocks - 1
        graphs = []
        try:
            for hc in layers:
                per_layer = []
                for ph in range(period):
                    gr = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(gr):
                        hc.append(*kv[ph % pool])
                        for s_ in range(STEPS_PER_BLOCK):
                            hc.attend(qs[s_], out)
                    per_layer.append(gr)
                graphs.append(per_layer)
            torch.cuda.synchronize()
            for per_layer in graphs:  # one warm replay of everything
                per_layer[0].replay()
            torch.cuda.synchronize()
            a, b = ev(), ev()
            a.record()
            for blk in range(args.blocks):
                for per_layer in graphs:
                    per_layer[blk % period].replay()
            b.record(); b.synchronize()
            t["headcast_graph_ms"] = a.elapsed_time(b)
            t["graph_launches"] = args.blocks * len(layers)
        except Exception as exc:  # report, do not hide
            t["headcast_graph_ms"] = None
            t["graph_error"] = str(exc)[:200]
        graphs = None
    a, b = ev(), ev()
    a.record()
    for blk in range(args.blocks):
        for hc in layers:
            for s_ in range(STEPS_PER_BLOCK):
                hc.full_attend(qs[s_], out)
    b.record(); b.synchronize()
    t["dense_ms"] = a.elapsed_time(b)
    for hc in layers:
        hc.check()
    n_steps = args.blocks * STEPS_PER_BLOCK
    per_step = t["headcast_ms"] / n_steps
    print(json.dumps({
        "metric": "headcast_rollout_attention_ms_per_block_step_all_layers", "value": per_step, "unit": "ms", "n_gpus": 1,
        "steps": n_steps, "warmup": 0, "ms_per_step": per_step, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic (seeded N(0,1) drawn on the device, shared by the layers)",
        "config": {"workload": "rollout-720p", "head_mix": args.mix, "ablation": args.ablation,
                   "head_counts_sink_dummy_spatial_global": [int(sum(1 for m in mixes for v in m if v == c)) for c in range(4)],
                   "layers": args.layers, "blocks": args.blocks, "steps_per_block": STEPS_PER_BLOCK,
                   "heads": H, "head_dim": D, "grid": [base.grid_h, base.grid_w], "l2": "working set of 30 layers (48 GB) exceeds L2"},
        "gpu_launches": int(launches),
        "rollout": {**t, "speedup_vs_dense": t["dense_ms"] / t["headcast_ms"],
                    "steady_state_tflops": flops * STEPS_PER_BLOCK / (t["headcast_ms"] / args.blocks) / 1e9,
                    "paper_end_to_end_speedup_720p": "1.31x (Self-Forcing 5 s) / 1.62x (LongLive 30 s), whole model, GPU unstated"},
    }))


def run_sharded(args, w):
    """Opt-in (`--shard heads`): ONE layer's heads spread over the ranks (paper_2607_20125_b200/sharding.py) instead of
    the default of one independent replica per GPU.  Every rank holds Q / K / V in full, attends its own heads and the
    outputs are all-gathered; total work is fixed, so the scaling is strong.  Prints the same metric as the default
    run, without the one-time phases."""
    import torch
    import torch.distributed as dist
    from paper_2607_20125_b200 import sharding

    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    else:  # a group of one rank, so that the same code path runs on one GPU
        dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%d" % (29500 + os.getpid() % 2000), rank=0, world_size=1)
    L, H, D = w.block_tokens, w.n_heads, w.head_dim
    n_cells = -(-w.grid_h // w.cell_h) * -(-w.grid_w // w.cell_w)
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    layer = sharding.HeadShardedHeadCast(H, D, L, n_cells, grid_h=w.grid_h, grid_w=w.grid_w, n_blocks=w.n_blocks,
                                         frames_per_block=w.frames_per_block, cell_h=w.cell_h, cell_w=w.cell_w,
                                         sd_mode=args.sd_mode, sd_blocks=1 + args.sd_mode)
    n_extra = 3
    kv = [tuple(to_dev(t, torch) for t in synth.make_kv(w, b)) for b in range(w.n_blocks + n_extra)]
    qs = [[to_dev(synth.make_q(w, w.n_blocks + e, s), torch) for s in range(STEPS_PER_BLOCK)] for e in range(n_extra)]
    out = torch.empty_like(qs[0][0])
    for b in range(w.n_blocks):
        layer.append(*kv[b])
    layer.split_cache(w.labels)  # the planted labels; heads are re-dealt by cost and the moved caches exchanged
    state = {"i": 0}

    def step():
        i = state["i"]
        e = (i // STEPS_PER_BLOCK) % n_extra
        if i % STEPS_PER_BLOCK == 0:
            layer.append(*kv[w.n_blocks + e])
        layer.attend(qs[e][i % STEPS_PER_BLOCK], out)
        state["i"] = i + 1

    for _ in range(args.warmup):
        step()
    times = []
    torch.cuda.synchronize()
    dist.barrier()
    with ClockSampler(local) as sampler:
        for _ in range(args.steps):
            flush_buf.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            step()
            b.record()
            b.synchronize()
            times.append(a.elapsed_time(b))
        torch.cuda.synchronize()
        dist.barrier()
    clocks = sampler.summary()
    ms = max_over_ranks(float(np.mean(times)), dist if world > 1 else None, torch, "cuda")
    owner = layer.owner_heads
    dist.destroy_process_group()
    if rank != 0:
        return
    print(json.dumps({
        "metric": METRIC, "value": ms, "unit": "ms", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": False, "scaling": "strong", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "parallelism": "heads/%d" % world, "heads_per_rank": [len(h) for h in owner],
                   "l2": "flushed between steps", "exchange": "all-gather of L x H x d bf16 per attend"},
        "clocks": clocks, "gpu_launches": None, "e2e": None, "roofline": None, "cpu_baseline": None}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--workload", default="480p", choices=["tiny", "480p", "720p", "1080p", "rollout"])
    ap.add_argument("--layers", type=int, default=30, help="rollout: attention layers (one context each)")
    ap.add_argument("--blocks", type=int, default=20, help="rollout: generated blocks after the warm-up")
    ap.add_argument("--impl", default="headcast", choices=["headcast", "reference"])
    ap.add_argument("--sd-mode", type=int, default=0, choices=[0, 1],
                    help="1: Sink / Dummy heads keep anchor + current block (Appendix B accounting) instead of one block")
    ap.add_argument("--mix", default="default", choices=["default", "reported"],
                    help="rollout: 2/3/4/3 heads per layer, or the 360-head distribution the paper reports for LongLive at 720P")
    ap.add_argument("--ablation", default="full", choices=["full", "all_global", "spatial_only", "sink_dummy_only"],
                    help="rollout: which archetypes stay sparse (the paper's archetype ablation); the rest become Global")
    ap.add_argument("--graphs", action="store_true",
                    help="rollout: also replay the steady-state blocks from CUDA graphs (one per layer and ring position)")
    ap.add_argument("--ablations", action="store_true",
                    help="single layer: also time headcast_attend for the label sets of the paper's archetype ablation")
    ap.add_argument("--shard", default="none", choices=["none", "heads"],
                    help="heads: one layer's heads spread over the ranks (strong scaling) instead of one replica per GPU")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-phases", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.workload == "rollout":
        if args.impl == "reference":
            args.workload = "720p"
        else:
            return run_rollout(args)
    w = workload_of(args.workload)
    if args.impl == "reference":
        return run_reference(args, w)
    if args.shard == "heads":
        return run_sharded(args, w)

    import torch
    from paper_2607_20125_b200.binding import HeadCast

    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    peaks = measured_peaks()

    L, H, D = w.block_tokens, w.n_heads, w.head_dim
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    flush = lambda: flush_buf.zero_()

    hc = HeadCast.from_workload(w, keep_monolithic=True, sd_mode=args.sd_mode)
    n_extra = 3  # generated blocks fed round-robin once the cache rolls, each with its own 4 denoise-step queries
    kv = [tuple(to_dev(t, torch) for t in synth.make_kv(w, b)) for b in range(w.n_blocks + n_extra)]
    q_fill = to_dev(synth.make_q(w, w.n_blocks - 1, 0), torch)
    q_extra = [[to_dev(synth.make_q(w, w.n_blocks + e, s), torch) for s in range(STEPS_PER_BLOCK)] for e in range(n_extra)]
    qs = [q_fill]
    out = torch.empty_like(q_fill)
    phases = {}

    # ---- one-time phases: warm-up appends, dense attention, classification, split
    for b in range(w.n_blocks):
        hc.append(*kv[b])
    torch.cuda.synchronize()
    block_bytes = 2 * L * H * D * 2
    if not args.no_phases:
        hc.set_kernel_timing(True)
        for _ in range(3):
            hc.full_attend(qs[0], out)
        dense_ms = timed(torch, lambda: hc.full_attend(qs[0], out), flush, 10)
        phases["dense_full_attend_ms"] = dense_ms
        phases["dense_tflops"] = hc.attend_flops(True) / dense_ms / 1e9
        t0 = time.perf_counter()
        labels, scores = hc.classify(qs[0])
        torch.cuda.synchronize()
        t_first = (time.perf_counter() - t0) * 1e3
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        flush()
        a.record()
        labels, scores = hc.classify(qs[0])
        b.record()
        b.synchronize()
        phases["classify_ms"] = a.elapsed_time(b)
        phases["classify_first_call_ms"] = t_first
        phases["labels_match_planted"] = bool(tuple(int(v) for v in labels) == tuple(w.labels))
        # how far every thresholded quantity of every head is from its threshold (cosines vs 0.95, score vs 0.755)
        sc = np.asarray(scores, dtype=np.float64)
        phases["classify_margins"] = {"min_abs_cos_minus_theta": float(np.abs(sc[:, :3] - 0.95).min()),
                                      "min_abs_score_minus_theta": float(np.abs(sc[:, 5] - 0.755).min())}
        t = timed(torch, lambda: hc.append(*kv[w.n_blocks]), flush, 5)  # monolithic ring append (rolls)
        phases["append_monolithic_ms"] = t
        phases["append_monolithic_gbs"] = 2 * block_bytes / t / 1e6
    else:
        hc.set_labels(w.labels)
        hc.set_kernel_timing(True)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    flush()
    a.record()
    hc.split_cache()
    b.record()
    b.synchronize()
    n_sd = sum(1 for v in w.labels if v in (synth.SINK, synth.DUMMY))
    kept_bytes = 2 * 2 * L * D * (n_sd + (H - n_sd) * w.n_blocks)
    phases["split_ms"] = a.elapsed_time(b)  # one gather launch per cached block
    phases["split_gbs"] = 2 * kept_bytes / phases["split_ms"] / 1e6

    n_sink = sum(1 for v in w.labels if v == synth.SINK)
    append_bytes = block_bytes + 2 * L * (H - n_sink) * D * 2 + block_bytes  # read + per-archetype writes + monolithic copy

    state = {"i": 0}

    def step():
        i = state["i"]
        e = (i // STEPS_PER_BLOCK) % n_extra
        if i % STEPS_PER_BLOCK == 0:
            hc.append(*kv[w.n_blocks + e])
        hc.attend(q_extra[e][i % STEPS_PER_BLOCK], out)
        state["i"] = i + 1

    for _ in range(args.warmup):
        step()
    hc.check()
    # append throughput without launch gaps: 200 launches back to back inside one event pair (16 GB at 480P, > L2)
    n_b2b = 200
    flush()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for i in range(n_b2b):
        hc.append(*kv[w.n_blocks + i % n_extra])
    b.record()
    b.synchronize()
    phases["append_split_back_to_back_ms"] = a.elapsed_time(b) / n_b2b
    phases["append_split_back_to_back_gbs"] = append_bytes / phases["append_split_back_to_back_ms"] / 1e6
    state["i"] = 0
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    launches0 = hc.launch_count()
    step_ms, kernel_ms, append_ms = [], [], []
    with ClockSampler(local) as clocks:
        for i in range(args.steps):
            flush()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            m = torch.cuda.Event(enable_timing=True)
            a.record()
            e = (i // STEPS_PER_BLOCK) % n_extra
            if i % STEPS_PER_BLOCK == 0:
                hc.append(*kv[w.n_blocks + e])
                m.record()
            hc.attend(q_extra[e][i % STEPS_PER_BLOCK], out)
            b.record()
            b.synchronize()
            step_ms.append(a.elapsed_time(b))
            if i % STEPS_PER_BLOCK == 0:
                append_ms.append(a.elapsed_time(m))
            kernel_ms.append(hc.last_attention_kernel_ms())
        torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    hc.check()
    launches = hc.launch_count() - launches0
    total_ms = max_over_ranks(float(np.sum(step_ms)), dist, torch, "cuda")
    ms_per_step = total_ms / args.steps
    attend_ms = float(np.mean([s - (append_ms[i // STEPS_PER_BLOCK] if i % STEPS_PER_BLOCK == 0 else 0.0)
                               for i, s in enumerate(step_ms)]))
    kern = float(np.mean(kernel_ms))
    flops = hc.attend_flops(False)
    phases["append_split_ms"] = float(np.mean(append_ms))
    phases["append_split_gbs"] = append_bytes / phases["append_split_ms"] / 1e6
    phases["attend_ms"] = attend_ms
    phases["attend_tflops"] = flops / attend_ms / 1e9
    if "dense_full_attend_ms" in phases:
        phases["speedup_vs_dense"] = phases["dense_full_attend_ms"] / attend_ms
        phases["ideal_speedup_by_flops"] = hc.attend_flops(True) / flops

    if args.ablations:
        # the paper's archetype ablation, attention only: a fresh context per label set, same cache content
        abl = {}
        for name, lab in synth.ablation_labels(w.labels).items():
            h2 = HeadCast.from_workload(w, keep_monolithic=False, sd_mode=args.sd_mode)
            for blk in range(w.n_blocks):
                h2.append(*kv[blk])
            h2.set_labels(lab)
            h2.split_cache()
            h2.set_kernel_timing(True)
            for _ in range(3):
                h2.attend(q_extra[0][0], out)
            abl[name + "_ms"] = timed(torch, lambda: h2.attend(q_extra[0][0], out), flush, 10)
            abl[name + "_gflop"] = h2.attend_flops(False) / 1e9
            h2.check()
            h2.destroy()
        for name in ("spatial_only", "sink_dummy_only", "full"):
            abl[name + "_speedup"] = abl["all_global_ms"] / abl[name + "_ms"]
        abl["paper_whole_model_speedups_720p"] = {"spatial_only": 1.19, "sink_dummy_only": 1.04, "full": 1.31}
        phases["ablation"] = abl

    # ---- end to end: the host-buffer entry points of the C ABI (pinned host tensors), every copy inside the timed
    # region: headcast_append_host every 4th step, headcast_attend_host (query columns in, outputs out, overlapped
    # with the kernels stage by stage), stream synchronised before the clock stops
    host_q = [q.cpu().pin_memory() for q in q_extra[0]]
    host_kv = [(k.cpu().pin_memory(), v.cpu().pin_memory()) for k, v in kv[w.n_blocks:w.n_blocks + 2]]
    host_out = torch.empty_like(host_q[0]).pin_memory()
    e2e_steps = min(args.steps, 40)
    e2e_ms = []
    for i in range(-STEPS_PER_BLOCK, e2e_steps):  # the warm-up includes one append
        flush()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        if i % STEPS_PER_BLOCK == 0:
            hc.append_host(*host_kv[(i // STEPS_PER_BLOCK) % 2])
        hc.attend_host(host_q[i % STEPS_PER_BLOCK], host_out)
        b.record()
        b.synchronize()
        if i >= 0:
            e2e_ms.append(a.elapsed_time(b))
    hc.check()
    e2e = max_over_ranks(float(np.sum(e2e_ms)) / e2e_steps, dist, torch, "cuda")
    q_bytes = L * H * D * 2

    if rank != 0:
        return
    achieved = flops / kern / 1e9
    pct = lambda xs: {"p10": float(np.percentile(xs, 10)), "p50": float(np.percentile(xs, 50)), "p90": float(np.percentile(xs, 90))}
    line = {
        "metric": METRIC, "value": ms_per_step, "unit": "ms", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "heads": H, "head_dim": D, "grid": [w.grid_h, w.grid_w], "block_tokens": L,
                   "kv_tokens": w.n_blocks * L, "head_mix_sink_dummy_spatial_global": [int(sum(1 for v in w.labels if v == c)) for c in range(4)],
                   "step": "1 attend per step + 1 append per 4 steps", "sd_mode": args.sd_mode, "l2": "flushed between steps (256 MiB memset outside the events)",
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "clocks": clocks.summary(),
        "e2e": {"value": e2e, "unit": "ms", "h2d_bytes_per_step": q_bytes + block_bytes // STEPS_PER_BLOCK, "d2h_bytes_per_step": q_bytes},
        "gpu_launches": int(launches),
        "spread": {"step_ms": pct(step_ms), "attention_kernel_ms": pct(kernel_ms), "e2e_ms": pct(e2e_ms)},
        "roofline": {"bound": "tensor", "kernel": "attn_kernel (tcgen05)", "achieved": achieved, "peak": peaks["tflops"],
                     "unit": "TFLOP/s", "frac": achieved / peaks["tflops"], "peak_source": peaks["source"] + " (burst bf16 GEMM)",
                     "frac_of_sustained": achieved / peaks["tflops_sustained"] if peaks["tflops_sustained"] else None,
                     "frac_of_nominal_2250": achieved / 2250.0, "kernel_ms": kern, "flops_per_launch": flops,
                     "traffic": NCU_TRAFFIC_BYTES.get(w.name)},
        "phases": phases,
        "hbm_peak_gbs": peaks["hbm_gbs"],
    }
    if not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(w)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
