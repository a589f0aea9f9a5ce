#!/usr/bin/env python
"""Benchmark of the HeadCast attention path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload all|480p|720p|1080p|tiny|rollout] [--impl reference]

Without --workload the three Wan-shaped configurations (480P, 720P, 1080P token grids) are measured one after the
other in one process; the printed line's value / config / roofline / e2e are the 1080P ones and `per_workload` holds
all three.

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
            "config": config_of(w, 1, args.sd_mode),
            "cpu_baseline": base, "e2e": {"value": value, "unit": "ms", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def run_rollout(args):
    """Streaming rollout at the 720P token grid (30 layers x 12 heads): per layer a 2-block dense warm-up, the third
    block appended and classified at its first denoise step, the split with 3 cached blocks, then `--blocks` generated
    blocks x 4 denoise steps, each block appended to (and rolled through) the per-archetype buffers of every layer.
    The dense arm repeats the generated blocks with headcast_full_attend on the monolithic caches kept alongside.
    Layer 0 is fed the seeded inputs with planted archetypes and keeps the labels its own classification returns
    (`labels_match_planted` says whether they are the planted ones); the other layers share seeded N(0,1) bf16 tensors
    drawn on the device and get their seeded 2/3/4/3 head mix through headcast_set_labels (their classification is
    timed, its labels replaced)."""
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
    w0 = synth.wan("720p", layer=0)
    from concurrent.futures import ThreadPoolExecutor
    with ThreadPoolExecutor(max_workers=8) as ex:
        kv0 = [tuple(to_dev(t, torch) for t in f.result()) for f in [ex.submit(synth.make_kv, w0, b) for b in range(3 + pool)]]
    q0 = to_dev(synth.make_q(w0, 2, 0), torch)
    planted_run = args.mix == "default" and args.ablation == "full"
    local = int(os.environ.get("LOCAL_RANK", "0"))
    layers = [HeadCast.from_workload(synth.wan("720p", layer=l), keep_monolithic=True) for l in range(args.layers)]
    mixes = (synth.reported_mixes("720p", args.layers) if args.mix == "reported"
             else [synth.wan("720p", layer=l).labels for l in range(args.layers)])
    if args.ablation != "full":
        mixes = [synth.ablation_labels(m)[args.ablation] for m in mixes]
    ev = lambda: torch.cuda.Event(enable_timing=True)
    t = {}
    a, b = ev(), ev()
    a.record()
    for li, hc in enumerate(layers):  # warm-up: two blocks, dense attention for their 4 steps each
        for blk in range(2):
            hc.append(*(kv0 if li == 0 else kv)[blk])
            for s_ in range(STEPS_PER_BLOCK):
                hc.full_attend(qs[s_], out)
    b.record(); b.synchronize()
    t["warmup_ms"] = a.elapsed_time(b)
    a, b = ev(), ev()
    a.record()
    labels_match_planted = None
    for li, (hc, mix) in enumerate(zip(layers, mixes)):
        hc.append(*(kv0 if li == 0 else kv)[2])
        labels, _ = hc.classify(q0 if li == 0 else qs[0])
        if li == 0:
            labels_match_planted = bool(tuple(int(v) for v in labels) == tuple(w0.labels))
        if not (li == 0 and planted_run):
            hc.set_labels(mix)
        hc.split_cache()
    b.record(); b.synchronize()
    t["classify_split_ms"] = a.elapsed_time(b)
    launches0 = sum(hc.launch_count() for hc in layers)
    a, b = ev(), ev()
    with ClockSampler(local) as hc_clocks:
        a.record()
        for blk in range(args.blocks):
            for li, hc in enumerate(layers):
                hc.append(*(kv0[3 + blk % pool] if li == 0 else kv[(3 + blk) % pool]))
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
    with ClockSampler(local) as dense_clocks:
        a.record()
        for blk in range(args.blocks):
            for hc in layers:
                for s_ in range(STEPS_PER_BLOCK):
                    hc.full_attend(qs[s_], out)
        b.record(); b.synchronize()
    t["dense_ms"] = a.elapsed_time(b)
    t["dense_clocks"] = dense_clocks.summary()
    t["labels_match_planted_layer0"] = labels_match_planted
    for hc in layers:
        hc.check()
    n_steps = args.blocks * STEPS_PER_BLOCK
    per_step = t["headcast_ms"] / n_steps
    print(json.dumps({
        "metric": "headcast_rollout_attention_ms_per_block_step_all_layers", "value": per_step, "unit": "ms", "n_gpus": 1,
        "steps": n_steps, "warmup": 0, "ms_per_step": per_step, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic (layer 0: seeded planted archetypes; other layers: seeded N(0,1) drawn on the device)",
        "config": {"workload": "rollout-720p", "head_mix": args.mix, "ablation": args.ablation,
                   "head_counts_sink_dummy_spatial_global": [int(sum(1 for m in mixes for v in m if v == c)) for c in range(4)],
                   "layers": args.layers, "blocks": args.blocks, "steps_per_block": STEPS_PER_BLOCK,
                   "heads": H, "head_dim": D, "grid": [base.grid_h, base.grid_w], "l2": "working set of 30 layers (48 GB) exceeds L2"},
        "gpu_launches": int(launches), "clocks": hc_clocks.summary(),
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


N_SM = 148
TENSOR_FLOP_PER_SM_CLK = 8192.0  # one SM retires a 128 x 128 x 16 bf16 product (524288 FLOP) in 64 clocks


def ncu_traffic_bytes(name: str):
    """dram__bytes_read.sum + dram__bytes_write.sum of one attention-kernel launch, as written down with the ncu
    capture under profiles/ (lines `workload bytes`); None where no capture of that size exists."""
    path = os.path.join(ROOT, "profiles", "attn_kernel_dram_traffic.txt")
    try:
        with open(path) as f:
            for line in f:
                parts = line.split("#")[0].split()
                if len(parts) >= 2 and parts[0] == name:
                    return float(parts[1])
    except OSError:
        pass
    return None


def gen_inputs(w, n_extra, torch):
    """Seeded K/V blocks (window + n_extra generated blocks) and queries, drawn on host threads, moved to the GPU."""
    from concurrent.futures import ThreadPoolExecutor
    with ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 4)) as ex:
        kv_f = [ex.submit(synth.make_kv, w, b) for b in range(w.n_blocks + n_extra)]
        q_fill_f = ex.submit(synth.make_q, w, w.n_blocks - 1, 0)
        q_f = [[ex.submit(synth.make_q, w, w.n_blocks + e, s) for s in range(STEPS_PER_BLOCK)] for e in range(n_extra)]
        kv = [tuple(to_dev(t, torch) for t in f.result()) for f in kv_f]
        q_fill = to_dev(q_fill_f.result(), torch)
        q_extra = [[to_dev(f.result(), torch) for f in row] for row in q_f]
    return kv, q_fill, q_extra


def algorithmic_bytes(w):
    """HBM bytes the method itself must move (bf16 K and V): one append after the split reads the block and writes
    every head but the Sink heads; the split reads and writes what is kept (Sink / Dummy heads one block, the others
    the whole window)."""
    L, H, D = w.block_tokens, w.n_heads, w.head_dim
    n_sink = sum(1 for v in w.labels if v == synth.SINK)
    n_sd = sum(1 for v in w.labels if v in (synth.SINK, synth.DUMMY))
    block = 2 * L * H * D * 2
    append = block + 2 * L * (H - n_sink) * D * 2
    kept = 2 * 2 * L * D * (n_sd + (H - n_sd) * w.n_blocks)
    return {"block": block, "append": append, "split": 2 * kept}


def measure_copy_path(w, kv, torch, HeadCast, flush, sd_mode):
    """Split and append on contexts that keep NO monolithic cache after the split: the method's own byte movement."""
    nbytes = algorithmic_bytes(w)
    res = {"append_bytes": nbytes["append"], "split_bytes": nbytes["split"]}
    split_ms = []
    hc = None
    for trial in range(3):
        if hc is not None:
            hc.destroy()
        hc = HeadCast.from_workload(w, keep_monolithic=False, sd_mode=sd_mode)
        for b in range(w.n_blocks):
            hc.append(*kv[b])
        hc.set_labels(w.labels)
        flush()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        hc.split_cache()
        b.record()
        b.synchronize()
        split_ms.append(a.elapsed_time(b))
    res["split_ms"] = float(np.median(split_ms))
    res["split_ms_trials"] = split_ms
    res["split_gbs"] = nbytes["split"] / res["split_ms"] / 1e6
    n_extra = len(kv) - w.n_blocks
    for i in range(3):
        hc.append(*kv[w.n_blocks + i % n_extra])
    res["append_ms"] = timed(torch, lambda: hc.append(*kv[w.n_blocks]), flush, 10)  # one launch, L2 flushed before
    res["append_gbs"] = nbytes["append"] / res["append_ms"] / 1e6
    n_b2b = 200
    flush()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for i in range(n_b2b):
        hc.append(*kv[w.n_blocks + i % n_extra])
    b.record()
    b.synchronize()
    res["append_back_to_back_ms"] = a.elapsed_time(b) / n_b2b
    res["append_back_to_back_gbs"] = nbytes["append"] / res["append_back_to_back_ms"] / 1e6
    # the same 200 appends as ONE CUDA graph launch: no host work between the kernels (the eager loop above pays a
    # Python call per 10-50 us kernel).  Capture records the launches and advances the host-side ring exactly as the
    # replay then advances the device-side one.
    try:
        graph = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                for i in range(n_b2b):
                    hc.append(*kv[w.n_blocks + i % n_extra])
        torch.cuda.synchronize()
        flush()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        graph.replay()
        b.record()
        b.synchronize()
        res["append_graph_ms"] = a.elapsed_time(b) / n_b2b
        res["append_graph_gbs"] = nbytes["append"] / res["append_graph_ms"] / 1e6
    except Exception as exc:  # report, do not hide
        res["append_graph_ms"] = None
        res["append_graph_error"] = str(exc)[:200]
    hc.check()
    hc.destroy()
    return res


def measure_workload(w, args, torch, HeadCast, peaks, dist, local, e2e_leg: bool):
    """Everything reported for one Wan-shaped workload: the K timed steps (attend + an append every 4th step), the
    one-time phases, a >= 2 s sustained leg for the clock sampler, the method-only copy path and, if asked, the
    end-to-end leg through the host-buffer entry points."""
    L, H, D = w.block_tokens, w.n_heads, w.head_dim
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    flush = lambda: flush_buf.zero_()
    n_extra = 2  # generated blocks fed round-robin once the cache rolls, each with its own 4 denoise-step queries
    kv, q_fill, q_extra = gen_inputs(w, n_extra, torch)
    out = torch.empty_like(q_fill)
    res, phases = {}, {}
    nbytes = algorithmic_bytes(w)

    hc = HeadCast.from_workload(w, keep_monolithic=True, sd_mode=args.sd_mode)
    for b in range(w.n_blocks):
        hc.append(*kv[b])
    torch.cuda.synchronize()
    hc.set_kernel_timing(True)
    if not args.no_phases:
        for _ in range(3):
            hc.full_attend(q_fill, out)
        dense_ms = timed(torch, lambda: hc.full_attend(q_fill, out), flush, 5 if w.name == "1080p" else 10)
        phases["dense_full_attend_ms"] = dense_ms
        phases["dense_tflops"] = hc.attend_flops(True) / dense_ms / 1e9
        t0 = time.perf_counter()
        labels, scores = hc.classify(q_fill)
        torch.cuda.synchronize()
        phases["classify_first_call_ms"] = (time.perf_counter() - t0) * 1e3
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        flush()
        a.record()
        labels, scores = hc.classify(q_fill)
        b.record()
        b.synchronize()
        phases["classify_ms"] = a.elapsed_time(b)
        phases["classify_over_dense"] = phases["classify_ms"] / dense_ms
        phases["labels_match_planted"] = bool(tuple(int(v) for v in labels) == tuple(w.labels))
        sc = np.asarray(scores, dtype=np.float64)
        phases["classify_margins"] = {"min_abs_cos_minus_theta": float(np.abs(sc[:, :3] - 0.95).min()),
                                      "min_abs_score_minus_theta": float(np.abs(sc[:, 5] - 0.755).min())}
        t = timed(torch, lambda: hc.append(*kv[w.n_blocks]), flush, 5)  # monolithic ring append (rolls)
        phases["append_monolithic_ms"] = t
        phases["append_monolithic_gbs"] = 2 * nbytes["block"] / t / 1e6
    else:
        hc.set_labels(w.labels)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    flush()
    a.record()
    hc.split_cache()
    b.record()
    b.synchronize()
    phases["split_with_monolithic_kept_ms"] = a.elapsed_time(b)

    def step(i):
        e = (i // STEPS_PER_BLOCK) % n_extra
        if i % STEPS_PER_BLOCK == 0:
            hc.append(*kv[w.n_blocks + e])
        hc.attend(q_extra[e][i % STEPS_PER_BLOCK], out)

    for i in range(args.warmup):
        step(i)
    hc.check()
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
    res["gpu_launches"] = int(hc.launch_count() - launches0)
    total_ms = max_over_ranks(float(np.sum(step_ms)), dist, torch, "cuda")
    res["ms_per_step"] = total_ms / args.steps
    attend_ms = float(np.mean([s - (append_ms[i // STEPS_PER_BLOCK] if i % STEPS_PER_BLOCK == 0 else 0.0)
                               for i, s in enumerate(step_ms)]))
    kern = float(np.mean(kernel_ms))
    flops = hc.attend_flops(False)
    res["clocks"] = clocks.summary()
    res["kernel_ms"] = kern
    res["flops_per_launch"] = flops
    res["attend_ms"] = attend_ms
    res["attend_tflops"] = flops / attend_ms / 1e9
    res["kernel_tflops"] = flops / kern / 1e9
    res["frac_of_measured_burst"] = res["kernel_tflops"] / peaks["tflops"]
    res["frac_of_measured_sustained"] = res["kernel_tflops"] / peaks["tflops_sustained"] if peaks["tflops_sustained"] else None
    res["frac_of_nominal_2250"] = res["kernel_tflops"] / 2250.0
    pct = lambda xs: {"p10": float(np.percentile(xs, 10)), "p50": float(np.percentile(xs, 50)), "p90": float(np.percentile(xs, 90))}
    res["spread"] = {"step_ms": pct(step_ms), "attention_kernel_ms": pct(kernel_ms)}
    if "dense_full_attend_ms" in phases:
        res["speedup_vs_dense"] = phases["dense_full_attend_ms"] / attend_ms
        res["ideal_speedup_by_flops"] = hc.attend_flops(True) / flops

    # ---- sustained leg: the same steps for >= 2 s of GPU time, so that the clock sampler sees the clocks the kernel
    # settles at under the power cap; the figure that compares workloads run at different clocks is FLOP per SM clock
    n_sus = 4 if args.no_sustained else int(min(20000, max(args.steps, 2000.0 / max(res["ms_per_step"], 1e-3))))
    sus_kernel = []
    with ClockSampler(local) as sus_clocks:
        for i in range(n_sus):
            flush()
            step(i)
            sus_kernel.append(hc.last_attention_kernel_ms())
        torch.cuda.synchronize()
    hc.check()
    sc_ = sus_clocks.summary()
    k_sus = float(np.mean(sus_kernel))
    res["sustained"] = {"steps": n_sus, "kernel_ms": k_sus, "kernel_tflops": flops / k_sus / 1e9,
                        "frac_of_measured_sustained": (flops / k_sus / 1e9) / peaks["tflops_sustained"] if peaks["tflops_sustained"] else None,
                        "clocks": sc_}
    for tag, k_ms, mhz in (("timed", kern, res["clocks"]["sm_mhz"]), ("sustained", k_sus, sc_["sm_mhz"])):
        if mhz:
            per_clk = flops / (k_ms * 1e-3 * mhz * 1e6 * N_SM)
            res["flop_per_sm_clk_" + tag] = per_clk
            res["tensor_pipe_frac_at_clock_" + tag] = per_clk / TENSOR_FLOP_PER_SM_CLK

    if args.ablations:
        # the paper's archetype ablation, attention only: a fresh context per label set, same cache content
        abl = {}
        for name, lab in synth.ablation_labels(w.labels).items():
            h2 = HeadCast.from_workload(w, keep_monolithic=False, sd_mode=args.sd_mode)
            for blk in range(w.n_blocks):
                h2.append(*kv[blk])
            h2.set_labels(lab)
            h2.split_cache()
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

    if e2e_leg:
        # end to end: the host-buffer entry points of the C ABI (pinned host tensors), every copy inside the timed
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
        q_bytes = L * H * D * 2
        res["e2e"] = {"value": max_over_ranks(float(np.sum(e2e_ms)) / e2e_steps, dist, torch, "cuda"), "unit": "ms",
                      "h2d_bytes_per_step": q_bytes + nbytes["block"] // STEPS_PER_BLOCK, "d2h_bytes_per_step": q_bytes,
                      "spread_ms": pct(e2e_ms)}
        del host_q, host_kv, host_out
    hc.destroy()
    if not args.no_phases:
        try:  # a side leg must not cost the run its headline line
            phases["copy_path_method_only"] = measure_copy_path(w, kv, torch, HeadCast, flush, args.sd_mode)
        except Exception as exc:
            phases["copy_path_method_only"] = {"error": repr(exc)[:300]}
    res["phases"] = phases
    del kv, q_fill, q_extra, out, flush_buf
    torch.cuda.empty_cache()
    return res


def write_pathway_table(w, args, torch, HeadCast, path, append):
    """Per-pathway accounting of one headcast_attend launch from the per-item trace: share of the key-tile work
    against share of the time CTAs spent on the items (markdown, appended to `path`)."""
    kv, q_fill, q_extra = gen_inputs(w, 1, torch)
    hc = HeadCast.from_workload(w, keep_monolithic=False, sd_mode=args.sd_mode)
    for b in range(w.n_blocks):
        hc.append(*kv[b])
    hc.set_labels(w.labels)
    hc.split_cache()
    out = torch.empty_like(q_fill)
    for _ in range(3):
        hc.attend(q_fill, out)
    hc.set_tracing(True)
    hc.attend(q_fill, out)
    hc.check()
    rows = hc.read_trace()
    hc.set_tracing(False)
    hc.destroy()
    names = {synth.SINK: "Sink+Dummy", synth.DUMMY: "Sink+Dummy", synth.GLOBAL: "Global", synth.SPATIAL: "Spatial"}
    acc = {}
    for cta, head, cell, n_rows, n_tiles, mode, t0, t1 in rows:
        lone = n_rows <= 128
        for key in (names[w.labels[head]], "lone query tiles (any pathway)" if lone else None):
            if key is None:
                continue
            a = acc.setdefault(key, [0, 0.0, 0.0, 0])
            a[0] += 1
            a[1] += float(n_rows) * n_tiles * 128 * 4 * w.head_dim  # FLOPs incl. the padding of the last key tile
            a[2] += (t1 - t0) * 1e-3
            a[3] += int(mode == 1)
    tot_f = sum(v[1] for k, v in acc.items() if not k.startswith("lone"))
    tot_t = sum(v[2] for k, v in acc.items() if not k.startswith("lone"))
    span = (rows[:, 7].max() - rows[:, 6].min()) * 1e-3
    with open(path, "a" if append else "w") as f:
        if not append:
            f.write("# headcast_attend: work items by pathway (per-item device timers, one launch)\n\n"
                    "Command: `python bench.py --pathways <this file>`.  FLOPs count rows x key tiles x 128 keys "
                    "(the padded last tile included);\nCTA time is the sum over items of (end - start) of query tile 0's warps.\n\n")
        f.write(f"## {w.name}: {len(rows)} items on {N_SM} CTAs, launch span {span:.1f} us, "
                f"CTA-time / (span x {N_SM}) = {tot_t / (span * N_SM):.3f}\n\n")
        f.write("| pathway | items | cut items (partials) | share of FLOPs | share of CTA time | time share / FLOP share |\n|---|---|---|---|---|---|\n")
        for key in ("Sink+Dummy", "Global", "Spatial", "lone query tiles (any pathway)"):
            if key in acc:
                n, fl, tm, cut = acc[key]
                f.write(f"| {key} | {n} | {cut} | {fl / tot_f:.3f} | {tm / tot_t:.3f} | {(tm / tot_t) / max(fl / tot_f, 1e-9):.2f} |\n")
        f.write("\n")


WAN_WORKLOADS = ("480p", "720p", "1080p")
HEADLINE = "1080p"


def roofline_of(r, w, args, peaks):
    """The `roofline` object of the headline workload.  Denominator: the measured cuBLAS bf16 rate of this machine - the
    sustained figure when the timed steps ran at the power cap (the clock sampler saw `sw_power_cap` and a median SM
    clock below 90 % of the maximum over a timed region of at least 50 ms: that is how the sustained figure itself was
    measured), else the burst figure; both fractions, and the one against the nominal 2250 TFLOP/s, are always given
    by name."""
    timed_s = args.steps * r["ms_per_step"] * 1e-3
    clocks = r["clocks"]
    capped = ("sw_power_cap" in (clocks.get("reasons") or []) and clocks.get("sm_mhz") and clocks.get("sm_max_mhz")
              and clocks["sm_mhz"] < 0.9 * clocks["sm_max_mhz"])
    sustained = bool(peaks["tflops_sustained"]) and timed_s >= 0.05 and bool(capped)
    peak = peaks["tflops_sustained"] if sustained else peaks["tflops"]
    return {"bound": "tensor", "kernel": "attn_kernel (tcgen05)", "achieved": r["kernel_tflops"], "peak": peak,
            "unit": "TFLOP/s", "frac": r["kernel_tflops"] / peak,
            "peak_source": peaks["source"] + (" (sustained bf16 GEMM: %.2f s of steps at %d MHz under sw_power_cap)" % (timed_s, clocks["sm_mhz"]) if sustained
                                               else " (burst bf16 GEMM)"),
            "frac_of_measured_burst": r["frac_of_measured_burst"], "frac_of_measured_sustained": r["frac_of_measured_sustained"],
            "frac_of_nominal": r["frac_of_nominal_2250"], "nominal_peak": 2250.0,
            "bar_met_nominal": bool(r["frac_of_nominal_2250"] > 0.5),
            "tensor_pipe_frac_at_sampled_clock": r.get("tensor_pipe_frac_at_clock_sustained"),
            "kernel_ms": r["kernel_ms"], "flops_per_launch": r["flops_per_launch"],
            "traffic": ncu_traffic_bytes(w.name)}


def config_of(w, world=1, sd_mode=0):
    """The `config` object both arms print (same keys, so that the two lines describe the same workload)."""
    return {"workload": w.name, "heads": w.n_heads, "head_dim": w.head_dim, "grid": [w.grid_h, w.grid_w],
            "block_tokens": w.block_tokens, "kv_tokens": w.n_blocks * w.block_tokens,
            "head_mix_sink_dummy_spatial_global": [int(sum(1 for v in w.labels if v == c)) for c in range(4)],
            "step": "1 attend per step + 1 append per 4 steps", "sd_mode": sd_mode,
            "l2": "flushed between steps (256 MiB memset outside the events)",
            "parallelism": "replicas only" if world > 1 else "single GPU"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--workload", default="all", choices=["all", "tiny", "480p", "720p", "1080p", "rollout"],
                    help="all (default): 480p, 720p and 1080p in one process, the 1080p line as the headline")
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
    ap.add_argument("--pathways", default=None, metavar="FILE",
                    help="also write a per-pathway table (share of FLOPs vs share of CTA time, from the per-item trace) to FILE")
    ap.add_argument("--copy-only", action="store_true",
                    help="only the method's byte movement of one workload (split and appends without a monolithic cache): "
                         "a short run for profiler captures of the copy kernel")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-phases", action="store_true")
    ap.add_argument("--no-sustained", action="store_true", help="skip the >= 2 s sustained leg (short runs for profiler captures)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.workload == "rollout":
        if args.impl == "reference":
            args.workload = "720p"
        else:
            return run_rollout(args)
    names = list(WAN_WORKLOADS) if args.workload == "all" else [args.workload]
    headline = HEADLINE if args.workload == "all" else args.workload
    if args.impl == "reference":
        return run_reference(args, workload_of(headline))
    if args.shard == "heads":
        return run_sharded(args, workload_of(headline))

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
    if args.copy_only:
        w = workload_of(headline)
        flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
        kv, _, _ = gen_inputs(w, 2, torch)
        res = measure_copy_path(w, kv, torch, HeadCast, lambda: flush_buf.zero_(), args.sd_mode)
        print(json.dumps({"workload": w.name, "copy_path_method_only": res, "hbm_peak_gbs": peaks["hbm_gbs"]}))
        return

    per = {}
    for name in names:
        w = workload_of(name)
        if name == headline or world > 1:
            per[name] = measure_workload(w, args, torch, HeadCast, peaks, dist, local, e2e_leg=(name == headline))
        else:
            try:  # the smaller workloads ride along; a failure there is reported and the headline still measured
                per[name] = measure_workload(w, args, torch, HeadCast, peaks, dist, local, e2e_leg=False)
            except Exception as exc:
                per[name] = {"error": repr(exc)[:300]}
                torch.cuda.empty_cache()
        if args.pathways and rank == 0:
            write_pathway_table(w, args, torch, HeadCast, args.pathways, append=(name != names[0]))
    if dist is not None:
        dist.barrier()
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    w = workload_of(headline)
    r = per[headline]
    line = {
        "metric": METRIC, "value": r["ms_per_step"], "unit": "ms", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": r["ms_per_step"], "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": config_of(w, world, args.sd_mode),
        "clocks": r["clocks"],
        "e2e": r.get("e2e"),
        "gpu_launches": r["gpu_launches"],
        "spread": r["spread"],
        "roofline": roofline_of(r, w, args, peaks),
        "speedup_vs_dense": r.get("speedup_vs_dense"),
        "phases": r["phases"],
        "per_workload": {n: {k: v for k, v in per[n].items() if k != "e2e"} for n in per},
        "hbm_peak_gbs": peaks["hbm_gbs"],
        "paper_reported_speedups": "up to 1.62x at 720P and 1.95x at 1080P, whole model end to end, GPU not stated",
    }
    if not args.no_cpu_baseline:
        try:
            line["cpu_baseline"] = cpu_baseline(w)
        except Exception as exc:  # reported, not hidden; the GPU numbers above stand on their own
            line["cpu_baseline"] = {"value": None, "unit": "ms", "cores": os.cpu_count(), "kind": "oracle", "sample": "failed: " + repr(exc)[:200]}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
