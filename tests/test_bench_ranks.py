"""The multi-process side of bench.py, on CPU: the path does not shard, `--gpus N` runs N independent replicas and
only the timing is reduced (maximum over ranks).  Two gloo ranks check that reduction, and two processes launched
the way the driver launches the reference arm check that rank 0 alone prints the JSON line."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

RANK_SCRIPT = r"""
import os, sys
sys.path.insert(0, os.environ["HC_ROOT"])
import torch
import torch.distributed as dist
import bench
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:" + os.environ["HC_PORT"],
                        rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
rank = dist.get_rank()
mine = [3.5, 7.25][rank]
got = bench.max_over_ranks(mine, dist, torch, "cpu")
assert got == 7.25, (rank, got)
assert bench.max_over_ranks(mine, None, torch, "cpu") == mine
dist.barrier()
dist.destroy_process_group()
print("rank", rank, "ok")
"""


def _free_port() -> int:
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _spawn(code_or_args, rank, world, port, code=True):
    env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
               MASTER_PORT=str(port), HC_PORT=str(port), HC_ROOT=ROOT)
    args = [sys.executable, "-c", code_or_args] if code else [sys.executable] + code_or_args
    return subprocess.Popen(args, cwd=ROOT, env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True)


def test_timing_is_the_maximum_over_two_gloo_ranks():
    port = _free_port()
    procs = [_spawn(RANK_SCRIPT, r, 2, port) for r in range(2)]
    outs = [p.communicate(timeout=240) for p in procs]
    for r, (p, (out, err)) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, err[-2000:]
        assert f"rank {r} ok" in out


def test_reference_arm_prints_one_line_from_rank_zero_only():
    port = _free_port()
    args = [os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny", "--gpus", "2", "--steps", "1",
            "--warmup", "3"]
    procs = [_spawn(args, r, 2, port, code=False) for r in range(2)]
    outs = [p.communicate(timeout=600) for p in procs]
    for p, (out, err) in zip(procs, outs):
        assert p.returncode == 0, err[-2000:]
    assert outs[1][0].strip() == "", "ranks other than 0 exit without work or output"
    lines = [l for l in outs[0][0].splitlines() if l.strip()]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["unit"] == "ms"
    assert line["higher_is_better"] is False and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"] == {"value": line["value"], "unit": "ms", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert line["config"]["workload"] == "tiny"


def test_both_arms_describe_the_same_workload_and_the_roofline_follows_the_regime():
    sys.path.insert(0, ROOT)
    import argparse
    import bench
    from paper_2607_20125_b200 import synth
    w = synth.wan("1080p")
    # the reference arm and the CUDA arm print the same `config` object (same keys, same values at one GPU)
    assert bench.config_of(w, 1, 0) == bench.config_of(w, 1, 0) and bench.config_of(w)["workload"] == "1080p"
    assert set(bench.config_of(w, 2, 0)) == set(bench.config_of(w, 1, 0))
    # algorithmic bytes of the copy path: append reads the block and writes every head but the two Sink heads
    nb = bench.algorithmic_bytes(synth.wan("480p"))
    assert abs(nb["append"] / 1e6 - 52.7) < 0.1 and abs(nb["split"] / 1e6 - 258.8) < 0.1 and abs(nb["block"] / 1e6 - 28.8) < 0.1
    # DRAM traffic comes from the capture written under profiles/, not from a literal
    assert bench.ncu_traffic_bytes("1080p") > bench.ncu_traffic_bytes("720p") > bench.ncu_traffic_bytes("480p") > 1e8
    assert bench.ncu_traffic_bytes("tiny") is None
    peaks = {"tflops": 1600.0, "tflops_sustained": 1400.0, "hbm_gbs": 6500.0, "source": "measured"}
    r = {"ms_per_step": 8.0, "kernel_tflops": 980.0, "kernel_ms": 8.0, "flops_per_launch": 8.0e12, "frac_of_measured_burst": 980 / 1600,
         "frac_of_measured_sustained": 0.7, "frac_of_nominal_2250": 980 / 2250,
         "clocks": {"reasons": ["sw_power_cap"], "sm_mhz": 1650.0, "sm_max_mhz": 1965}}
    long_run = bench.roofline_of(r, w, argparse.Namespace(steps=40), peaks)
    assert long_run["peak"] == 1400.0 and abs(long_run["frac"] - 0.7) < 1e-12 and "sustained" in long_run["peak_source"]
    assert long_run["bar_met_nominal"] is False and long_run["frac_of_nominal"] < 0.5
    short = bench.roofline_of(dict(r, ms_per_step=0.35), w, argparse.Namespace(steps=40), peaks)
    assert short["peak"] == 1600.0 and "burst" in short["peak_source"]  # 14 ms of steps: a burst
    cool = bench.roofline_of(dict(r, clocks={"reasons": [], "sm_mhz": 1965.0, "sm_max_mhz": 1965}), w, argparse.Namespace(steps=40), peaks)
    assert cool["peak"] == 1600.0
    fast = bench.roofline_of(dict(r, clocks={"reasons": ["sw_power_cap"], "sm_mhz": 1900.0, "sm_max_mhz": 1965}), w,
                             argparse.Namespace(steps=40), peaks)
    assert fast["peak"] == 1600.0  # the cap touched, the clock not held down: still the burst figure
