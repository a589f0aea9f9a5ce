"""Head sharding (paper_2607_20125_b200/sharding.py) on CPU: the dealing of heads, and two gloo ranks that run the
whole sequence - warm-up appends, dense attention, classification, re-dealing with cache transfer, split, a rolled
append, head-specific attention - against the unsharded oracle.  The ranks' local engine here is a stand-in built on
the oracle (test infrastructure only; the product's engine is the CUDA library)."""
import os
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2607_20125_b200 import sharding  # noqa: E402
from oracle import headcast_oracle as orc  # noqa: E402


def test_contiguous_split_covers_every_head_once():
    for n, w in [(12, 1), (12, 2), (12, 5), (12, 8), (64, 8), (7, 7)]:
        parts = sharding.contiguous_split(n, w)
        assert sorted(h for p in parts for h in p) == list(range(n))
        sizes = [len(p) for p in parts]
        assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)
        assert all(p == list(range(p[0], p[0] + len(p))) for p in parts)
    with pytest.raises(ValueError):
        sharding.contiguous_split(3, 4)


def test_partition_is_balanced_deterministic_and_leaves_no_rank_empty():
    rng = np.random.default_rng(0)
    for trial in range(200):
        world = int(rng.integers(1, 9))
        n = int(rng.integers(world, 65))
        costs = rng.choice([4680.0, 9360.0, 327.6, 32760.0], size=n).tolist()
        parts = sharding.partition_heads(costs, world)
        assert parts == sharding.partition_heads(list(costs), world)
        assert sorted(h for p in parts for h in p) == list(range(n))
        assert all(len(p) >= 1 and p == sorted(p) for p in parts)
        loads = [sum(costs[h] for h in p) for p in parts]
        # greedy bound: no rank carries more than the mean plus one (largest) head
        assert max(loads) <= sum(costs) / world + max(costs) + 1e-9
    # the paper's 480P mix on two ranks: contiguous runs would be 3:1 out of balance, the dealt heads are even
    labels = [orc.GLOBAL] * 3 + [orc.SPATIAL] * 4 + [orc.SINK] * 2 + [orc.DUMMY] * 3
    costs = [sharding.effective_keys(l, 4680, 8, 100) for l in labels]
    loads = [sum(costs[h] for h in p) for p in sharding.partition_heads(costs, 2)]
    naive = [sum(costs[h] for h in p) for p in sharding.contiguous_split(12, 2)]
    assert max(loads) / min(loads) < 1.6 < max(naive) / min(naive)


def test_effective_keys_follow_the_flop_count_of_the_oracle():
    geom = orc.Geometry.make(30, 50, 3, 10, 10)   # cells of equal size, so the cell share is exact
    L, d, n_filled = geom.block_tokens, 128, 5
    for labels in ([orc.GLOBAL], [orc.SINK], [orc.DUMMY], [orc.SPATIAL], [orc.GLOBAL, orc.SPATIAL, orc.SINK, orc.DUMMY]):
        keys = sum(sharding.effective_keys(l, L, n_filled, geom.n_cells) for l in labels)
        assert 4.0 * L * keys * d == pytest.approx(orc.attend_flops(geom, labels, n_filled, d), rel=1e-12)
    assert sharding.effective_keys(orc.SINK, L, 1, geom.n_cells, sd_blocks=2) == L
    assert sharding.effective_keys(orc.DUMMY, L, 5, geom.n_cells, sd_blocks=2) == 2 * L


RANK_SCRIPT = r"""
import os, sys
sys.path.insert(0, os.environ["HC_ROOT"])
import numpy as np
import torch
import torch.distributed as dist
from paper_2607_20125_b200 import sharding, synth
from oracle import headcast_oracle as orc

def bits(t):
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)

def to_bf16(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16)

class OracleEngine:
    # stand-in for binding.HeadCast over a subset of heads, built on the float64 oracle
    def __init__(self, n_heads, head_dim, geom, n_blocks):
        self.geom, self.cache, self.n_heads = geom, orc.CacheModel(n_blocks, n_heads), n_heads
    def append(self, k, v):
        assert k.shape[1] == self.n_heads
        self.cache.append(bits(k).copy(), bits(v).copy())
    def n_filled(self):
        return len(self.cache.blocks)
    def full_attend(self, q, out):
        out.copy_(to_bf16(orc.full_attend(bits(q), self.cache)[0]))
    def classify(self, q):
        return orc.classify(bits(q), self.cache, self.geom)
    def set_labels(self, labels):
        self.labels = list(labels)
    def split_cache(self):
        self.cache.split(self.labels)
    def attend(self, q, out):
        out.copy_(to_bf16(orc.attend(bits(q), self.cache, self.geom)))
    def export_cache_device(self, i):
        k, v = self.cache.mono_kv_bits(i)
        f = lambda a: torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16)
        return f(k), f(v)

dist.init_process_group("gloo", init_method="tcp://127.0.0.1:" + os.environ["HC_PORT"],
                        rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
rank = dist.get_rank()
w = synth.tiny()
geom = orc.Geometry.make(w.grid_h, w.grid_w, w.frames_per_block, w.cell_h, w.cell_w)
L, H, d = w.block_tokens, w.n_heads, w.head_dim
as_t = lambda a: torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16)

layer = sharding.HeadShardedHeadCast(H, d, L, geom.n_cells, engine_factory=OracleEngine, geom=geom, n_blocks=w.n_blocks)
whole = OracleEngine(H, d, geom, w.n_blocks)                 # the unsharded layer, same inputs
assert layer.heads == sharding.contiguous_split(H, 2)[rank]

n_warm = w.n_blocks + 1                                      # the ring has rolled once before the classification
for b in range(n_warm):
    k, v = synth.make_kv(w, b)
    layer.append(as_t(k), as_t(v)); whole.append(as_t(k), as_t(v))
q = as_t(synth.make_q(w, n_warm - 1, 0))
out, ref = torch.zeros((L, H, d), dtype=torch.bfloat16), torch.zeros((L, H, d), dtype=torch.bfloat16)
layer.full_attend(q, out); whole.full_attend(q, ref)
assert torch.equal(out.view(torch.int16), ref.view(torch.int16))

labels, scores = layer.classify(q)
ref_labels, ref_scores = whole.classify(q)
assert list(labels) == list(ref_labels) == list(w.labels), (labels, ref_labels, w.labels)
assert np.allclose(scores, ref_scores, rtol=1e-6, atol=1e-7)

costs = [sharding.effective_keys(int(l), L, whole.n_filled(), geom.n_cells) for l in labels]
want = sharding.partition_heads(costs, 2)
assert want != sharding.contiguous_split(H, 2), "the test should move at least one head"
layer.split_cache(labels)
assert layer.owner_heads == want and layer.engine.n_heads == len(want[rank])
whole.set_labels(ref_labels); whole.split_cache()
for i, h in enumerate(layer.heads):                          # the moved caches are the heads' caches, bit for bit
    for a, b in zip(layer.engine.cache.head_kv_bits(i), whole.cache.head_kv_bits(h)):
        assert np.array_equal(a, b)

for b in range(n_warm, n_warm + 2):                          # generation: rolled appends, four attends each
    k, v = synth.make_kv(w, b)
    layer.append(as_t(k), as_t(v)); whole.append(as_t(k), as_t(v))
    for step in range(2):
        q = as_t(synth.make_q(w, b, step))
        layer.attend(q, out); whole.attend(q, ref)
        assert torch.equal(out.view(torch.int16), ref.view(torch.int16))
dist.barrier()
dist.destroy_process_group()
print("rank", rank, "ok", layer.owner_heads)
"""


def _free_port() -> int:
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_match_the_unsharded_oracle():
    port = _free_port()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE="2", HC_PORT=str(port), HC_ROOT=ROOT, OMP_NUM_THREADS="2")
        procs.append(subprocess.Popen([sys.executable, "-c", RANK_SCRIPT], cwd=ROOT, env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=600) for p in procs]
    for r, (p, (out, err)) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, err[-3000:]
        assert f"rank {r} ok" in out
