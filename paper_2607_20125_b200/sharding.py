"""Head-sharded HeadCast layer over several GPUs, one process per GPU.

The pathways of Sec. 3 are per head: a head's cache, its classification (Eq. 2-5), the split and the attention never
look at another head.  A layer therefore shards by head.  Every rank owns a ``HeadCast`` context over its own heads,
takes its columns of Q / K / V (which every rank holds in full, as after a tensor-parallel QKV projection with the
weights replicated), and the outputs are all-gathered along the head dimension: one exchange of L x H x d bf16 per
attend, nothing else on the data path.

Before the classification the heads are dealt in equal, contiguous runs.  The classification tells what each head
will cost from then on (its effective key count, App. B), so the heads are dealt again, heaviest first onto the
least loaded rank, and the monolithic caches of the heads that change owner move once, point to point.  Only then
is the cache split.

The module holds no arithmetic of the method: it calls a local engine (``HeadCast`` by default, i.e. the CUDA
library; nothing here falls back to the CPU) and ``torch.distributed``.
"""
from __future__ import annotations

from typing import Callable, List, Optional, Sequence

SINK, DUMMY, SPATIAL, GLOBAL = 0, 1, 2, 3


def contiguous_split(n_heads: int, world_size: int) -> List[List[int]]:
    """Heads 0..n_heads-1 in world_size contiguous runs whose lengths differ by at most one (longer runs first)."""
    if world_size < 1 or n_heads < world_size:
        raise ValueError("need at least one head per rank")
    base, extra = divmod(n_heads, world_size)
    out, h = [], 0
    for r in range(world_size):
        n = base + (1 if r < extra else 0)
        out.append(list(range(h, h + n)))
        h += n
    return out


def effective_keys(label: int, block_tokens: int, n_filled: int, n_cells: int, sd_blocks: int = 1) -> float:
    """Keys one query of a head of this class attends to (App. B): one block (two in the appendix variant) for Sink
    and Dummy, the cell's share of the cache for Spatial, the whole cache for Global."""
    cache = float(block_tokens) * n_filled
    if label in (SINK, DUMMY):
        return float(block_tokens) * min(sd_blocks, n_filled)
    if label == SPATIAL:
        return cache / max(1, n_cells)
    if label == GLOBAL:
        return cache
    raise ValueError(f"unknown class {label}")


def partition_heads(costs: Sequence[float], world_size: int) -> List[List[int]]:
    """Deals heads to ranks so that the summed cost per rank is about equal: heaviest head first (ties by head index)
    onto the least loaded rank (ties by rank), every rank getting at least one head.  Deterministic, so every rank
    computes the same answer without talking.  Each rank's heads are returned in ascending order."""
    n = len(costs)
    if world_size < 1 or n < world_size:
        raise ValueError("need at least one head per rank")
    order = sorted(range(n), key=lambda h: (-float(costs[h]), h))
    load = [0.0] * world_size
    out: List[List[int]] = [[] for _ in range(world_size)]
    for i, h in enumerate(order):
        left = n - i                                  # heads not placed yet, this one included
        empty = [r for r in range(world_size) if not out[r]]
        cand = empty if len(empty) >= left else range(world_size)   # keep enough heads for the ranks still empty
        r = min(cand, key=lambda x: (load[x], x))
        out[r].append(h)
        load[r] += float(costs[h])
    return [sorted(hs) for hs in out]


class HeadShardedHeadCast:
    """One attention layer, its heads spread over the ranks of a process group.

    ``engine_factory(n_heads=..., **engine_kw)`` builds the local engine; it must offer ``append``, ``full_attend``,
    ``classify``, ``set_labels``, ``split_cache``, ``attend``, ``n_filled`` and ``export_cache_device`` with the
    meaning they have in ``binding.HeadCast``.  All tensors are ``[L, H, d]`` bf16 on the engine's device, the same
    on every rank; outputs are complete on every rank when a call returns.
    """

    def __init__(self, n_heads: int, head_dim: int, block_tokens: int, n_cells: int, group=None,
                 engine_factory: Optional[Callable] = None, sd_blocks: int = 1, **engine_kw):
        import torch.distributed as dist
        if engine_factory is None:
            from .binding import HeadCast
            engine_factory = HeadCast
        self.dist, self.group = dist, group
        self.rank, self.world = dist.get_rank(group), dist.get_world_size(group)
        self.n_heads, self.head_dim, self.block_tokens, self.n_cells = n_heads, head_dim, block_tokens, n_cells
        self.sd_blocks = sd_blocks
        self._factory, self._kw = engine_factory, dict(engine_kw)
        self.owner_heads = contiguous_split(n_heads, self.world)
        self.engine = self._factory(n_heads=len(self.heads), head_dim=head_dim, **self._kw)
        self.labels: Optional[List[int]] = None
        self._idx = {}

    # ------------------------------------------------------------------ helpers
    @property
    def heads(self) -> List[int]:
        return self.owner_heads[self.rank]

    def _index(self, r: int, device):
        """Head indices of rank r as a tensor on `device` (built once per dealing: no host copy per call)."""
        key = (r, str(device))
        if key not in self._idx:
            import torch
            self._idx[key] = torch.tensor(self.owner_heads[r], dtype=torch.long, device=device)
        return self._idx[key]

    def _mine(self, t):
        """This rank's head columns of an [L, H, d] tensor, contiguous."""
        hs = self.heads
        if hs == list(range(hs[0], hs[0] + len(hs))):
            return t if len(hs) == t.shape[1] else t[:, hs[0]:hs[0] + len(hs), :].contiguous()
        return t.index_select(1, self._index(self.rank, t.device))

    def _gather_heads(self, local, out) -> None:
        """all-gather of [L, H_local, d] pieces (padded to the largest piece) into out[L, H, d]."""
        import torch
        if self.world == 1:
            out.copy_(local)
            return
        h_max = max(len(hs) for hs in self.owner_heads)
        if local.shape[1] == h_max:
            piece = local
        else:
            piece = local.new_zeros((local.shape[0], h_max, local.shape[2]))
            piece[:, : local.shape[1]] = local
        pieces = [torch.empty_like(piece) for _ in range(self.world)]
        # moved as bytes: the exchange only copies, and not every backend knows bf16
        self.dist.all_gather([p.view(torch.uint8) for p in pieces], piece.view(torch.uint8), group=self.group)
        for r, hs in enumerate(self.owner_heads):
            out.index_copy_(1, self._index(r, out.device), pieces[r][:, : len(hs)])

    # ------------------------------------------------------------------ the layer's calls
    def append(self, k_new, v_new) -> None:
        self._device = k_new.device
        self.engine.append(self._mine(k_new), self._mine(v_new))

    def full_attend(self, q, out) -> None:
        local = self._mine(q)
        res = local.new_empty(local.shape)
        self.engine.full_attend(local, res)
        self._gather_heads(res, out)

    def classify(self, q):
        """Labels and scores of ALL heads, identical on every rank (each rank classifies its own heads)."""
        import numpy as np
        import torch
        labels, scores = self.engine.classify(self._mine(q))
        n_sc = scores.shape[1]
        h_max = max(len(hs) for hs in self.owner_heads)
        mine = torch.zeros((h_max, 1 + n_sc), dtype=torch.float64)
        mine[: len(self.heads), 0] = torch.from_numpy(np.asarray(labels, dtype=np.float64))
        mine[: len(self.heads), 1:] = torch.from_numpy(np.asarray(scores, dtype=np.float64))
        mine = mine.to(q.device)
        if self.world == 1:
            pieces = [mine]
        else:
            pieces = [torch.empty_like(mine) for _ in range(self.world)]
            self.dist.all_gather(pieces, mine, group=self.group)
        all_labels = np.zeros(self.n_heads, dtype=np.int32)
        all_scores = np.zeros((self.n_heads, n_sc), dtype=np.float32)
        for r, hs in enumerate(self.owner_heads):
            p = pieces[r].cpu().numpy()
            all_labels[hs] = p[: len(hs), 0].astype(np.int32)
            all_scores[hs] = p[: len(hs), 1:].astype(np.float32)
        return all_labels, all_scores

    def split_cache(self, labels: Sequence[int], rebalance: bool = True) -> None:
        """Fixes the labels of all heads, re-deals the heads by cost (unless ``rebalance`` is off), moves the caches
        of the heads that change owner, and splits every rank's cache into the per-archetype buffers."""
        labels = [int(v) for v in labels]
        if len(labels) != self.n_heads:
            raise ValueError("one label per head")
        if rebalance and self.world > 1:
            n_filled = self.engine.n_filled()
            costs = [effective_keys(l, self.block_tokens, n_filled, self.n_cells, self.sd_blocks) for l in labels]
            self._redeal(partition_heads(costs, self.world))
        self.labels = labels
        self.engine.set_labels([labels[h] for h in self.heads])
        self.engine.split_cache()

    def attend(self, q, out) -> None:
        local = self._mine(q)
        res = local.new_empty(local.shape)
        self.engine.attend(local, res)
        self._gather_heads(res, out)

    # ------------------------------------------------------------------ re-dealing the heads
    def _redeal(self, new_owner_heads: List[List[int]]) -> None:
        """Moves every head whose owner changes (its monolithic K and V, logical order) and rebuilds the local engine
        over the new head set by appending the blocks again.  Transfers go head by head in index order, so the
        blocking send / recv pairs of all ranks form one sequence and cannot wait on each other in a cycle."""
        import torch
        old_of = {h: r for r, hs in enumerate(self.owner_heads) for h in hs}
        new_of = {h: r for r, hs in enumerate(new_owner_heads) for h in hs}
        if old_of == new_of:
            return
        n_filled = self.engine.n_filled()
        rows = n_filled * self.block_tokens
        kept = {}
        for h in range(self.n_heads):
            src, dst = old_of[h], new_of[h]
            if src == self.rank:
                k, v = self.engine.export_cache_device(self.heads.index(h))   # [rows, d] bf16 each
                if dst == self.rank:
                    kept[h] = (k, v)
                else:
                    self.dist.send(k.view(torch.uint8), dst, group=self.group)
                    self.dist.send(v.view(torch.uint8), dst, group=self.group)
            elif dst == self.rank:
                k = torch.empty((rows, self.head_dim), dtype=torch.bfloat16, device=self._device)
                v = torch.empty_like(k)
                self.dist.recv(k.view(torch.uint8), src, group=self.group)
                self.dist.recv(v.view(torch.uint8), src, group=self.group)
                kept[h] = (k, v)
        self.owner_heads = new_owner_heads
        self._idx = {}
        self._rebuild(kept, n_filled)

    def _rebuild(self, kept, n_filled: int) -> None:
        """A fresh local engine over this rank's heads, filled by appending the blocks of ``kept`` (head -> (K, V),
        [n_filled * L, d] in logical order: sink block first, newest last) once more.  Later appends roll the new
        ring exactly as they would have rolled the old one."""
        import torch
        old_engine = self.engine
        self.engine = self._factory(n_heads=len(self.heads), head_dim=self.head_dim, **self._kw)
        L = self.block_tokens
        for b in range(n_filled):
            k_b = torch.stack([kept[h][0][b * L:(b + 1) * L] for h in self.heads], dim=1).contiguous()
            v_b = torch.stack([kept[h][1][b * L:(b + 1) * L] for h in self.heads], dim=1).contiguous()
            self.engine.append(k_b, v_b)
        if hasattr(old_engine, "destroy"):
            old_engine.destroy()
