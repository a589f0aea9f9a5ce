"""Seeded synthetic workloads for the HeadCast attention path.

This module only *draws inputs*: bf16 Q/K/V bytes with the shapes of an
autoregressive video DiT attention layer (3-frame blocks over a G_h x G_w
latent token grid, sink block + sliding window) and, per head, a planted
pattern that makes the head behave like one of the paper's four archetypes
(Observations 1-2, Appendix A).  It holds none of the method's arithmetic (no
attention, no scoring, no cache policy), so the CPU oracle and the CUDA path
can both be fed from it without sharing any code of the method itself.

All tensors are returned as ``numpy.uint16`` arrays holding bf16 bit patterns,
so that both sides consume exactly the same bytes.

Token order inside a block is frame-major, then grid row, then grid column:
``t = f * (G_h * G_w) + y * G_w + x``.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Sequence, Tuple

import numpy as np

SINK, DUMMY, SPATIAL, GLOBAL = 0, 1, 2, 3
LABEL_NAMES = ("sink", "dummy", "spatial", "global")
BASE_SEED = 20260720


@dataclass(frozen=True)
class Workload:
    """Shape of one attention layer plus the planted head mix."""

    name: str
    n_heads: int
    head_dim: int
    grid_h: int
    grid_w: int
    n_blocks: int  # cache capacity in blocks, sink block and newest block included
    frames_per_block: int = 3
    cell_h: int = 10
    cell_w: int = 10
    labels: Tuple[int, ...] = ()  # planted archetype per head (original head order)
    # strengths of the planted patterns (see plant_* below)
    sink_alpha: float = 6.0
    dummy_lift: float = 20.0  # logit lift (nats) of same-block keys for a Dummy head
    spatial_peak: float = 32.0  # logit (nats) of a key at the query's own grid position
    spatial_len: float = 1.25  # length scale (tokens) of the positional code
    seed: int = BASE_SEED

    @property
    def tokens_per_frame(self) -> int:
        return self.grid_h * self.grid_w

    @property
    def block_tokens(self) -> int:
        return self.frames_per_block * self.tokens_per_frame


def _mix(n_heads: int, counts: Sequence[int], seed: int) -> Tuple[int, ...]:
    """Seeded interleaving of ``counts`` = (n_sink, n_dummy, n_spatial, n_global)."""
    labels = np.repeat(np.arange(4), counts)
    assert labels.size == n_heads
    rng = np.random.Generator(np.random.PCG64([seed, 0xC1A55]))
    return tuple(int(v) for v in rng.permutation(labels))


def tiny(cell: int = 10, seed: int = BASE_SEED) -> Workload:
    """4 heads x d=64, 8x8 grid, one head per archetype, 5-block cache (sink + 4)."""
    return Workload("tiny", 4, 64, 8, 8, 5, cell_h=cell, cell_w=cell,
                    labels=(SINK, DUMMY, SPATIAL, GLOBAL), sink_alpha=10.0,
                    dummy_lift=20.0, spatial_peak=36.0, seed=seed)


def wan(resolution: str, seed: int = BASE_SEED, layer: int = 0) -> Workload:
    """12 heads x d=128 layer at the 480P / 720P / 1080P token grids, 7-block cache,
    head mix 2 Sink / 3 Dummy / 4 Spatial / 3 Global in a seeded interleaved order."""
    grids = {"480p": (30, 52), "720p": (45, 80), "1080p": (68, 120)}
    gh, gw = grids[resolution.lower()]
    return Workload(resolution.lower(), 12, 128, gh, gw, 7,
                    labels=_mix(12, (2, 3, 4, 3), seed + 7919 * layer), seed=seed + 7919 * layer)


# Head counts out of 30 layers x 12 heads that the paper reports for LongLive at t = 1000 (appendix table of the
# archetype distribution), rounded so that each row sums to 360: (Sink, Dummy, Spatial, Global).
REPORTED_HEAD_COUNTS = {"480p": (2, 94, 168, 96), "720p": (2, 98, 167, 93), "1080p": (2, 92, 203, 63)}


def reported_mixes(resolution: str, n_layers: int = 30, seed: int = BASE_SEED):
    """Per-layer label tuples whose totals follow REPORTED_HEAD_COUNTS: the 360 labels are shuffled (seeded) over
    the layers, so layers differ in their mix and some have no Sink or no Dummy head at all."""
    counts = REPORTED_HEAD_COUNTS[resolution.lower()]
    labels = np.repeat(np.arange(4), counts)
    rng = np.random.Generator(np.random.PCG64([seed, 0x7AB1E6]))
    labels = rng.permutation(labels).reshape(30, 12)
    return [tuple(int(v) for v in labels[l % 30]) for l in range(n_layers)]


def ablation_labels(labels: Sequence[int]):
    """The label sets of the paper's archetype ablation: all heads Global; only the Spatial heads sparse; only the
    Sink and Dummy heads sparse; everything."""
    lab = np.asarray(labels)
    return {
        "all_global": tuple(int(GLOBAL) for _ in lab),
        "spatial_only": tuple(int(v) if v == SPATIAL else int(GLOBAL) for v in lab),
        "sink_dummy_only": tuple(int(v) if v in (SINK, DUMMY) else int(GLOBAL) for v in lab),
        "full": tuple(int(v) for v in lab),
    }


def small(seed: int = BASE_SEED, **kw) -> Workload:
    """A mid-size case for CPU-speed parity runs: ragged tiles, several cells, d=128."""
    base = Workload("small", 6, 128, 13, 22, 4, cell_h=5, cell_w=7,
                    labels=(GLOBAL, SPATIAL, SINK, DUMMY, SPATIAL, GLOBAL),
                    sink_alpha=8.0, seed=seed)
    return replace(base, **kw)


# --------------------------------------------------------------------------- bf16 helpers


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (round to nearest even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


# --------------------------------------------------------------------------- draws


def _rng(w: Workload, *stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64([w.seed, *[int(s) & 0xFFFFFFFF for s in stream]]))


_TAG_Q, _TAG_K, _TAG_V, _TAG_DIR, _TAG_POS = 1, 2, 3, 4, 5


def _normal(w: Workload, tag: int, block: int, step: int) -> np.ndarray:
    g = _rng(w, tag, block, step)
    return g.standard_normal((w.block_tokens, w.n_heads, w.head_dim), dtype=np.float32)


def _block_direction(w: Workload, head: int, block: int) -> np.ndarray:
    """Unit direction shared by the queries and keys of one absolute block (Dummy plant)."""
    g = _rng(w, _TAG_DIR, head, block)
    v = g.standard_normal(w.head_dim)
    return (v / np.linalg.norm(v)).astype(np.float32)


def _position_code(w: Workload, head: int) -> np.ndarray:
    """[T_f, d] random Fourier features of a Gaussian kernel over grid positions, so that
    code(p) . code(p') ~= exp(-|p - p'|^2 / (2 len^2)) (Spatial plant)."""
    g = _rng(w, _TAG_POS, head)
    d = w.head_dim
    omega = g.standard_normal((d, 2)) / w.spatial_len
    phase = g.uniform(0.0, 2.0 * np.pi, size=d)
    ys, xs = np.divmod(np.arange(w.tokens_per_frame), w.grid_w)
    pos = np.stack([ys, xs], axis=1).astype(np.float64)
    code = np.sqrt(2.0 / d) * np.cos(pos @ omega.T + phase)
    return code.astype(np.float32)


def make_kv(w: Workload, block: int) -> Tuple[np.ndarray, np.ndarray]:
    """K and V of absolute block index ``block``: uint16 [L, H, d] bf16 bit patterns."""
    k = _normal(w, _TAG_K, block, 0)
    v = _normal(w, _TAG_V, block, 0)
    tf = w.tokens_per_frame
    for h, lab in enumerate(w.labels):
        if lab == SINK and block == 0:
            # keys of the very first frame are scaled up: every query's softmax collapses
            # onto a few of them, i.e. onto the first cached block
            k[:tf, h, :] *= np.float32(w.sink_alpha)
        elif lab == DUMMY:
            beta = np.sqrt(w.dummy_lift * np.sqrt(w.head_dim))
            k[:, h, :] += np.float32(beta) * _block_direction(w, h, block)
        elif lab == SPATIAL:
            c = np.sqrt(w.spatial_peak * np.sqrt(w.head_dim))
            code = _position_code(w, h)
            k[:, h, :] += np.float32(c) * np.tile(code, (w.frames_per_block, 1))
    return f32_to_bf16_bits(k), f32_to_bf16_bits(v)


def make_q(w: Workload, block: int, step: int = 0) -> np.ndarray:
    """Q of absolute block ``block`` at denoise step ``step``: uint16 [L, H, d]."""
    q = _normal(w, _TAG_Q, block, step)
    for h, lab in enumerate(w.labels):
        if lab == DUMMY:
            beta = np.sqrt(w.dummy_lift * np.sqrt(w.head_dim))
            q[:, h, :] += np.float32(beta) * _block_direction(w, h, block)
        elif lab == SPATIAL:
            c = np.sqrt(w.spatial_peak * np.sqrt(w.head_dim))
            code = _position_code(w, h)
            q[:, h, :] += np.float32(c) * np.tile(code, (w.frames_per_block, 1))
    return f32_to_bf16_bits(q)


def sample_rows(w: Workload, n_random: int = 256, seed: int = 1) -> np.ndarray:
    """Query rows used where the oracle cannot afford every row: tile-boundary rows of the
    128-row tiling, every row on the edge of a corner / border / interior deployed cell, and
    ``n_random`` uniformly drawn rows.  Sorted, unique."""
    L = w.block_tokens
    rows = set()
    for t in range(0, L, 128):
        rows.update(r for r in (t - 1, t, t + 1, t + 127) if 0 <= r < L)
    rows.update((0, L - 1, L - 2))
    tf, gw, gh = w.tokens_per_frame, w.grid_w, w.grid_h
    for (y0, y1, x0, x1) in ((0, w.cell_h, 0, w.cell_w),
                             (gh - w.cell_h, gh, gw - w.cell_w, gw),
                             (gh // 2 - 1, gh // 2 + 1, gw // 2 - 1, gw // 2 + 1)):
        for f in range(w.frames_per_block):
            for y in range(max(y0, 0), min(y1, gh)):
                for x in (max(x0, 0), min(x1, gw) - 1):
                    rows.add(f * tf + y * gw + x)
    g = _rng(w, 0x5A3F1E, seed)
    rows.update(int(r) for r in g.integers(0, L, size=n_random))
    return np.array(sorted(rows), dtype=np.int64)
