"""CPU oracle for the HeadCast attention path.  TEST INFRASTRUCTURE ONLY.

A plain, slow float64 restatement of what the paper defines, written to be
checked against the paper by eye.  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may call it; it shares no code with the CUDA
library and never imports it.

What each function follows:

* ``softmax_attention``   - Eq. 2's ``Attention(Q, K, V)``: scaled dot-product
  softmax attention over an explicit key set, one row at a time (no tiling,
  no running max; the whole row of logits is formed first).
* ``full_attend``         - Sec. 3.1 / "Global Path" (Sec. 4.4): every cached token.
* ``attend``              - Sec. 4.4: Sink -> first block, Dummy -> newest block,
  Global -> whole window, Spatial -> keys of the query's own non-overlapping
  grid cell in every cached frame (Fig. 3).
* ``classify``            - Sec. 4.2: Eq. 2 reference output, the three proxies,
  Eq. 3 mean cosine, Eq. 4 score (5th percentile minus gamma * MSE), Eq. 5 rule.
* ``CacheModel``          - Sec. 4.3: split along the head dimension, Sink freeze,
  Dummy rolling overwrite, Global/Spatial sliding window that keeps the sink block.
* ``flops_ratio`` / ``kv_reduction`` - the closed forms of Appendix B and C.

Readings taken where the paper is silent:
softmax scale 1/sqrt(d); Sink/Dummy use exactly one block (Sec. 4.4), the
appendix's "anchor + current block" accounting is only used by the two
closed-form helpers; cells: n = max(1, floor(G/cell + 1/2)) per axis with edges
floor(i*G/n); proxy neighbourhood clipped at frame borders and applied to
every cached frame; percentile = linear interpolation at rank 0.05*(L-1);
MSE = mean over all L*d elements; cosine denominator clamped at 1e-12.

Parity unpinned (the paper prints no worked example): the percentile
interpolation rule, the cell rounding rule, and the attention-mass auxiliary
outputs' "rest" partition, and the threshold of the optional mass rule (``decide_mass``).  Everything else is pinned by the CPU test suite.
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import numpy as np

SINK, DUMMY, SPATIAL, GLOBAL = 0, 1, 2, 3

# score vector layout (per head)
SCORE_NAMES = ("cos_sink", "cos_dummy", "cos_spatial", "p5_spatial", "mse_spatial", "score",
               "mass_first", "mass_last", "mass_spatial", "mass_rest")
N_SCORES = len(SCORE_NAMES)


def widen_bf16(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> float64, exactly."""
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


# --------------------------------------------------------------------------- geometry


def cell_edges(grid: int, cell: int) -> np.ndarray:
    """Edges of the non-overlapping cells along one axis ("the boundary remainder is
    rounded", Sec. 5.1): n = max(1, floor(grid/cell + 1/2)) cells, edge i = floor(i*grid/n)."""
    n = max(1, int(math.floor(grid / cell + 0.5)))
    return np.array([(i * grid) // n for i in range(n + 1)], dtype=np.int64)


@dataclass(frozen=True)
class Geometry:
    grid_h: int
    grid_w: int
    frames_per_block: int
    row_edges: Tuple[int, ...]
    col_edges: Tuple[int, ...]

    @staticmethod
    def make(grid_h: int, grid_w: int, frames_per_block: int = 3, cell_h: int = 10,
             cell_w: int = 10, row_edges: Optional[Sequence[int]] = None,
             col_edges: Optional[Sequence[int]] = None) -> "Geometry":
        re = tuple(int(v) for v in (row_edges if row_edges is not None else cell_edges(grid_h, cell_h)))
        ce = tuple(int(v) for v in (col_edges if col_edges is not None else cell_edges(grid_w, cell_w)))
        assert re[0] == 0 and re[-1] == grid_h and ce[0] == 0 and ce[-1] == grid_w
        return Geometry(grid_h, grid_w, frames_per_block, re, ce)

    @property
    def tokens_per_frame(self) -> int:
        return self.grid_h * self.grid_w

    @property
    def block_tokens(self) -> int:
        return self.frames_per_block * self.tokens_per_frame

    def yx(self, tokens: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
        """Grid position of block-local (or cache-global) token indices."""
        p = np.asarray(tokens) % self.tokens_per_frame
        return p // self.grid_w, p % self.grid_w

    def cell_of(self, tokens: np.ndarray) -> np.ndarray:
        """Index of the deployed cell holding each token's grid position."""
        y, x = self.yx(tokens)
        cy = np.searchsorted(np.asarray(self.row_edges), y, side="right") - 1
        cx = np.searchsorted(np.asarray(self.col_edges), x, side="right") - 1
        return cy * (len(self.col_edges) - 1) + cx

    @property
    def n_cells(self) -> int:
        return (len(self.row_edges) - 1) * (len(self.col_edges) - 1)


# --------------------------------------------------------------------------- Eq. 2


def softmax_attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, scale: float,
                      allowed: Optional[np.ndarray] = None, want_p: bool = False):
    """Attention(Q, K, V) of Eq. 2 for query rows ``q`` [n, d] over keys ``k`` [m, d]
    and values ``v`` [m, d]; ``allowed`` [n, m] (bool) removes keys from a row's key set.
    Returns (o [n, d], lse [n]) and, if asked, the normalised probabilities [n, m]."""
    s = scale * (q @ k.T)
    if allowed is not None:
        s = np.where(allowed, s, -np.inf)
    m = s.max(axis=1, keepdims=True)
    p = np.exp(s - m)
    ell = p.sum(axis=1, keepdims=True)
    p /= ell
    o = p @ v
    lse = m[:, 0] + np.log(ell[:, 0])
    return (o, lse, p) if want_p else (o, lse)


def _chunks(n: int, size: int):
    for a in range(0, n, size):
        yield a, min(n, a + size)


def _attend_keys(q: np.ndarray, k: np.ndarray, v: np.ndarray, scale: float, chunk: int = 512):
    """softmax_attention over one shared key set, a few rows at a time (rows are independent)."""
    o = np.empty((q.shape[0], v.shape[1]))
    lse = np.empty(q.shape[0])
    for a, b in _chunks(q.shape[0], chunk):
        o[a:b], lse[a:b] = softmax_attention(q[a:b], k, v, scale)
    return o, lse


# --------------------------------------------------------------------------- cache model


class CacheModel:
    """List model of the KV cache (Sec. 3.1, 4.3).  ``blocks`` holds (K, V) pairs of
    uint16 [L, H, d] arrays in logical order: index 0 is the sink block, the last is the newest."""

    def __init__(self, n_blocks: int, n_heads: int, sd_mode: int = 0):
        self.n_blocks = n_blocks
        self.n_heads = n_heads
        # 0: Sink / Dummy heads keep exactly one block (Sec. 4.3, 4.4); 1: the appendix's accounting (App. B, C):
        # Sink keeps its anchor block plus the current block, Dummy the previous plus the current block (2L tokens)
        self.sd_mode = sd_mode
        self.blocks: List[Tuple[np.ndarray, np.ndarray]] = []
        self.labels: Optional[np.ndarray] = None
        self.per_head: Optional[List[List[Tuple[np.ndarray, np.ndarray]]]] = None

    # sliding window that keeps the sink block (Sec. 3.1; "Global Cache", Sec. 4.3)
    @staticmethod
    def _roll(lst: list, item, capacity: int) -> None:
        if len(lst) >= capacity:
            del lst[1]
        lst.append(item)

    def append(self, k: np.ndarray, v: np.ndarray) -> None:
        if self.per_head is None:
            self._roll(self.blocks, (k, v), self.n_blocks)
            return
        self._roll(self.blocks, (k, v), self.n_blocks)  # kept for the dense baseline
        for h in range(self.n_heads):
            item = (k[:, h, :], v[:, h, :])
            lab = self.labels[h]
            if lab == SINK:
                if self.sd_mode == 1:
                    self.per_head[h] = [self.per_head[h][0], item]  # anchor stays frozen, current block follows
                # else: frozen initial block
            elif lab == DUMMY:
                self.per_head[h] = [self.per_head[h][-1], item] if self.sd_mode == 1 else [item]  # rolling overwrite
            else:
                self._roll(self.per_head[h], item, self.n_blocks)

    def split(self, labels: Sequence[int]) -> None:
        """Slice the monolithic cache along the head dimension into per-archetype buffers."""
        self.labels = np.asarray(labels, dtype=np.int64)
        self.per_head = []
        for h in range(self.n_heads):
            all_blocks = [(k[:, h, :], v[:, h, :]) for k, v in self.blocks]
            lab = self.labels[h]
            if lab == SINK:
                both = self.sd_mode == 1 and len(all_blocks) > 1
                self.per_head.append([all_blocks[0], all_blocks[-1]] if both else all_blocks[:1])
            elif lab == DUMMY:
                self.per_head.append(all_blocks[-2:] if self.sd_mode == 1 else all_blocks[-1:])
            else:
                self.per_head.append(all_blocks)

    def overwrite_last(self, k: np.ndarray, v: np.ndarray) -> None:
        """Per-denoise-step refresh: the newest block is replaced wherever it is kept as the newest block (the
        monolithic cache, the windows, a Dummy head's current block, a Sink head's current block in sd_mode 1).
        A Sink head's anchor block stays frozen."""
        self.blocks[-1] = (k, v)
        if self.per_head is None:
            return
        for h in range(self.n_heads):
            lab = self.labels[h]
            if lab == SINK and not (self.sd_mode == 1 and len(self.per_head[h]) > 1):
                continue
            self.per_head[h][-1] = (k[:, h, :], v[:, h, :])

    def head_kv_bits(self, h: int) -> Tuple[np.ndarray, np.ndarray]:
        """Logical content kept for head ``h`` as uint16 [n_tokens, d] (oldest block first)."""
        src = self.per_head[h] if self.per_head is not None else [(k[:, h, :], v[:, h, :]) for k, v in self.blocks]
        return (np.concatenate([k for k, _ in src], axis=0), np.concatenate([v for _, v in src], axis=0))

    def mono_kv_bits(self, h: int) -> Tuple[np.ndarray, np.ndarray]:
        return (np.concatenate([k[:, h, :] for k, _ in self.blocks], axis=0),
                np.concatenate([v[:, h, :] for _, v in self.blocks], axis=0))


# --------------------------------------------------------------------------- attention paths


def _scale(d: int, softmax_scale: float) -> float:
    return softmax_scale if softmax_scale > 0 else 1.0 / math.sqrt(d)


def full_attend(q_bits: np.ndarray, cache: CacheModel, rows: Optional[np.ndarray] = None,
                softmax_scale: float = 0.0, heads: Optional[Sequence[int]] = None):
    """Dense attention of every head over every cached token.  Returns (o [n, H, d], lse [n, H])."""
    L, H, d = q_bits.shape
    rows = np.arange(L) if rows is None else np.asarray(rows)
    o = np.zeros((rows.size, H, d))
    lse = np.zeros((rows.size, H))
    for h in (range(H) if heads is None else heads):
        kb, vb = cache.mono_kv_bits(h)
        o[:, h, :], lse[:, h] = _attend_keys(widen_bf16(q_bits[rows, h, :]), widen_bf16(kb),
                                             widen_bf16(vb), _scale(d, softmax_scale))
    return o, lse


def attend(q_bits: np.ndarray, cache: CacheModel, geom: Geometry, rows: Optional[np.ndarray] = None,
           softmax_scale: float = 0.0, heads: Optional[Sequence[int]] = None) -> np.ndarray:
    """Head-specific attention after the split.  Returns o [n, H, d] for the requested rows."""
    assert cache.per_head is not None
    L, H, d = q_bits.shape
    rows = np.arange(L) if rows is None else np.asarray(rows)
    scale = _scale(d, softmax_scale)
    o = np.zeros((rows.size, H, d))
    for h in (range(H) if heads is None else heads):
        kb, vb = cache.head_kv_bits(h)  # Sink: first block; Dummy: newest block; else the window
        k, v = widen_bf16(kb), widen_bf16(vb)
        q = widen_bf16(q_bits[rows, h, :])
        if cache.labels[h] != SPATIAL:
            o[:, h, :], _ = _attend_keys(q, k, v, scale)
            continue
        key_cell = geom.cell_of(np.arange(k.shape[0]))
        row_cell = geom.cell_of(rows)
        for c in np.unique(row_cell):
            sel = np.nonzero(row_cell == c)[0]
            keys = np.nonzero(key_cell == c)[0]
            o[sel, h, :], _ = _attend_keys(q[sel], k[keys], v[keys], scale)
    return o


# --------------------------------------------------------------------------- classification


def percentile_linear(values: np.ndarray, pct: float) -> float:
    """pct-th percentile with linear interpolation between order statistics."""
    s = np.sort(np.asarray(values, dtype=np.float64))
    rank = pct / 100.0 * (s.size - 1)
    lo = int(math.floor(rank))
    hi = min(lo + 1, s.size - 1)
    return float(s[lo] + (rank - lo) * (s[hi] - s[lo]))


def decide(cos_sink: float, cos_dummy: float, cos_spatial: float, score: float,
           theta_s: float = 0.95, theta_d: float = 0.95, theta_sp: float = 0.95,
           theta_sc: float = 0.755) -> int:
    """Eq. 5, in the order written, with >= ; a NaN fails every comparison."""
    if cos_sink >= theta_s:
        return SINK
    if cos_dummy >= theta_d:
        return DUMMY
    if cos_spatial >= theta_sp and score >= theta_sc:
        return SPATIAL
    return GLOBAL


def decide_mass(mass_first: float, mass_last: float, mass_spatial: float, tau: float = 0.9) -> int:
    """The cascade of Eq. 5 applied to the mean attention masses instead of the cosines (not in the paper, which
    gives no threshold for it: parity unpinned beyond the truth table): same order, same >=, NaN fails every test."""
    if mass_first >= tau:
        return SINK
    if mass_last >= tau:
        return DUMMY
    if mass_spatial >= tau:
        return SPATIAL
    return GLOBAL


def _row_cosine(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    num = (a * b).sum(axis=1)
    den = np.maximum(np.linalg.norm(a, axis=1) * np.linalg.norm(b, axis=1), 1e-12)
    return num / den


def proxy_allowed(geom: Geometry, rows: np.ndarray, n_keys: int, r: int) -> np.ndarray:
    """[n, n_keys] mask of the Spatial proxy: key (y', x') of any cached frame is allowed for
    the query at (y, x) iff |y' - y| <= r and |x' - x| <= r (clipped at the frame border)."""
    qy, qx = geom.yx(rows)
    ky, kx = geom.yx(np.arange(n_keys))
    return (np.abs(ky[None, :] - qy[:, None]) <= r) & (np.abs(kx[None, :] - qx[:, None]) <= r)


def classify(q_bits: np.ndarray, cache: CacheModel, geom: Geometry, r: int = 2, gamma: float = 5.0,
             thetas: Tuple[float, float, float, float] = (0.95, 0.95, 0.95, 0.755),
             softmax_scale: float = 0.0, rows: Optional[np.ndarray] = None,
             heads: Optional[Sequence[int]] = None, chunk: int = 256, want_tokens: bool = False,
             rule: int = 0, mass_tau: float = 0.9):
    """One-time head classification (Sec. 4.2).  Returns (labels [H] int32, scores [H, N_SCORES]).
    With ``rows`` given, the per-token quantities are only formed for those rows (the per-head
    statistics are then statistics of that sample).  ``want_tokens`` also returns the per-token
    cosines and squared errors as a dict."""
    L, H, d = q_bits.shape
    Lb = geom.block_tokens
    assert L == Lb and len(cache.blocks) >= 2
    rows = np.arange(L) if rows is None else np.asarray(rows)
    scale = _scale(d, softmax_scale)
    labels = np.full(H, GLOBAL, dtype=np.int32)
    scores = np.zeros((H, N_SCORES))
    tokens = {}
    for h in (range(H) if heads is None else heads):
        kb, vb = cache.mono_kv_bits(h)
        k, v = widen_bf16(kb), widen_bf16(vb)
        n_keys = k.shape[0]
        first = np.arange(n_keys) < Lb  # first temporal block
        last = np.arange(n_keys) >= n_keys - Lb  # current (newest) block
        cos = np.empty((3, rows.size))
        sqerr = np.empty(rows.size)
        mass = np.empty((4, rows.size))
        for a, b in _chunks(rows.size, chunk):
            q = widen_bf16(q_bits[rows[a:b], h, :])
            o_ref, _, p = softmax_attention(q, k, v, scale, want_p=True)  # Eq. 2
            o_sink, _ = softmax_attention(q, k[first], v[first], scale)  # Sink proxy
            o_dummy, _ = softmax_attention(q, k[last], v[last], scale)  # Dummy proxy
            near = proxy_allowed(geom, rows[a:b], n_keys, r)
            o_sp, _ = softmax_attention(q, k, v, scale, allowed=near)  # Spatial proxy
            cos[0, a:b] = _row_cosine(o_sink, o_ref)
            cos[1, a:b] = _row_cosine(o_dummy, o_ref)
            cos[2, a:b] = _row_cosine(o_sp, o_ref)
            sqerr[a:b] = ((o_sp - o_ref) ** 2).sum(axis=1)
            mass[0, a:b] = p[:, first].sum(axis=1)
            mass[1, a:b] = p[:, last].sum(axis=1)
            mass[2, a:b] = np.where(near, p, 0.0).sum(axis=1)
            mass[3, a:b] = np.where(near | first[None, :] | last[None, :], 0.0, p).sum(axis=1)
        cs, cd, csp = cos.mean(axis=1)  # Eq. 3
        p5 = percentile_linear(cos[2], 5.0)
        mse = sqerr.sum() / (rows.size * d)
        score = p5 - gamma * mse  # Eq. 4
        mean_mass = mass.mean(axis=1)
        if rule == 0:
            labels[h] = decide(cs, cd, csp, score, *thetas)  # Eq. 5
        else:
            labels[h] = decide_mass(mean_mass[0], mean_mass[1], mean_mass[2], mass_tau)
        scores[h] = (cs, cd, csp, p5, mse, score, *mean_mass)
        if want_tokens:
            tokens[h] = dict(cos=cos, sqerr=sqerr, mass=mass)
    return (labels, scores, tokens) if want_tokens else (labels, scores)


# --------------------------------------------------------------------------- closed forms


def flops_ratio(n_sink: float, n_dummy: float, n_spatial: float, n_global: float,
                window: float = 8.0, sd_blocks: float = 2.0, spatial_blocks: float = 0.5) -> float:
    """Appendix B: attention FLOPs of HeadCast over full attention, in units of B*L^2*d per head
    (full = ``window``, Sink = Dummy = ``sd_blocks``, Spatial = ``spatial_blocks``)."""
    total = n_sink + n_dummy + n_spatial + n_global
    return (sd_blocks * (n_sink + n_dummy) + spatial_blocks * n_spatial + window * n_global) / (window * total)


def spatial_fraction(geom: Geometry) -> float:
    """Fraction of a frame's keys a Spatial query reads, averaged over queries
    (= sum of squared cell areas / T_f^2); Appendix B quotes ~1/16 at 30x52."""
    h = np.diff(np.asarray(geom.row_edges))
    w = np.diff(np.asarray(geom.col_edges))
    areas = np.outer(h, w).astype(np.float64)
    return float((areas ** 2).sum() / geom.tokens_per_frame ** 2)


def kv_reduction(n_sink_dummy: float, n_total: float, window: float = 8.0, kept: float = 2.0) -> float:
    """Appendix C: expected steady-state KV-cache reduction."""
    return n_sink_dummy / n_total * (1.0 - kept / window)


def attend_flops(geom: Geometry, labels: Sequence[int], n_filled: int, d: int, sd_blocks: int = 1) -> float:
    """Algorithmic FLOPs (4 * L_q * L_k * d per head, Appendix B) of one head-specific attend.
    ``sd_blocks`` = blocks a Sink / Dummy head reads: 1 (Sec. 4.4) or 2 (the appendix's accounting),
    never more than are cached."""
    L = geom.block_tokens
    total = 0.0
    for lab in labels:
        if lab in (SINK, DUMMY):
            total += 4.0 * L * min(sd_blocks, n_filled) * L * d
        elif lab == GLOBAL:
            total += 4.0 * L * n_filled * L * d
        else:
            total += 4.0 * L * n_filled * L * d * spatial_fraction(geom)
    return total
