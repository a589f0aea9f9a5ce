"""Host-only checks of the tile scheduler (no GPU): the work list must cover every (head, query row) once, give it
exactly the key set the paper's pathways prescribe (Sec. 4.4), cut key ranges without gaps or overlaps, and spread
the work evenly over the persistent CTAs."""
import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

from oracle import headcast_oracle as orc
from paper_2607_20125_b200 import binding, synth

F = {n: i for i, n in enumerate(binding.ITEM_FIELDS)}
MONO, SD, GLOBAL_BUF, SPATIAL_BUF = 0, 1, 2, 3


def config_of(w, **kw):
    return binding.default_config(n_heads=w.n_heads, head_dim=w.head_dim, grid_h=w.grid_h, grid_w=w.grid_w,
                                  n_blocks=w.n_blocks, frames_per_block=w.frames_per_block, cell_h=w.cell_h,
                                  cell_w=w.cell_w, **kw)


def query_tokens(item, t, geom, cells):
    """Block-local tokens of query tile t of an item."""
    start, count = item[F["q_start0"] + t], item[F["q_count0"] + t]
    idx = np.arange(start, start + count)
    if item[F["cell"]] < 0:
        return idx
    y0, x0, ch, cw = cells[item[F["cell"]]]
    nc = ch * cw
    f, i = idx // nc, idx % nc
    return f * geom.tokens_per_frame + (y0 + i // cw) * geom.grid_w + x0 + i % cw


def check_plan(w, labels, n_filled, n_ctas, dense=False):
    cfg = config_of(w)
    items, first = binding.plan_schedule(cfg, labels, n_filled, n_ctas, dense)
    geom = orc.Geometry.make(w.grid_h, w.grid_w, w.frames_per_block, w.cell_h, w.cell_w)
    cells = [(geom.row_edges[i], geom.col_edges[j], geom.row_edges[i + 1] - geom.row_edges[i],
              geom.col_edges[j + 1] - geom.col_edges[j])
             for i in range(len(geom.row_edges) - 1) for j in range(len(geom.col_edges) - 1)]
    L, H = geom.block_tokens, w.n_heads
    assert first[0] == 0 and first[-1] <= len(items) and np.all(np.diff(first) >= 0)
    covered = np.zeros((H, L), dtype=np.int64)   # key tiles seen by every (head, row)
    finals = np.zeros((H, L), dtype=np.int64)
    groups = {}
    for it in items:
        n_tiles = it[F["tiles_per_seg"]]
        assert it[F["seg_stride"]] == 0 and n_tiles == -(-it[F["seg_len"]] // 128)
        assert 0 <= it[F["tile_begin"]] < it[F["tile_end"]] <= n_tiles
        assert 1 <= it[F["q_count0"]] <= 128 and 0 <= it[F["q_count1"]] <= 128
        h = it[F["head"]]
        lab = orc.GLOBAL if dense else labels[h]
        # key set: which buffer, how many keys
        if dense:
            assert it[F["kv_map"]] == MONO and it[F["seg_len"]] == n_filled * L and it[F["kv_x0"]] == h * w.head_dim
        elif lab in (orc.SINK, orc.DUMMY):
            assert it[F["kv_map"]] == SD and it[F["seg_len"]] == L and it[F["cell"]] < 0
        elif lab == orc.GLOBAL:
            assert it[F["kv_map"]] == GLOBAL_BUF and it[F["seg_len"]] == n_filled * L and it[F["cell"]] < 0
        else:
            nc = cells[it[F["cell"]]][2] * cells[it[F["cell"]]][3]
            assert it[F["kv_map"]] == SPATIAL_BUF and it[F["seg_len"]] == n_filled * w.frames_per_block * nc
        for t in range(2):
            tok = query_tokens(it, t, geom, cells)
            if tok.size == 0:
                continue
            assert tok.min() >= 0 and tok.max() < L
            if it[F["cell"]] >= 0:  # Spatial queries sit in the cell whose keys they read
                assert np.all(geom.cell_of(tok) == it[F["cell"]])
            covered[h, tok] += it[F["tile_end"]] - it[F["tile_begin"]]
            finals[h, tok] += 1 if it[F["out_mode"]] == 0 else 0
        key = (h, it[F["cell"]], it[F["q_start0"]])
        groups.setdefault(key, []).append(it)
    # every row exists once as a final result or as a set of partials that tile the key range exactly
    for key, parts in groups.items():
        parts = sorted(parts, key=lambda x: x[F["tile_begin"]])
        assert parts[0][F["tile_begin"]] == 0 and parts[-1][F["tile_end"]] == parts[0][F["tiles_per_seg"]]
        for a, b in zip(parts, parts[1:]):
            assert a[F["tile_end"]] == b[F["tile_begin"]]
        if len(parts) == 1:
            assert parts[0][F["out_mode"]] == 0
        else:
            assert all(p[F["out_mode"]] == 1 for p in parts)
            slots = [p[F["out_slot"]] for p in parts]
            assert slots == list(range(slots[0], slots[0] + len(parts)))  # combine_kernel reads consecutive slots
    want_tiles = np.zeros((H, L), dtype=np.int64)
    for h in range(H):
        lab = orc.GLOBAL if dense else labels[h]
        if lab in (orc.SINK, orc.DUMMY):
            want_tiles[h] = -(-L // 128)
        elif lab == orc.GLOBAL:
            want_tiles[h] = -(-(n_filled * L) // 128)
        else:
            cell = geom.cell_of(np.arange(L))
            sizes = np.array([c[2] * c[3] for c in cells])
            want_tiles[h] = -(-(n_filled * w.frames_per_block * sizes[cell]) // 128)
    assert np.array_equal(covered, want_tiles)
    assert np.all(finals <= 1)
    # load balance under the scheduler's own cost model: per key tile 1 (query pair) or 0.86 (lone query tile), times
    # 1.02 for Spatial items; per item 2.4 or 1.0, +0.75 per partial result
    pair = items[:, F["q_count1"]] > 0
    cost = np.where(pair, 1.0, 0.86) * np.where(items[:, F["cell"]] >= 0, 1.02, 1.0) \
        * (items[:, F["tile_end"]] - items[:, F["tile_begin"]]) + np.where(pair, 2.4, 1.0) + 0.75 * (items[:, F["out_mode"]] == 1)
    per_cta = np.array([cost[first[b]:first[b + 1]].sum() for b in range(n_ctas)])
    # what lies after the last CTA's list is the shared queue that CTAs draw from once their own lists are done: a
    # small part of the launch, in pieces small enough that the last one drawn cannot delay the end by much
    queue = cost[first[-1]:]
    if queue.size:
        # (2 % of the launch by design, plus the cost of the cuts that the equal static shares did not allow for, which
        # weighs more the shorter the launch)
        assert queue.sum() <= (0.08 if cost.sum() > 200.0 * n_ctas else 0.15) * cost.sum() + 40.0
        q_tiles = (items[first[-1]:, F["tile_end"]] - items[first[-1]:, F["tile_begin"]]).max()
        assert q_tiles <= max(8, 0.02 * cost.sum() / (4 * n_ctas)) + 4  # a piece, plus a remainder too short to stand alone
    return items, per_cta


@pytest.mark.parametrize("res", ["480p", "720p", "1080p"])
def test_paper_workloads_are_covered_and_balanced(res):
    w = synth.wan(res)
    for dense in (False, True):
        items, per_cta = check_plan(w, list(w.labels), w.n_blocks, 148, dense)
        assert (per_cta == 0).sum() <= 2  # the last CTA takes what is left of the line
        assert per_cta.max() <= 1.06 * per_cta.mean(), (res, dense, per_cta.max() / per_cta.mean())


def test_long_key_streams_are_swept_chunk_by_chunk_by_all_ctas():
    """1080P: one Global head's K/V (88 MB) does not fit L2 next to everything else, so its sweep is cut into key
    chunks of at most 30 MB and every CTA works through the chunks in the same order: what the CTAs read at the same
    time stays a fraction of L2."""
    w = synth.wan("1080p")
    items, first = binding.plan_schedule(config_of(w), list(w.labels), w.n_blocks, 148)
    tile_bytes = 128 * w.head_dim * 2 * 2  # one key tile of K and V
    for h in [i for i, lab in enumerate(w.labels) if lab == orc.GLOBAL]:
        mine = items[:, F["head"]] == h
        total_tiles = int(items[mine][0][F["tiles_per_seg"]])
        n_chunks = -(-total_tiles * tile_bytes // (30 << 20))
        assert n_chunks == 3
        bounds = [total_tiles * k // n_chunks for k in range(n_chunks + 1)]
        chunk_of = lambda it: next(k for k in range(n_chunks) if bounds[k] <= it[F["tile_begin"]] < bounds[k + 1])
        busy = 0
        for it in items[first[-1]:]:  # pieces in the shared queue keep to the chunk boundaries too
            if it[F["head"]] == h:
                k = chunk_of(it)
                assert bounds[k] <= it[F["tile_begin"]] < it[F["tile_end"]] <= bounds[k + 1]
        for b in range(148):
            seq = [chunk_of(it) for it in items[first[b]:first[b + 1]] if it[F["head"]] == h]
            for it in items[first[b]:first[b + 1]]:
                if it[F["head"]] == h:  # no piece straddles a chunk boundary
                    k = chunk_of(it)
                    assert bounds[k] <= it[F["tile_begin"]] < it[F["tile_end"]] <= bounds[k + 1]
            assert seq == sorted(seq)
            busy += len(set(seq)) == n_chunks
        assert busy >= 140  # (nearly) every CTA takes part in every chunk


def test_growth_phase_and_odd_cta_counts():
    w = synth.small()
    for n_filled in (1, 2, 4):
        for n_ctas in (1, 7, 148):
            check_plan(w, list(w.labels), n_filled, n_ctas)
            check_plan(w, list(w.labels), n_filled, n_ctas, dense=True)


def test_tiny_single_cell_and_empty_groups():
    check_plan(synth.tiny(), [0, 1, 2, 3], 5, 148)
    check_plan(synth.tiny(cell=4), [2, 2, 2, 2], 3, 148)
    check_plan(synth.small(), [orc.GLOBAL] * 6, 4, 148)
    check_plan(synth.small(), [orc.SINK] * 6, 4, 148)


@settings(max_examples=40, deadline=None)
@given(gh=st.integers(1, 24), gw=st.integers(1, 24), ch=st.integers(1, 12), cw=st.integers(1, 12),
       n_blocks=st.integers(2, 6), fill=st.integers(1, 6), heads=st.lists(st.integers(0, 3), min_size=1, max_size=8),
       n_ctas=st.sampled_from([1, 3, 148]), d=st.sampled_from([64, 128]))
def test_random_geometries(gh, gw, ch, cw, n_blocks, fill, heads, n_ctas, d):
    w = synth.Workload("rand", len(heads), d, gh, gw, n_blocks, cell_h=ch, cell_w=cw, labels=tuple(heads))
    check_plan(w, heads, min(fill, n_blocks), n_ctas)


@settings(max_examples=40, deadline=None)
@given(gh=st.integers(20, 70), gw=st.integers(30, 120), n_blocks=st.integers(3, 8),
       heads=st.lists(st.integers(0, 3), min_size=6, max_size=16), n_ctas=st.sampled_from([37, 148, 160]))
def test_large_workloads_are_spread_evenly(gh, gw, n_blocks, heads, n_ctas):
    """Whatever the grid and the head mix, a workload much larger than the machine is spread evenly: no CTA carries
    much more than the mean (the share search falls back to an upward scan when its bisection goes astray)."""
    w = synth.Workload("big", len(heads), 128, gh, gw, n_blocks, labels=tuple(heads))
    items, per_cta = check_plan(w, heads, n_blocks, n_ctas)
    if per_cta.sum() > 40.0 * n_ctas:  # several items' worth of work per CTA
        # the busiest CTA decides the launch: it may not carry much more than an equal share (whole items of about
        # half a share cannot be dealt more evenly without paying for cuts, hence the slack; some CTAs may then idle)
        assert per_cta.max() <= 1.15 * per_cta.mean(), (per_cta.max(), per_cta.mean(), (per_cta == 0).sum())


def test_planner_rejects_bad_input():
    w = synth.tiny()
    cfg = config_of(w)
    with pytest.raises(binding.HeadCastError):
        binding.plan_schedule(cfg, [0, 1, 2, 9], 3, 148)
    with pytest.raises(binding.HeadCastError):
        binding.plan_schedule(cfg, [0, 1, 2, 3], 9, 148)  # more blocks than the cache holds
    with pytest.raises(binding.HeadCastError):
        binding.plan_schedule(cfg, None, 3, 148)
