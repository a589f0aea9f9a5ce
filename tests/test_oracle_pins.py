"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU)."""
import math
import os

import numpy as np
import pytest

from oracle import headcast_oracle as orc
from paper_2607_20125_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_closed_forms.txt")


def golden():
    out = {}
    with open(GOLDEN) as f:
        for line in f:
            line = line.split("#")[0].split()
            if line:
                out[line[0]] = [float(v) for v in line[1:]]
    return out


def rand_bits(rng, shape, scale=1.0):
    return synth.f32_to_bf16_bits((scale * rng.standard_normal(shape)).astype(np.float32))


def fill(w, n=None, labels=None):
    geom = orc.Geometry.make(w.grid_h, w.grid_w, w.frames_per_block, w.cell_h, w.cell_w)
    cache = orc.CacheModel(w.n_blocks, w.n_heads)
    for b in range(w.n_blocks if n is None else n):
        cache.append(*synth.make_kv(w, b))
    return geom, cache


# ---- Eq. 2: softmax attention ------------------------------------------------------------


def brute_force_attention(q, k, v, scale):
    """Independent restatement: key-outer loops, long double accumulation, explicit matrix."""
    n, m = q.shape[0], k.shape[0]
    out = np.zeros((n, v.shape[1]), dtype=np.longdouble)
    for i in range(n):
        logits = [math.fsum(float(q[i, c]) * float(k[j, c]) for c in range(q.shape[1])) * scale for j in range(m)]
        top = max(logits)
        w = [np.longdouble(math.exp(s - top)) for s in logits]
        z = sum(w)
        for j in range(m):
            out[i] += (w[j] / z) * v[j].astype(np.longdouble)
    return out.astype(np.float64)


def test_rows_sum_to_one_and_match_brute_force():
    rng = np.random.default_rng(0)
    q, k, v = rng.standard_normal((5, 8)), rng.standard_normal((11, 8)), rng.standard_normal((11, 8))
    o, lse, p = orc.softmax_attention(q, k, v, 0.37, want_p=True)
    assert np.abs(p.sum(axis=1) - 1).max() < 1e-12
    assert np.abs(o - brute_force_attention(q, k, v, 0.37)).max() < 1e-12
    # lse is the log of the softmax normaliser
    s = 0.37 * q @ k.T
    assert np.abs(lse - np.log(np.exp(s).sum(axis=1))).max() < 1e-12


def test_transposed_or_unscaled_operands_would_fail():
    # asymmetric shapes and a scale far from 1: K^T vs K, q.k vs k.q, missing scale all differ
    rng = np.random.default_rng(1)
    q, k, v = rng.standard_normal((3, 4)), rng.standard_normal((6, 4)), rng.standard_normal((6, 2))
    o, _ = orc.softmax_attention(q, k, v, 2.5)
    assert o.shape == (3, 2)
    assert np.abs(o - brute_force_attention(q, k, v, 2.5)).max() < 1e-12
    assert np.abs(o - brute_force_attention(q, k, v, 1.0)).max() > 1e-3


def test_closed_forms_zero_query_constant_value_single_key():
    rng = np.random.default_rng(2)
    k, v = rng.standard_normal((9, 4)), rng.standard_normal((9, 4))
    o, _ = orc.softmax_attention(np.zeros((2, 4)), k, v, 0.5)
    assert np.abs(o - v.mean(axis=0)).max() < 1e-14  # uniform weights
    o, _ = orc.softmax_attention(rng.standard_normal((2, 4)), k, np.full((9, 4), 3.25), 0.5)
    assert np.abs(o - 3.25).max() < 1e-14
    o, _ = orc.softmax_attention(rng.standard_normal((2, 4)), k[:1], v[:1], 0.5)
    assert np.abs(o - v[0]).max() < 1e-14
    allowed = np.zeros((2, 9), bool)
    allowed[0, 4] = allowed[1, 7] = True
    o, _ = orc.softmax_attention(rng.standard_normal((2, 4)), k, v, 0.5, allowed=allowed)
    assert np.abs(o - v[[4, 7]]).max() < 1e-14


# ---- geometry ----------------------------------------------------------------------------


def test_cell_partition_matches_paper_counts():
    g = golden()
    ch, cw = (int(x) for x in g["cell"])
    geom = orc.Geometry.make(30, 52, 3, ch, cw)
    assert geom.n_cells == 15  # 3 x 5 cells, i.e. "about 1/16 of the frame" each
    assert abs(orc.spatial_fraction(geom) - g["cell_fraction_480p"][0]) < 0.01
    assert list(orc.cell_edges(30, 10)) == [0, 10, 20, 30]
    assert list(orc.cell_edges(52, 10)) == [0, 10, 20, 31, 41, 52]
    assert list(np.diff(orc.cell_edges(68, 10))) == [9, 10, 10, 9, 10, 10, 10]
    assert list(np.diff(orc.cell_edges(45, 10))) == [9] * 5
    assert list(orc.cell_edges(8, 10)) == [0, 8]  # grid smaller than the cell: one cell
    # cells tile the frame: every token has exactly one cell, areas add up
    cells = geom.cell_of(np.arange(geom.tokens_per_frame))
    assert cells.min() == 0 and cells.max() == 14
    assert np.bincount(cells).sum() == 1560 and set(np.bincount(cells)) <= {100, 110}
    # token order is frame-major, then row, then column
    y, x = geom.yx(np.array([0, 51, 52, 1559, 1560 + 53]))
    assert list(y) == [0, 0, 1, 29, 1] and list(x) == [0, 51, 0, 51, 1]


def test_proxy_neighbourhood_clipping():
    geom = orc.Geometry.make(6, 7, 3, 10, 10)
    tf = geom.tokens_per_frame
    allowed = orc.proxy_allowed(geom, np.array([0, 3 * 7 + 3, tf + 5 * 7 + 6]), 2 * tf, 2)
    # corner: 3x3 survive, in each of the 2 cached frames; interior: 5x5; other frames too
    assert allowed[0].sum() == 2 * 9 and allowed[1].sum() == 2 * 25 and allowed[2].sum() == 2 * 9
    assert allowed[1, 3 * 7 + 3] and allowed[1, tf + 1 * 7 + 1] and not allowed[1, 0]
    narrow = orc.Geometry.make(3, 2, 3, 10, 10)  # grid narrower than 2r+1: whole frame
    assert orc.proxy_allowed(narrow, np.array([0]), 12, 2).all()


# ---- pathways ----------------------------------------------------------------------------


def small_case(seed=3, H=4, d=16, gh=4, gw=6, n=3, cell=(2, 3)):
    rng = np.random.default_rng(seed)
    geom = orc.Geometry.make(gh, gw, 3, *cell)
    L = geom.block_tokens
    cache = orc.CacheModel(n, H)
    for _ in range(n):
        cache.append(rand_bits(rng, (L, H, d)), rand_bits(rng, (L, H, d)))
    q = rand_bits(rng, (L, H, d), 2.0)
    return geom, cache, q


def test_sink_dummy_global_equal_full_attention_on_the_kept_blocks():
    geom, cache, q = small_case()
    H = cache.n_heads
    ref_all, _ = orc.full_attend(q, cache)
    only_first = orc.CacheModel(3, H)
    only_first.append(*cache.blocks[0])
    only_last = orc.CacheModel(3, H)
    only_last.append(*cache.blocks[-1])
    ref_first, _ = orc.full_attend(q, only_first)
    ref_last, _ = orc.full_attend(q, only_last)
    cache.split([orc.SINK, orc.DUMMY, orc.GLOBAL, orc.GLOBAL])
    o = orc.attend(q, cache, geom)
    assert np.array_equal(o[:, 0], ref_first[:, 0])
    assert np.array_equal(o[:, 1], ref_last[:, 1])
    assert np.array_equal(o[:, 2:], ref_all[:, 2:])


def test_spatial_with_one_cell_equals_global_and_cells_are_independent():
    geom, cache, q = small_case(cell=(10, 10))
    assert geom.n_cells == 1
    ref, _ = orc.full_attend(q, cache)
    cache.split([orc.SPATIAL] * 4)
    o = orc.attend(q, cache, geom)
    assert np.abs(o - ref).max() < 1e-13
    # several cells: brute force per query over explicitly enumerated same-cell keys
    geom, cache, q = small_case(seed=5, cell=(2, 3))
    assert geom.n_cells == 4
    cache.split([orc.SPATIAL] * 4)
    o = orc.attend(q, cache, geom)
    h = 2
    kb, vb = cache.head_kv_bits(h)
    k, v = orc.widen_bf16(kb), orc.widen_bf16(vb)
    for t in (0, 5, 13, 24 + 17, 71):
        f, rem = divmod(t, 24)
        y, x = divmod(rem, 6)
        keys = [j for j in range(k.shape[0])
                if ((j % 24) // 6) // 2 == y // 2 and ((j % 24) % 6) // 3 == x // 3]
        assert len(keys) == 9 * 6
        want = brute_force_attention(orc.widen_bf16(q[t:t + 1, h]), k[keys], v[keys], 0.25)
        assert np.abs(o[t, h] - want[0]).max() < 1e-12


def test_zero_query_gives_mean_of_values_over_each_key_set():
    geom, cache, q = small_case(seed=7, cell=(2, 3))
    q0 = np.zeros_like(q)
    labels = [orc.SINK, orc.DUMMY, orc.SPATIAL, orc.GLOBAL]
    cache.split(labels)
    o = orc.attend(q0, cache, geom)
    L = geom.block_tokens
    v = [orc.widen_bf16(cache.mono_kv_bits(h)[1]) for h in range(4)]
    assert np.abs(o[:, 0] - v[0][:L].mean(axis=0)).max() < 1e-14
    assert np.abs(o[:, 1] - v[1][-L:].mean(axis=0)).max() < 1e-14
    assert np.abs(o[:, 3] - v[3].mean(axis=0)).max() < 1e-14
    cells = geom.cell_of(np.arange(v[2].shape[0]))
    for t in (0, 4, 23, 50):
        want = v[2][cells == geom.cell_of(np.array([t]))[0]].mean(axis=0)
        assert np.abs(o[t, 2] - want).max() < 1e-14


def test_key_order_invariance_justifies_a_ring():
    geom, cache, q = small_case(seed=9)
    ref, _ = orc.full_attend(q, cache)
    rolled = orc.CacheModel(3, cache.n_heads)
    for i in (2, 0, 1):
        rolled.append(*cache.blocks[i])
    o, _ = orc.full_attend(q, rolled)
    assert np.abs(o - ref).max() < 1e-13


def test_rows_argument_selects_rows():
    geom, cache, q = small_case(seed=10)
    rows = np.array([0, 7, 33, 71])
    full, lse = orc.full_attend(q, cache)
    part, lse_p = orc.full_attend(q, cache, rows=rows)
    assert np.array_equal(full[rows], part) and np.array_equal(lse[rows], lse_p)
    cache.split([orc.SINK, orc.SPATIAL, orc.SPATIAL, orc.DUMMY])
    assert np.abs(orc.attend(q, cache, geom)[rows] - orc.attend(q, cache, geom, rows=rows)).max() < 1e-13


# ---- cache model -------------------------------------------------------------------------


def test_cache_split_append_roll_follow_the_list_model():
    H, d, L, cap = 4, 2, 3, 4
    labels = [orc.GLOBAL, orc.SINK, orc.DUMMY, orc.SPATIAL]
    blocks = [(np.full((L, H, d), 10 * b + 1, np.uint16) + np.arange(H, dtype=np.uint16)[None, :, None],
               np.full((L, H, d), 10 * b + 5, np.uint16)) for b in range(9)]
    cache = orc.CacheModel(cap, H)
    for b in range(3):
        cache.append(*blocks[b])
    cache.split(labels)  # split during the growth phase: 3 of 4 blocks filled

    def ids(h):
        return [int(v) // 10 for v in cache.head_kv_bits(h)[0][::L, 0]]

    assert ids(0) == [0, 1, 2] and ids(1) == [0] and ids(2) == [2] and ids(3) == [0, 1, 2]
    expect = [0, 1, 2]
    for b in range(3, 9):
        cache.append(*blocks[b])
        expect.append(b)
        if len(expect) > cap:
            del expect[1]  # the sink block stays, the oldest rolling block goes
        assert ids(0) == expect and ids(3) == expect
        assert ids(1) == [0] and ids(2) == [b]
        assert [int(v) // 10 for v in cache.mono_kv_bits(0)[0][::L, 0]] == expect
    # values are copied, never recomputed; head slices are the right heads
    assert cache.head_kv_bits(3)[0][0, 0] == 10 * 0 + 1 + 3
    assert cache.head_kv_bits(2)[1][0, 0] == 10 * 8 + 5


# ---- Eq. 3-5 -----------------------------------------------------------------------------


def test_decision_rule_truth_table():
    g = golden()
    th = tuple(g["thresholds"])
    assert th == (0.95, 0.95, 0.95, 0.755)
    d = lambda *a: orc.decide(*a, *th)
    assert d(0.95, 0.99, 0.99, 0.9) == orc.SINK  # >= and first branch wins
    assert d(0.9499, 0.95, 0.99, 0.9) == orc.DUMMY
    assert d(0.1, 0.9499, 0.95, 0.755) == orc.SPATIAL  # both equalities
    assert d(0.1, 0.1, 0.95, 0.7549) == orc.GLOBAL  # mean cosine passes, worst-case score fails
    assert d(0.1, 0.1, 0.9499, 0.99) == orc.GLOBAL
    assert d(float("nan"), 0.2, 0.3, 0.1) == orc.GLOBAL
    assert d(float("nan"), 0.96, 0.3, 0.1) == orc.DUMMY


def test_mass_rule_truth_table_and_planted_heads():
    d = orc.decide_mass
    assert d(0.9, 0.95, 0.95, 0.9) == orc.SINK  # >= and the first branch wins
    assert d(0.8999, 0.9, 0.95, 0.9) == orc.DUMMY
    assert d(0.1, 0.8999, 0.9, 0.9) == orc.SPATIAL
    assert d(0.1, 0.1, 0.8999, 0.9) == orc.GLOBAL
    assert d(float("nan"), 0.95, 0.1, 0.9) == orc.DUMMY and d(float("nan"), float("nan"), float("nan"), 0.9) == orc.GLOBAL
    assert d(0.5, 0.1, 0.1, 0.5) == orc.SINK  # the threshold is the argument, not a constant
    # planted archetypes concentrate their mass where Appendix A says they do: both rules give the planted labels
    w = synth.tiny(cell=4)
    geom, cache = fill(w)
    q = synth.make_q(w, w.n_blocks - 1, 0)
    by_cos, s = orc.classify(q, cache, geom)
    by_mass, s2 = orc.classify(q, cache, geom, rule=1, mass_tau=0.9)
    assert tuple(by_cos) == tuple(by_mass) == w.labels and np.array_equal(s, s2)
    # the rule really reads the masses: with a threshold nobody reaches every head is Global
    assert tuple(orc.classify(q, cache, geom, rule=1, mass_tau=1.0 + 1e-9)[0]) == (orc.GLOBAL,) * 4


def test_percentile_rule():
    assert orc.percentile_linear(np.arange(21.0)[::-1], 5.0) == 1.0  # rank 0.05*20 = 1
    assert abs(orc.percentile_linear(np.array([0.0, 10.0, 20.0]), 5.0) - 1.0) < 1e-12  # rank 0.1
    rng = np.random.default_rng(4)
    x = rng.standard_normal(1001)
    assert abs(orc.percentile_linear(x, 5.0) - np.sort(x)[50]) < 1e-15
    assert orc.percentile_linear(np.array([3.0]), 5.0) == 3.0


def test_scores_follow_their_definitions_on_a_hand_case():
    # one head, d=2, a 1x1 grid with 3 frames per block and 2 cached blocks: every key is in
    # every query's neighbourhood, so the Spatial proxy is the reference itself
    geom = orc.Geometry.make(1, 1, 3, 10, 10)
    cache = orc.CacheModel(2, 1)
    one = synth.f32_to_bf16_bits(np.ones((3, 1, 2), np.float32))
    zero = np.zeros((3, 1, 2), np.uint16)
    v0 = synth.f32_to_bf16_bits(np.tile(np.array([1.0, 0.0], np.float32), (3, 1, 1)))
    v1 = synth.f32_to_bf16_bits(np.tile(np.array([0.0, 1.0], np.float32), (3, 1, 1)))
    cache.append(zero, v0)
    cache.append(zero, v1)
    labels, s = orc.classify(one, cache, geom)
    # all logits are 0: uniform weights; O_ref = (1/2, 1/2), O_sink = (1, 0), O_dummy = (0, 1)
    assert abs(s[0, 0] - math.sqrt(0.5)) < 1e-12 and abs(s[0, 1] - math.sqrt(0.5)) < 1e-12
    assert abs(s[0, 2] - 1) < 1e-12 and abs(s[0, 3] - 1) < 1e-12 and s[0, 4] < 1e-30
    assert abs(s[0, 5] - 1) < 1e-12
    assert np.allclose(s[0, 6:], [0.5, 0.5, 1.0, 0.0])
    assert labels[0] == orc.SPATIAL


def _hand_case(v_blocks, r=0, gamma=2.0):
    """1 x 3 grid, one frame per block, one head, d = 2, every key zero (uniform weights over a key set)."""
    geom = orc.Geometry.make(1, 3, 1, 10, 10)
    cache = orc.CacheModel(len(v_blocks), 1)
    zero = np.zeros((3, 1, 2), np.uint16)
    for vb in v_blocks:
        cache.append(zero, synth.f32_to_bf16_bits(np.asarray(vb, np.float32).reshape(3, 1, 2)))
    q = synth.f32_to_bf16_bits(np.ones((3, 1, 2), np.float32))
    return orc.classify(q, cache, geom, r=r, gamma=gamma)


def test_masked_proxy_and_error_term_on_a_hand_case_with_nonzero_error():
    # three cached frames (first / middle / newest block); with r = 0 the proxy of the query at column x sees the
    # three keys of column x only.  Weights are uniform, so every output is a plain average of value rows:
    #   O_ref  = (4.5, 4.5) / 9 = (1/2, 1/2) for every query
    #   O_sp   = (2.5, 0.5)/3, (1.25, 1.5)/3, (0.75, 2.5)/3   (column sums of the three blocks)
    #   O_sink = (2.75, 0.75)/3, O_dummy = (0.25, 2.25)/3
    v_first = [(2, 0), (0.5, 0.25), (0.25, 0.5)]
    v_mid = [(0.5, 0.5)] * 3
    v_last = [(0, 0), (0.25, 0.75), (0, 1.5)]
    labels, s = _hand_case([v_first, v_mid, v_last], r=0, gamma=2.0)
    r2 = math.sqrt(2.0)
    # the cosine with a vector along (1, 1) is (a0 + a1) / (sqrt(2) |a|)
    cos_sp = [3.0 / (r2 * math.sqrt(6.5)), 2.75 / (r2 * math.sqrt(3.8125)), 3.25 / (r2 * math.sqrt(6.8125))]
    cos_sink = 3.5 / (r2 * math.sqrt(2.75 ** 2 + 0.75 ** 2))
    cos_dummy = 2.5 / (r2 * math.sqrt(0.25 ** 2 + 2.25 ** 2))
    lo, mid = sorted(cos_sp)[:2]
    p5 = lo + 0.1 * (mid - lo)  # rank 0.05 * (3 - 1)
    # squared errors per query: |O_sp - (1/2, 1/2)|^2, averaged over L * d = 6 elements
    sq = [(2.5 / 3 - 0.5) ** 2 + (0.5 / 3 - 0.5) ** 2, (1.25 / 3 - 0.5) ** 2 + 0.0, (0.25 - 0.5) ** 2 + (2.5 / 3 - 0.5) ** 2]
    mse = sum(sq) / 6.0
    assert abs(mse - (1 / 9 + 1 / 9 + 1 / 144 + 1 / 16 + 1 / 9) / 6) < 1e-15 and mse > 0.06
    want = [cos_sink, cos_dummy, sum(cos_sp) / 3, p5, mse, p5 - 2.0 * mse, 1 / 3, 1 / 3, 1 / 3, 2 / 9]
    assert np.abs(s[0] - np.array(want)).max() < 1e-12
    assert labels[0] == orc.GLOBAL
    # gamma enters once, with a minus sign, and multiplies the error only
    _, s5 = _hand_case([v_first, v_mid, v_last], r=0, gamma=5.0)
    assert abs(s5[0, 5] - (p5 - 5.0 * mse)) < 1e-12 and abs(s5[0, 3] - p5) < 1e-12
    # r = 1: the middle column sees the whole frame (error 0 there), the outer columns two of three columns
    _, s1 = _hand_case([v_first, v_mid, v_last], r=1, gamma=2.0)
    o_left = np.array([2.5 + 1.25, 0.5 + 1.5]) / 6
    o_right = np.array([1.25 + 0.75, 1.5 + 2.5]) / 6
    mse1 = (((o_left - 0.5) ** 2).sum() + ((o_right - 0.5) ** 2).sum()) / 6.0
    assert abs(s1[0, 4] - mse1) < 1e-15 and abs(s1[0, 8] - (6 + 9 + 6) / 27) < 1e-15 and abs(s1[0, 9] - 2 / 27) < 1e-15


def test_zero_norm_output_gives_cosine_zero():
    # the proxy output of column 0 is exactly the zero vector: its cosine is 0 (clamped denominator), not NaN
    v_first = [(1, 0), (0.5, 0.25), (0.25, 0.5)]
    v_last = [(-1, 0), (0.25, 0.75), (0, 1.5)]
    labels, s = _hand_case([v_first, v_last], r=0)
    assert np.isfinite(s).all()
    o_ref = np.array([1.0, 3.0]) / 6
    cos = [0.0] + [float(a @ o_ref / np.linalg.norm(a) / np.linalg.norm(o_ref)) for a in (np.array([0.75, 1.0]), np.array([0.25, 2.0]))]
    assert abs(s[0, 2] - sum(cos) / 3) < 1e-12 and abs(s[0, 3] - 0.1 * min(cos[1:])) < 1e-12


def test_total_probability_identity_and_mass_partition():
    w = synth.small(n_blocks=3)
    geom, cache = fill(w)
    q = synth.make_q(w, w.n_blocks - 1, 0)
    rows = np.array([0, 17, 300, 857])
    h = 5  # a Global head: mass is spread, so every term matters
    labels, scores, tok = orc.classify(q, cache, geom, rows=rows, heads=[h], want_tokens=True)
    mass = tok[h]["mass"]
    assert (mass >= 0).all() and (mass[:3] <= 1 + 1e-12).all()
    # mass of a key subset equals exp(lse_subset - lse_full), and the reference output is the
    # mass-weighted mix of the restricted outputs (first / middle / last blocks)
    L = geom.block_tokens
    kb, vb = cache.mono_kv_bits(h)
    k, v = orc.widen_bf16(kb), orc.widen_bf16(vb)
    qq = orc.widen_bf16(q[rows, h])
    sc = 1 / math.sqrt(w.head_dim)
    o_ref, lse = orc.softmax_attention(qq, k, v, sc)
    parts = [orc.softmax_attention(qq, k[a:b], v[a:b], sc) for a, b in ((0, L), (L, 2 * L), (2 * L, 3 * L))]
    m = [np.exp(p[1] - lse) for p in parts]
    assert np.abs(m[0] - mass[0]).max() < 1e-12 and np.abs(m[2] - mass[1]).max() < 1e-12
    mix = sum(mi[:, None] * p[0] for mi, p in zip(m, parts))
    assert np.abs(mix - o_ref).max() < 1e-12
    # six-cell partition: in-neighbourhood + (first or last, outside it) + rest = 1
    near = orc.proxy_allowed(geom, rows, 3 * L, 2)
    p = orc.softmax_attention(qq, k, v, sc, want_p=True)[2]
    edge = np.zeros(3 * L, bool)
    edge[:L] = edge[2 * L:] = True
    outside_edge = np.where(~near & edge[None, :], p, 0).sum(axis=1)
    assert np.abs(mass[2] + outside_edge + mass[3] - 1).max() < 1e-12


@pytest.mark.parametrize("cell", [10, 4])
def test_planted_heads_get_their_labels_with_margin(cell):
    w = synth.tiny(cell=cell)
    geom, cache = fill(w)
    q = synth.make_q(w, w.n_blocks - 1, 0)
    labels, s = orc.classify(q, cache, geom)
    assert tuple(labels) == w.labels == (orc.SINK, orc.DUMMY, orc.SPATIAL, orc.GLOBAL)
    margin = 0.02
    assert s[0, 0] >= 0.95 + margin
    assert s[1, 0] <= 0.95 - margin and s[1, 1] >= 0.95 + margin
    assert max(s[2, 0], s[2, 1]) <= 0.95 - margin and s[2, 2] >= 0.95 + margin and s[2, 5] >= 0.755 + margin
    assert max(s[3, 0], s[3, 1]) <= 0.95 - margin and s[3, 2] <= 0.95 - margin
    # masses tell the same story (Appendix A's description of the archetypes)
    assert s[0, 6] > 0.9 and s[1, 7] > 0.9 and s[2, 8] > 0.9 and s[3, 9] > 0.3
    # a Global head's restricted outputs look like random subsets of a flat distribution
    assert abs(s[3, 0] - math.sqrt(1 / 5)) < 0.15


def test_planted_heads_small_workload_sampled_rows():
    w = synth.small()
    geom, cache = fill(w)
    q = synth.make_q(w, w.n_blocks - 1, 0)
    rows = synth.sample_rows(w, n_random=96)
    labels, s = orc.classify(q, cache, geom, rows=rows)
    assert tuple(labels) == w.labels


# ---- Appendix B / C closed forms ---------------------------------------------------------


def test_flops_and_memory_closed_forms_match_the_appendix():
    g = golden()
    W = g["window_blocks"][0]
    assert abs((1 - orc.flops_ratio(1, 0, 0, 0, W)) - g["sink_reduction"][0]) < 1e-12
    assert abs((1 - orc.flops_ratio(0, 1, 0, 0, W)) - g["dummy_reduction"][0]) < 1e-12
    assert abs((1 - orc.flops_ratio(0, 0, 1, 0, W)) - g["spatial_reduction_480p"][0]) < 0.005
    assert orc.flops_ratio(0, 0, 0, 1, W) == 1.0
    assert abs((1 - orc.flops_ratio(*g["dist_480p"], W)) - g["aggregate_reduction_480p"][0]) < 0.01
    # the Spatial term from the geometry itself: 8 blocks x 1/16 of each frame = 1/2
    geom = orc.Geometry.make(30, 52, 3, 10, 10)
    assert abs(W * orc.spatial_fraction(geom) - 0.5) < 0.04
    # higher resolution -> smaller fraction -> larger reduction (Sec. 5.3)
    fr = [orc.spatial_fraction(orc.Geometry.make(*gr, 3, 10, 10)) for gr in ((30, 52), (45, 80), (68, 120))]
    assert fr[0] > fr[1] > fr[2]
    sd, tot = g["kv_sink_dummy_share"]
    assert abs(orc.kv_reduction(sd, tot, W) - g["kv_reduction"][0]) < 0.01
    # this build's one-block reading with a 7-block cache: (5/12) * (6/7)
    assert abs(orc.kv_reduction(5, 12, 7, 1) - 5 / 12 * 6 / 7) < 1e-15


def test_attend_flops_counts():
    geom = orc.Geometry.make(30, 52, 3, 10, 10)
    labels = [orc.SINK] * 2 + [orc.DUMMY] * 3 + [orc.SPATIAL] * 4 + [orc.GLOBAL] * 3
    L = geom.block_tokens
    dense = 12 * 4.0 * L * 7 * L * 128
    assert abs(dense / 1e9 - 942.0) < 0.5
    assert abs(orc.attend_flops(geom, labels, 7, 128) / 1e9 - 312.5) < 0.5
    # the appendix's accounting: Sink / Dummy read two blocks, i.e. one more L x L product per such head
    two = orc.attend_flops(geom, labels, 7, 128, sd_blocks=2)
    assert two - orc.attend_flops(geom, labels, 7, 128) == 5 * 4.0 * L * L * 128
    assert orc.attend_flops(geom, labels, 1, 128, sd_blocks=2) == orc.attend_flops(geom, labels, 1, 128)


# ---- the input generator -----------------------------------------------------------------


def test_generator_is_deterministic_and_bf16_rounding_is_rne():
    w = synth.tiny()
    a, b = synth.make_kv(w, 2), synth.make_kv(w, 2)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    assert not np.array_equal(synth.make_kv(w, 1)[0], a[0])
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 0.0], np.float32)  # ties go to even
    assert list(synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(x))) == [1.0, 1.0, 1.015625, -2.5, 0.0]
    assert orc.widen_bf16(np.array([0x3F80, 0xC020], np.uint16)).tolist() == [1.0, -2.5]
    rows = synth.sample_rows(synth.wan("480p"))
    assert rows.min() >= 0 and rows.max() < 4680 and np.all(np.diff(rows) > 0) and rows.size >= 256


# ---- appendix variant: Sink / Dummy keep two blocks (App. B, C) ---------------------------


def test_two_block_variant_of_sink_and_dummy():
    rng = np.random.default_rng(21)
    geom = orc.Geometry.make(4, 6, 3, 2, 3)
    L, H, d = geom.block_tokens, 3, 16
    blocks = [(rand_bits(rng, (L, H, d)), rand_bits(rng, (L, H, d))) for _ in range(7)]
    q = rand_bits(rng, (L, H, d), 2.0)
    cache = orc.CacheModel(4, H, sd_mode=1)
    for b in blocks[:3]:
        cache.append(*b)
    cache.split([orc.SINK, orc.DUMMY, orc.GLOBAL])

    def ids(h):
        kb = cache.head_kv_bits(h)[0]
        return [next(i for i, b in enumerate(blocks) if np.array_equal(b[0][:, h], kb[j * L:(j + 1) * L])) for j in range(kb.shape[0] // L)]

    assert ids(0) == [0, 2] and ids(1) == [1, 2] and ids(2) == [0, 1, 2]
    for n in range(3, 6):
        cache.append(*blocks[n])
        assert ids(0) == [0, n] and ids(1) == [n - 1, n]
    # attention of a Sink head = dense attention over {anchor, current}; of a Dummy head over {previous, current}
    two = orc.CacheModel(4, H)
    two.append(*blocks[0]); two.append(*blocks[5])
    prev = orc.CacheModel(4, H)
    prev.append(*blocks[4]); prev.append(*blocks[5])
    o = orc.attend(q, cache, geom)
    assert np.array_equal(o[:, 0], orc.full_attend(q, two)[0][:, 0])
    assert np.array_equal(o[:, 1], orc.full_attend(q, prev)[0][:, 1])
    # per-denoise-step refresh replaces the current block, never the Sink anchor
    cache.overwrite_last(*blocks[6])
    assert ids(0) == [0, 6] and ids(1) == [4, 6] and ids(2)[-1] == 6 and len(ids(2)) == 4
    # one cached block: anchor and current coincide
    one = orc.CacheModel(4, H, sd_mode=1)
    one.append(*blocks[0])
    one.split([orc.SINK, orc.DUMMY, orc.GLOBAL])
    assert one.head_kv_bits(0)[0].shape[0] == L and one.head_kv_bits(1)[0].shape[0] == L
    one.append(*blocks[1])
    assert one.head_kv_bits(0)[0].shape[0] == 2 * L and one.head_kv_bits(1)[0].shape[0] == 2 * L
    # memory: the appendix's formula with W = 8 and 2 kept blocks
    g = golden()
    sd, tot = g["kv_sink_dummy_share"]
    assert abs(orc.kv_reduction(sd, tot, 8, 2) - (sd / tot) * 0.75) < 1e-15


def test_one_block_mode_refresh_leaves_the_sink_frozen():
    rng = np.random.default_rng(22)
    L, H, d = 6, 3, 4
    blocks = [(rand_bits(rng, (L, H, d)), rand_bits(rng, (L, H, d))) for _ in range(4)]
    cache = orc.CacheModel(3, H)
    cache.append(*blocks[0]); cache.append(*blocks[1])
    cache.split([orc.SINK, orc.DUMMY, orc.SPATIAL])
    cache.overwrite_last(*blocks[3])
    assert np.array_equal(cache.head_kv_bits(0)[0], blocks[0][0][:, 0])
    assert np.array_equal(cache.head_kv_bits(1)[0], blocks[3][0][:, 1])
    assert np.array_equal(cache.head_kv_bits(2)[0][L:], blocks[3][0][:, 2])
    assert np.array_equal(cache.mono_kv_bits(0)[0][L:], blocks[3][0][:, 0])
