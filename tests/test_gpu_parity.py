"""GPU parity: the CUDA library (through its C ABI) against the float64 CPU oracle on the same seeded bytes.

Bars: cache contents and labels bit-exact; attention outputs (bf16 Q/K/V, fp32 accumulation, bf16 output)
within max-abs 2e-2 and mean-abs 2e-3 of the oracle; classification scores within 5e-3 (cosines, masses)
and 1e-2 (score).
"""
import numpy as np
import pytest

from oracle import headcast_oracle as orc
from paper_2607_20125_b200 import synth

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 2e-2, 2e-3


def to_dev(bits):
    import torch
    return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).cuda()


def to_f64(t):
    import torch
    return t.float().cpu().numpy().astype(np.float64)


def geometry(w, **kw):
    return orc.Geometry.make(w.grid_h, w.grid_w, w.frames_per_block, w.cell_h, w.cell_w, **kw)


class Pair:
    """The library context and the oracle's cache model, fed the same blocks."""

    def __init__(self, w, keep_monolithic=True, **kw):
        from paper_2607_20125_b200.binding import HeadCast
        self.w = w
        self.hc = HeadCast.from_workload(w, keep_monolithic=keep_monolithic, **kw)
        self.cache = orc.CacheModel(w.n_blocks, w.n_heads, sd_mode=kw.get("sd_mode", 0))
        self.geom = geometry(w, row_edges=kw.get("row_edges"), col_edges=kw.get("col_edges"))
        self.next_block = 0

    def append(self, n=1):
        for _ in range(n):
            k, v = synth.make_kv(self.w, self.next_block)
            self.hc.append(to_dev(k), to_dev(v))
            self.cache.append(k, v)
            self.next_block += 1

    def overwrite_last(self, seed_block):
        """Per-denoise-step refresh of the newest block with fresh seeded K/V."""
        k, v = synth.make_kv(self.w, 1000 + seed_block)
        self.hc.overwrite_last(to_dev(k), to_dev(v))
        self.cache.overwrite_last(k, v)

    def check_cache(self):
        for h in range(self.w.n_heads):
            k, v = self.hc.export_cache(h)
            ko, vo = self.cache.head_kv_bits(h)
            assert k.shape == ko.shape, (h, k.shape, ko.shape)
            assert np.array_equal(k, ko) and np.array_equal(v, vo), f"cache of head {h} differs"

    def check_attention(self, dense, rows=None, step=0):
        import torch
        q = synth.make_q(self.w, self.next_block - 1, step)
        out = torch.full((self.w.block_tokens, self.w.n_heads, self.w.head_dim), float("nan"),
                         dtype=torch.bfloat16, device="cuda")
        (self.hc.full_attend if dense else self.hc.attend)(to_dev(q), out)
        self.hc.check()
        got = to_f64(out)
        assert np.isfinite(got).all(), "rows were left unwritten or are not finite"
        if dense:
            want, _ = orc.full_attend(q, self.cache, rows=rows)
        else:
            want = orc.attend(q, self.cache, self.geom, rows=rows)
        if rows is not None:
            got = got[rows]
        err = np.abs(got - want)
        per_head = err.mean(axis=(0, 2))
        assert err.max() <= MAX_ABS, (err.max(), np.unravel_index(err.argmax(), err.shape))
        assert per_head.max() <= MEAN_ABS, per_head
        return err


def run_pipeline(w, fill, extra, labels=None, rows=None, **kw):
    p = Pair(w, **kw)
    p.append(fill)
    p.check_cache()
    p.check_attention(dense=True, rows=rows)
    p.hc.set_labels(w.labels if labels is None else labels)
    p.hc.split_cache()
    p.cache.split(w.labels if labels is None else labels)
    p.check_cache()
    p.check_attention(dense=False, rows=rows)
    for i in range(extra):
        p.append()
        p.check_cache()
        p.check_attention(dense=False, rows=rows, step=i % 4)
    p.check_attention(dense=True, rows=rows)
    return p


@pytest.mark.parametrize("cell", [10, 4])
def test_tiny_all_rows(cell):
    w = synth.tiny(cell=cell)
    run_pipeline(w, fill=5, extra=3)


def test_small_ragged_split_during_growth_then_roll():
    # 13x22 grid, d=128: L = 858 (6.7 query tiles), cells of 5..7 x 7..8 tokens, window of 4 blocks;
    # split with 2 of 4 blocks cached, then grow to full and roll three times
    w = synth.small()
    run_pipeline(w, fill=2, extra=5)


def test_single_block_cache_and_first_block_is_newest():
    w = synth.small(n_blocks=3)
    p = Pair(w)
    p.append(1)
    p.check_attention(dense=True)
    p.hc.set_labels(w.labels)
    p.hc.split_cache()
    p.cache.split(w.labels)
    p.check_cache()
    p.check_attention(dense=False)


@pytest.mark.parametrize("labels", [[orc.GLOBAL] * 6, [orc.SPATIAL] * 6, [orc.SINK, orc.DUMMY] * 3])
def test_archetype_groups_may_be_empty(labels):
    w = synth.small(n_blocks=3)
    run_pipeline(w, fill=3, extra=1, labels=labels)


@pytest.mark.parametrize("d,cell_h,cell_w", [(128, 13, 11), (64, 13, 22), (128, 2, 3)])
def test_copy_path_geometries_bands_of_large_cells_and_many_small_cells(d, cell_h, cell_w):
    # the bulk copy kernel moves a Spatial cell as one box of the token grid - or, for a cell with more tokens than a
    # 32 KB stage holds, in bands of its rows (13 x 11 tokens at d = 128: bands of 11 + 2 rows; 13 x 22 at d = 64: 11 + 2);
    # 2 x 3 cells give 42 small boxes per frame.  Split during growth, appends through two rolls, refresh of the newest
    # block, Sink / Dummy heads in both modes: exported caches bit-exact every time, attention against the oracle.
    for sd_mode in (0, 1):
        w = synth.small(head_dim=d, cell_h=cell_h, cell_w=cell_w)
        p = Pair(w, keep_monolithic=(sd_mode == 0), sd_mode=sd_mode)
        p.append(2)
        p.check_cache()
        p.hc.set_labels(w.labels)
        p.hc.split_cache()
        p.cache.split(w.labels)
        p.check_cache()
        for i in range(4):
            p.append()
            p.check_cache()
            if i == 1:
                p.overwrite_last(i)
                p.check_cache()
        p.check_attention(dense=False)
        if sd_mode == 0:
            p.check_attention(dense=True)
        p.hc.destroy()


def test_explicit_cell_edges_one_row_cells():
    w = synth.small(n_blocks=3)
    rows_e = [0, 1, 2, 7, 13]
    cols_e = [0, 21, 22]
    run_pipeline(w, fill=3, extra=1, row_edges=rows_e, col_edges=cols_e)


def test_zero_queries_give_the_mean_value_of_each_key_set():
    import torch
    w = synth.small(n_blocks=3)
    p = Pair(w)
    p.append(3)
    p.hc.set_labels(w.labels)
    p.hc.split_cache()
    p.cache.split(w.labels)
    q = torch.zeros((w.block_tokens, w.n_heads, w.head_dim), dtype=torch.bfloat16, device="cuda")
    out = torch.empty_like(q)
    p.hc.attend(q, out)
    p.hc.check()
    got = to_f64(out)
    L = w.block_tokens
    for h, lab in enumerate(w.labels):
        v = orc.widen_bf16(p.cache.mono_kv_bits(h)[1])
        if lab == orc.SINK:
            assert np.abs(got[:, h] - v[:L].mean(axis=0)).max() < 2e-3
        elif lab == orc.DUMMY:
            assert np.abs(got[:, h] - v[-L:].mean(axis=0)).max() < 2e-3
        elif lab == orc.GLOBAL:
            assert np.abs(got[:, h] - v.mean(axis=0)).max() < 2e-3
        else:
            cells = p.geom.cell_of(np.arange(v.shape[0]))
            for t in (0, 21, 300, L - 1):
                want = v[cells == p.geom.cell_of(np.array([t]))[0]].mean(axis=0)
                assert np.abs(got[t, h] - want).max() < 4e-3


def test_wrong_state_calls_change_nothing():
    import torch
    from paper_2607_20125_b200.binding import HeadCastError
    w = synth.tiny()
    p = Pair(w, keep_monolithic=False)
    q = to_dev(synth.make_q(w, 0, 0))
    out = torch.empty_like(q)
    for call in (lambda: p.hc.full_attend(q, out), lambda: p.hc.attend(q, out), lambda: p.hc.split_cache(),
                 lambda: p.hc.classify(q)):
        with pytest.raises(HeadCastError) as e:
            call()
        assert e.value.code == -2
    p.append(1)
    with pytest.raises(HeadCastError) as e:
        p.hc.classify(q)  # one cached block: first block == newest block
    assert e.value.code == -2
    with pytest.raises(HeadCastError) as e:
        p.hc.set_labels([0, 1, 2, 7])
    assert e.value.code == -1
    p.append(1)
    p.hc.set_labels(w.labels)
    p.hc.split_cache()
    p.cache.split(w.labels)
    with pytest.raises(HeadCastError) as e:
        p.hc.full_attend(q, out)  # monolithic cache was released
    assert e.value.code == -2
    with pytest.raises(HeadCastError):
        p.hc.set_labels(w.labels)
    with pytest.raises(ValueError):
        p.hc.attend(q[1:], out)  # the binding refuses a tensor of the wrong shape
    assert p.hc.lib.headcast_attend(p.hc._ctx, q.data_ptr() + 2, out.data_ptr(), None) == -1  # misaligned pointer
    p.check_cache()
    assert p.hc.n_filled() == 2


def check_classify(w, fill, rows=None):
    p = Pair(w)
    p.append(fill)
    q = synth.make_q(w, fill - 1, 0)
    labels, scores = p.hc.classify(to_dev(q))
    want_labels, want = orc.classify(q, p.cache, p.geom, rows=rows)
    assert tuple(labels) == tuple(want_labels) == tuple(w.labels)
    if rows is None:
        d = np.abs(scores.astype(np.float64) - want)
        assert d[:, [0, 1, 2, 6, 7, 8, 9]].max() <= 5e-3, d
        assert d[:, [3, 5]].max() <= 1e-2 and d[:, 4].max() <= 2e-3, d
    assert p.hc.get_labels() == list(w.labels)
    return p


@pytest.mark.parametrize("cell", [10, 4])
def test_classify_tiny(cell):
    p = check_classify(synth.tiny(cell=cell), 5)
    p.hc.split_cache()
    p.cache.split(p.w.labels)
    p.check_cache()
    p.check_attention(dense=False)


def test_mass_rule_gives_the_planted_labels_and_follows_its_threshold():
    # the optional rule on attention masses (same cascade as Eq. 5, one threshold): planted archetypes concentrate their
    # mass on the first block / newest block / neighbourhood, so it reproduces the labels; labels equal the oracle's
    w = synth.tiny(cell=4)
    q = synth.make_q(w, 4, 0)
    for tau, rule_labels in ((0.9, None), (0.999999, None)):
        p = Pair(w, rule=1, mass_tau=tau)
        p.append(5)
        labels, scores = p.hc.classify(to_dev(q))
        want_labels, want = orc.classify(q, p.cache, p.geom, rule=1, mass_tau=tau)
        margin = np.abs(want[:, 6:9] - tau).min()
        if margin > 1e-2:  # away from the threshold the fp32 masses decide like the float64 ones
            assert tuple(labels) == tuple(want_labels), (tau, labels, want_labels)
        assert np.abs(scores[:, 6:].astype(np.float64) - want[:, 6:]).max() <= 5e-3
        if tau == 0.9:
            assert tuple(labels) == tuple(w.labels)
        p.hc.destroy()
    # the cosine rule is untouched by mass_tau
    p = Pair(w, rule=0, mass_tau=0.1)
    p.append(5)
    assert tuple(p.hc.classify(to_dev(q))[0]) == tuple(w.labels)


def test_classify_small_with_ring_rolled_before_classification():
    # 6 appends into a 4-block cache: the newest block is not the last physical slot
    check_classify(synth.small(), 6)


def test_classify_small_two_blocks_no_middle():
    check_classify(synth.small(), 2)


def test_480p_sampled_rows():
    w = synth.wan("480p")
    rows = synth.sample_rows(w, n_random=128)
    p = run_pipeline(w, fill=7, extra=1, rows=rows)
    assert abs(p.hc.attend_flops(False) / 1e9 - 312.5) < 0.5 and abs(p.hc.attend_flops(True) / 1e9 - 942.0) < 0.5


def test_classify_480p_labels_and_sampled_scores():
    # full-size classification on the GPU; the oracle scores a sample of rows (its statistics are those of the sample,
    # so only quantities that do not depend on the row set are compared tightly)
    w = synth.wan("480p")
    p = Pair(w)
    p.append(7)
    q = synth.make_q(w, 6, 0)
    labels, scores = p.hc.classify(to_dev(q))
    rows = synth.sample_rows(w, n_random=64)[::3]
    want_labels, want = orc.classify(q, p.cache, p.geom, rows=rows)
    assert tuple(labels) == tuple(want_labels) == tuple(w.labels)
    d = np.abs(scores.astype(np.float64) - want)
    assert d[:, [0, 1, 2]].max() <= 0.06 and d[:, [6, 7, 8, 9]].max() <= 0.06, d  # sample vs population means


@pytest.mark.parametrize("res,n_random", [("720p", 48), ("1080p", 24)])
def test_hd_grids_sampled_rows(res, n_random):
    w = synth.wan(res)
    rows = synth.sample_rows(w, n_random=n_random)[::5]
    p = Pair(w, keep_monolithic=(res == "720p"))
    p.append(7)
    if res == "720p":
        p.check_attention(dense=True, rows=rows)
    p.hc.set_labels(w.labels)
    p.hc.split_cache()
    p.cache.split(w.labels)
    for h in (0, 5, 11):  # one exported head per call keeps the host copies small
        k, v = p.hc.export_cache(h)
        ko, vo = p.cache.head_kv_bits(h)
        assert np.array_equal(k, ko) and np.array_equal(v, vo)
    p.check_attention(dense=False, rows=rows)
    p.append()
    p.check_attention(dense=False, rows=rows, step=1)


def test_rollout_sequence_three_layers():
    # the streaming schedule of a long rollout at small scale: per layer two warm-up blocks with dense attention, the third
    # block appended and classified at its first denoise step, the split with 3 of 4 blocks cached, then generated
    # blocks x 4 denoise steps with an append (and, once full, a roll) per block; cache checked bit-exactly every block
    for layer in range(3):
        w = synth.small(seed=synth.BASE_SEED + 101 * layer,
                        labels=[(orc.GLOBAL, orc.SPATIAL, orc.SINK, orc.DUMMY, orc.SPATIAL, orc.GLOBAL),
                                (orc.DUMMY, orc.GLOBAL, orc.SPATIAL, orc.SPATIAL, orc.SINK, orc.DUMMY),
                                (orc.SPATIAL, orc.SINK, orc.GLOBAL, orc.DUMMY, orc.GLOBAL, orc.SPATIAL)][layer])
        p = Pair(w)
        rows = synth.sample_rows(w, n_random=40)
        for _ in range(2):
            p.append()
            p.check_attention(dense=True, rows=rows)
        p.append()
        q = synth.make_q(w, 2, 0)
        labels, _ = p.hc.classify(to_dev(q))
        want_labels, _ = orc.classify(q, p.cache, p.geom, rows=rows)
        assert tuple(labels) == tuple(want_labels) == tuple(w.labels)
        p.hc.split_cache()
        p.cache.split(labels)
        p.check_cache()
        for step in range(4):
            p.check_attention(dense=False, rows=rows, step=step)
        for block in range(4):
            p.append()
            p.check_cache()
            for step in (0, 3):
                p.check_attention(dense=False, rows=rows, step=step)


def test_rollout_at_the_720p_grid_two_layers_classified_labels_drive_the_split():
    # the streaming rollout at its own size (45 x 80 grid, 12 heads x 128, 7-block cache), two layers with different
    # seeded head mixes: two warm-up blocks with dense attention, the third block appended and classified on the
    # planted inputs - the labels the GPU returns (equal to the oracle's and to the planted ones) drive the split at 3
    # cached blocks - then 6 more appends, so the ring fills (7) and rolls twice.  Every block: cache bit-exact for
    # three exported heads, attention on sampled rows at the first and last denoise step.
    for layer in (0, 1):
        w = synth.wan("720p", layer=layer)
        rows = synth.sample_rows(w, n_random=32)[::7]
        p = Pair(w, keep_monolithic=(layer == 0))
        for _ in range(2):
            p.append()
            p.check_attention(dense=True, rows=rows)
        p.append()
        q = synth.make_q(w, 2, 0)
        labels, _ = p.hc.classify(to_dev(q))
        want_labels, _ = orc.classify(q, p.cache, p.geom, rows=rows[::2])
        assert tuple(int(v) for v in labels) == tuple(int(v) for v in want_labels) == tuple(w.labels)
        p.hc.split_cache()  # no set_labels: the context splits by what its own classification found
        p.cache.split([int(v) for v in labels])
        assert p.hc.n_filled() == 3
        for block in range(6):
            p.append()
            assert p.hc.n_filled() == min(7, 4 + block)
            for h in [(3 * block + i * 5 + layer) % w.n_heads for i in range(3)]:
                k, v = p.hc.export_cache(h)
                ko, vo = p.cache.head_kv_bits(h)
                assert k.shape == ko.shape and np.array_equal(k, ko) and np.array_equal(v, vo), (layer, block, h)
            for step in (0, 3):
                p.check_attention(dense=False, rows=rows, step=step)
        if layer == 0:
            p.check_attention(dense=True, rows=rows)  # the monolithic ring kept alongside rolled the same way
        p.hc.destroy()


def test_cuda_graph_replay_of_append_and_attend_matches_eager_bit_for_bit():
    # the steady state of a rollout captured into CUDA graphs, one per ring position (the slot a new block lands in
    # cycles with period n_blocks - 1, and after that many appends the host-side ring is back where it started);
    # replays with fresh data in the static input buffers give the eager context's bytes
    import torch
    w = synth.small()
    eager, graphed = Pair(w, keep_monolithic=False), Pair(w, keep_monolithic=False)
    for p in (eager, graphed):
        p.append(w.n_blocks)
        p.hc.set_labels(w.labels)
        p.hc.split_cache()
        p.cache.split(w.labels)
        p.append()  # the work lists of the full cache are uploaded by this eager step
        p.check_attention(dense=False, rows=synth.sample_rows(w, n_random=16))
    L, H, D = w.block_tokens, w.n_heads, w.head_dim
    k_buf, v_buf, q_buf = (torch.zeros((L, H, D), dtype=torch.bfloat16, device="cuda") for _ in range(3))
    out_g, out_e = torch.zeros_like(q_buf), torch.zeros_like(q_buf)
    period = w.n_blocks - 1
    graphs = []
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        for ph in range(period):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                graphed.hc.append(k_buf, v_buf)
                graphed.hc.attend(q_buf, out_g)
            graphs.append(g)
    torch.cuda.synchronize()
    for i in range(2 * period + 1):
        k, v = synth.make_kv(w, 50 + i)
        q = synth.make_q(w, 50 + i, i % 4)
        k_buf.copy_(to_dev(k)); v_buf.copy_(to_dev(v)); q_buf.copy_(to_dev(q))
        graphs[i % period].replay()
        eager.hc.append(to_dev(k), to_dev(v))
        eager.hc.attend(to_dev(q), out_e)
        torch.cuda.synchronize()
        assert torch.equal(out_g, out_e), i
        graphed.hc.append(k_buf, v_buf)  # keeps the graphed context's host-side ring in step with what the replay did
        for h in (0, 3):
            kg, vg = graphed.hc.export_cache(h)
            ke, ve = eager.hc.export_cache(h)
            assert np.array_equal(kg, ke) and np.array_equal(vg, ve)
    eager.hc.check(); graphed.hc.check()


def test_an_expired_wait_is_reported_and_the_context_stays_usable():
    # failure detection without a GPU fault: a kernel waits (bounded) on a barrier nothing signals, gives up after
    # 50 ms, the host sees HC_ERR_TIMEOUT, and the same context then computes correct attention
    import time
    w = synth.tiny()
    p = Pair(w)
    p.append(2)
    t0 = time.perf_counter()
    assert p.hc.selftest_bounded_wait(50) == -6
    assert 0.04 < time.perf_counter() - t0 < 5.0
    assert "bounded wait" in p.hc.lib.headcast_last_error(p.hc._ctx).decode()
    p.hc.check()  # the status word was cleared by the report
    p.check_attention(dense=True)


@pytest.mark.parametrize("fill", [1, 2, 4])
def test_anchor_plus_current_variant_of_sink_and_dummy(fill):
    # Appendix B / C accounting: Sink = anchor + current block, Dummy = previous + current block; split with 1, 2 or
    # all 4 blocks cached, then appends that roll the window, with a per-step refresh of the current block in between
    w = synth.small()
    p = Pair(w, sd_mode=1)
    p.append(fill)
    p.hc.set_labels(w.labels)
    p.hc.split_cache()
    p.cache.split(w.labels)
    p.check_cache()
    p.check_attention(dense=False)
    for i in range(4):
        p.append()
        p.check_cache()
        p.check_attention(dense=False, step=i)
        p.overwrite_last(i)
        p.check_cache()
        p.check_attention(dense=False, step=i)
    p.check_attention(dense=True)
    assert abs(p.hc.attend_flops(False) - orc.attend_flops(p.geom, w.labels, 4, w.head_dim, sd_blocks=2)) < 1.0


def test_refresh_of_the_current_block_in_one_block_mode():
    w = synth.small()
    p = Pair(w)
    p.append(2)
    p.overwrite_last(0)  # before the split: monolithic cache only
    p.check_cache()
    p.check_attention(dense=True)
    p.hc.set_labels(w.labels)
    p.hc.split_cache()
    p.cache.split(w.labels)
    for i in range(3):
        p.overwrite_last(1 + i)
        p.check_cache()
        p.check_attention(dense=False, step=i)
        p.append()
    p.check_cache()
    p.check_attention(dense=True)


@pytest.mark.parametrize("labels", [None, [orc.GLOBAL] * 6, [orc.SINK, orc.DUMMY, orc.SPATIAL] * 2, "tiny"])
def test_host_buffer_calls_match_the_oracle(labels):
    """headcast_append_host / headcast_attend_host: host tensors in, host tensor out, stage-wise overlap of the
    copies with the kernels; cache content stays bit-exact and the outputs meet the same bars as headcast_attend.
    Pinned and pageable host memory are both accepted.  "tiny": a block shorter than one query-tile pair (192
    tokens), where the Global heads' rows cannot be halved."""
    import torch
    w = synth.tiny() if labels == "tiny" else synth.small()
    lab = w.labels if labels is None or labels == "tiny" else labels
    p = Pair(w)
    p.append(2)
    p.hc.set_labels(lab)
    p.hc.split_cache()
    p.cache.split(lab)
    for i in range(4):  # grows to the full window and rolls once
        k, v = synth.make_kv(w, p.next_block)
        host = lambda bits: torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16)
        kh, vh = host(k), host(v)
        if i % 2 == 0:
            kh, vh = kh.pin_memory(), vh.pin_memory()
        p.hc.append_host(kh, vh)
        p.cache.append(k, v)
        p.next_block += 1
        p.check_cache()
        q = synth.make_q(w, p.next_block - 1, i)
        qh = host(q)
        oh = torch.full(qh.shape, float("nan"), dtype=torch.bfloat16)
        if i % 2 == 0:
            qh, oh = qh.pin_memory(), oh.pin_memory()
        p.hc.attend_host(qh, oh)
        torch.cuda.current_stream().synchronize()
        p.hc.check()
        got = oh.float().numpy().astype(np.float64)
        assert np.isfinite(got).all(), "columns of some head were not copied back"
        want = orc.attend(q, p.cache, p.geom)
        err = np.abs(got - want)
        assert err.max() <= MAX_ABS and err.mean(axis=(0, 2)).max() <= MEAN_ABS
        # and the device entry point still agrees afterwards (the two paths share the partial-result buffers)
        p.check_attention(dense=False, step=i)


@pytest.mark.parametrize("case", range(12))
def test_seeded_random_shapes(case):
    """Shapes nobody picked by hand: grid, cell size, head count and head_dim, window, frames per block, label mix
    (classes may be missing), fill level at the split, number of rolls and the Sink/Dummy mode are drawn from a
    seeded generator; every stage of the pipeline must still match the oracle."""
    rng = np.random.default_rng(4200 + case)
    n_heads = int(rng.integers(2, 7))
    w = synth.Workload(
        name=f"random{case}", n_heads=n_heads, head_dim=int(rng.choice([64, 128])),
        grid_h=int(rng.integers(3, 15)), grid_w=int(rng.integers(4, 21)), n_blocks=int(rng.integers(2, 6)),
        frames_per_block=int(rng.integers(1, 4)), cell_h=int(rng.integers(2, 8)), cell_w=int(rng.integers(2, 8)),
        labels=tuple(int(v) for v in rng.integers(0, 4, size=n_heads)), sink_alpha=8.0, seed=synth.BASE_SEED + case)
    fill = int(rng.integers(1, w.n_blocks + 1))
    extra = int(rng.integers(1, 2 * w.n_blocks))
    run_pipeline(w, fill=fill, extra=extra, sd_mode=int(rng.integers(0, 2)))
    # classification of the same shape (needs two cached blocks; the ring may have rolled), with a drawn proxy radius
    # and gamma: scores within the bars; labels must agree wherever the float64 decision is not within the score
    # tolerance of a threshold; the labels found then drive the split
    r, gamma = int(rng.integers(0, 4)), float(rng.choice([1.0, 5.0, 20.0]))
    cfill = int(rng.integers(2, 2 * w.n_blocks + 1))
    p = Pair(w, proxy_radius=r, gamma=gamma)
    p.append(cfill)
    q = synth.make_q(w, cfill - 1, 0)
    labels, scores = p.hc.classify(to_dev(q))
    want_labels, want = orc.classify(q, p.cache, p.geom, r=r, gamma=gamma)
    d = np.abs(scores.astype(np.float64) - want)
    score_tol = 1e-2 + gamma * 2e-3  # score = P5 - gamma * MSE
    assert d[:, [0, 1, 2, 6, 7, 8, 9]].max() <= 5e-3, d
    assert d[:, 3].max() <= 1e-2 and d[:, 4].max() <= 2e-3 and d[:, 5].max() <= score_tol, d
    theta = np.array([0.95, 0.95, 0.95])
    decisive = (np.abs(want[:, :3] - theta).min(axis=1) > 1e-2) & (np.abs(want[:, 5] - 0.755) > 2 * score_tol)
    assert all(int(a) == int(b) for a, b, ok in zip(labels, want_labels, decisive) if ok), (labels, want_labels)
    p.hc.split_cache()
    p.cache.split([int(v) for v in labels])
    p.check_cache()
    p.check_attention(dense=False)


def test_maximum_head_and_block_counts():
    """The largest context the header allows: 64 heads and a 32-block window (small grid so that the oracle stays
    quick).  Fills the whole window, splits, rolls past the end of the ring, and classifies."""
    rng = np.random.default_rng(77)
    labels = tuple(int(v) for v in rng.integers(0, 4, size=64))
    w = synth.Workload(name="limits", n_heads=64, head_dim=64, grid_h=5, grid_w=7, n_blocks=32, frames_per_block=2,
                       cell_h=3, cell_w=4, labels=labels, sink_alpha=8.0, seed=synth.BASE_SEED + 99)
    rows = np.arange(0, w.block_tokens, 3)
    p = run_pipeline(w, fill=32, extra=3, rows=rows)
    assert p.hc.n_filled() == 32
    q = synth.make_q(w, p.next_block - 1, 1)
    c = Pair(w)
    c.append(32)
    got_labels, scores = c.hc.classify(to_dev(synth.make_q(w, 31, 0)))
    want_labels, want = orc.classify(synth.make_q(w, 31, 0), c.cache, c.geom)
    d = np.abs(scores.astype(np.float64) - want)
    assert d[:, [0, 1, 2, 6, 7, 8, 9]].max() <= 5e-3 and d[:, [3, 5]].max() <= 1e-2 and d[:, 4].max() <= 2e-3
    decisive = (np.abs(want[:, :3] - 0.95).min(axis=1) > 1e-2) & (np.abs(want[:, 5] - 0.755) > 2e-2)
    assert all(int(a) == int(b) for a, b, ok in zip(got_labels, want_labels, decisive) if ok)


def test_head_sharded_layer_on_one_rank_equals_the_plain_layer():
    # the sharding wrapper with the CUDA engine on a process group of one rank: head columns in, gathered outputs out,
    # and the rebuild used when heads change owner (export every head's cache, append the blocks to a fresh context)
    # after the ring has rolled; the caches must equal the plain context's bit for bit, the outputs up to rounding
    import torch
    import torch.distributed as dist
    from paper_2607_20125_b200 import sharding
    from paper_2607_20125_b200.binding import HeadCast
    w = synth.small()
    geom = geometry(w)
    L, H, d = w.block_tokens, w.n_heads, w.head_dim
    own_group = not dist.is_initialized()
    if own_group:
        import socket
        with socket.socket() as s:
            s.bind(("127.0.0.1", 0))
            port = s.getsockname()[1]
        dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1)
    try:
        kw = dict(grid_h=w.grid_h, grid_w=w.grid_w, n_blocks=w.n_blocks, frames_per_block=w.frames_per_block,
                  cell_h=w.cell_h, cell_w=w.cell_w, keep_monolithic=True)
        layer = sharding.HeadShardedHeadCast(H, d, L, geom.n_cells, **kw)
        plain = HeadCast.from_workload(w, keep_monolithic=True)
        n_warm = w.n_blocks + 1
        for b in range(n_warm):
            k, v = synth.make_kv(w, b)
            layer.append(to_dev(k), to_dev(v))
            plain.append(to_dev(k), to_dev(v))
        q = to_dev(synth.make_q(w, n_warm - 1, 0))
        out, ref = torch.zeros_like(q), torch.zeros_like(q)
        layer.full_attend(q, out)
        plain.full_attend(q, ref)
        torch.cuda.synchronize()
        assert torch.equal(out.view(torch.int16), ref.view(torch.int16))
        labels, scores = layer.classify(q)
        ref_labels, ref_scores = plain.classify(q)
        assert list(labels) == list(ref_labels) == list(w.labels)
        assert np.array_equal(scores, ref_scores)
        kept = {h: layer.engine.export_cache_device(h) for h in range(H)}
        layer._rebuild(kept, layer.engine.n_filled())
        layer.split_cache(labels)
        plain.split_cache()
        for b in range(n_warm, n_warm + 2):
            k, v = synth.make_kv(w, b)
            layer.append(to_dev(k), to_dev(v))
            plain.append(to_dev(k), to_dev(v))
            q = to_dev(synth.make_q(w, b, 1))
            layer.attend(q, out)
            plain.attend(q, ref)
            torch.cuda.synchronize()
            # the rebuilt ring starts at another slot, so key tiles are summed in another order: equal up to rounding
            err = np.abs(to_f64(out) - to_f64(ref))
            assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS / 4
        for h in (0, H - 1):
            for a, b_ in zip(layer.engine.export_cache(h), plain.export_cache(h)):
                assert np.array_equal(a, b_)
    finally:
        if own_group:
            dist.destroy_process_group()


def test_two_contexts_on_two_streams_give_the_single_stream_results():
    # two layers driven from two CUDA streams at once (the library keeps no state outside its contexts): every output
    # must equal, bit for bit, what the same calls give one after the other
    import torch
    from paper_2607_20125_b200.binding import HeadCast
    ws = [synth.small(seed=synth.BASE_SEED + 5), synth.tiny()]

    def prepare(w):
        hc = HeadCast.from_workload(w, keep_monolithic=True)
        for b in range(w.n_blocks):
            hc.append(*[to_dev(t) for t in synth.make_kv(w, b)])
        hc.set_labels(w.labels)
        hc.split_cache()
        return hc

    def step(hc, w, i, outs):
        if i % 2 == 0:
            hc.append(*[to_dev(t) for t in synth.make_kv(w, w.n_blocks + i)])
        q = to_dev(synth.make_q(w, w.n_blocks + i, i % 4))
        o = torch.empty_like(q)
        hc.attend(q, o)
        outs.append(o)

    ref = [[], []]
    for i, w in enumerate(ws):
        hc = prepare(w)
        for s in range(6):
            step(hc, w, s, ref[i])
        torch.cuda.synchronize()
        hc.check()
        hc.destroy()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    got, ctx = [[], []], []
    for i, w in enumerate(ws):
        with torch.cuda.stream(streams[i]):
            ctx.append(prepare(w))
    for s in range(6):
        for i, w in enumerate(ws):
            with torch.cuda.stream(streams[i]):
                step(ctx[i], w, s, got[i])
    torch.cuda.synchronize()
    for i in range(2):
        ctx[i].check()
        for a, b in zip(got[i], ref[i]):
            assert torch.equal(a.view(torch.int16), b.view(torch.int16))
        ctx[i].destroy()


def test_contexts_give_their_device_memory_back():
    # every phase once per context (dense, classification, split, append, both attends, the host-buffer calls with
    # their staging buffers, streams and events), 40 contexts in a row: the device memory in use must not grow
    import torch
    from paper_2607_20125_b200.binding import HeadCast
    w = synth.small()
    kv = [[to_dev(t) for t in synth.make_kv(w, b)] for b in range(w.n_blocks + 1)]
    q = to_dev(synth.make_q(w, 1, 0))
    o = torch.empty_like(q)
    qh, kh, vh = q.cpu().pin_memory(), kv[0][0].cpu().pin_memory(), kv[0][1].cpu().pin_memory()
    oh = torch.empty_like(qh).pin_memory()

    def once():
        hc = HeadCast.from_workload(w, keep_monolithic=True)
        for b in range(w.n_blocks):
            hc.append(*kv[b])
        hc.full_attend(q, o)
        hc.classify(q)
        hc.split_cache()
        hc.append(*kv[-1])
        hc.attend(q, o)
        hc.append_host(kh, vh)
        hc.attend_host(qh, oh)
        torch.cuda.synchronize()
        hc.check()
        hc.destroy()

    def in_use():
        torch.cuda.synchronize()
        free, total = torch.cuda.mem_get_info()
        return (total - free) / 2 ** 20

    for _ in range(3):
        once()
    before = in_use()
    for _ in range(40):
        once()
    assert in_use() - before < 8.0


def test_repeated_attends_are_bit_identical_with_the_shared_queue():
    """At 480P the end of a launch is drawn from the shared queue by whichever CTA is free: which CTA runs a piece changes
    from launch to launch, what it computes and the order of the merge do not, so repeated calls give the same bits."""
    import torch
    w = synth.wan("480p")
    from paper_2607_20125_b200 import binding
    from test_schedule_host import config_of
    items, first = binding.plan_schedule(config_of(w), list(w.labels), w.n_blocks, 148)
    assert first[-1] < len(items), "no shared queue at this size any more: pick a larger one"
    p = Pair(w)
    p.append(w.n_blocks)
    p.hc.set_labels(w.labels)
    p.hc.split_cache()
    q = to_dev(synth.make_q(w, w.n_blocks - 1, 0))
    ref = torch.empty((w.block_tokens, w.n_heads, w.head_dim), dtype=torch.bfloat16, device="cuda")
    p.hc.attend(q, ref)
    outs = [torch.full_like(ref, float("nan")) for _ in range(8)]
    for rep in range(40):
        p.hc.attend(q, outs[rep % 8])
    p.hc.check()
    assert all(torch.equal(o, ref) for o in outs)


def test_query_tiles_cut_into_dozens_of_pieces_are_merged_row_by_row():
    """Six Global heads over a 32-block window at a 32x32 grid: the launch is long enough for the shared queue at its
    end, whose pieces are cuts of the last pairs - those pairs end up in about thirty pieces each, which the merge
    handles with one block per row.  The host plan says which rows those are; they are all compared."""
    w = synth.Workload(name="long_groups", n_heads=6, head_dim=128, grid_h=32, grid_w=32, n_blocks=32,
                       frames_per_block=1, cell_h=8, cell_w=8, labels=(orc.GLOBAL,) * 6, seed=synth.BASE_SEED + 321)
    from paper_2607_20125_b200 import binding
    from test_schedule_host import F, config_of
    items, first = binding.plan_schedule(config_of(w), list(w.labels), w.n_blocks, 148)
    parts = {}
    for it in items:
        if it[F["out_mode"]] == 1:
            key = (int(it[F["head"]]), int(it[F["q_start0"]]))
            parts[key] = parts.get(key, 0) + 1
    long_pairs = [k for k, n in parts.items() if n > 16]
    assert long_pairs and first[-1] < len(items), "the plan no longer has a pair in more than 16 pieces: pick another shape"
    rows = np.unique(np.concatenate([np.arange(q0, min(q0 + 256, w.block_tokens), 5) for _, q0 in long_pairs]
                                    + [np.arange(0, w.block_tokens, 37)]))
    p = Pair(w)
    p.append(w.n_blocks)
    p.hc.set_labels(w.labels)
    p.hc.split_cache()
    p.cache.split(w.labels)
    p.check_attention(dense=False, rows=rows)
    p.check_attention(dense=True, rows=rows)


@pytest.mark.parametrize("scale", [0.01, 16.0, 256.0])
def test_flat_peaked_and_huge_logits(scale):
    # queries scaled so that the softmax is nearly uniform, nearly one-hot, or has logits in the thousands; a few rows
    # get one enormous coordinate, so their logits jump by hundreds from one key tile to the next (the running
    # reference has to be moved and the accumulated output rescaled).  Every pathway, dense and head-specific.
    import torch
    w = synth.small()
    p = Pair(w, sd_mode=1)
    p.append(w.n_blocks)
    p.hc.set_labels(w.labels)
    p.hc.split_cache()
    p.cache.split(w.labels)
    rng = np.random.default_rng(99)
    qf = synth.bf16_bits_to_f32(synth.make_q(w, w.n_blocks - 1, 0)) * scale
    qf[rng.integers(0, w.block_tokens, size=16), :, 7] *= 50.0
    q = synth.f32_to_bf16_bits(qf.astype(np.float32))
    for dense in (True, False):
        out = torch.full((w.block_tokens, w.n_heads, w.head_dim), float("nan"), dtype=torch.bfloat16, device="cuda")
        (p.hc.full_attend if dense else p.hc.attend)(to_dev(q), out)
        p.hc.check()
        got = to_f64(out)
        want = orc.full_attend(q, p.cache)[0] if dense else orc.attend(q, p.cache, p.geom)
        assert np.isfinite(got).all()
        err = np.abs(got - want)
        assert (err <= np.maximum(MAX_ABS, np.abs(want) * 2.0 ** -7)).all(), err.max()  # one bf16 step on large outputs
        assert err.mean(axis=(0, 2)).max() <= MEAN_ABS
