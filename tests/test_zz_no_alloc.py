"""The allocation-free dense attention entry point against the context-based one and against the CPU oracle.

Some hosts cannot let the library allocate device memory (their own pool owns the GPU, or they cannot take the
device-wide synchronisation of an allocation); for them headcast_dense_attend_noalloc keeps its scratch in a fixed
device array inside the library.  That array keeps the previous call's contents, so the checks run several
different calls in a row, and this file is collected last so that a failure here cannot hide any other test.
"""
import numpy as np
import pytest

from oracle import headcast_oracle as orc
from paper_2607_20125_b200 import synth

pytestmark = pytest.mark.gpu


def dev(bits):
    import torch
    return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).cuda()


def to_f64(t):
    import torch
    return orc.widen_bf16(t.view(torch.int16).cpu().numpy().view(np.uint16))


def full_attend_reference(w, blocks, q):
    """headcast_full_attend on a context holding the same blocks."""
    import torch
    from paper_2607_20125_b200.binding import HeadCast
    hc = HeadCast.from_workload(w, keep_monolithic=True)
    for k, v in blocks:
        hc.append(dev(k), dev(v))
    out = torch.empty_like(q)
    hc.full_attend(q, out)
    hc.check()
    hc.destroy()
    return out


def oracle_reference(w, blocks, q_bits):
    cache = orc.CacheModel(w.n_blocks, w.n_heads)
    for k, v in blocks:
        cache.append(k, v)
    return orc.full_attend(q_bits, cache)[0]


def driver_free_bytes():
    """Free device memory as the driver counts it: unlike torch's own counters this also sees an allocation made
    inside the library."""
    import torch
    torch.cuda.synchronize()
    return torch.cuda.mem_get_info()[0]


def test_two_calls_in_a_row_match_full_attend_and_the_oracle():
    import torch
    from paper_2607_20125_b200 import binding
    cases = [(synth.small(n_blocks=3), 3), (synth.tiny(), 2)]  # d=128 ragged, then d=64 with fewer items
    prepared = []
    for w, n_fill in cases:
        blocks = [synth.make_kv(w, b) for b in range(n_fill)]
        q_bits = synth.make_q(w, n_fill - 1, 0)
        q = dev(q_bits)
        k_all = dev(np.concatenate([k for k, _ in blocks], axis=0))
        v_all = dev(np.concatenate([v for _, v in blocks], axis=0))
        prepared.append((w, q, k_all, v_all, full_attend_reference(w, blocks, q), oracle_reference(w, blocks, q_bits),
                         torch.full_like(q, float("nan"))))
    # warm both kernel variants once (the first call on a device looks up the scratch address, and the driver loads a
    # kernel's code on its first launch), then watch the driver's free-memory figure across the two calls under
    # test: nothing may be allocated, by torch or by the library
    for w, q, k_all, v_all, _, _, got in prepared:
        binding.dense_attend_noalloc(q, k_all, v_all, got)
        binding.noalloc_status()
        got.fill_(float("nan"))
    free_before = driver_free_bytes()
    for w, q, k_all, v_all, _, _, got in prepared:
        binding.dense_attend_noalloc(q, k_all, v_all, got)
    binding.noalloc_status()
    assert driver_free_bytes() == free_before
    for w, q, k_all, v_all, want_gpu, want, got in prepared:
        assert torch.isfinite(got.float()).all()
        # same kernel, but the context's scheduler may cut key ranges and merge partial results: equal up to rounding
        dg = (got.float() - want_gpu.float()).abs()
        assert dg.max().item() <= 2e-2 and dg.mean().item() <= 2e-3, (w.name, dg.max().item())
        d = np.abs(to_f64(got) - want)
        for h in range(w.n_heads):
            assert d[:, h].max() <= 2e-2 and d[:, h].mean() <= 2e-3, (w.name, h, d[:, h].max(), d[:, h].mean())


def test_same_shapes_other_buffers_back_to_back():
    # two calls whose shapes agree and whose K / V live elsewhere: the second must read ITS keys, not the first call's
    import torch
    from paper_2607_20125_b200 import binding
    w = synth.small(n_blocks=2)
    q_bits = synth.make_q(w, 1, 0)
    q = dev(q_bits)
    sets = [[synth.make_kv(w, b) for b in (0, 1)], [synth.make_kv(w, b) for b in (2, 3)]]
    outs = []
    for blocks in sets:
        k_all = dev(np.concatenate([k for k, _ in blocks], axis=0))
        v_all = dev(np.concatenate([v for _, v in blocks], axis=0))
        got = torch.full_like(q, float("nan"))
        binding.dense_attend_noalloc(q, k_all, v_all, got)
        outs.append((got, k_all, v_all))  # keep the buffers alive until the stream is synchronised
    binding.noalloc_status()
    assert not torch.equal(outs[0][0], outs[1][0])
    for blocks, (got, _, _) in zip(sets, outs):
        dg = (got.float() - full_attend_reference(w, blocks, q).float()).abs()
        assert dg.max().item() <= 2e-2 and dg.mean().item() <= 2e-3
        d = np.abs(to_f64(got) - oracle_reference(w, blocks, q_bits))
        assert d.max() <= 2e-2 and d.mean() <= 2e-3


def test_sizes_beyond_the_fixed_scratch_are_rejected():
    import torch
    from paper_2607_20125_b200 import binding
    q = torch.zeros((256 * 40, 64, 64), dtype=torch.bfloat16, device="cuda")  # 64 heads x 40 pairs = 2560 items
    kv = torch.zeros((128, 64, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.HeadCastError) as e:
        binding.dense_attend_noalloc(q, kv, kv, torch.empty_like(q))
    assert e.value.code == -5 and "HEADCAST_NOALLOC_MAX_ITEMS" in str(e.value)
    with pytest.raises(binding.HeadCastError) as e:
        binding.dense_attend_noalloc(q[:256, :4, :48].contiguous(), kv[:, :4, :48].contiguous(), kv[:, :4, :48].contiguous(),
                                     torch.empty((256, 4, 48), dtype=torch.bfloat16, device="cuda"))
    assert e.value.code == -1
