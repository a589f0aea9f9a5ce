"""The allocation-free dense attention entry point against the context-based one.

Some hosts cannot let the library allocate device memory (their own pool owns the GPU, or they cannot take the
device-wide synchronisation of an allocation); for them headcast_dense_attend_noalloc keeps its scratch in a fixed
device array inside the library.  That array keeps the previous call's contents, so the check runs two different
calls in a row, and this file is collected last so that a failure here cannot hide any other test.
"""
import numpy as np
import pytest

from paper_2607_20125_b200 import synth

pytestmark = pytest.mark.gpu


def dev(bits):
    import torch
    return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).cuda()


def reference(w, n_fill, q):
    """headcast_full_attend on a context holding the same blocks."""
    import torch
    from paper_2607_20125_b200.binding import HeadCast
    hc = HeadCast.from_workload(w, keep_monolithic=True)
    blocks = [synth.make_kv(w, b) for b in range(n_fill)]
    for k, v in blocks:
        hc.append(dev(k), dev(v))
    out = torch.empty_like(q)
    hc.full_attend(q, out)
    hc.check()
    k_all = dev(np.concatenate([k for k, _ in blocks], axis=0))
    v_all = dev(np.concatenate([v for _, v in blocks], axis=0))
    hc.destroy()
    return out, k_all, v_all


def test_two_calls_in_a_row_match_full_attend():
    import torch
    from paper_2607_20125_b200 import binding
    cases = [(synth.small(n_blocks=3), 3), (synth.tiny(), 2)]  # d=128 ragged, then d=64 with fewer items
    for w, n_fill in cases:
        q = dev(synth.make_q(w, n_fill - 1, 0))
        want, k_all, v_all = reference(w, n_fill, q)
        got = torch.full_like(q, float("nan"))
        before = torch.cuda.memory_allocated()
        binding.dense_attend_noalloc(q, k_all, v_all, got)
        binding.noalloc_status()
        assert torch.cuda.memory_allocated() == before
        d = (got.float() - want.float()).abs()
        assert torch.isfinite(got.float()).all()
        assert d.max().item() <= 2e-2 and d.mean().item() <= 2e-3, (w.name, d.max().item(), d.mean().item())


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
