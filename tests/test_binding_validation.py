"""The binding rejects tensors that would make a kernel run past the caller's buffer (no GPU needed: every check
happens before the library is called)."""
import pytest
import torch

from paper_2607_20125_b200 import binding


def test_validate_rejects_wrong_dtype_rank_shape_layout_and_device():
    ok = torch.zeros((6, 2, 64), dtype=torch.bfloat16)
    binding._validate(ok, "q", (6, 2, 64), cuda=False)
    binding._validate(ok, "q", (None, 2, 64), cuda=False)
    with pytest.raises(ValueError, match="dtype"):
        binding._validate(ok.float(), "q", (6, 2, 64), cuda=False)
    with pytest.raises(ValueError, match="shape"):
        binding._validate(ok, "q", (6, 2, 128), cuda=False)
    with pytest.raises(ValueError, match="shape"):
        binding._validate(ok[0], "q", (6, 2, 64), cuda=False)
    with pytest.raises(ValueError, match="contiguous"):
        binding._validate(ok.transpose(0, 1), "q", (2, 6, 64), cuda=False)
    with pytest.raises(ValueError, match="CUDA"):
        binding._validate(ok, "q", (6, 2, 64), cuda=True)
    with pytest.raises(ValueError, match="torch tensor"):
        binding._validate([1, 2, 3], "q", (3,), cuda=False)


def test_entry_points_validate_before_calling_the_library():
    q = torch.zeros((6, 2, 64), dtype=torch.bfloat16)
    with pytest.raises(ValueError):
        binding.dense_attend_noalloc(q, q, q, q)  # CPU tensors
    with pytest.raises(ValueError):
        binding.dense_attend_noalloc(q[0], q, q, q)

    class Stub(binding.HeadCast):  # the methods' checks, without a context
        def __init__(self):
            self.lib, self._ctx = binding.load_library(), None  # arguments are checked before the call is made
            self.n_heads, self.head_dim, self.block_tokens, self.n_blocks = 2, 64, 6, 3

        def destroy(self):
            pass

    hc = Stub()
    for call in (lambda: hc.append(q, q), lambda: hc.overwrite_last(q, q), lambda: hc.attend(q, q), lambda: hc.full_attend(q, q),
                 lambda: hc.classify(q), lambda: hc.attend_host(q[:4], q), lambda: hc.append_host(q.float(), q),
                 lambda: hc.set_labels([0, 1, 2])):
        with pytest.raises(ValueError):
            call()
