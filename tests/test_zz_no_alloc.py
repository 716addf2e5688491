"""The no-allocation forward (scratch inside the library image) against the regular forward.

Collected last on purpose: a run that stops at the first failure has already run every other test.
It serves callers that cannot allocate device memory at the call site (a serving loop that must not hit
cudaMalloc after start-up, a plug-in inside a host that owns all device memory); they still own q, k, v, o."""
import numpy as np
import pytest
import torch

from paper_2609_09721_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def _dev(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def test_static_scratch_forward_matches_workspace_forward_twice():
    """Two calls in a row on different problems: the second must not see anything of the first in the
    shared scratch.  Both are compared with efq_attention_fwd on a caller-owned workspace."""
    cases = [inputs.AttentionCase("a", 1, 4, 2, 640, 640, 128, True, 31, "k_outliers"),
             inputs.AttentionCase("b", 1, 2, 1, 300, 900, 128, False, 32, "iid")]
    for case in cases:
        q, k, v = (_dev(t) for t in inputs.make_qkv(case))
        want = binding.efq_attention_fwd(q, k, v, case.causal)
        o = torch.full_like(want, float("nan"))          # caller-owned output, allocated before the call
        before = torch.cuda.memory_stats()["allocation.all.allocated"]
        got = binding.efq_attention_fwd_static(q, k, v, case.causal, o=o)
        torch.cuda.synchronize()
        assert torch.cuda.memory_stats()["allocation.all.allocated"] == before   # no request reached torch's allocator either
        assert got.data_ptr() == o.data_ptr()
        assert torch.isfinite(got).all()
        assert torch.equal(got, want)       # the same kernels on the same operands: not a tolerance, the same bits
    # same problem again, back to back: results repeat exactly
    again = binding.efq_attention_fwd_static(q, k, v, case.causal, o=torch.empty_like(want))
    torch.cuda.synchronize()
    assert torch.equal(again, got)


def test_static_scratch_limit_is_reported():
    S = 16384       # 8 query heads of 16384 tokens need far more than the built-in 4 MiB
    assert binding.efq_attention_workspace_bytes(1, 8, 8, S, S, 128) > binding.STATIC_SCRATCH_BYTES
    q = torch.zeros((1, 8, S, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.EfqError) as e:
        binding.efq_attention_fwd_static(q, q, q, True, o=torch.empty((1, 8, S, 128), dtype=torch.float32, device="cuda"))
    assert e.value.status == binding.STATUS_NAMES.index("EFQ_ERR_STATIC_LIMIT")
    assert "built-in scratch" in str(e.value)


def test_static_entry_applies_the_argument_rules_of_the_regular_forward():
    q = torch.zeros((1, 3, 128, 128), dtype=torch.bfloat16, device="cuda")
    k = torch.zeros((1, 2, 128, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.EfqError) as e:       # Hq % Hkv != 0 is an invalid argument here too
        binding.efq_attention_fwd_static(q, k, k, False, o=torch.empty((1, 3, 128, 128), dtype=torch.float32, device="cuda"))
    assert e.value.status == binding.STATUS_NAMES.index("EFQ_ERR_INVALID_ARG")
