"""szo_select_mask_static: the variant of the mask selection for callers that cannot allocate device
memory (they pass inputs and outputs only; the scratch is a fixed array inside the library).

Collected last on purpose (file name), so a run that stops at the first failure has already run
everything else.  The check is against the existing entry point, szo_select_mask, on two calls in a
row with different sizes and k, so that whatever the first call leaves in the shared scratch must not
leak into the second.  Index results are integers: the comparison is exact, as in the other mask
tests."""
import numpy as np
import pytest
import torch

from paper_2406_02913_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2406_02913_b200 import binding
    binding.lib()
    return binding


def test_static_scratch_matches_workspace_variant_twice_in_a_row(B):
    cases = [(3_000_017, 2999, 21), (70_001, 35_000, 22)]      # big then small: stale counts would show
    for n, k, seed in cases:
        g = wl.student_t_gradient(n, 3.0, seed=seed)
        scores = torch.from_numpy(np.round(g * g, 2).astype(np.float32)).cuda()     # rounding makes ties
        out = torch.full((k + 8,), -1, dtype=torch.int64, device="cuda")           # caller-owned output
        got = B.szo_select_mask_static(scores, k, out)
        ref = B.szo_select_mask(scores, k)
        assert torch.equal(got, ref)
        assert (out[k:] == -1).all()                                                # nothing past k written
    # the same call again gives the same answer (the array is shared and reused)
    got2 = B.szo_select_mask_static(scores, k, torch.empty(k, dtype=torch.int64, device="cuda"))
    assert torch.equal(got2, ref)


def test_static_scratch_limits_and_errors(B):
    out = torch.empty(16, dtype=torch.int64, device="cuda")
    small = torch.ones(16, device="cuda")
    assert torch.equal(B.szo_select_mask_static(small, 4, out), torch.arange(4, device="cuda"))
    assert B.szo_select_mask_static(small, 0, out).numel() == 0
    # beyond the built-in maximum: rejected on the host before anything is launched or read
    rc = B.lib().szo_select_mask_static(small.data_ptr(), (1 << 26) + 1, 4, out.data_ptr(), None)
    assert rc == -5 and b"exceeds the built-in scratch" in B.lib().szo_last_error()
    bad = small.clone()
    bad[3] = float("nan")
    with pytest.raises(B.SzoError) as ei:
        B.szo_select_mask_static(bad, 2, out)
    assert ei.value.name == "SZO_ERR_NONFINITE"
