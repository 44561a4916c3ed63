"""The scratch-free mean entropy entry point against the regular one.

e3_masked_mean_entropy_static serves callers that may not allocate device memory (code running
inside another engine's stream, processes with a fixed memory pool): its partial sums sit in an
array built into the library instead of a caller workspace.  This file is collected last on
purpose, so that a run that stops at the first failure has already been through every other
test; it must also pass when run on its own in a fresh process.
"""
import math

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def e3():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2505_18573_b200 import binding
    binding.lib()
    return binding


def test_static_scratch_mean_matches_workspace_mean_twice_in_a_row(e3):
    dev = "cuda"
    rng = np.random.default_rng(2024)
    # two calls back to back: the second is smaller, so partials left by the first are still in
    # the shared array and must not reach the result
    for n, with_mask in ((1_000_003, True), (5_000, True), (131_072, False), (1, True), (0, False)):
        ent = torch.from_numpy(rng.random(n).astype(np.float32)).to(dev)
        mask = torch.from_numpy((rng.random(n) < 0.56).astype(np.uint8)).to(dev) if with_mask else None
        out = torch.full((2,), -1.0, dtype=torch.float64, device=dev)     # caller-owned output, no allocation inside
        got = e3.e3_masked_mean_entropy_static(ent, mask, out=out)
        ref = e3.e3_masked_mean_entropy(ent, mask)
        torch.cuda.synchronize()
        assert float(got[1]) == float(ref[1])
        if float(ref[1]) == 0:
            assert math.isnan(float(got[0])) and math.isnan(float(ref[0]))
        else:
            assert float(got[0]) == pytest.approx(float(ref[0]), rel=1e-12)
            sel = ent.cpu().numpy().astype(np.float64)
            if mask is not None:
                sel = sel[mask.cpu().numpy() != 0]
            assert float(got[0]) == pytest.approx(math.fsum(sel) / sel.size, rel=1e-12)


def test_static_scratch_mean_rejects_oversize_and_bad_arguments(e3):
    L = e3.lib()
    assert L.e3_masked_mean_entropy_static(1024, None, e3.E3_STATIC_MEAN_MAX_TOKENS + 1, 1024, 1032, None) == 4
    assert L.e3_masked_mean_entropy_static(1024, None, -1, 1024, 1032, None) == 1
    assert L.e3_masked_mean_entropy_static(1024, None, 8, None, 1032, None) == 1
    assert L.e3_masked_mean_entropy_static(1026, None, 8, 1024, 1032, None) == 3
