"""Backward of the training-side pass (gradient of log-probability and entropy with respect to the logits):
the CUDA kernel, fed with the CUDA forward's own outputs, against the fp64 oracle entry by entry.

Tolerance.  fp32 logits: 2e-5 * beta * (|g_logp| + |g_ent| (1 + H)) absolute (the forward outputs the kernel
starts from are good to 1e-5, `ex2.approx` to 2^-22).  bf16: the same with 2e-3, plus half a bf16 ulp of the
value (the gradient is stored in the element type of the logits)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_18573_b200 import inputs

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(scope="module")
def e3():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2505_18573_b200 import binding
    binding.lib()
    return binding


def _check(e3, logits, targets, g_lp, g_en, mask=None, temps=None, temp_scalar=1.0):
    rows, V = logits.shape
    lp, en = e3.e3_token_logp_entropy(logits, targets, mask=mask, temps=temps, temp_scalar=temp_scalar)
    pad = 3
    buf = torch.full((rows + 2 * pad, logits.stride(0)), 7.0, dtype=logits.dtype, device=DEV)   # canary rows
    out = buf[pad:pad + rows, :V]
    e3.e3_token_logp_entropy_backward(logits, targets, lp, en, g_lp, g_en, mask=mask, temps=temps,
                                      temp_scalar=temp_scalar, out=out)
    torch.cuda.synchronize()
    assert torch.all(buf[:pad] == 7.0) and torch.all(buf[pad + rows:] == 7.0) and torch.all(buf[pad:pad + rows, V:] == 7.0)
    ref = oracle.token_logp_entropy_backward(inputs.to_oracle_array(logits), targets.cpu().numpy(),
                                             None if g_lp is None else g_lp.cpu().numpy(),
                                             None if g_en is None else g_en.cpu().numpy(),
                                             mask=None if mask is None else mask.cpu().numpy(),
                                             temps=None if temps is None else temps.cpu().numpy(), temp_scalar=temp_scalar)
    got = out.float().cpu().numpy().astype(np.float64)
    tau = temps.cpu().numpy().astype(np.float64) if temps is not None else np.full(rows, float(np.float32(temp_scalar)))
    gl = np.zeros(rows) if g_lp is None else np.abs(g_lp.cpu().numpy().astype(np.float64))
    ge = np.zeros(rows) if g_en is None else np.abs(g_en.cpu().numpy().astype(np.float64))
    H = np.nan_to_num(en.cpu().numpy().astype(np.float64))
    base = 2e-5 if logits.dtype == torch.float32 else 2e-3
    bound = (base * (gl + ge * (1 + H)) / np.where(tau > 0, tau, 1.0))[:, None] + 1e-12
    if logits.dtype == torch.bfloat16:
        bound = bound + np.abs(np.nan_to_num(ref)) * 2.0 ** -8
    nan_ok = np.isnan(ref) & np.isnan(got)
    bad = ~nan_ok & ~(np.abs(got - ref) <= bound)
    assert not bad.any(), (int(bad.sum()), np.argwhere(bad)[:3], got[bad][:3], ref[bad][:3])
    if mask is not None:
        assert torch.all(out[mask == 0] == 0)
    return got


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("V", [1, 7, 8, 9, 1000, 8191, 8192, 8193, 33333, 151936])
def test_backward_matches_the_oracle(e3, dtype, V):
    rows = 5 if V > 50000 else 37
    g = torch.Generator(device=DEV); g.manual_seed(V)
    logits = inputs.zipf_gaussian_logits(rows, V, seed=V, dtype=dtype, device=DEV)
    targets = inputs.uniform_targets(rows, V, seed=1, device=DEV)
    temps = inputs.uniform_temps(rows, seed=2, device=DEV)
    g_lp = torch.randn(rows, generator=g, device=DEV)
    g_en = torch.randn(rows, generator=g, device=DEV)
    mask = (torch.arange(rows, device=DEV) % 4 != 1).to(torch.uint8)
    got = _check(e3, logits, targets, g_lp, g_en, mask=mask, temps=temps)
    live = mask.cpu().numpy() != 0
    tol = 1e-3 if dtype == torch.float32 else 0.5 * V ** 0.5 * 2.0 ** -8 + 1e-2
    assert np.abs(got[live].sum(axis=1)).max() < tol       # the gradient is orthogonal to the all-ones direction
    _check(e3, logits, targets, g_lp, None, temp_scalar=0.8)   # log-probability term alone, scalar temperature
    _check(e3, logits, targets, None, g_en, temp_scalar=1.7)   # entropy term alone


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_backward_layouts_and_unusable_rows(e3, dtype):
    rows, V = 6, 5000
    base = inputs.zipf_gaussian_logits(rows, V + 11, seed=3, dtype=dtype, device=DEV)
    targets = inputs.uniform_targets(rows, V, seed=4, device=DEV)
    g_lp = torch.ones(rows, device=DEV); g_en = torch.full((rows,), 0.5, device=DEV)
    _check(e3, base[:, :V], targets, g_lp, g_en)            # odd stride: rows not 16-byte aligned
    _check(e3, base[:, 1:V + 1], targets, g_lp, g_en)       # base pointer off by one element
    z = base[:, :V].clone()
    z[0, ::3] = -float("inf")                               # entries without mass
    t2 = targets.clone(); t2[0] = 1; t2[2] = V              # row 2: target out of range
    temps = torch.tensor([1.0, 0.0, 1.0, float("nan"), 0.5, 2.0], device=DEV)   # rows 1 and 3: unusable temperature
    got = _check(e3, z.contiguous(), t2, g_lp, g_en, temps=temps)
    assert np.isnan(got[1]).all() and np.isnan(got[2]).all() and np.isnan(got[3]).all()
    assert np.all(got[0, ::3] == 0) and np.isfinite(got[[0, 4, 5]]).all()
    out = e3.e3_token_logp_entropy_backward(torch.zeros((0, 8), dtype=dtype, device=DEV), torch.zeros(0, dtype=torch.int32, device=DEV),
                                            torch.zeros(0, device=DEV), torch.zeros(0, device=DEV))
    assert out.numel() == 0


def test_backward_training_chunk_at_full_width(e3):
    """One 2,048-row chunk of the training pass (151,936 bf16, response mask, scalar temperature): sampled rows."""
    rows = 2048
    logits = inputs.zipf_gaussian_logits(rows, 151936, seed=100, dtype=torch.bfloat16, device=DEV)
    targets = inputs.uniform_targets(rows, 151936, seed=4, device=DEV)
    mask, _ = inputs.response_mask(1, rows, seed=5, min_len=1500, device=DEV)
    g = torch.Generator(device=DEV); g.manual_seed(9)
    g_lp = torch.randn(rows, generator=g, device=DEV); g_en = 1e-2 * torch.randn(rows, generator=g, device=DEV)
    lp, en = e3.e3_token_logp_entropy(logits, targets, mask=mask)
    out = e3.e3_token_logp_entropy_backward(logits, targets, lp, en, g_lp, g_en, mask=mask)
    torch.cuda.synchronize()
    pick = np.array([0, 1, 777, 1499, int(mask.sum().item()) - 1, rows - 1])
    sub = torch.as_tensor(pick, device=DEV)
    ref = oracle.token_logp_entropy_backward(inputs.to_oracle_array(logits[sub]), targets.cpu().numpy()[pick],
                                             g_lp.cpu().numpy()[pick], g_en.cpu().numpy()[pick],
                                             mask=mask.cpu().numpy()[pick])
    got = out[sub].float().cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - ref) <= 2e-3 * (np.abs(g_lp.cpu().numpy()[pick]) + 1)[:, None] + np.abs(ref) * 2.0 ** -8)
    assert torch.all(out[mask == 0] == 0)
