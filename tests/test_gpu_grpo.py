"""GRPO objective (Sec. 3.1, no KL term) on the device against the fp64 oracle: value, clipped fraction and the
per-token gradient.  Both sides compute in fp64 from the same fp32 inputs, so the tolerance is 1e-12 on J
(summation order) and one fp32 rounding on the stored gradient; the clip decision must agree token by token."""
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


def _case(seed, sizes, seq_len, min_len=0, with_mask=True):
    rng = np.random.default_rng(seed)
    off = inputs.group_offsets(sizes)
    n_seq = int(off[-1])
    lengths = rng.integers(min_len, seq_len + 1, size=n_seq)
    mask = (np.arange(seq_len)[None, :] < lengths[:, None]).astype(np.uint8)
    logp_old = (-rng.random((n_seq, seq_len)) * 4).astype(np.float32)
    logp = (logp_old + rng.normal(size=(n_seq, seq_len)) * 0.25).astype(np.float32)
    rewards = (rng.random(n_seq) < 0.5).astype(np.float32)
    adv, _ = oracle.group_advantage(rewards, off.numpy())
    return logp, logp_old, (mask if with_mask else None), adv.astype(np.float32), off.numpy()


@pytest.mark.parametrize("sizes,seq_len,min_len,with_mask", [
    ([8] * 8, 64, 0, True), ([2, 32, 1, 5, 17, 8, 3], 300, 0, True), ([4] * 3, 1, 0, True), ([6, 2], 1000, 500, False),
    ([int(x) for x in np.random.default_rng(7).integers(2, 33, size=64)], 2048, 256, True)])
def test_grpo_objective_matches_the_oracle(e3, sizes, seq_len, min_len, with_mask):
    logp, logp_old, mask, adv, off = _case(len(sizes) + seq_len, sizes, seq_len, min_len, with_mask)
    n_seq = logp.shape[0]
    t = lambda a: None if a is None else torch.from_numpy(a).to(DEV)
    pad = 16
    gbuf = torch.full((n_seq * seq_len + 2 * pad,), 9.0, dtype=torch.float32, device=DEV)
    g_view = gbuf[pad:pad + n_seq * seq_len].view(n_seq, seq_len)
    m = None if mask is None else t(mask).reshape(-1)
    for _ in range(2):                                     # twice: scratch contents from the first call must not matter
        out, g = e3.e3_grpo_objective(t(logp), t(logp_old), t(adv), t(off), mask=m, clip_eps=0.2, out_g_logp=g_view)
    torch.cuda.synchronize()
    assert torch.all(gbuf[:pad] == 9.0) and torch.all(gbuf[-pad:] == 9.0)
    J, grad, frac = oracle.grpo_objective(logp, logp_old, mask, adv, off, 0.2)
    assert float(out[0]) == pytest.approx(J, abs=1e-12)
    assert float(out[1]) == pytest.approx(frac, abs=1e-12)
    got = g.cpu().numpy().astype(np.float64)
    assert np.array_equal(got == 0, grad == 0)             # same clip decisions, same masked tokens
    assert np.all(np.abs(got - grad) <= np.abs(grad) * 2.0 ** -23 + 1e-30)
    if frac > 0:
        assert 0 < frac < 0.6


def test_grpo_objective_edge_cases(e3):
    z = lambda *s: torch.zeros(*s, device=DEV)
    off0 = torch.zeros(1, dtype=torch.int64, device=DEV)
    out, g = e3.e3_grpo_objective(z(0, 5), z(0, 5), z(0), off0)
    torch.cuda.synchronize()
    assert float(out[0]) == 0.0 and float(out[1]) == 0.0 and g.numel() == 0
    # at the old policy the objective is the mean advantage of the responses that have tokens, gradient = weight * A
    logp, logp_old, mask, adv, off = _case(3, [3, 5], 20)
    t = lambda a: torch.from_numpy(a).to(DEV)
    out, g = e3.e3_grpo_objective(t(logp_old), t(logp_old), t(adv), t(off), mask=t(mask).reshape(-1))
    J, grad, frac = oracle.grpo_objective(logp_old, logp_old, mask, adv, off, 0.2)
    torch.cuda.synchronize()
    assert float(out[0]) == pytest.approx(J, abs=1e-12) and float(out[1]) == 0.0
    L = e3.lib()
    assert L.e3_grpo_objective(1024, 1024, None, 4, 4, 1024, 1024, 1, 0.2, None, 1024, None, None, 0, None) == 4   # workspace
    assert L.e3_grpo_objective(1024, 1024, None, -1, 4, 1024, 1024, 1, 0.2, None, 1024, None, 1024, 1 << 20, None) == 1
    assert L.e3_grpo_objective(1024, 1024, None, 4, 4, 1024, 1024, 1, -0.1, None, 1024, None, 1024, 1 << 20, None) == 1


def test_training_step_chain_objective_feeds_the_backward(e3):
    """Forward (log-probabilities) -> objective gradient -> backward of the vocabulary pass, against the oracle chain."""
    n_groups, G, seq_len, V = 3, 4, 6, 3000
    n_seq = n_groups * G
    rows = n_seq * seq_len
    logits = inputs.zipf_gaussian_logits(rows, V, seed=5, dtype=torch.float32, device=DEV)
    targets = inputs.uniform_targets(rows, V, seed=6, device=DEV)
    mask, _ = inputs.response_mask(n_seq, seq_len, seed=7, min_len=1, device=DEV)
    lp, en = e3.e3_token_logp_entropy(logits, targets, mask=mask, temp_scalar=1.0)
    g = torch.Generator(device=DEV); g.manual_seed(1)
    lp_old = lp + 0.2 * torch.randn(rows, generator=g, device=DEV) * mask
    rewards = inputs.bernoulli_rewards([G] * n_groups, 0.5, seed=8, device=DEV)
    off = inputs.group_offsets([G] * n_groups, device=DEV)
    adv, _ = e3.e3_group_advantage(rewards, off)
    out, g_lp = e3.e3_grpo_objective(lp.view(n_seq, seq_len), lp_old.view(n_seq, seq_len).contiguous(), adv, off, mask=mask)
    dz = e3.e3_token_logp_entropy_backward(logits, targets, lp, en, g_lp.reshape(-1), None, mask=mask)
    torch.cuda.synchronize()
    # oracle chain on the host, from the same logits and old log-probabilities
    olp, oen, _ = oracle.token_logp_entropy(logits.cpu().numpy(), targets.cpu().numpy(), mask=mask.cpu().numpy())
    oadv, _ = oracle.group_advantage(rewards.cpu().numpy(), off.cpu().numpy())
    J, ograd, _ = oracle.grpo_objective(olp.astype(np.float32).reshape(n_seq, seq_len), lp_old.cpu().numpy().reshape(n_seq, seq_len),
                                        mask.cpu().numpy().reshape(n_seq, seq_len), oadv.astype(np.float32), off.cpu().numpy(), 0.2)
    odz = oracle.token_logp_entropy_backward(logits.cpu().numpy(), targets.cpu().numpy(), ograd.reshape(-1).astype(np.float32),
                                             None, mask=mask.cpu().numpy())
    assert float(out[0]) == pytest.approx(J, abs=1e-5)
    assert np.abs(dz.cpu().numpy() - odz).max() < 1e-5
