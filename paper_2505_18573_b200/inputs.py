"""Seeded synthetic inputs shaped like the paper's rollout and training batches.

This module holds input generators only: none of the method's arithmetic (no
softmax, no entropy, no sampler, no advantage, no Philox).  The CUDA path and
the CPU oracle are both fed the bytes produced here, so the generator is not
part of either.  Everything is a pure function of its seed on a given device
(``torch.Generator``); values differ between CPU and CUDA generators, which is
fine because a test always hands the same tensor to both sides.

Logit rows follow the shape the paper cites for LLM logits (App. A: a Gaussian
"noisy region" plus a few informative outliers): a Gaussian body with a
Zipf-like bias over a per-row random ranking of the vocabulary.
"""
from __future__ import annotations

import math

import numpy as np
import torch


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def zipf_gaussian_logits(rows: int, V: int, seed: int, dtype=torch.float32, device="cpu",
                         chunk_rows: int = 1024) -> torch.Tensor:
    """z_i = 3 N(0,1) - 1.2 ln(1 + rank_i); rank = per-row random permutation of [0, V)."""
    g = _gen(seed, device)
    out = torch.empty((rows, V), dtype=dtype, device=device)
    for r0 in range(0, rows, chunk_rows):
        r1 = min(rows, r0 + chunk_rows)
        noise = torch.randn((r1 - r0, V), generator=g, device=device, dtype=torch.float32)
        keys = torch.rand((r1 - r0, V), generator=g, device=device, dtype=torch.float32)
        rank = torch.argsort(torch.argsort(keys, dim=1), dim=1).to(torch.float32)
        z = 3.0 * noise - 1.2 * torch.log1p(rank)
        out[r0:r1] = z.to(dtype)
    return out


def onehot_flat_logits(rows: int, V: int, seed: int, dtype=torch.float32, device="cpu",
                       chunk_rows: int = 512) -> torch.Tensor:
    """Even rows: N(0,1) with one random index raised to (row max + 25).  Odd rows: N(0, sigma=0.1)."""
    g = _gen(seed, device)
    out = torch.empty((rows, V), dtype=dtype, device=device)
    for r0 in range(0, rows, chunk_rows):
        r1 = min(rows, r0 + chunk_rows)
        n = r1 - r0
        z = torch.randn((n, V), generator=g, device=device, dtype=torch.float32)
        hot = torch.randint(0, V, (n,), generator=g, device=device)
        ridx = torch.arange(r0, r1, device=device)
        even = (ridx % 2) == 0
        z[~even] *= 0.1
        peak = z.max(dim=1).values + 25.0
        rows_even = torch.nonzero(even).flatten()
        z[rows_even, hot[rows_even]] = peak[rows_even]
        out[r0:r1] = z.to(dtype)
    return out


def uniform_temps(rows: int, seed: int, lo: float = 0.6, hi: float = 1.4, device="cpu") -> torch.Tensor:
    g = _gen(seed, device)
    return (lo + (hi - lo) * torch.rand(rows, generator=g, device=device, dtype=torch.float32)).contiguous()


def loguniform_temps(rows: int, seed: int, lo: float = 0.1, hi: float = 2.0, device="cpu") -> torch.Tensor:
    g = _gen(seed, device)
    u = torch.rand(rows, generator=g, device=device, dtype=torch.float32)
    return torch.exp(math.log(lo) + (math.log(hi) - math.log(lo)) * u).contiguous()


def uniform_targets(rows: int, V: int, seed: int, device="cpu") -> torch.Tensor:
    g = _gen(seed, device)
    return torch.randint(0, V, (rows,), generator=g, device=device, dtype=torch.int32)


def response_mask(n_seq: int, seq_len: int, seed: int, min_len: int = 256, device="cpu"):
    """Per-sequence response length uniform in [min_len, seq_len]; mask = first L_s tokens.

    Returns (mask uint8 [n_seq * seq_len], lengths int64 [n_seq])."""
    g = _gen(seed, device)
    lengths = torch.randint(min_len, seq_len + 1, (n_seq,), generator=g, device=device)
    pos = torch.arange(seq_len, device=device).unsqueeze(0)
    mask = (pos < lengths.unsqueeze(1)).to(torch.uint8).reshape(-1).contiguous()
    return mask, lengths


def bernoulli_rewards(group_sizes, p, seed: int, device="cpu") -> torch.Tensor:
    """One 0/1 reward per rollout; ``p`` is a scalar or one success probability per group."""
    g = _gen(seed, device)
    sizes = torch.as_tensor(group_sizes, dtype=torch.int64)
    n = int(sizes.sum())
    probs = torch.as_tensor(p, dtype=torch.float32)
    if probs.ndim == 0:
        probs = probs.expand(sizes.numel())
    per_row = torch.repeat_interleave(probs, sizes).to(device)
    return (torch.rand(n, generator=g, device=device) < per_row).to(torch.float32).contiguous()


def group_offsets(group_sizes, device="cpu") -> torch.Tensor:
    sizes = torch.as_tensor(group_sizes, dtype=torch.int64)
    off = torch.zeros(sizes.numel() + 1, dtype=torch.int64)
    off[1:] = torch.cumsum(sizes, 0)
    return off.to(device)


def beta22_difficulty(n: int, seed: int) -> np.ndarray:
    """Per-prompt difficulty in (0,1) ~ Beta(2,2), host side (feeds the host budget call)."""
    rng = np.random.default_rng(seed)
    return rng.beta(2.0, 2.0, size=n).astype(np.float64)


def force_extreme_groups(rewards: torch.Tensor, offsets: torch.Tensor, n_each: int = 4) -> torch.Tensor:
    """Overwrite the first ``n_each`` groups with all-0 rewards and the next ``n_each`` with all-1."""
    r = rewards.clone()
    off = offsets.tolist()
    ng = len(off) - 1
    for gi in range(min(n_each, ng)):
        r[off[gi]:off[gi + 1]] = 0.0
    for gi in range(n_each, min(2 * n_each, ng)):
        r[off[gi]:off[gi + 1]] = 1.0
    return r


def to_oracle_array(t: torch.Tensor) -> np.ndarray:
    """Host numpy view of a tensor; bf16 becomes uint16 bit patterns (what the oracle reads)."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()
