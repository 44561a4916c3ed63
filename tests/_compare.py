"""Comparison rules between the CUDA path and the fp64 oracle.

Tolerances (absolute): 2e-3 for bf16 logits, 1e-5 for fp32 logits, on log-probabilities,
entropies, advantages and the mean entropy.  The outputs are fp32, so one rounding of the
output itself (2^-24 relative) is allowed on top: a log-probability of -300 cannot be stored
in fp32 to better than 1.5e-5.
Tokens must be bit-exact, except rows whose two best perturbed scores in the oracle differ by
less than 1e-6 (sampler 1 also: in-block threshold within 1e-6 of a prefix boundary); such rows
are counted and reported, not failed.
"""
import numpy as np
import torch

ATOL = {torch.float32: 1e-5, torch.bfloat16: 2e-3}


def assert_close(name, got, ref, atol):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (name, got.shape, ref.shape)
    both_nan = np.isnan(got) & np.isnan(ref)
    both_same_inf = np.isinf(ref) & (got == ref)
    ok = both_nan | both_same_inf
    fin = ~ok
    err = np.abs(got[fin] - ref[fin])
    bound = atol + np.abs(ref[fin]) * 2.0**-23
    bad = ~(err <= bound)
    if bad.any():
        i = np.flatnonzero(fin)[np.flatnonzero(bad)[0]]
        raise AssertionError(f"{name}: {bad.sum()} of {got.size} outside tolerance {atol}; first at {i}: "
                             f"got {got[i]!r} ref {ref[i]!r}; max err {np.nanmax(err)}")
    return float(err.max()) if err.size else 0.0


def assert_tokens(name, got_tok, oracle_res, sampler=0):
    got_tok = np.asarray(got_tok)
    ref = oracle_res.tok
    diff = np.flatnonzero(got_tok != ref)
    near = (oracle_res.y1 - oracle_res.y2) < 1e-6
    if sampler == 1:
        near = near | (oracle_res.cdf_margin < 1e-6)
    real = [int(i) for i in diff if not near[i]]
    assert not real, f"{name}: token mismatch on rows {real[:8]} (got {got_tok[real[:8]]}, ref {ref[real[:8]]})"
    return {"mismatch_near_tie": int(len(diff)), "near_tie_rows": int(near.sum())}
