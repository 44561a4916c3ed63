"""The benchmark configurations at full size, in the launch shape bench.py times: the CUDA path against
the fp64 oracle on every row where the oracle finishes in seconds, on sampled rows otherwise."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_18573_b200 import inputs
from _compare import ATOL, assert_close, assert_tokens

pytestmark = pytest.mark.gpu
DEV = "cuda"
V_LM = 151936


@pytest.fixture(scope="module")
def e3():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2505_18573_b200 import binding
    binding.lib()
    return binding


def _sample_parity(e3, logits, temps, seed, counter, row_base, sampler, name, rows_idx=None):
    tok, lp, en = e3.e3_sample(logits, temps, seed, counter, row_base, sampler)
    torch.cuda.synchronize()
    tok, lp, en = tok.cpu().numpy(), lp.cpu().numpy(), en.cpu().numpy()
    if rows_idx is None:
        rows_idx = np.arange(logits.shape[0])
    sub = inputs.to_oracle_array(logits[torch.as_tensor(rows_idx, device=logits.device)])
    t_sub = temps.cpu().numpy()[rows_idx]
    # the oracle addresses the random streams by global row: one call per run of consecutive rows
    ref_tok = np.empty(len(rows_idx), np.int32); ref_lp = np.empty(len(rows_idx)); ref_en = np.empty(len(rows_idx))
    y1 = np.empty(len(rows_idx)); y2 = np.empty(len(rows_idx)); cm = np.empty(len(rows_idx))
    start = 0
    while start < len(rows_idx):
        stop = start + 1
        while stop < len(rows_idx) and rows_idx[stop] == rows_idx[stop - 1] + 1:
            stop += 1
        r = oracle.sample(sub[start:stop], t_sub[start:stop], seed, counter, row_base + int(rows_idx[start]), sampler)
        ref_tok[start:stop] = r.tok; ref_lp[start:stop] = r.logp; ref_en[start:stop] = r.ent
        y1[start:stop] = r.y1; y2[start:stop] = r.y2; cm[start:stop] = r.cdf_margin
        start = stop

    class R:
        pass
    ref = R(); ref.tok = ref_tok; ref.y1 = y1; ref.y2 = y2; ref.cdf_margin = cm
    info = assert_tokens(name, tok[rows_idx], ref, sampler)
    same = tok[rows_idx] == ref_tok
    atol = ATOL[logits.dtype]
    info["max_err_ent"] = assert_close(name + ".ent", en[rows_idx], ref_en, atol)
    info["max_err_logp"] = assert_close(name + ".logp", lp[rows_idx][same], ref_lp[same], atol)
    info["rows_checked"] = int(len(rows_idx))
    _report(name, info)
    return info


def _report(name, info):
    """Parity counts of every configuration: printed (pytest -rP shows them) and, when E3_REPORT_DIR names a
    directory, appended as one JSON line per case to parity_counts.jsonl there."""
    import json, os
    line = json.dumps({"case": name, **info})
    print("parity:", line)
    out_dir = os.environ.get("E3_REPORT_DIR")
    if out_dir:
        os.makedirs(out_dir, exist_ok=True)
        with open(os.path.join(out_dir, "parity_counts.jsonl"), "a") as f:
            f.write(line + "\n")


@pytest.mark.parametrize("sampler", [0, 1])
def test_config2_rollout_decode_steps(e3, sampler):
    """512 rows (64 prompts x 8 rollouts) x 151,936 bf16, advancing step counter; all rows at steps 0, 1, 255."""
    rows = 512
    temps = inputs.uniform_temps(rows, seed=2, device=DEV)
    for step in (0, 1, 2, 127, 255):
        logits = inputs.zipf_gaussian_logits(rows, V_LM, seed=10 + step % 8, dtype=torch.bfloat16, device=DEV)
        _sample_parity(e3, logits, temps, 0, step, 0, sampler, f"c2.step{step}")


def test_config3_training_pass_full_size(e3):
    """64 sequences x 2,048 tokens x 151,936 bf16 (39.8 GB) in one call, response mask with lengths in
    [256, 2048], uniform targets; the first and last response token of every sequence and 128 more response
    tokens of every sequence (8,192 rows stratified by sequence, plus the 128 end points) against the oracle,
    masked rows exactly zero, mean entropy against the oracle's reduction."""
    n_seq, seq_len = 64, 2048
    rows = n_seq * seq_len
    free, _ = torch.cuda.mem_get_info()
    if free < 60 * 2**30:
        pytest.skip("needs 60 GB of free device memory")
    logits = torch.empty((rows, V_LM), dtype=torch.bfloat16, device=DEV)
    for c in range(rows // 8192):          # generated on the device chunk by chunk from a seed
        logits[c * 8192:(c + 1) * 8192] = inputs.zipf_gaussian_logits(8192, V_LM, seed=100 + c, dtype=torch.bfloat16,
                                                                       device=DEV)
    targets = inputs.uniform_targets(rows, V_LM, seed=4, device=DEV)
    mask, lengths = inputs.response_mask(n_seq, seq_len, seed=5, min_len=256, device=DEV)
    lp, en = e3.e3_token_logp_entropy(logits, targets, mask=mask, temp_scalar=1.0)
    out = e3.e3_masked_mean_entropy(en, mask)
    torch.cuda.synchronize()
    m = mask.cpu().numpy()
    assert torch.all(lp[mask == 0] == 0) and torch.all(en[mask == 0] == 0)
    L = lengths.cpu().numpy()
    pick = [s * seq_len for s in range(n_seq)] + [s * seq_len + int(L[s]) - 1 for s in range(n_seq)]
    rng = np.random.default_rng(6)
    for s_ in range(n_seq):                # 128 response tokens of every sequence
        pick += list(s_ * seq_len + rng.choice(int(L[s_]), size=128, replace=False))
    pick = np.unique(np.asarray(pick))
    assert len(pick) >= 8192
    tg = targets.cpu().numpy()
    e_lp = e_en = 0.0
    for c0 in range(0, len(pick), 2048):   # the oracle works through the sample in chunks of 2,048 rows
        pc = pick[c0:c0 + 2048]
        sub = inputs.to_oracle_array(logits[torch.as_tensor(pc, device=DEV)])
        rlp, ren, _ = oracle.token_logp_entropy(sub, tg[pc], temp_scalar=1.0)
        e_lp = max(e_lp, assert_close("c3.logp", lp.cpu().numpy()[pc], rlp, ATOL[torch.bfloat16]))
        e_en = max(e_en, assert_close("c3.ent", en.cpu().numpy()[pc], ren, ATOL[torch.bfloat16]))
    _report("c3", {"rows_checked": int(len(pick)), "max_err_logp": e_lp, "max_err_ent": e_en,
                   "unmasked_rows": int(L.sum()), "rows": rows})
    rmean, rcnt = oracle.masked_mean_entropy(en.cpu().numpy(), m)
    assert float(out[1]) == rcnt == float(L.sum())
    assert float(out[0]) == pytest.approx(rmean, rel=1e-12)
    s = e3.make_sched(tau=1.0, H_init=1.1 * float(out[0]), V=V_LM)
    so = oracle.make_sched(tau=1.0, H_init=1.1 * rmean, V=V_LM)
    assert e3.e3_update_temperature(s, float(out[0])) == pytest.approx(oracle.update_temperature(so, rmean), rel=1e-12)
    del logits


@pytest.mark.parametrize("sampler", [0, 1])
def test_config4_variable_budget_rollout(e3, sampler):
    """256 prompts, budgets from Algorithm 1 (difficulty ~ Beta(2,2), 2..32 rollouts, 4,096 rows in all) x
    151,936 bf16; fused sample step on every row, then the advantage over the ragged groups."""
    k = inputs.beta22_difficulty(256, seed=6)
    budgets = e3.e3_allocate_budget(k, 16, 2, 32)
    assert budgets == list(oracle.allocate_budget(k, 16, 2, 32)) and sum(budgets) == 4096
    rows = 4096
    logits = inputs.zipf_gaussian_logits(rows, V_LM, seed=40, dtype=torch.bfloat16, device=DEV)
    temps = inputs.uniform_temps(rows, seed=41, device=DEV)
    _sample_parity(e3, logits, temps, 3, 17, 0, sampler, "c4")
    rewards = inputs.bernoulli_rewards(budgets, 1.0 - k, seed=7, device=DEV)
    off = inputs.group_offsets(budgets, device=DEV)
    rewards = inputs.force_extreme_groups(rewards, off.cpu(), n_each=4)
    adv, flags = e3.e3_group_advantage(rewards, off)
    radv, rflags = oracle.group_advantage(rewards.cpu().numpy(), off.cpu().numpy())
    assert_close("c4.adv", adv.cpu().numpy(), radv, 1e-5)
    assert np.array_equal(flags.cpu().numpy(), rflags)
    assert (rflags[:4] == 3).all() and (rflags[4:8] == 1).all()
    a, o = adv.cpu().numpy(), off.cpu().numpy()
    for g in range(256):
        assert abs(a[o[g]:o[g + 1]].sum()) < 1e-4 * budgets[g]
        if rflags[g] & 1:
            assert np.all(a[o[g]:o[g + 1]] == 0.0)


def test_config5_large_batch_stress(e3):
    """4,096 rows x 256,000 fp32 (4.2 GB), half near-one-hot, half flat, temperatures log-uniform in
    [0.1, 2]: one launch over all rows, every row against the oracle (both samplers and the training pass)."""
    rows, V = 4096, 256000
    logits = inputs.onehot_flat_logits(rows, V, seed=20, device=DEV)
    temps = inputs.loguniform_temps(rows, seed=21, device=DEV)
    for sampler in (0, 1):
        _sample_parity(e3, logits, temps, 4, 1, 0, sampler, f"c5.s{sampler}")
    targets = inputs.uniform_targets(rows, V, seed=22, device=DEV)
    lp, en = e3.e3_token_logp_entropy(logits, targets, temps=temps)
    e_lp = e_en = 0.0
    for c0 in range(0, rows, 1024):
        sub = logits[c0:c0 + 1024].cpu().numpy()
        rlp, ren, _ = oracle.token_logp_entropy(sub, targets.cpu().numpy()[c0:c0 + 1024], temps=temps.cpu().numpy()[c0:c0 + 1024])
        e_lp = max(e_lp, assert_close("c5.logp", lp.cpu().numpy()[c0:c0 + 1024], rlp, 1e-5))
        e_en = max(e_en, assert_close("c5.ent", en.cpu().numpy()[c0:c0 + 1024], ren, 1e-5))
    _report("c5.train", {"rows_checked": rows, "max_err_logp": e_lp, "max_err_ent": e_en})
    e = en.cpu().numpy()
    assert np.all(e[1::2] > 11.8) and np.all(e[0::2] < 11.8)   # flat rows near ln V = 12.45, peaked rows below
