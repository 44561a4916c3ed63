"""Parity of the CUDA path (called through the C ABI) with the fp64 CPU oracle, element by element,
on the same seeded inputs."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2505_18573_b200 import inputs
from _compare import ATOL, assert_close, assert_tokens

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def e3():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2505_18573_b200 import binding
    binding.lib()   # raises when the CUDA library has not been built: no fallback
    return binding


DEV = "cuda"


def _guarded(n, dtype, fill):
    """Output buffer with canary bands on both sides; returns (view, check)."""
    pad = 64
    buf = torch.full((n + 2 * pad,), fill, dtype=dtype, device=DEV)
    view = buf[pad:pad + n]

    def check():
        assert torch.all(buf[:pad] == fill) and torch.all(buf[pad + n:] == fill), "write outside the output"
    return view, check


def _run_sample(e3, logits, temps, seed, counter, row_base=0, sampler=0):
    rows = logits.shape[0]
    tok, c1 = _guarded(rows, torch.int32, -7)
    lp, c2 = _guarded(rows, torch.float32, 123.0)
    en, c3 = _guarded(rows, torch.float32, 123.0)
    e3.e3_sample(logits, temps, seed, counter, row_base, sampler, out_tok=tok, out_logp=lp, out_ent=en)
    torch.cuda.synchronize()
    c1(); c2(); c3()
    return tok.cpu().numpy(), lp.cpu().numpy(), en.cpu().numpy()


def _check_sample(e3, logits, temps, seed, counter, row_base=0, sampler=0, name="sample"):
    tok, lp, en = _run_sample(e3, logits, temps, seed, counter, row_base, sampler)
    ref = oracle.sample(inputs.to_oracle_array(logits), temps.cpu().numpy(), seed, counter, row_base, sampler)
    atol = ATOL[logits.dtype]
    info = assert_tokens(name, tok, ref, sampler)
    same = tok == ref.tok
    assert_close(name + ".ent", en, ref.ent, atol)
    assert_close(name + ".logp", lp[same], ref.logp[same], atol)
    return info


# ----------------------------------------------------------------------------------------------
# configuration 1: 64 rows (8 prompts x 8 rollouts) x 32,000 fp32, full parity incl. advantages
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("sampler", [0, 1])
def test_config1_tiny_sampling_step(e3, sampler):
    rows, V = 64, 32000
    logits = inputs.zipf_gaussian_logits(rows, V, seed=1, dtype=torch.float32, device=DEV)
    temps = inputs.uniform_temps(rows, seed=2, device=DEV)
    info = _check_sample(e3, logits, temps, seed=0, counter=0, sampler=sampler, name="c1")
    print("parity:", {"case": f"c1.s{sampler}", "rows_checked": rows, **info})
    assert info["mismatch_near_tie"] == 0
    sizes = [8] * 8
    rewards = inputs.bernoulli_rewards(sizes, 0.5, seed=3, device=DEV)
    off = inputs.group_offsets(sizes, device=DEV)
    adv, flags = e3.e3_group_advantage(rewards, off)
    radv, rflags = oracle.group_advantage(rewards.cpu().numpy(), off.cpu().numpy())
    assert_close("c1.adv", adv.cpu().numpy(), radv, 1e-5)
    assert np.array_equal(flags.cpu().numpy(), rflags)
    for g in range(8):
        assert abs(float(adv[8 * g:8 * g + 8].sum())) < 1e-4


@pytest.mark.parametrize("sampler", [0, 1])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_rollout_shape_rows_full_vocab(e3, dtype, sampler):
    """Rows at V = 151,936: rows cut between thread blocks (few rows) and whole rows per block (many rows)."""
    for rows, seed in ((3, 10), (41, 11), (150, 12), (700, 13)):
        logits = inputs.zipf_gaussian_logits(rows, 151936, seed=seed, dtype=dtype, device=DEV)
        temps = inputs.uniform_temps(rows, seed=seed + 50, device=DEV)
        _check_sample(e3, logits, temps, seed=5, counter=seed, sampler=sampler, name=f"rollout{rows}")


# ----------------------------------------------------------------------------------------------
# ragged sizes and layouts
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("V", [1, 2, 3, 7, 8, 9, 15, 16, 17, 127, 128, 129, 511, 512, 513, 1000, 4097, 33333])
def test_ragged_vocab_sizes(e3, dtype, V):
    for rows in (1, 2, 149):
        logits = inputs.zipf_gaussian_logits(rows, V, seed=V + rows, dtype=dtype, device=DEV)
        temps = inputs.uniform_temps(rows, seed=V, device=DEV)
        for sampler in (0, 1):
            _check_sample(e3, logits, temps, seed=V, counter=(1 << 33) + rows, row_base=7, sampler=sampler,
                          name=f"V{V}r{rows}s{sampler}")
        targets = inputs.uniform_targets(rows, V, seed=3, device=DEV)
        lp, en = e3.e3_token_logp_entropy(logits, targets, temps=temps)
        rlp, ren, _ = oracle.token_logp_entropy(inputs.to_oracle_array(logits), targets.cpu().numpy(),
                                                temps=temps.cpu().numpy())
        assert_close("logp", lp.cpu().numpy(), rlp, ATOL[dtype])
        assert_close("ent", en.cpu().numpy(), ren, ATOL[dtype])


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_padded_stride_and_unaligned_rows(e3, dtype):
    rows, V = 13, 5000
    base = inputs.zipf_gaussian_logits(rows, V + 24, seed=77, dtype=dtype, device=DEV)
    temps = inputs.uniform_temps(rows, seed=78, device=DEV)
    # stride > V, rows still 16-byte aligned
    view = base[:, :V]
    assert view.stride(0) == V + 24
    odd = inputs.zipf_gaussian_logits(rows, V + 3, seed=79, dtype=dtype, device=DEV)
    for sampler in (0, 1):
        _check_sample(e3, view, temps, seed=1, counter=2, sampler=sampler, name="padded")
        # stride that breaks 16-byte row alignment, and a base pointer offset by one element
        _check_sample(e3, odd[:, :V], temps, seed=1, counter=3, sampler=sampler, name="oddstride")
        _check_sample(e3, odd[:, 1:V + 1], temps, seed=1, counter=4, sampler=sampler, name="offset1")


def test_audit_sampler_settles_rows_in_fp64_and_agrees(e3):
    """E3_SAMPLER_TOKEN_AUDIT distrusts the fp32 scores of the fast path (slack x 1000), so rows whose two or
    three leaders lie within ~0.35 of each other are settled by the fp64 path (two contenders) or by the
    second look at the whole row (three or more): both must give the token of the definition."""
    for rows, V, dtype, seed in ((256, 4000, torch.float32, 90), (64, 151936, torch.bfloat16, 91),
                                 (40, 33333, torch.bfloat16, 92), (300, 129, torch.float32, 93)):
        logits = inputs.zipf_gaussian_logits(rows, V, seed=seed, dtype=dtype, device=DEV)
        temps = inputs.uniform_temps(rows, seed=seed + 1, device=DEV)
        ref = oracle.sample(inputs.to_oracle_array(logits), temps.cpu().numpy(), 7, seed, 0, 0)
        gap = ref.y1 - ref.y2
        assert (gap < 0.3).sum() >= 5, "the case must contain rows that take the exact path"
        tok, lp, en = _run_sample(e3, logits, temps, 7, seed, 0, e3.E3_SAMPLER_TOKEN_AUDIT)
        fast, lp0, en0 = _run_sample(e3, logits, temps, 7, seed, 0, e3.E3_SAMPLER_TOKEN)
        assert_tokens("audit", tok, ref, 0)
        assert np.array_equal(tok, fast)
        assert_close("audit.logp", lp, ref.logp, ATOL[dtype])
        assert_close("audit.ent", en, ref.ent, ATOL[dtype])
    # flat rows: many entries within the widened slack of the leader
    logits = inputs.onehot_flat_logits(16, 256000, seed=94, device=DEV)
    temps = inputs.loguniform_temps(16, seed=95, device=DEV)
    ref = oracle.sample(logits.cpu().numpy(), temps.cpu().numpy(), 1, 2, 0, 0)
    tok, lp, en = _run_sample(e3, logits, temps, 1, 2, 0, e3.E3_SAMPLER_TOKEN_AUDIT)
    assert_tokens("audit.flat", tok, ref, 0)


def test_empty_batch_is_a_noop(e3):
    logits = torch.zeros((0, 100), dtype=torch.float32, device=DEV)
    tok, lp, en = e3.e3_sample(logits, torch.zeros(0, device=DEV), 0, 0)
    assert tok.numel() == 0
    lp, en = e3.e3_token_logp_entropy(logits, torch.zeros(0, dtype=torch.int32, device=DEV))
    assert lp.numel() == 0
    adv, flags = e3.e3_group_advantage(torch.zeros(0, device=DEV), torch.zeros(1, dtype=torch.int64, device=DEV))
    assert adv.numel() == 0
    out = e3.e3_masked_mean_entropy(torch.zeros(0, device=DEV))
    torch.cuda.synchronize()
    assert math.isnan(float(out[0])) and float(out[1]) == 0.0


# ----------------------------------------------------------------------------------------------
# rows with a closed form, degenerate and invalid rows
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_special_rows(e3, dtype):
    V = 151936
    z = torch.zeros((8, V), dtype=torch.float32)
    z[0] = 0.375                                        # uniform: H = ln V
    z[1, 1234] = 12.0                                   # two-level rows
    z[2, 99999] = 25.0
    z[3] = torch.linspace(-4, 4, V); z[3, ::3] = -float("inf")   # -inf entries carry no mass
    z[4, 5] = float("nan")                              # invalid
    z[5, 6] = float("inf")                              # invalid
    z[6] = -float("inf")                                # invalid (no mass at all)
    z[7] = torch.linspace(-2, 2, V)                     # sampled at tau = 0: greedy
    logits = z.to(dtype).to(DEV)
    temps = torch.tensor([0.9, 1.0, 1.0, 0.7, 1.0, 1.0, 1.0, 0.0], dtype=torch.float32, device=DEV)
    tok1, lp1, en1 = _run_sample(e3, logits, temps, seed=3, counter=9, sampler=1)
    ref1 = oracle.sample(inputs.to_oracle_array(logits), temps.cpu().numpy(), 3, 9, sampler=1)
    assert np.array_equal(tok1, ref1.tok)
    assert_close("ent.s1", en1, ref1.ent, ATOL[dtype])
    assert_close("logp.s1", lp1, ref1.logp, ATOL[dtype])
    tok, lp, en = _run_sample(e3, logits, temps, seed=3, counter=9)
    ref = oracle.sample(inputs.to_oracle_array(logits), temps.cpu().numpy(), 3, 9)
    assert np.array_equal(tok, ref.tok)
    assert_close("ent", en, ref.ent, ATOL[dtype])
    assert_close("logp", lp, ref.logp, ATOL[dtype])
    assert en[0] == pytest.approx(math.log(V), abs=ATOL[dtype])
    assert tok[4] == -1 and tok[5] == -1 and tok[6] == -1 and np.isnan(lp[4:7]).all() and np.isnan(en[4:7]).all()
    assert lp[7] == 0 and en[7] == 0 and (dtype != torch.float32 or tok[7] == V - 1)
    assert tok[3] % 3 != 0
    # negative / NaN temperature marks the row only
    temps2 = torch.tensor([-1.0, float("nan"), 1.0, float("inf"), 1.0, 1.0, 1.0, 1.0], dtype=torch.float32, device=DEV)
    tok2, lp2, en2 = _run_sample(e3, logits, temps2, seed=3, counter=9)
    assert tok2[0] == -1 and tok2[1] == -1 and tok2[3] == -1 and tok2[2] >= 0
    ref2 = oracle.sample(inputs.to_oracle_array(logits), temps2.cpu().numpy(), 3, 9)
    assert np.array_equal(tok2, ref2.tok)
    # training side on the same rows
    targets = torch.tensor([7, 1234, 5, 1, 0, 0, 0, 3], dtype=torch.int32, device=DEV)
    t1 = torch.tensor([0.9, 1.0, 1.0, 0.7, 1.0, 1.0, 1.0, 1.3], dtype=torch.float32, device=DEV)
    lp3, en3 = e3.e3_token_logp_entropy(logits, targets, temps=t1)
    rlp, ren, _ = oracle.token_logp_entropy(inputs.to_oracle_array(logits), targets.cpu().numpy(), temps=t1.cpu().numpy())
    assert_close("logp3", lp3.cpu().numpy(), rlp, ATOL[dtype])
    assert_close("ent3", en3.cpu().numpy(), ren, ATOL[dtype])


def test_dominant_logit_and_tiny_temperature(e3):
    V = 40000
    logits = inputs.zipf_gaussian_logits(32, V, seed=5, device=DEV)
    arg = logits.argmax(dim=1).cpu().numpy()
    temps = torch.full((32,), 1e-3, device=DEV)
    for counter in range(4):
        tok, lp, en = _run_sample(e3, logits, temps, seed=8, counter=counter)
        assert np.array_equal(tok, arg)
    _check_sample(e3, logits, temps, seed=8, counter=0, name="tiny_tau")


def test_stress_rows_one_hot_and_flat(e3):
    """Configuration 5 at reduced row count: V = 256,000 fp32, near-one-hot and flat rows,
    temperatures log-uniform in [0.1, 2]."""
    rows, V = 24, 256000
    logits = inputs.onehot_flat_logits(rows, V, seed=20, device=DEV)
    temps = inputs.loguniform_temps(rows, seed=21, device=DEV)
    _check_sample(e3, logits, temps, seed=4, counter=1, name="c5")
    _check_sample(e3, logits, temps, seed=4, counter=1, sampler=1, name="c5.s1")
    targets = inputs.uniform_targets(rows, V, seed=22, device=DEV)
    lp, en = e3.e3_token_logp_entropy(logits, targets, temps=temps)
    rlp, ren, _ = oracle.token_logp_entropy(logits.cpu().numpy(), targets.cpu().numpy(), temps=temps.cpu().numpy())
    assert_close("c5.logp", lp.cpu().numpy(), rlp, 1e-5)
    assert_close("c5.ent", en.cpu().numpy(), ren, 1e-5)
    assert np.all(ren[1::2] > 12.0) and np.all(ren[0::2] < 12.0)


# ----------------------------------------------------------------------------------------------
# reproducibility, streams, batch splitting
# ----------------------------------------------------------------------------------------------
def test_bitwise_reproducible_and_row_base(e3):
    rows, V = 96, 20000
    logits = inputs.zipf_gaussian_logits(rows, V, seed=30, dtype=torch.bfloat16, device=DEV)
    temps = inputs.uniform_temps(rows, seed=31, device=DEV)
    a = _run_sample(e3, logits, temps, 12, 34)
    b = _run_sample(e3, logits, temps, 12, 34)
    for x, y in zip(a, b):
        assert x.tobytes() == y.tobytes()
    # the batch split over two calls draws the same tokens (row_base carries the row index)
    lo = _run_sample(e3, logits[:40], temps[:40].contiguous(), 12, 34, row_base=0)
    hi = _run_sample(e3, logits[40:], temps[40:].contiguous(), 12, 34, row_base=40)
    assert np.array_equal(np.concatenate([lo[0], hi[0]]), a[0])
    # (the split changes the launch shape, hence the summation order: values agree, not their last bits)
    assert np.allclose(np.concatenate([lo[1], hi[1]]), a[1], rtol=0, atol=1e-5)
    assert np.allclose(np.concatenate([lo[2], hi[2]]), a[2], rtol=0, atol=1e-5)
    # another step counter or seed draws differently
    assert not np.array_equal(_run_sample(e3, logits, temps, 12, 35)[0], a[0])
    assert not np.array_equal(_run_sample(e3, logits, temps, 13, 34)[0], a[0])
    # non-default stream
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        tok, lp, en = e3.e3_sample(logits, temps, 12, 34)
    s.synchronize()
    assert np.array_equal(tok.cpu().numpy(), a[0])


@pytest.mark.parametrize("sampler", [0, 1])
def test_sampler_distribution_on_device(e3, sampler):
    """Chi-square of 200k device draws (advancing step counter) against softmax(z / tau)."""
    import scipy.special
    import scipy.stats
    V, tau, rows = 300, 0.8, 2000
    row = inputs.zipf_gaussian_logits(1, V, seed=41, device=DEV)
    logits = row.expand(rows, V).contiguous()
    temps = torch.full((rows,), tau, device=DEV)
    toks = []
    for step in range(100):
        toks.append(e3.e3_sample(logits, temps, 77, step, sampler=sampler, want_logp=False, want_ent=False)[0])
    toks = torch.cat(toks).cpu().numpy()
    p = scipy.special.softmax(row.cpu().numpy()[0].astype(np.float64) / float(np.float32(tau)))
    counts = np.bincount(toks, minlength=V).astype(np.float64)
    keep = p * toks.size >= 20
    obs = np.append(counts[keep], counts[~keep].sum())
    exp = np.append(p[keep], p[~keep].sum()) * toks.size
    assert scipy.stats.chisquare(obs, exp).pvalue > 1e-3


# ----------------------------------------------------------------------------------------------
# training side, masked mean, advantages
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_training_pass_with_mask_and_scheduler(e3, dtype):
    n_seq, seq_len, V = 6, 64, 50000
    rows = n_seq * seq_len
    logits = inputs.zipf_gaussian_logits(rows, V, seed=60, dtype=dtype, device=DEV)
    targets = inputs.uniform_targets(rows, V, seed=61, device=DEV)
    mask, _ = inputs.response_mask(n_seq, seq_len, seed=62, min_len=8, device=DEV)
    # poison the masked rows: they must not be read
    poisoned = logits.clone()
    poisoned[mask == 0] = float("nan")
    lp, en = e3.e3_token_logp_entropy(poisoned, targets, mask=mask, temp_scalar=1.0)
    rlp, ren, _ = oracle.token_logp_entropy(inputs.to_oracle_array(logits), targets.cpu().numpy(),
                                            mask=mask.cpu().numpy(), temp_scalar=1.0)
    assert_close("logp", lp.cpu().numpy(), rlp, ATOL[dtype])
    assert_close("ent", en.cpu().numpy(), ren, ATOL[dtype])
    assert torch.all(lp[mask == 0] == 0) and torch.all(en[mask == 0] == 0)
    out = e3.e3_masked_mean_entropy(en, mask)
    torch.cuda.synchronize()
    rmean, rcnt = oracle.masked_mean_entropy(en.cpu().numpy(), mask.cpu().numpy())
    assert float(out[1]) == rcnt
    assert float(out[0]) == pytest.approx(rmean, abs=1e-9)
    # against the oracle's own entropies the mean stays inside the per-token tolerance
    omean, _ = oracle.masked_mean_entropy(ren.astype(np.float32), mask.cpu().numpy())
    assert float(out[0]) == pytest.approx(omean, abs=ATOL[dtype])
    # feed the scheduler (host): same update as the oracle's
    s = e3.make_sched(tau=1.0, H_init=1.1 * float(out[0]), V=V)
    so = oracle.make_sched(tau=1.0, H_init=1.1 * rmean, V=V)
    assert e3.e3_update_temperature(s, float(out[0])) == pytest.approx(oracle.update_temperature(so, rmean), rel=1e-9)


def test_masked_mean_sizes(e3):
    rng = np.random.default_rng(0)
    for n in (1, 31, 256, 4097, 131072, 1_000_003):
        ent = torch.from_numpy(rng.random(n).astype(np.float32)).to(DEV)
        mask = torch.from_numpy((rng.random(n) < 0.56).astype(np.uint8)).to(DEV)
        for m in (mask, None):
            out = e3.e3_masked_mean_entropy(ent, m)
            torch.cuda.synchronize()
            rmean, rcnt = oracle.masked_mean_entropy(ent.cpu().numpy(), None if m is None else m.cpu().numpy())
            assert float(out[1]) == rcnt
            assert float(out[0]) == pytest.approx(rmean, rel=1e-12)
    z = e3.e3_masked_mean_entropy(torch.ones(10, device=DEV), torch.zeros(10, dtype=torch.uint8, device=DEV))
    torch.cuda.synchronize()
    assert math.isnan(float(z[0])) and float(z[1]) == 0


def test_group_advantage_ragged(e3):
    rng = np.random.default_rng(1)
    sizes = [2, 32, 1, 0, 5, 8, 8, 17, 100, 3] + [int(x) for x in rng.integers(2, 33, size=300)]
    off = inputs.group_offsets(sizes, device=DEV)
    rewards = inputs.bernoulli_rewards(sizes, 0.5, seed=70, device=DEV)
    rewards = inputs.force_extreme_groups(rewards, off.cpu(), n_each=4)
    for unbiased in (True, False):
        adv, c = _guarded(rewards.numel(), torch.float32, 55.0)
        _, flags = e3.e3_group_advantage(rewards, off, eps=1e-6, unbiased=unbiased, out_adv=adv)
        torch.cuda.synchronize(); c()
        radv, rflags = oracle.group_advantage(rewards.cpu().numpy(), off.cpu().numpy(), 1e-6, unbiased)
        assert_close("adv", adv.cpu().numpy(), radv, 1e-5)
        assert np.array_equal(flags.cpu().numpy(), rflags)
        a = adv.cpu().numpy()
        o = off.cpu().numpy()
        for g in range(len(sizes)):
            seg = a[o[g]:o[g + 1]]
            if rflags[g] & 1:
                assert np.all(seg == 0.0)          # identical rewards -> exactly zero advantage
            assert abs(seg.sum()) < 1e-4 * max(1, len(seg))
    # real-valued rewards
    r = torch.from_numpy(rng.normal(size=int(off[-1])).astype(np.float32)).to(DEV)
    adv, _ = e3.e3_group_advantage(r, off)
    radv, _ = oracle.group_advantage(r.cpu().numpy(), off.cpu().numpy())
    assert_close("adv.real", adv.cpu().numpy(), radv, 1e-5)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_first_pieces_masked_or_invalid(e3, dtype):
    """Every CTA's first row piece is masked out or has an unusable temperature (the finishing warp's dry run
    then has nothing to walk through), in the split that cuts rows and in the one that hands out whole rows."""
    V = 151936
    for rows in (40, 1300):
        logits = inputs.zipf_gaussian_logits(rows, V, seed=70 + rows, dtype=dtype, device=DEV)
        targets = inputs.uniform_targets(rows, V, seed=71, device=DEV)
        mask = torch.ones(rows, dtype=torch.uint8, device=DEV)
        mask[::2] = 0
        mask[: rows // 3] = 0
        temps = inputs.uniform_temps(rows, seed=72, device=DEV)
        temps[1::4] = float("nan")
        lp, en = e3.e3_token_logp_entropy(logits, targets, mask=mask, temps=temps)
        torch.cuda.synchronize()
        rlp, ren, _ = oracle.token_logp_entropy(inputs.to_oracle_array(logits), targets.cpu().numpy(),
                                                mask=mask.cpu().numpy(), temps=temps.cpu().numpy())
        assert_close("logp", lp.cpu().numpy(), rlp, ATOL[dtype])
        assert_close("ent", en.cpu().numpy(), ren, ATOL[dtype])
        if rows == 40:
            t2 = temps.clone()
            t2[: rows // 2] = -1.0
            for sampler in (0, 1):
                _check_sample(e3, logits, t2, seed=5, counter=rows, sampler=sampler, name=f"s{sampler}")
