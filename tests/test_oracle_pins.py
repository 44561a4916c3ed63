"""Pins of the fp64 CPU oracle against what the paper and the mathematics fix.

None of these tests uses the CUDA path.  Each one ties an oracle function to
something other than itself: a closed form, an invariant, a library routine
(scipy / numpy / an independent Philox implementation), a statistical test or
brute force on tiny inputs.
"""
import itertools
import json
import math
import os
import subprocess
import sys

import numpy as np
import pytest
import scipy.special
import scipy.stats
import torch

import oracle
from paper_2505_18573_b200 import inputs

HERE = os.path.dirname(os.path.abspath(__file__))
GOLDEN = json.load(open(os.path.join(HERE, "golden", "paper_settings.json")))


# ----------------------------------------------------------------------------------------------
# Philox4x32-10
# ----------------------------------------------------------------------------------------------
_TRITON_SCRIPT = r"""
import os, sys, json
os.environ["TRITON_INTERPRET"] = "1"
import numpy as np, torch, triton, triton.language as tl

@triton.jit
def k(out, seed, c0, c1, c2, c3, N: tl.constexpr):
    i = tl.arange(0, N)
    a, b, c, d = tl.philox(seed, tl.load(c0 + i), tl.load(c1 + i), tl.load(c2 + i), tl.load(c3 + i))
    tl.store(out + i, a); tl.store(out + N + i, b); tl.store(out + 2 * N + i, c); tl.store(out + 3 * N + i, d)

N = 256
rng = np.random.default_rng(12345)
res = []
for seed in [0, 1, 0x9E3779B97F4A7C15 & ((1 << 63) - 1), 0x00000001FFFFFFFF]:
    ctr = rng.integers(0, 1 << 32, size=(4, N), dtype=np.uint64).astype(np.uint32)
    ctr[:, 0] = 0
    ctr[:, 1] = 0xFFFFFFFF
    cs = [torch.from_numpy(ctr[j].view(np.int32).copy()) for j in range(4)]
    out = torch.zeros(4 * N, dtype=torch.int32)
    k[(1,)](out, seed, cs[0], cs[1], cs[2], cs[3], N=N)
    res.append({"seed": seed, "ctr": ctr.tolist(), "out": out.numpy().view(np.uint32).reshape(4, N).tolist()})
json.dump(res, open(sys.argv[1], "w"))
"""


def test_philox_matches_independent_library(tmp_path):
    """Bit equality with Triton's Philox4x32-10 (CPU interpreter): an implementation written by others."""
    pytest.importorskip("triton")
    script, out = tmp_path / "tri.py", tmp_path / "out.json"
    script.write_text(_TRITON_SCRIPT)
    subprocess.run([sys.executable, str(script), str(out)], check=True, timeout=600)
    cases = json.load(open(out))
    n = 0
    for case in cases:
        seed = case["seed"]
        ctr = np.array(case["ctr"], dtype=np.uint32)
        exp = np.array(case["out"], dtype=np.uint32)
        for j in range(ctr.shape[1]):
            got = oracle.philox4x32_10(seed & 0xFFFFFFFF, seed >> 32, ctr[:, j])
            assert np.array_equal(got, exp[:, j]), (seed, ctr[:, j])
            n += 1
    assert n == 1024


def test_philox_equidistribution():
    """Bytes and words of consecutive counters are uniform (chi-square on 2^18 bytes)."""
    words = np.concatenate([oracle.philox4x32_10(7, 9, [j, 3, 5, 1]) for j in range(1 << 14)])
    counts = np.bincount(words.view(np.uint8), minlength=256)
    p = scipy.stats.chisquare(counts).pvalue
    assert p > 1e-4, p
    top = np.bincount(words >> 24, minlength=256)
    assert scipy.stats.chisquare(top).pvalue > 1e-4
    # changing any counter word or key word changes the output
    base = oracle.philox4x32_10(7, 9, [1, 2, 3, 4])
    for alt in ([0, 2, 3, 4], [1, 0, 3, 4], [1, 2, 0, 4], [1, 2, 3, 0]):
        assert not np.array_equal(base, oracle.philox4x32_10(7, 9, alt))
    assert not np.array_equal(base, oracle.philox4x32_10(8, 9, [1, 2, 3, 4]))
    assert not np.array_equal(base, oracle.philox4x32_10(7, 8, [1, 2, 3, 4]))


def test_token_uniform_layout_and_range():
    """u_i = (c_i + (x_i + 1/2) 2^-32) / 256 with the documented byte / word addressing."""
    seed, counter, row = 0x1234567890ABCDEF, (5 << 32) | 77, 11
    klo, khi = seed & 0xFFFFFFFF, seed >> 32
    for i in [0, 1, 3, 4, 15, 16, 17, 63, 64, 151935]:
        coarse = oracle.philox4x32_10(klo, khi, [i >> 4, row, 77, (5 << 8) | 0])
        fine = oracle.philox4x32_10(klo, khi, [i >> 2, row, 77, (5 << 8) | 1])
        c = int(coarse.view(np.uint8)[i & 15])  # little-endian byte i%16 of the 16-byte output
        x = int(fine[i & 3])
        u = (c + (x + 0.5) / 2.0**32) / 256.0
        assert oracle.token_uniform(seed, counter, row, i) == u
        assert 0.0 < u < 1.0
    blk = oracle.philox4x32_10(klo, khi, [9 >> 2, row, 77, (5 << 8) | 2])
    assert oracle.block_uniform(seed, counter, row, 9) == (int(blk[9 & 3]) + 0.5) / 2.0**32
    inb = oracle.philox4x32_10(klo, khi, [0, row, 77, (5 << 8) | 3])
    assert oracle.inblock_uniform(seed, counter, row) == (int(inb[0]) + 0.5) / 2.0**32
    # extreme Gumbel values reachable with a 40-bit uniform
    assert -math.log(-math.log(2.0**-41)) == pytest.approx(-3.347059, abs=1e-6)
    assert -math.log(-math.log1p(-(2.0**-41))) == pytest.approx(28.419034, abs=1e-6)


# ----------------------------------------------------------------------------------------------
# Row statistics (App. A softmax, Eq. "entropy" and its decomposition, log-prob)
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("V", [32000, 151936, 256000])
@pytest.mark.parametrize("tau", [0.6, 1.0, 1.4])
def test_uniform_row_gives_ln_V(V, tau):
    z = np.full((1, V), 0.37, np.float32)
    lp, ent, ent_dec = oracle.token_logp_entropy(z, np.array([V // 3]), temp_scalar=tau)
    assert ent[0] == pytest.approx(math.log(V), abs=1e-9)
    assert ent_dec[0] == pytest.approx(math.log(V), abs=1e-9)
    assert lp[0] == pytest.approx(-math.log(V), abs=1e-9)
    assert math.log(V) == pytest.approx(GOLDEN["ln_V"][str(V)], abs=1e-6)


@pytest.mark.parametrize("N,delta,tau", [(151936, 12.0, 1.0), (151936, 25.0, 1.0), (256000, 25.0, 2.0), (1000, 3.0, 0.5)])
def test_two_level_row_closed_form(N, delta, tau):
    """One logit at +Delta, N-1 at 0 (the row model of App. A, without its approximations):
    Z = 1 + (N-1) e^{-beta Delta}; H = ln Z + beta Delta (N-1) e^{-beta Delta} / Z; logp_max = -ln Z."""
    z = np.zeros((1, N), np.float32)
    hot = N // 7
    z[0, hot] = delta
    beta = 1.0 / float(np.float32(tau))
    q = (N - 1) * math.exp(-beta * delta)
    Z = 1.0 + q
    H = math.log(Z) + beta * delta * q / Z
    lp, ent, ent_dec = oracle.token_logp_entropy(z, np.array([hot]), temp_scalar=tau)
    # plain fp64 summation of N terms next to a leading 1 carries up to N 2^-53 ~ 3e-11 of rounding
    assert ent[0] == pytest.approx(H, rel=1e-10, abs=1e-10)
    assert ent_dec[0] == pytest.approx(H, rel=1e-10, abs=1e-10)
    assert lp[0] == pytest.approx(-math.log(Z), rel=1e-10, abs=1e-10)
    lp_other, _, _ = oracle.token_logp_entropy(z, np.array([(hot + 1) % N]), temp_scalar=tau)
    assert lp_other[0] == pytest.approx(-beta * delta - math.log(Z), rel=1e-12)
    # the paper's small-entropy approximation H ~ (N-1) beta Delta e^{-beta Delta} holds when Z ~ 1
    if q < 1e-3:
        assert ent[0] == pytest.approx(beta * delta * q, rel=5e-2)


def test_entropy_identity_and_library_softmax():
    """-sum p ln p equals beta sum p Delta + ln Z, and both equal scipy's softmax / entropy / log_softmax."""
    z = inputs.zipf_gaussian_logits(6, 5000, seed=21).numpy()
    temps = inputs.uniform_temps(6, seed=22).numpy()
    targets = inputs.uniform_targets(6, 5000, seed=23).numpy()
    lp, ent, ent_dec = oracle.token_logp_entropy(z, targets, temps=temps)
    for r in range(6):
        s = z[r].astype(np.float64) / float(temps[r])
        p = scipy.special.softmax(s)
        assert ent[r] == pytest.approx(scipy.stats.entropy(p), rel=1e-11)
        assert ent_dec[r] == pytest.approx(ent[r], abs=1e-9)
        assert lp[r] == pytest.approx(scipy.special.log_softmax(s)[targets[r]], rel=1e-12)


def test_row_invariances():
    z = inputs.zipf_gaussian_logits(1, 3000, seed=31).numpy().astype(np.float64)
    tgt = np.array([1234])
    base = oracle.token_logp_entropy(z.astype(np.float32), tgt, temp_scalar=0.8)
    # shift by a constant (exactly representable so that the inputs are the same numbers shifted)
    zq = np.round(z * 64) / 64
    a = oracle.token_logp_entropy(zq.astype(np.float32), tgt, temp_scalar=0.8)
    b = oracle.token_logp_entropy((zq + 16.0).astype(np.float32), tgt, temp_scalar=0.8)
    assert a[0][0] == pytest.approx(b[0][0], abs=1e-10) and a[1][0] == pytest.approx(b[1][0], abs=1e-10)
    # permutation: entropy unchanged, logp follows the token
    perm = np.random.default_rng(3).permutation(3000)
    c = oracle.token_logp_entropy(z[:, perm].astype(np.float32), np.array([int(np.where(perm == 1234)[0][0])]), temp_scalar=0.8)
    assert c[1][0] == pytest.approx(base[1][0], abs=1e-10) and c[0][0] == pytest.approx(base[0][0], abs=1e-10)
    # scaling logits and temperature together (by a power of two, exact) changes nothing
    d = oracle.token_logp_entropy((z * 2).astype(np.float32), tgt, temp_scalar=1.6)
    assert d[1][0] == pytest.approx(base[1][0], abs=1e-6) and d[0][0] == pytest.approx(base[0][0], abs=1e-6)
    # temperature matters: higher tau -> higher entropy on a peaked row
    hi = oracle.token_logp_entropy(z.astype(np.float32), tgt, temp_scalar=1.4)
    assert hi[1][0] > base[1][0]


def test_degenerate_rows():
    one = np.array([[3.5]], np.float32)
    lp, ent, _ = oracle.token_logp_entropy(one, np.array([0]))
    assert lp[0] == 0.0 and ent[0] == 0.0
    r = oracle.sample(one, np.array([0.9], np.float32), 1, 2)
    assert r.tok[0] == 0 and r.logp[0] == 0.0 and r.ent[0] == 0.0
    # -inf entries carry no mass and are never drawn
    z = np.array([[0.0, -np.inf, 0.0, -np.inf]], np.float32)
    lp, ent, _ = oracle.token_logp_entropy(z, np.array([0]))
    assert ent[0] == pytest.approx(math.log(2)) and lp[0] == pytest.approx(-math.log(2))
    lp1, _, _ = oracle.token_logp_entropy(z, np.array([1]))
    assert lp1[0] == -np.inf
    for sampler in (0, 1):
        toks = oracle.sample_repeat(z[0], 1.0, 5, 0, 0, sampler, 2000)
        assert set(toks.tolist()) == {0, 2}
    # invalid rows
    for bad in ([0.0, np.nan], [0.0, np.inf], [-np.inf, -np.inf]):
        zb = np.array([bad], np.float32)
        rr = oracle.sample(zb, np.array([1.0], np.float32), 0, 0)
        assert rr.tok[0] == -1 and np.isnan(rr.logp[0]) and np.isnan(rr.ent[0])
        lpb, entb, _ = oracle.token_logp_entropy(zb, np.array([0]))
        assert np.isnan(lpb[0]) and np.isnan(entb[0])
    rr = oracle.sample(np.zeros((1, 4), np.float32), np.array([-1.0], np.float32), 0, 0)
    assert rr.tok[0] == -1
    # target out of range: entropy still defined
    lp, ent, _ = oracle.token_logp_entropy(np.zeros((1, 4), np.float32), np.array([4]))
    assert np.isnan(lp[0]) and ent[0] == pytest.approx(math.log(4))
    # masked rows give zeros and are not read (NaN row behind a zero mask)
    zz = np.array([[np.nan, 1.0], [0.0, 0.0]], np.float32)
    lp, ent, _ = oracle.token_logp_entropy(zz, np.array([0, 1]), mask=np.array([0, 1], np.uint8))
    assert lp[0] == 0.0 and ent[0] == 0.0 and ent[1] == pytest.approx(math.log(2))


def test_bf16_widening_is_exact():
    t = inputs.zipf_gaussian_logits(3, 777, seed=5, dtype=torch.bfloat16)
    as_bits = inputs.to_oracle_array(t)
    as_f32 = t.to(torch.float32).numpy()
    tg = np.array([0, 5, 776])
    a = oracle.token_logp_entropy(as_bits, tg, temp_scalar=0.9)
    b = oracle.token_logp_entropy(as_f32, tg, temp_scalar=0.9)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


def test_strided_rows():
    z = inputs.zipf_gaussian_logits(4, 300, seed=8).numpy()
    padded = np.full((4, 320), np.nan, np.float32)
    padded[:, :300] = z
    tg = np.array([1, 2, 3, 299])
    a = oracle.token_logp_entropy(z, tg)
    b = oracle.token_logp_entropy(padded[:, :300], tg)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


# ----------------------------------------------------------------------------------------------
# Sampler
# ----------------------------------------------------------------------------------------------
def _chisq_pvalue(tokens, p, min_expected=20.0):
    n = tokens.size
    counts = np.bincount(tokens, minlength=p.size).astype(np.float64)
    order = np.argsort(p)
    exp, obs, acc_e, acc_o = [], [], 0.0, 0.0
    for i in order:  # merge the low-expectation tail into bins of >= min_expected
        acc_e += p[i] * n
        acc_o += counts[i]
        if acc_e >= min_expected:
            exp.append(acc_e); obs.append(acc_o); acc_e = acc_o = 0.0
    if acc_e > 0:
        exp[-1] += acc_e; obs[-1] += acc_o
    exp = np.array(exp); obs = np.array(obs)
    return scipy.stats.chisquare(obs, exp * obs.sum() / exp.sum()).pvalue


@pytest.mark.parametrize("sampler", [0, 1])
@pytest.mark.parametrize("V,tau", [(48, 0.7), (700, 1.3)])
def test_sampler_chi_square_million_draws(sampler, V, tau):
    """10^6 draws (advancing step counter) follow softmax(z / tau); fixed seeds make the statistic a constant."""
    z = inputs.zipf_gaussian_logits(1, V, seed=41).numpy()[0]
    toks = oracle.sample_repeat(z, tau, seed=2024, counter0=0, grow=3, sampler=sampler, n=1_000_000)
    assert toks.min() >= 0 and toks.max() < V
    p = scipy.special.softmax(z.astype(np.float64) / float(np.float32(tau)))
    assert _chisq_pvalue(toks, p) > 1e-3
    # the test has teeth: the same draws are incompatible with a wrong temperature or an unscaled row
    assert _chisq_pvalue(toks, scipy.special.softmax(z.astype(np.float64))) < 1e-12
    assert _chisq_pvalue(toks, scipy.special.softmax(z.astype(np.float64) / (tau * 1.05))) < 1e-6


def test_two_samplers_agree_in_distribution():
    z = inputs.zipf_gaussian_logits(1, 600, seed=43).numpy()[0]
    a = oracle.sample_repeat(z, 1.0, 7, 0, 0, 0, 300_000)
    b = oracle.sample_repeat(z, 1.0, 7, 0, 0, 1, 300_000)
    ca, cb = np.bincount(a, minlength=600), np.bincount(b, minlength=600)
    keep = (ca + cb) >= 40
    table = np.stack([np.append(ca[keep], ca[~keep].sum()), np.append(cb[keep], cb[~keep].sum())])
    assert scipy.stats.chi2_contingency(table)[1] > 1e-3


def test_dominant_logit_always_wins_and_zero_temperature_is_argmax():
    """With a 40-bit uniform g lies in [-3.3471, 28.4191]: a logit ahead by more than 31.7661 tau can never lose."""
    V = 500
    z = inputs.zipf_gaussian_logits(1, V, seed=44).numpy()[0]
    z[123] = z.max() + 31.77 * 0.5
    toks = oracle.sample_repeat(z, 0.5, 9, 0, 0, 0, 20000)
    assert np.all(toks == 123)
    r = oracle.sample(z.reshape(1, -1), np.array([0.5], np.float32), 9, 0)
    assert r.ent[0] < 1e-10 and r.logp[0] > -1e-10
    # tau -> 0 (tiny tau) and tau == 0 (greedy) both return the arg-max
    z2 = inputs.zipf_gaussian_logits(4, V, seed=45).numpy()
    arg = z2.argmax(axis=1)
    r = oracle.sample(z2, np.full(4, 1e-3, np.float32), 1, 1)
    assert np.array_equal(r.tok, arg)
    r0 = oracle.sample(z2, np.zeros(4, np.float32), 1, 1)
    assert np.array_equal(r0.tok, arg) and np.all(r0.logp == 0) and np.all(r0.ent == 0)
    # ties at tau == 0 go to the lowest index
    zt = np.array([[1.0, 5.0, 5.0, 2.0]], np.float32)
    assert oracle.sample(zt, np.zeros(1, np.float32), 0, 0).tok[0] == 1


def test_token_sampler_brute_force_small_rows():
    """Sampler 0 equals an arg-max over s_i + g_i computed in numpy from the documented uniforms."""
    rng = np.random.default_rng(1)
    for V in (1, 2, 3, 17, 33, 100):
        z = rng.normal(size=(5, V)).astype(np.float32)
        temps = np.array([0.6, 0.8, 1.0, 1.2, 1.4], np.float32)
        r = oracle.sample(z, temps, seed=99, counter=(1 << 40) + 5, row_base=1000)
        for row in range(5):
            u = np.array([oracle.token_uniform(99, (1 << 40) + 5, 1000 + row, i) for i in range(V)])
            y = z[row].astype(np.float64) / float(temps[row]) - np.log(-np.log(u))
            assert r.tok[row] == int(np.argmax(y))
            ys = np.sort(y)
            assert r.y1[row] == pytest.approx(ys[-1], rel=1e-14)
            if V > 1:
                assert r.y2[row] == pytest.approx(ys[-2], rel=1e-14)
            assert r.logp[row] == pytest.approx(scipy.special.log_softmax(z[row].astype(np.float64) / float(temps[row]))[r.tok[row]], abs=1e-12)


def test_block_sampler_small_vocab_is_textbook_inverse_cdf():
    """V <= 256: one block, so sampler 1 is inverse-CDF sampling with the in-block uniform."""
    rng = np.random.default_rng(2)
    for V in (1, 2, 5, 255, 256):
        z = rng.normal(size=(3, V)).astype(np.float32) * 2
        temps = np.array([0.7, 1.0, 1.3], np.float32)
        r = oracle.sample(z, temps, seed=5, counter=17, row_base=4, sampler=1)
        for row in range(3):
            s = z[row].astype(np.float64) / float(temps[row])
            w = np.exp(s - s.max())
            v = oracle.inblock_uniform(5, 17, 4 + row)
            tok = int(np.searchsorted(np.cumsum(w), v * w.sum(), side="right"))
            assert r.tok[row] == min(tok, V - 1)


def test_block_sampler_brute_force_multi_block():
    rng = np.random.default_rng(3)
    V = 256 * 3 + 57
    z = (rng.normal(size=(4, V)) * 3).astype(np.float32)
    temps = np.array([0.6, 0.9, 1.1, 1.4], np.float32)
    r = oracle.sample(z, temps, seed=11, counter=3, row_base=0, sampler=1)
    for row in range(4):
        s = z[row].astype(np.float64) / float(temps[row])
        Y = []
        for b in range(4):
            blk = s[b * 256:(b + 1) * 256]
            L = scipy.special.logsumexp(blk)
            Y.append(L - math.log(-math.log(oracle.block_uniform(11, 3, row, b))))
        bstar = int(np.argmax(Y))
        blk = s[bstar * 256:(bstar + 1) * 256]
        w = np.exp(blk - blk.max())
        tok = bstar * 256 + int(np.searchsorted(np.cumsum(w), oracle.inblock_uniform(11, 3, row) * w.sum(), side="right"))
        assert r.tok[row] == tok
        assert r.y1[row] == pytest.approx(max(Y), rel=1e-13)


def test_rows_and_steps_use_distinct_streams():
    z = np.zeros((64, 1000), np.float32)
    t = np.ones(64, np.float32)
    a = oracle.sample(z, t, 0, 0).tok
    assert len(set(a.tolist())) > 55                      # rows differ
    assert not np.array_equal(a, oracle.sample(z, t, 0, 1).tok)   # step counter matters
    assert not np.array_equal(a, oracle.sample(z, t, 1, 0).tok)   # seed matters
    # row_base shifts the row index: rows [8, 64) of one call = rows [0, 56) of a call with row_base 8
    b = oracle.sample(z[:56], t[:56], 0, 0, row_base=8).tok
    assert np.array_equal(a[8:], b)


# ----------------------------------------------------------------------------------------------
# Masked mean entropy
# ----------------------------------------------------------------------------------------------
def test_masked_mean_entropy():
    rng = np.random.default_rng(4)
    ent = rng.random(1000).astype(np.float32)
    mask = (rng.random(1000) < 0.5).astype(np.uint8)
    mean, cnt = oracle.masked_mean_entropy(ent, mask)
    assert cnt == mask.sum()
    assert mean == pytest.approx(math.fsum(float(e) for e, m in zip(ent, mask) if m) / mask.sum(), rel=1e-13)
    mean1, cnt1 = oracle.masked_mean_entropy(ent, np.ones(1000, np.uint8))
    assert cnt1 == 1000 and mean1 == pytest.approx(float(np.mean(ent.astype(np.float64))), rel=1e-13)
    assert oracle.masked_mean_entropy(ent, None)[0] == mean1
    m0, c0 = oracle.masked_mean_entropy(ent, np.zeros(1000, np.uint8))
    assert math.isnan(m0) and c0 == 0
    m0, c0 = oracle.masked_mean_entropy(np.zeros(0, np.float32), None)
    assert math.isnan(m0) and c0 == 0


def test_sequence_mean_entropy_brute_force_and_readings():
    rng = np.random.default_rng(31)
    n_seq, seq_len = 9, 37
    ent = rng.random((n_seq, seq_len)).astype(np.float32)
    lens = rng.integers(0, seq_len + 1, size=n_seq)
    lens[2] = 0                                                    # a sequence without tokens takes no part
    mask = (np.arange(seq_len)[None, :] < lens[:, None]).astype(np.uint8)
    mean, used = oracle.sequence_mean_entropy(ent, mask)
    per_seq = [ent[s, :lens[s]].astype(np.float64).mean() for s in range(n_seq) if lens[s] > 0]
    assert used == len(per_seq) and mean == pytest.approx(float(np.mean(per_seq)), rel=1e-14)
    # equal lengths (or no mask): the two readings of "average entropy" coincide
    m2, u2 = oracle.sequence_mean_entropy(ent, None)
    t2, c2 = oracle.masked_mean_entropy(ent.reshape(-1), None)
    assert u2 == n_seq and c2 == n_seq * seq_len and m2 == pytest.approx(t2, rel=1e-13)
    # hand case where they differ: one token of entropy 1, three tokens of entropy 0
    e = np.array([[1, 9, 9], [0, 0, 0]], np.float32)
    k = np.array([[1, 0, 0], [1, 1, 1]], np.uint8)
    assert oracle.sequence_mean_entropy(e, k) == (0.5, 2.0)
    assert oracle.masked_mean_entropy(e.reshape(-1), k.reshape(-1)) == (0.25, 4.0)
    nan_mean, zero = oracle.sequence_mean_entropy(e, np.zeros_like(k))
    assert math.isnan(nan_mean) and zero == 0.0


# ----------------------------------------------------------------------------------------------
# Mean logit gap (App. A: beta sum p_i Delta_i, the first term of H = beta sum p Delta + ln Z)
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("N,delta,tau", [(151936, 12.0, 1.0), (151936, 25.0, 1.0), (256000, 25.0, 2.0), (1000, 3.0, 0.5),
                                          (32000, 6.0, 0.7)])
def test_row_gap_two_level_closed_form(N, delta, tau):
    """One logit at +Delta, N-1 at 0: gap = beta Delta q / (1 + q) with q = (N-1) e^{-beta Delta}."""
    z = np.zeros((1, N), np.float32)
    z[0, N // 5] = delta
    beta = 1.0 / float(np.float32(tau))
    q = (N - 1) * math.exp(-beta * delta)
    gap = oracle.row_gap(z, temp_scalar=tau)
    assert gap[0] == pytest.approx(beta * delta * q / (1.0 + q), rel=1e-10, abs=1e-12)


def test_row_gap_special_cases_and_entropy_identity():
    rng = np.random.default_rng(21)
    V = 5003
    z = (3.0 * rng.normal(size=(6, V))).astype(np.float32)
    z[1, 17:900] = -np.inf                       # entries without mass
    temps = np.array([0.6, 1.0, 1.4, 0.3, 2.0, 1.0], np.float32)
    gap = oracle.row_gap(z, temps=temps)
    # H from -sum p ln p (its own routine) equals ln Z + gap, with ln Z from a library log-sum-exp
    _, ent, _ = oracle.token_logp_entropy(z, np.zeros(6, np.int32), temps=temps)
    for r in range(6):
        s = z[r].astype(np.float64) / float(temps[r])
        lnZ = scipy.special.logsumexp(s - s.max())
        assert ent[r] == pytest.approx(lnZ + gap[r], rel=1e-11, abs=1e-11)
        # the gap is the softmax-weighted mean of s_max - s_i: a library softmax gives the same
        p = scipy.special.softmax(s)
        keep = np.isfinite(s)
        assert gap[r] == pytest.approx(float(np.sum(p[keep] * (s.max() - s[keep]))), rel=1e-11, abs=1e-12)
    # shifting a row changes nothing (multiples of 1/8: adding 32 is exact)
    zs = np.round(z[:1] * 8) / 8
    assert oracle.row_gap(zs + np.float32(32.0), temp_scalar=1.0)[0] == pytest.approx(oracle.row_gap(zs, temp_scalar=1.0)[0], rel=1e-12)
    # a uniform row has no gap; a single entry has none either
    assert oracle.row_gap(np.full((1, 777), -2.5, np.float32), temp_scalar=0.7)[0] == 0.0
    assert oracle.row_gap(np.array([[4.0]], np.float32), temp_scalar=0.7)[0] == 0.0
    # two entries at distance d: gap = beta d e^{-beta d} / (1 + e^{-beta d})
    d, tau = 1.5, 0.5
    g2 = oracle.row_gap(np.array([[0.25, 0.25 - d]], np.float32), temp_scalar=tau)[0]
    assert g2 == pytest.approx((d / tau) * math.exp(-d / tau) / (1.0 + math.exp(-d / tau)), rel=1e-13)
    # masked rows give 0; greedy rows (tau == 0 where the caller allows it) give 0; bad rows NaN
    zz = np.array([[0.0, 1.0, 2.0], [0.0, np.nan, 1.0], [np.inf, 0.0, 0.0], [-np.inf, -np.inf, -np.inf], [0.0, 1.0, 2.0]], np.float32)
    g = oracle.row_gap(zz, temps=np.array([1.0, 1.0, 1.0, 1.0, 0.0], np.float32), mask=np.array([0, 1, 1, 1, 1], np.uint8), greedy=True)
    assert g[0] == 0.0 and np.isnan(g[1]) and np.isnan(g[2]) and np.isnan(g[3]) and g[4] == 0.0
    g = oracle.row_gap(zz[4:], temps=np.array([0.0], np.float32), greedy=False)
    assert np.isnan(g[0])
    assert np.isnan(oracle.row_gap(zz[:1], temp_scalar=-1.0)[0])


def test_row_gap_estimates_the_gap_of_the_two_level_model():
    """Eq. "tp_relation_1" wants Delta / tau_0 of the two-level model; for such a row in the small-entropy regime the
    measured gap statistic divided by the mass off the leader, (gap / (1 - p_max)), is exactly beta Delta."""
    N, delta, tau = 151936, 20.0, 1.25
    z = np.zeros((1, N), np.float32)
    z[0, 3] = delta
    gap = oracle.row_gap(z, temp_scalar=tau)[0]
    lp, _, _ = oracle.token_logp_entropy(z, np.array([3]), temp_scalar=tau)
    assert gap / (1.0 - math.exp(lp[0])) == pytest.approx(delta / tau, rel=1e-9)


# ----------------------------------------------------------------------------------------------
# Group advantage (Eq. "adv")
# ----------------------------------------------------------------------------------------------
def test_group_advantage_worked_example():
    r = np.array([1, 0, 0, 0, 0, 0, 0, 0], np.float32)
    adv, flags = oracle.group_advantage(r, [0, 8], eps=0.0, unbiased=True)
    sd = math.sqrt((0.875**2 + 7 * 0.125**2) / 7)
    assert sd == pytest.approx(GOLDEN["adv_example"]["sample_std"], abs=1e-6)
    assert adv[0] == pytest.approx(0.875 / sd, rel=1e-14) and np.allclose(adv[1:], -0.125 / sd, rtol=1e-14)
    advp, _ = oracle.group_advantage(r, [0, 8], eps=0.0, unbiased=False)
    assert advp[0] == pytest.approx(GOLDEN["adv_example"]["population_adv0"], abs=1e-6)
    assert flags[0] == 0


def test_group_advantage_matches_textbook_zscore_and_invariants():
    rng = np.random.default_rng(5)
    sizes = [2, 3, 8, 32, 1, 5, 0, 7]
    off = np.concatenate([[0], np.cumsum(sizes)])
    r = rng.normal(size=off[-1]).astype(np.float32)
    r[off[3]:off[4]] = 1.0       # all equal (ones)
    r[off[5]:off[6]] = 0.0       # all zero
    for unbiased in (True, False):
        adv, flags = oracle.group_advantage(r, off, eps=1e-6, unbiased=unbiased)
        for g, n in enumerate(sizes):
            seg = adv[off[g]:off[g + 1]]
            if n == 0:
                continue
            assert abs(seg.sum()) < 1e-6 * max(n, 1)                 # zero mean inside a group
            if g in (3, 5) or n == 1:
                assert np.all(seg == 0.0)                              # identical rewards -> exactly zero
            else:
                exact, _ = oracle.group_advantage(r[off[g]:off[g + 1]], [0, n], eps=0.0, unbiased=unbiased)
                ref = scipy.stats.zscore(r[off[g]:off[g + 1]].astype(np.float64), ddof=1 if unbiased else 0)
                assert np.allclose(exact, ref, rtol=1e-12)
                assert np.allclose(seg, ref, rtol=1e-5)
        assert flags.tolist() == [0, 0, 0, 1, 1, 3, 0, 0]
    # eps is added to the standard deviation
    a0, _ = oracle.group_advantage(np.array([0, 1], np.float32), [0, 2], eps=0.0)
    a1, _ = oracle.group_advantage(np.array([0, 1], np.float32), [0, 2], eps=0.5)
    sd = math.sqrt(0.5)
    assert a0[1] == pytest.approx(0.5 / sd) and a1[1] == pytest.approx(0.5 / (sd + 0.5))
    # identical rewards give exactly zero also without eps (Sec. 4.2: such groups carry no signal), never 0/0
    for unbiased in (True, False):
        az, fz = oracle.group_advantage(np.array([1, 1, 1, 0.5, 0.5], np.float32), [0, 3, 5], eps=0.0, unbiased=unbiased)
        assert np.all(az == 0.0) and fz.tolist() == [1, 1]


# ----------------------------------------------------------------------------------------------
# Algorithm 1
# ----------------------------------------------------------------------------------------------
def test_budget_invariants_random():
    rng = np.random.default_rng(6)
    for trial in range(300):
        B = int(rng.integers(1, 70))
        G = int(rng.integers(2, 17))
        G_min = int(rng.integers(0, G + 1))
        G_max = int(rng.integers(G, 2 * G + 5))
        k = rng.beta(2, 2, size=B) if trial % 3 else rng.integers(1, B + 1, size=B) / B
        for mode in (0, 1):
            out = oracle.allocate_budget(k, G, G_min, G_max, mode)
            assert out.sum() == B * G                                   # "total rollout budget ... remains constant"
            assert out.min() >= G_min and out.max() <= G_max


def test_budget_is_monotone_in_difficulty_fill_to_cap():
    rng = np.random.default_rng(7)
    for _ in range(200):
        B = int(rng.integers(2, 40))
        k = rng.random(B)
        out = oracle.allocate_budget(k, 8, 2, 14, 0)
        order = np.argsort(k, kind="stable")
        assert np.all(np.diff(out[order]) >= 0), (k, out)


def test_budget_special_cases():
    # the paper's first-epoch state: G_min = G_max = G
    assert oracle.allocate_budget(np.linspace(0.1, 1, 64), 8, 8, 8).tolist() == [8] * 64
    # all difficulty zero -> default budget
    assert oracle.allocate_budget(np.zeros(5), 8, 4, 12).tolist() == [8] * 5
    # example where the two readings of "greedily" differ
    ex = GOLDEN["budget_example"]
    assert oracle.allocate_budget(ex["k"], ex["G"], ex["G_min"], ex["G_max"], 0).tolist() == ex["fill_to_cap"]
    assert oracle.allocate_budget(ex["k"], ex["G"], ex["G_min"], ex["G_max"], 1).tolist() == ex["round_robin"]
    with pytest.raises(ArithmeticError):
        oracle.allocate_budget([0.5], 8, 9, 12)
    with pytest.raises(ArithmeticError):
        oracle.allocate_budget([0.5], 8, 4, 7)
    with pytest.raises(ValueError):
        oracle.allocate_budget([1.5], 8, 4, 12)
    with pytest.raises(ValueError):
        oracle.allocate_budget([float("nan")], 8, 4, 12)
    assert oracle.allocate_budget([], 8, 4, 12).size == 0


def test_budget_brute_force_tiny_batches():
    """Every ordering of k for B <= 4: follow Algorithm 1 by hand with exact rationals."""
    from fractions import Fraction
    base = [Fraction(1, 10), Fraction(3, 10), Fraction(6, 10), Fraction(1)]
    for B in (1, 2, 3, 4):
        for ks in itertools.permutations(base[:B]):
            G, G_min, G_max = 8, 4, 12
            tot = B * G
            rem = tot - B * G_min
            out = [min(G_max, G_min + (rem * kk / sum(ks)).__floor__()) for kk in ks]
            left = tot - sum(out)
            for i in sorted(range(B), key=lambda i: (-ks[i], i)):
                give = min(left, G_max - out[i]); out[i] += give; left -= give
            got = oracle.allocate_budget([float(x) for x in ks], G, G_min, G_max, 0)
            assert got.tolist() == out


# ----------------------------------------------------------------------------------------------
# Temperature scheduler (Eq. "tp_adj") and annealing
# ----------------------------------------------------------------------------------------------
def test_temperature_update_values():
    V = 151936
    denom = math.log(V) + math.log(math.log(V))
    assert denom == pytest.approx(GOLDEN["tp_adj"]["denominator_V151936"], abs=1e-6)
    s = oracle.make_sched(tau=1.0, H_init=0.2, V=V)
    assert oracle.update_temperature(s, 0.1) == pytest.approx(1 + math.log(2) / denom, rel=1e-14)  # alpha = 2
    assert s.tau == pytest.approx(GOLDEN["tp_adj"]["tau_alpha2"], abs=1e-6) and s.t == 1
    s = oracle.make_sched(tau=1.0, H_init=0.2, V=V)
    assert oracle.update_temperature(s, 0.4) == pytest.approx(GOLDEN["tp_adj"]["tau_alpha_half"], abs=1e-6)
    # alpha = 1 is a fixed point; the sign of the change follows ln(alpha)
    s = oracle.make_sched(tau=0.83, H_init=0.3, V=V)
    assert oracle.update_temperature(s, 0.3) == 0.83
    s = oracle.make_sched(tau=0.83, H_init=0.3, V=V)
    assert oracle.update_temperature(s, 0.25) > 0.83
    s = oracle.make_sched(tau=0.83, H_init=0.3, V=V)
    assert oracle.update_temperature(s, 0.35) < 0.83
    # tau enters squared: tau' - tau = tau^2 ln(alpha) / denom
    s = oracle.make_sched(tau=2.0, H_init=0.2, V=V)
    assert oracle.update_temperature(s, 0.1) - 2.0 == pytest.approx(4 * math.log(2) / denom, rel=1e-12)
    # first call records H_init ("average entropy of the first batch") and keeps tau
    s = oracle.make_sched(tau=1.0, V=V)
    assert oracle.update_temperature(s, 0.17) == 1.0 and s.H_init == 0.17 and s.t == 1
    for bad in (0.0, -1.0, float("nan"), float("inf")):
        with pytest.raises(ValueError):
            oracle.update_temperature(oracle.make_sched(tau=1.0, H_init=0.2), bad)
    # clamp
    s = oracle.make_sched(tau=1.0, H_init=0.2, V=V, tau_min=0.5, tau_max=1.01)
    assert oracle.update_temperature(s, 0.1) == 1.01


def test_annealing_schedule_end_points():
    st = GOLDEN["settings"]
    t_max, eta = st["train_steps"], st["eta"]
    t_a = math.floor(st["anneal_start_fraction"] * t_max)
    assert t_a == 288
    H0 = 0.25
    def target(t):
        return oracle.anneal_target(oracle.make_sched(H_init=H0, t=t, t_anneal=t_a, t_max=t_max, eta=eta))
    assert target(0) == H0 and target(t_a - 1) == H0 and target(t_a) == H0
    assert target(t_max) == pytest.approx(eta * H0, rel=1e-14)
    assert target((t_a + t_max) // 2) == pytest.approx(H0 * (eta + (1 - eta) / 2), rel=1e-12)
    assert target(t_max + 50) == pytest.approx(eta * H0, rel=1e-14)
    vals = [target(t) for t in range(t_a, t_max + 1)]
    assert all(a >= b for a, b in zip(vals, vals[1:]))
    # the annealed target is the numerator of alpha once t >= t_anneal
    s = oracle.make_sched(tau=1.0, H_init=H0, t=t_max, t_anneal=t_a, t_max=t_max, eta=eta, V=151936)
    denom = math.log(151936) + math.log(math.log(151936))
    assert oracle.update_temperature(s, H0) == pytest.approx(1 + math.log(eta) / denom, rel=1e-13)


# ----------------------------------------------------------------------------------------------
# gradient of log-probability and entropy with respect to the logits
# ----------------------------------------------------------------------------------------------
def test_backward_matches_central_differences_of_the_forward_oracle(oracle_mod):
    o = oracle_mod
    rng = np.random.default_rng(5)
    rows, V = 3, 9
    z = rng.normal(size=(rows, V)).astype(np.float32) * 2
    z[1, 4] = -np.inf                                   # an entry without mass
    targets = np.array([2, 0, 8], np.int32)
    temps = np.array([0.7, 1.0, 1.9], np.float32)
    g_lp = np.array([1.0, -0.5, 2.0], np.float32)
    g_en = np.array([0.25, 1.0, -3.0], np.float32)
    d = o.token_logp_entropy_backward(z, targets, g_lp, g_en, temps=temps)
    h = 2.0 ** -7                                       # exactly representable step, fp32 logits stay exact
    for r in range(rows):
        for i in range(V):
            if not np.isfinite(z[r, i]):
                assert d[r, i] == 0.0
                continue
            zp, zm = z.copy(), z.copy()
            zp[r, i] += h; zm[r, i] -= h
            lp_p, en_p, _ = o.token_logp_entropy(zp, targets, temps=temps)
            lp_m, en_m, _ = o.token_logp_entropy(zm, targets, temps=temps)
            num = (g_lp[r] * (lp_p[r] - lp_m[r]) + g_en[r] * (en_p[r] - en_m[r])) / (2 * h)
            assert d[r, i] == pytest.approx(num, abs=2e-4), (r, i)   # O(h^2) truncation


def test_backward_sums_to_zero_and_matches_autograd(oracle_mod):
    import torch
    o = oracle_mod
    rng = np.random.default_rng(6)
    rows, V = 4, 50
    z = rng.normal(size=(rows, V)).astype(np.float32) * 3
    targets = rng.integers(0, V, size=rows).astype(np.int32)
    g_lp = rng.normal(size=rows).astype(np.float32)
    g_en = rng.normal(size=rows).astype(np.float32)
    mask = np.array([1, 0, 1, 1], np.uint8)
    d = o.token_logp_entropy_backward(z, targets, g_lp, g_en, mask=mask, temp_scalar=1.3)
    assert np.all(d[1] == 0.0)
    assert np.abs(d.sum(axis=1)).max() < 1e-12          # both terms are orthogonal to the all-ones direction
    zt = torch.tensor(z, dtype=torch.float64, requires_grad=True)
    logp_all = torch.log_softmax(zt / float(np.float32(1.3)), dim=1)
    lp = logp_all[torch.arange(rows), torch.tensor(targets, dtype=torch.long)]
    H = -(logp_all.exp() * logp_all).sum(dim=1)
    m = torch.tensor(mask, dtype=torch.float64)
    (m * (torch.tensor(g_lp, dtype=torch.float64) * lp + torch.tensor(g_en, dtype=torch.float64) * H)).sum().backward()
    assert np.abs(d - zt.grad.numpy()).max() < 1e-12
    # out-of-range target and invalid temperature
    bad = o.token_logp_entropy_backward(z[:1], np.array([V], np.int32), g_lp[:1], g_en[:1])
    assert np.isnan(bad).all()


# ----------------------------------------------------------------------------------------------
# difficulty model and G_min / G_max curriculum (Sec. 4.1, Sec. 5.2)
# ----------------------------------------------------------------------------------------------
def test_difficulty_rank_against_a_library_sort_and_by_hand(oracle_mod):
    o = oracle_mod
    # by hand: averages 0.5, 1.0, 0.0, 0.5 -> descending order q1, q0, q3, q2 -> ranks 2, 1, 4, 3 (tie: earlier first)
    k = o.difficulty_rank(np.array([4, 2, 8, 2]), np.array([2.0, 2.0, 0.0, 1.0]))
    assert list(k) == [2 / 4, 1 / 4, 4 / 4, 3 / 4]
    rng = np.random.default_rng(3)
    D = 500
    n = rng.integers(0, 40, size=D)                      # some questions never rolled out: average 0
    r = np.floor(rng.random(D) * (n + 1)).astype(np.float64)
    k = o.difficulty_rank(n, r)
    avg = np.where(n > 0, r / np.maximum(n, 1), 0.0)
    order = np.argsort(-avg, kind="stable")              # library routine: descending, stable
    expect = np.empty(D); expect[order] = np.arange(1, D + 1) / D
    assert np.array_equal(k, expect)
    assert sorted(k) == [(i + 1) / D for i in range(D)]  # a permutation of 1/D ... 1
    harder = avg[:, None] < avg[None, :]                 # i strictly harder than j -> k_i > k_j
    assert np.all((k[:, None] > k[None, :])[harder])


def test_difficulty_accumulate_adds_counts_and_rewards(oracle_mod):
    o = oracle_mod
    n = np.zeros(5, np.int64); r = np.zeros(5, np.float64)
    o.difficulty_accumulate(n, r, [3, 0, 3], [2, 3, 1], [1, 0, 1, 1, 1, 0])
    assert list(n) == [3, 0, 0, 3, 0] and list(r) == [3.0, 0.0, 0.0, 1.0, 0.0]
    with pytest.raises(ValueError):
        o.difficulty_accumulate(n, r, [5], [1], [1.0])


def test_curriculum_follows_the_papers_setting(oracle_mod):
    o = oracle_mod
    # G = 8, +-2 per epoch (Sec. 5.2), limits 2 and 16
    assert [o.budget_curriculum(8, 2, 2, 16, e) for e in range(6)] == [(8, 8), (6, 10), (4, 12), (2, 14), (2, 16), (2, 16)]
    assert o.budget_curriculum(8, 2, 5, 9, 1) == (6, 9) and o.budget_curriculum(8, 2, 5, 9, 2) == (5, 9)
    assert o.budget_curriculum(8, 0, 2, 16, 10) == (8, 8)
    with pytest.raises(ValueError):
        o.budget_curriculum(8, 2, 9, 16, 1)


# ----------------------------------------------------------------------------------------------
# GRPO objective (Sec. 3.1, no KL term)
# ----------------------------------------------------------------------------------------------
def _grpo_case(seed=0, n_groups=5, seq_len=12):
    rng = np.random.default_rng(seed)
    sizes = rng.integers(1, 5, size=n_groups)
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    n_seq = int(off[-1])
    lengths = rng.integers(0, seq_len + 1, size=n_seq)
    lengths[0] = 0                                                     # a response without tokens
    mask = (np.arange(seq_len)[None, :] < lengths[:, None]).astype(np.uint8)
    logp_old = -rng.random((n_seq, seq_len)).astype(np.float32) * 3
    logp = (logp_old + rng.normal(size=(n_seq, seq_len)).astype(np.float32) * 0.3).astype(np.float32)
    adv = rng.normal(size=n_seq).astype(np.float32)
    return logp, logp_old, mask, adv, off


def test_grpo_objective_hand_cases(oracle_mod):
    o = oracle_mod
    ln = np.log
    # one question, two responses of 2 and 1 tokens, eps = 0.2
    logp_old = np.zeros((2, 2), np.float32)
    logp = np.array([[ln(1.5), ln(0.5)], [ln(1.1), 0.0]], np.float32)
    mask = np.array([[1, 1], [1, 0]], np.uint8)
    adv = np.array([1.0, -2.0], np.float32)
    J, g, frac = o.grpo_objective(logp, logp_old, mask, adv, [0, 2], 0.2)
    # response 0 (A = 1): r = 1.5 -> min(1.5, 1.2) = 1.2 (clipped, no gradient); r = 0.5 -> min(0.5, 0.8) = 0.5
    # response 1 (A = -2): r = 1.1 -> min(-2.2, -2.2) = -2.2
    assert J == pytest.approx(0.5 * ((1.2 + 0.5) / 2 + (-2.2) / 1), abs=1e-6)
    assert g[0, 0] == 0.0 and g[0, 1] == pytest.approx(0.5 * 1.0 / (2 * 2), abs=1e-7)
    assert g[1, 0] == pytest.approx(1.1 * -2.0 / (1 * 2), abs=1e-6) and g[1, 1] == 0.0
    assert frac == pytest.approx(1 / 3)
    # negative advantage, ratio below the range: the clipped term (0.8 A) is smaller than r A: no gradient
    J2, g2, _ = o.grpo_objective(np.full((1, 1), ln(0.5), np.float32), np.zeros((1, 1), np.float32), None,
                                 np.array([-1.0], np.float32), [0, 1], 0.2)
    assert J2 == pytest.approx(-0.8, abs=1e-6) and g2[0, 0] == 0.0


def test_grpo_objective_at_the_old_policy_is_the_mean_advantage(oracle_mod):
    o = oracle_mod
    logp, logp_old, mask, adv, off = _grpo_case(1)
    J, g, frac = o.grpo_objective(logp_old, logp_old, mask, adv, off, 0.2)
    adv = adv.astype(np.float64)
    has = mask.sum(axis=1) > 0
    expect = np.mean([np.sum(adv[off[q]:off[q + 1]][has[off[q]:off[q + 1]]]) / (off[q + 1] - off[q]) for q in range(off.size - 1)])
    assert J == pytest.approx(expect, abs=1e-9) and frac == 0.0
    w = 1.0 / (np.maximum(mask.sum(axis=1), 1) * np.repeat(np.diff(off), np.diff(off)) * (off.size - 1))
    assert np.allclose(g, mask * (adv * w)[:, None], atol=1e-12)


def test_grpo_objective_gradient_against_central_differences_and_autograd(oracle_mod):
    import torch
    o = oracle_mod
    logp, logp_old, mask, adv, off = _grpo_case(2)
    J, g, _ = o.grpo_objective(logp, logp_old, mask, adv, off, 0.2)
    r = np.exp(logp.astype(np.float64) - logp_old)
    h = 2.0 ** -10
    for (i, t) in [(1, 0), (2, 3), (5, 1), (7, 0)]:
        if not mask[i, t] or min(abs(r[i, t] - 0.8), abs(r[i, t] - 1.2)) < 0.02:
            continue                                                   # off the response or next to a kink
        lp, lm = logp.copy(), logp.copy()
        lp[i, t] += h; lm[i, t] -= h
        num = (o.grpo_objective(lp, logp_old, mask, adv, off, 0.2)[0] - o.grpo_objective(lm, logp_old, mask, adv, off, 0.2)[0]) / (2 * h)
        assert g[i, t] == pytest.approx(num, abs=1e-6)
    x = torch.tensor(logp, dtype=torch.float64, requires_grad=True)
    ratio = torch.exp(x - torch.tensor(logp_old, dtype=torch.float64))
    A = torch.tensor(adv, dtype=torch.float64)[:, None]
    eps = float(np.float32(0.2))
    sur = torch.minimum(ratio * A, torch.clamp(ratio, 1 - eps, 1 + eps) * A) * torch.tensor(mask, dtype=torch.float64)
    per_seq = sur.sum(dim=1) / torch.clamp(torch.tensor(mask.sum(axis=1), dtype=torch.float64), min=1)
    Jt = sum(per_seq[off[q]:off[q + 1]].sum() / (off[q + 1] - off[q]) for q in range(off.size - 1)) / (off.size - 1)
    Jt.backward()
    assert J == pytest.approx(float(Jt), abs=1e-12)
    assert np.abs(g - x.grad.numpy()).max() < 1e-12


# ----------------------------------------------------------------------------------------------
# Delta-aware temperature update (Eq. tp_relation_1 with Delta estimated from the entropy, App. A)
# ----------------------------------------------------------------------------------------------
def _two_level_entropy(N, delta, tau):
    b = 1.0 / tau
    w = (N - 1) * math.exp(-b * delta)
    return math.log(1 + w) + b * delta * w / (1 + w)      # exact entropy of one logit at +delta over N-1 at 0


def test_entropy_gap_is_the_root_of_the_two_level_model(oracle_mod):
    o = oracle_mod
    for N, H in ((151936, 0.1), (151936, 2.5), (32000, 0.01), (256000, 0.7), (10, 0.5)):
        x = o.entropy_gap(H, N)
        assert x >= 1 and (N - 1) * x * math.exp(-x) == pytest.approx(H, rel=1e-12)
        assert x == pytest.approx(math.log(N - 1) + math.log(x) - math.log(H), abs=1e-10)   # the paper's fixed-point form
    assert math.isnan(o.entropy_gap(0.0, 100)) and math.isnan(o.entropy_gap(50.0, 100))
    # on exact two-level rows of low entropy the root recovers beta * Delta
    for delta in (16.0, 18.0, 20.0):
        for tau in (0.8, 1.0, 1.2):
            H = _two_level_entropy(151936, delta, tau)
            if H < 0.5:
                assert o.entropy_gap(H, 151936) == pytest.approx(delta / tau, rel=5e-3)


def test_gap_update_scales_the_entropy_of_two_level_rows_by_alpha(oracle_mod):
    o = oracle_mod
    N = 151936
    worse = 0
    for delta in (16.0, 18.0, 20.0):
        for tau in (0.8, 1.0, 1.2):
            H0 = _two_level_entropy(N, delta, tau)
            if H0 > 0.5:
                continue
            for alpha in (0.8, 1.25):
                s = o.make_sched(tau=tau, H_init=alpha * H0, V=N)
                t_gap = o.update_temperature_gap(s, H0)
                s2 = o.make_sched(tau=tau, H_init=alpha * H0, V=N)
                t_sur = o.update_temperature(s2, H0)
                r_gap = _two_level_entropy(N, delta, t_gap) / H0
                r_sur = _two_level_entropy(N, delta, t_sur) / H0
                assert abs(r_gap - alpha) < 0.04, (delta, tau, alpha, r_gap)
                assert (t_gap - tau) * (alpha - 1) > 0                  # the temperature moves the right way
                if delta >= 18.0:      # away from Delta = ln N + ln ln N = 14.4, where the simplified formula is at home
                    worse += abs(r_gap - alpha) > abs(r_sur - alpha)
    assert worse == 0
    s = o.make_sched(tau=1.0, H_init=0.3, V=N)
    assert o.update_temperature_gap(s, 0.3) == 1.0 and s.t == 1         # alpha = 1: fixed point
    s = o.make_sched(tau=1.0, V=N)
    assert o.update_temperature_gap(s, 0.2) == 1.0 and s.H_init == 0.2  # first call records H_init
