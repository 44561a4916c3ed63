"""GPU tests of the optional outputs of the row calls (mean logit gap, fused sum of entropies, status word),
of replays from a captured graph, and of the closed loop temperature -> entropy that the scheduler relies on.
Everything goes through the C ABI; expected values come from the fp64 CPU oracle."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2505_18573_b200 import inputs
from _compare import ATOL, assert_close

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(scope="module")
def e3():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2505_18573_b200 import binding
    binding.lib()   # raises when the CUDA library has not been built: no fallback
    return binding


# ----------------------------------------------------------------------------------------------
# mean logit gap (App. A): beta sum_i p_i Delta_i per row, from the same pass
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_gap_matches_oracle_on_both_row_calls(e3, dtype):
    rows, V = 96, 151936 if dtype == torch.bfloat16 else 40007   # cut rows, several tiles, a ragged tail
    logits = inputs.zipf_gaussian_logits(rows, V, seed=31, dtype=dtype, device=DEV)
    temps = inputs.uniform_temps(rows, seed=32, device=DEV)
    ref = oracle.row_gap(inputs.to_oracle_array(logits), temps=temps.cpu().numpy())
    atol = ATOL[dtype]
    # training side, with a mask
    mask = (torch.arange(rows, device=DEV) % 5 != 2).to(torch.uint8)
    targets = inputs.uniform_targets(rows, V, seed=33, device=DEV)
    lp, en, gap = e3.e3_token_logp_entropy(logits, targets, mask=mask, temps=temps, want_gap=True)
    lp0, en0 = e3.e3_token_logp_entropy(logits, targets, mask=mask, temps=temps)
    torch.cuda.synchronize()
    m = mask.cpu().numpy().astype(bool)
    assert_close("gap.train", gap.cpu().numpy()[m], ref[m], atol)
    assert np.all(gap.cpu().numpy()[~m] == 0.0)
    # the variant that tracks the maximum gives the same other outputs, bit for bit
    assert torch.equal(lp, lp0) and torch.equal(en, en0)
    # H = ln Z(beta) + gap: the entropy of the same call minus the gap is ln sum exp(-beta Delta)
    rlp, rent, _ = oracle.token_logp_entropy(inputs.to_oracle_array(logits), targets.cpu().numpy(), temps=temps.cpu().numpy())
    assert_close("gap.identity", (en - gap).cpu().numpy()[m], (rent - ref)[m], 2 * atol)
    # rollout side, all three samplers
    for sampler in (0, 1, 2):
        tok, slp, sen, sgap = e3.e3_sample(logits, temps, 5, 9, 0, sampler, want_gap=True)
        tok0, slp0, sen0 = e3.e3_sample(logits, temps, 5, 9, 0, sampler)
        torch.cuda.synchronize()
        assert_close(f"gap.sample{sampler}", sgap.cpu().numpy(), ref, atol)
        assert torch.equal(tok, tok0) and torch.equal(slp, slp0) and torch.equal(sen, sen0)


def test_gap_two_level_rows_closed_form_and_special_rows(e3):
    N = 151936
    cases = [(12.0, 1.0), (25.0, 1.0), (6.0, 0.7), (20.0, 1.25)]
    z = torch.zeros(len(cases) + 4, N, dtype=torch.float32, device=DEV)
    temps = torch.ones(len(cases) + 4, device=DEV)
    for r, (delta, tau) in enumerate(cases):
        z[r, 1000 * r + 3] = delta
        temps[r] = tau
    k = len(cases)
    z[k, 5] = float("nan")            # invalid row
    z[k + 1] = 0.25                   # uniform: no gap
    temps[k + 2] = 0.0                # greedy
    z[k + 2, 77] = 3.0
    temps[k + 3] = -1.0               # unusable temperature
    tok, lp, en, gap = e3.e3_sample(z, temps, 1, 2, 0, 1, want_gap=True)
    torch.cuda.synchronize()
    g = gap.cpu().numpy().astype(np.float64)
    for r, (delta, tau) in enumerate(cases):
        beta = 1.0 / float(np.float32(tau))
        q = (N - 1) * math.exp(-beta * delta)
        assert g[r] == pytest.approx(beta * delta * q / (1.0 + q), abs=1e-5)
    assert np.isnan(g[k]) and g[k + 1] == pytest.approx(0.0, abs=1e-6) and g[k + 2] == 0.0 and np.isnan(g[k + 3])
    assert int(tok[k]) == -1 and int(tok[k + 2]) == 77 and int(tok[k + 3]) == -1


# ----------------------------------------------------------------------------------------------
# fused batch entropy (Sec. 4.2): sum of entropies and count from the training call itself
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("rows,V", [(1, 33), (257, 4099), (4096 + 17, 1000), (20000, 64)])
def test_fused_entropy_sum_is_bit_equal_to_the_separate_mean(e3, rows, V):
    logits = inputs.zipf_gaussian_logits(rows, V, seed=41, dtype=torch.float32, device=DEV)
    targets = inputs.uniform_targets(rows, V, seed=42, device=DEV)
    g = torch.Generator(device="cpu").manual_seed(43)
    mask = (torch.rand(rows, generator=g) < 0.7).to(torch.uint8).to(DEV)
    for m in (mask, None):
        out_sum = torch.full((2,), -1.0, dtype=torch.float64, device=DEV)
        lp, en = e3.e3_token_logp_entropy(logits, targets, mask=m, temp_scalar=0.9, out_sum=out_sum)
        mean = e3.e3_masked_mean_entropy(en, m)
        torch.cuda.synchronize()
        s, c = float(out_sum[0]), float(out_sum[1])
        assert c == float(mean[1]) == (rows if m is None else int(mask.sum()))
        if c > 0:
            assert s / c == float(mean[0])          # bit for bit: same blocks, same order
        omean, ocnt = oracle.masked_mean_entropy(en.cpu().numpy(), None if m is None else m.cpu().numpy())
        assert ocnt == c and (c == 0 or s / c == pytest.approx(omean, rel=1e-12))
    # nothing unmasked: sum 0, count 0
    out_sum = torch.full((2,), -1.0, dtype=torch.float64, device=DEV)
    e3.e3_token_logp_entropy(logits, targets, mask=torch.zeros(rows, dtype=torch.uint8, device=DEV), out_sum=out_sum)
    torch.cuda.synchronize()
    assert out_sum.tolist() == [0.0, 0.0]


def test_fused_entropy_sum_feeds_the_scheduler(e3):
    rows, V = 3000, 32000
    logits = inputs.zipf_gaussian_logits(rows, V, seed=44, dtype=torch.bfloat16, device=DEV)
    targets = inputs.uniform_targets(rows, V, seed=45, device=DEV)
    mask = inputs.response_mask(6, 500, seed=46, min_len=100, device=DEV)[0].reshape(-1)
    out_sum = torch.zeros(2, dtype=torch.float64, device=DEV)
    e3.e3_token_logp_entropy(logits, targets, mask=mask, temp_scalar=1.0, out_sum=out_sum)
    torch.cuda.synchronize()
    H_t = float(out_sum[0] / out_sum[1])
    _, rent, _ = oracle.token_logp_entropy(inputs.to_oracle_array(logits), targets.cpu().numpy(), mask=mask.cpu().numpy())
    assert H_t == pytest.approx(float(rent[mask.cpu().numpy() != 0].mean()), abs=2e-3)
    s = e3.make_sched(tau=1.0, H_init=1.1 * H_t, V=V)
    so = oracle.make_sched(tau=1.0, H_init=1.1 * H_t, V=V)
    assert e3.e3_update_temperature(s, H_t) == pytest.approx(oracle.update_temperature(so, H_t), rel=1e-12)


def test_sequence_mean_entropy_matches_oracle(e3):
    rng = np.random.default_rng(7)
    for n_seq, seq_len in ((1, 1), (5, 300), (64, 2048), (300, 33)):
        ent = torch.from_numpy(rng.random((n_seq, seq_len)).astype(np.float32)).to(DEV)
        lens = rng.integers(0, seq_len + 1, size=n_seq)
        mask = torch.from_numpy((np.arange(seq_len)[None, :] < lens[:, None]).astype(np.uint8)).to(DEV)
        for m in (mask, None):
            out = e3.e3_sequence_mean_entropy(ent, m)
            torch.cuda.synchronize()
            rmean, rused = oracle.sequence_mean_entropy(ent.cpu().numpy(), None if m is None else m.cpu().numpy())
            assert float(out[1]) == rused
            if rused == 0:
                assert math.isnan(float(out[0]))
            else:
                assert float(out[0]) == pytest.approx(rmean, rel=1e-12)
    # the two readings differ when lengths differ
    e = torch.tensor([[1, 9, 9], [0, 0, 0]], dtype=torch.float32, device=DEV)
    k = torch.tensor([[1, 0, 0], [1, 1, 1]], dtype=torch.uint8, device=DEV)
    a = e3.e3_sequence_mean_entropy(e, k)
    b = e3.e3_masked_mean_entropy(e.reshape(-1), k.reshape(-1))
    torch.cuda.synchronize()
    assert a.tolist() == [0.5, 2.0] and b.tolist() == [0.25, 4.0]
    z = e3.e3_sequence_mean_entropy(torch.zeros((0, 8), device=DEV))
    torch.cuda.synchronize()
    assert math.isnan(float(z[0])) and float(z[1]) == 0.0


# ----------------------------------------------------------------------------------------------
# group advantage with eps == 0: identical rewards give 0, not 0/0
# ----------------------------------------------------------------------------------------------
def test_group_advantage_without_eps(e3):
    sizes = [3, 2, 8, 1, 4]
    r = torch.tensor([1, 1, 1, 0.5, 0.5, 1, 0, 0, 0, 0, 0, 0, 0, 2.0, 0, 0, 0, 0], dtype=torch.float32, device=DEV)
    off = inputs.group_offsets(sizes, device=DEV)
    for unbiased in (True, False):
        adv, flags = e3.e3_group_advantage(r, off, eps=0.0, unbiased=unbiased)
        radv, rflags = oracle.group_advantage(r.cpu().numpy(), off.cpu().numpy(), eps=0.0, unbiased=unbiased)
        torch.cuda.synchronize()
        a = adv.cpu().numpy()
        assert not np.isnan(a).any()
        assert np.all(a[:5] == 0.0) and np.all(a[13:] == 0.0)
        assert_close("adv.eps0", a, radv, 1e-5)
        assert np.array_equal(flags.cpu().numpy(), rflags)


# ----------------------------------------------------------------------------------------------
# replay from a captured graph: cut rows keep their partial states in the workspace, tagged per call;
# a replay re-runs the very same launch (same tag) on new data and must not pick up an old state
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("which", ["train", "sample1", "sample0"])
def test_graph_replay_on_cut_rows(e3, which):
    rows, V = 40, 151936                       # far fewer rows than thread blocks: every row is cut
    dt = torch.bfloat16
    data = [inputs.zipf_gaussian_logits(rows, V, seed=80 + i, dtype=dt, device=DEV) for i in range(3)]
    logits = data[0].clone()
    temps = inputs.uniform_temps(rows, seed=84, device=DEV)
    targets = inputs.uniform_targets(rows, V, seed=85, device=DEV)
    sampler = {"train": -1, "sample1": 1, "sample0": 0}[which]
    call = e3.E3_CALL_TOKEN_LOGP_ENTROPY if sampler < 0 else e3.E3_CALL_SAMPLE
    ws = torch.zeros(e3.e3_workspace_bytes(call, rows, V, e3.E3_BF16), dtype=torch.uint8, device=DEV)
    tok = torch.empty(rows, dtype=torch.int32, device=DEV)
    lp = torch.empty(rows, device=DEV)
    en = torch.empty(rows, device=DEV)

    def run(stream):
        if sampler < 0:
            e3.e3_token_logp_entropy(logits, targets, temps=temps, out_logp=lp, out_ent=en, workspace=ws, stream=stream)
        else:
            e3.e3_sample(logits, temps, 3, 4, 0, sampler, out_tok=tok, out_logp=lp, out_ent=en, workspace=ws, stream=stream)

    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        run(side)                              # first use outside the capture (sets up the kernel)
    side.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        run(side)
    for i in (1, 2, 0, 2):
        logits.copy_(data[i])
        graph.replay()
        torch.cuda.synchronize()
        got = (tok.clone(), lp.clone(), en.clone())
        run(None)                              # the same data through a fresh call
        torch.cuda.synchronize()
        assert torch.equal(got[1], lp) and torch.equal(got[2], en), (which, i)
        if sampler >= 0:
            assert torch.equal(got[0], tok)
        if sampler < 0:
            rlp, ren, _ = oracle.token_logp_entropy(inputs.to_oracle_array(data[i]), targets.cpu().numpy(), temps=temps.cpu().numpy())
            assert_close("replay.logp", got[1].cpu().numpy(), rlp, ATOL[dt])
            assert_close("replay.ent", got[2].cpu().numpy(), ren, ATOL[dt])
        else:
            ref = oracle.sample(inputs.to_oracle_array(data[i]), temps.cpu().numpy(), 3, 4, 0, sampler)
            assert np.array_equal(got[0].cpu().numpy(), ref.tok)
            assert_close("replay.ent", got[2].cpu().numpy(), ref.ent, ATOL[dt])


# ----------------------------------------------------------------------------------------------
# a bounded wait that runs out: the call returns, the thread block concerned marks its rows, the status
# word says so, and the context stays usable
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("which", ["train", "sample1"])
def test_wait_that_runs_out_sets_the_status_word(e3, which):
    rows, V = 600, 151936
    dt = torch.bfloat16
    logits = inputs.zipf_gaussian_logits(rows, V, seed=90, dtype=dt, device=DEV)
    temps = inputs.uniform_temps(rows, seed=91, device=DEV)
    targets = inputs.uniform_targets(rows, V, seed=92, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)

    def run():
        if which == "train":
            lp, en = e3.e3_token_logp_entropy(logits, targets, temps=temps, status=status)
            return None, lp, en
        return e3.e3_sample(logits, temps, 3, 4, 0, 1, status=status)

    tok0, lp0, en0 = run()
    torch.cuda.synchronize()
    assert int(status[0]) == 0 and not torch.isnan(en0).any()
    tiles_per_row = (V * 2 + 4095) // 4096
    victim = 300
    e3.e3_test_arm_stall(victim * tiles_per_row + 5, 20_000_000)      # 20 ms instead of two seconds
    tok1, lp1, en1 = run()
    torch.cuda.synchronize()                                          # the kernel returned
    assert int(status[0]) & e3.E3_STATUS_TIMEOUT
    bad = torch.isnan(en1)
    assert bool(bad[victim]) and 1 <= int(bad.sum()) <= 8             # only rows of the thread block concerned
    assert torch.isnan(lp1[bad]).all()
    if tok1 is not None:
        assert torch.all(tok1[bad] == -1) and torch.equal(tok1[~bad], tok0[~bad])
    assert torch.equal(en1[~bad], en0[~bad]) and torch.equal(lp1[~bad], lp0[~bad])
    # the hook is one shot and the context is intact: the next call is clean (the status word is never cleared)
    status.zero_()
    tok2, lp2, en2 = run()
    torch.cuda.synchronize()
    assert int(status[0]) == 0 and torch.equal(en2, en0) and torch.equal(lp2, lp0)
    if tok2 is not None:
        assert torch.equal(tok2, tok0)


# ----------------------------------------------------------------------------------------------
# closed loop (Sec. 4.2 under Eq. "tp_adj", App. A): update tau with alpha, run the kernel again on the same
# logits, and see how the measured entropy scales
# ----------------------------------------------------------------------------------------------
def test_closed_loop_entropy_scaling_with_alpha(e3):
    rows, V = 256, 151936
    dt = torch.bfloat16
    logits = inputs.zipf_gaussian_logits(rows, V, seed=95, dtype=dt, device=DEV)
    targets = inputs.uniform_targets(rows, V, seed=96, device=DEV)
    host = inputs.to_oracle_array(logits)
    tau0 = 1.0

    def measure(tau):
        out_sum = torch.zeros(2, dtype=torch.float64, device=DEV)
        lp, en, gap = e3.e3_token_logp_entropy(logits, targets, temp_scalar=tau, want_gap=True, out_sum=out_sum)
        gmean = e3.e3_masked_mean_entropy(gap)          # masked mean of the gap statistic: same reduction
        torch.cuda.synchronize()
        return float(out_sum[0] / out_sum[1]), float(gmean[0])

    def oracle_entropy(tau):
        _, ent, _ = oracle.token_logp_entropy(host, targets.cpu().numpy(), temp_scalar=tau)
        return float(ent.mean())

    H0, gap0 = measure(tau0)
    assert H0 == pytest.approx(oracle_entropy(tau0), abs=ATOL[dt])
    assert gap0 == pytest.approx(float(oracle.row_gap(host, temp_scalar=tau0).mean()), abs=ATOL[dt])
    report = {}
    for alpha in (0.8, 1.25):
        # surrogate update (Eq. "tp_adj") and the update with the logit gap estimated (Eq. "tp_relation_1")
        s = e3.make_sched(tau=tau0, H_init=alpha * H0, V=V)
        t_sur = e3.e3_update_temperature(s, H0)
        sg = e3.make_sched(tau=tau0, H_init=alpha * H0, V=V)
        t_gap = e3.e3_update_temperature_gap(sg, H0)
        so = oracle.make_sched(tau=tau0, H_init=alpha * H0, V=V)
        assert t_sur == pytest.approx(oracle.update_temperature(so, H0), rel=1e-12)
        sog = oracle.make_sched(tau=tau0, H_init=alpha * H0, V=V)
        assert t_gap == pytest.approx(oracle.update_temperature_gap(sog, H0), rel=1e-12)
        # the gap measured by the kernel gives a third update: tau (1 + ln(alpha) / gap), gap = beta Delta measured
        t_meas = tau0 * (1.0 + math.log(alpha) / gap0)
        for name, t1 in (("surrogate", t_sur), ("two_level_root", t_gap), ("measured_gap", t_meas)):
            H1, _ = measure(t1)
            assert H1 == pytest.approx(oracle_entropy(t1), abs=ATOL[dt])      # kernel == oracle at the new tau
            report[(alpha, name)] = H1 / H0
        # direction and size: the entropy moves towards alpha H0, by less than the full factor for the surrogate
        # (ln V + ln ln V over-estimates the gap of these rows), and every update is monotone in alpha
        for name in ("surrogate", "two_level_root", "measured_gap"):
            ratio = report[(alpha, name)]
            assert (ratio < 1.0) == (alpha < 1.0), (alpha, name, ratio)
            assert abs(math.log(ratio)) <= abs(math.log(alpha)) * 1.6, (alpha, name, ratio)
        assert abs(math.log(report[(alpha, "surrogate")])) > 0.02 * abs(math.log(alpha))
    print("closed loop H1/H0:", {f"alpha={a} {n}": round(v, 4) for (a, n), v in report.items()})


# ----------------------------------------------------------------------------------------------
# measurement aid: the read-only probe really reads every word once
# ----------------------------------------------------------------------------------------------
def test_probe_read_checksum(e3):
    rng = np.random.default_rng(3)
    for n_words in (4, 4 * 1000, 4 * 123457):       # multiples of 16 bytes, smaller and larger than one pass of the grid
        host = rng.integers(0, 1 << 32, size=n_words, dtype=np.uint64).astype(np.uint32)
        buf = torch.from_numpy(host.view(np.int32)).to(DEV)
        scratch = torch.zeros(e3.E3_PROBE_SCRATCH_BYTES, dtype=torch.uint8, device=DEV)
        e3.e3_probe_read(buf, scratch=scratch)
        torch.cuda.synchronize()
        per_cta = scratch.cpu().numpy().view(np.uint64)
        v = host.reshape(-1, 4).astype(np.uint64)
        want = int(((v[:, 0] ^ v[:, 1]) + (v[:, 2] ^ v[:, 3])).sum() % (1 << 32))
        assert int(per_cta.sum() % (1 << 32)) == want
    with pytest.raises(e3.E3Error):
        e3.e3_probe_read(torch.zeros(3, dtype=torch.int32, device=DEV))     # not a multiple of 16 bytes
