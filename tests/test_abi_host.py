"""CPU-side checks of the C-ABI library: it loads, exports every symbol the header declares,
and its host entry points (Algorithm 1, temperature scheduler) agree with the oracle.
No device call is made here."""
import ctypes as C
import math
import os
import re

import numpy as np
import pytest

import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def e3():
    from paper_2505_18573_b200 import build, binding
    build.build()
    binding.lib()
    return binding


def test_library_exports_every_declared_symbol(e3):
    header = open(os.path.join(ROOT, "include", "e3.h")).read()
    declared = set(re.findall(r"E3_API[^;(]*?\b(e3_\w+)\s*\(", header))
    assert declared == set(e3.EXPORTS)
    L = C.CDLL(e3.LIB_PATH)
    for name in declared:
        assert hasattr(L, name), name


def test_status_strings_and_workspace(e3):
    assert e3.status_string(0) == "E3_OK"
    assert e3.status_string(5) == "E3_ERR_INFEASIBLE"
    assert e3.e3_workspace_bytes(e3.E3_CALL_SAMPLE, 512, 151936, e3.E3_BF16) >= 1024 * 256 + 512 * 75 * 132 + 512 * 16
    assert e3.e3_workspace_bytes(e3.E3_CALL_SAMPLE, 512, 151936, e3.E3_BF16) < 16 * 512 * 151936 * 2 // 256
    assert e3.e3_workspace_bytes(e3.E3_CALL_TOKEN_LOGP_ENTROPY, 131072, 151936, e3.E3_BF16) >= 1024 * 256 + 16
    assert e3.e3_workspace_bytes(e3.E3_CALL_MASKED_MEAN_ENTROPY, 131072) >= 16
    assert e3.e3_workspace_bytes(e3.E3_CALL_MASKED_MEAN_ENTROPY, 0) >= 16


def test_device_calls_reject_bad_arguments_on_the_host(e3):
    L = e3.lib()
    # checked before any CUDA call is made, so these run without a device
    def sample(logits, dt, rows, V, stride, temps=None, counter=0, row_base=0, sampler=0, out_tok=None,
               ws=None, ws_bytes=0):
        return L.e3_sample(logits, dt, rows, V, stride, temps, 0, counter, row_base, sampler, out_tok, None, None,
                           None, None, ws, ws_bytes, None)

    def token(logits, dt, rows, V, stride, targets=None, out_ent=None, out_sum=None, out_count=None, ws=None,
              ws_bytes=0):
        return L.e3_token_logp_entropy(logits, dt, rows, V, stride, targets, None, None, 1.0, None, out_ent, None,
                                       out_sum, out_count, None, ws, ws_bytes, None)

    assert sample(None, 7, 1, 8, 8) == 2                      # dtype
    assert sample(None, 0, -1, 8, 8) == 1                     # rows < 0
    assert sample(None, 0, 1, 8, 4) == 1                      # stride < V
    assert sample(None, 0, 1, 1 << 31, 1 << 31) == 1          # V too large
    assert sample(None, 0, 0, 8, 8) == 0                      # rows == 0
    assert sample(None, 0, 0, 8, 8, counter=1 << 56) == 1
    assert sample(None, 0, 0, 8, 8, sampler=3) == 1           # sampler
    assert sample(1024, 0, 1, 8, 8) == 1                      # temps NULL
    assert sample(1026, 0, 1, 8, 8, temps=1024, out_tok=1024) == 3   # misaligned
    # the row number is one 32-bit word of the Philox counter
    assert sample(None, 0, 0, 8, 8, row_base=-1) == 1
    assert sample(None, 0, 0, 8, 8, row_base=1 << 32) == 0            # no rows: nothing exceeds the range
    assert sample(1024, 0, 1, 8, 8, temps=1024, out_tok=1024, row_base=1 << 32) == 1
    assert sample(1024, 0, 2, 8, 8, temps=1024, out_tok=1024, row_base=(1 << 32) - 1) == 1
    # the blocked sampler needs its workspace
    assert sample(1024, 0, 1, 8, 8, temps=1024, out_tok=1024, sampler=1) == 4
    assert sample(1024, 0, 1, 8, 8, temps=1024, out_tok=1024, sampler=1, ws=4096, ws_bytes=1 << 18) == 4
    assert token(None, 0, 0, 8, 8) == 0
    assert token(1024, 0, 1, 8, 8) == 1                       # targets NULL
    # fused mean entropy: both scalars or none, needs out_ent and the workspace
    assert token(1024, 0, 1, 8, 8, targets=1024, out_ent=1024, out_sum=2048) == 1
    assert token(1024, 0, 1, 8, 8, targets=1024, out_sum=2048, out_count=2056) == 1
    assert token(1024, 0, 1, 8, 8, targets=1024, out_ent=1024, out_sum=2048, out_count=2056) == 4
    assert token(1024, 0, 1, 8, 8, targets=1024, out_ent=1024, out_sum=2052, out_count=2056) == 3
    assert L.e3_masked_mean_entropy(None, None, -1, None, None, None, 0, None) == 1
    assert L.e3_masked_mean_entropy(1024, None, 4, 1024, 1032, None, 0, None) == 4                  # workspace
    assert L.e3_sequence_mean_entropy(None, None, -1, 4, 1024, 1032, 1024, 64, None) == 1
    assert L.e3_sequence_mean_entropy(1024, None, 2, 4, None, 1032, 1024, 64, None) == 1
    assert L.e3_sequence_mean_entropy(1024, None, 2, 4, 1024, 1032, None, 0, None) == 4               # workspace
    assert L.e3_sequence_mean_entropy(1024, None, 2, 4, 1024, 1032, 1024, 16, None) == 4              # too small
    assert L.e3_sequence_mean_entropy(1026, None, 2, 4, 1024, 1032, 1024, 64, None) == 3
    assert L.e3_group_advantage(None, None, 0, 1e-6, 1, None, None, None) == 0
    assert L.e3_group_advantage(None, None, 2, 1e-6, 1, None, None, None) == 1
    assert L.e3_group_advantage(None, None, 2, -1.0, 1, None, None, None) == 1                       # eps < 0
    assert L.e3_group_advantage(None, None, 2, float("inf"), 1, None, None, None) == 1
    with pytest.raises(ValueError):
        import torch
        e3.e3_sample(torch.zeros(2, 8), torch.ones(2), 0, 0)   # CPU tensors: there is no CPU path


def test_allocate_budget_matches_oracle(e3):
    rng = np.random.default_rng(11)
    for trial in range(400):
        B = int(rng.integers(1, 80))
        G = int(rng.integers(1, 20))
        G_min = int(rng.integers(0, G + 1))
        G_max = int(rng.integers(G, 2 * G + 6))
        if trial % 4 == 0:
            k = rng.integers(1, B + 1, size=B) / B     # normalised ranks, with ties
        elif trial % 4 == 1:
            k = np.round(rng.random(B), 1)
        else:
            k = rng.beta(2, 2, size=B)
        for mode in (0, 1):
            got = e3.e3_allocate_budget(k.tolist(), G, G_min, G_max, mode)
            ref = oracle.allocate_budget(k, G, G_min, G_max, mode)
            assert got == ref.tolist(), (B, G, G_min, G_max, mode)
            assert sum(got) == B * G
    assert e3.e3_allocate_budget([], 8, 4, 12) == []
    assert e3.e3_allocate_budget([0.0, 0.0], 8, 4, 12) == [8, 8]
    for args in (([0.5], 8, 9, 12), ([0.5], 8, 4, 7)):
        with pytest.raises(e3.E3Error) as ei:
            e3.e3_allocate_budget(*args)
        assert ei.value.status == 5
    for bad in ([1.5], [-0.1], [float("nan")]):
        with pytest.raises(e3.E3Error) as ei:
            e3.e3_allocate_budget(bad, 8, 4, 12)
        assert ei.value.status == 1


def test_update_temperature_matches_oracle(e3):
    rng = np.random.default_rng(12)
    for trial in range(200):
        kw = dict(tau=float(rng.uniform(0.3, 2.0)), H_init=float(rng.uniform(0.05, 1.0)) if trial % 5 else float("nan"),
                  t=int(rng.integers(0, 500)), t_anneal=288, t_max=480, eta=float(rng.uniform(0.5, 0.99)),
                  V=int(rng.choice([32000, 151936, 256000])))
        if trial % 7 == 0:
            kw.update(tau_min=0.5, tau_max=1.5)
        a, b = e3.make_sched(**kw), oracle.make_sched(**kw)
        for _ in range(5):
            H = float(rng.uniform(0.02, 1.5))
            ta = e3.e3_update_temperature(a, H)
            tb = oracle.update_temperature(b, H)
            assert ta == pytest.approx(tb, rel=1e-12)
            assert a.t == b.t and a.H_init == b.H_init
            assert e3.e3_anneal_target(a) == pytest.approx(oracle.anneal_target(b), rel=1e-12)
    s = e3.make_sched(tau=1.0, H_init=0.2)
    for bad in (0.0, -1.0, float("nan"), float("inf")):
        with pytest.raises(e3.E3Error):
            e3.e3_update_temperature(s, bad)
    assert s.tau == 1.0 and s.t == 0
    # an update that would push tau below zero is refused and leaves the state alone
    s = e3.make_sched(tau=4.0, H_init=1e-9, V=3)
    with pytest.raises(e3.E3Error):
        e3.e3_update_temperature(s, 1e3)
    assert s.tau == 4.0 and s.t == 0


def test_gap_based_temperature_update_matches_oracle(e3):
    """App. A with the gap estimated from the entropy (Eq. "tp_relation_1"): root and update against the oracle."""
    rng = np.random.default_rng(31)
    for N in (3, 17, 32000, 151936, 256000):
        top = (N - 1) / np.e
        for H in list(rng.uniform(1e-6, 1.0, 20) * top) + [1e-12 * top, 1e-3, 0.3, 0.999999 * top]:
            x = e3.e3_entropy_gap(float(H), N)
            xo = oracle.entropy_gap(float(H), N)
            # close to the double root at H = (N-1)/e the root is only determined to sqrt(rounding)
            assert x == pytest.approx(xo, rel=1e-9 if H < 0.99 * top else 1e-5)
            assert x >= 1.0
        for bad in (0.0, -1.0, float("nan"), float("inf"), 1.001 * top):
            assert np.isnan(e3.e3_entropy_gap(bad, N)) and np.isnan(oracle.entropy_gap(bad, N))
    assert np.isnan(e3.e3_entropy_gap(0.1, 2))
    for trial in range(200):
        kw = dict(tau=float(rng.uniform(0.3, 2.0)), H_init=float(rng.uniform(0.05, 1.0)) if trial % 5 else float("nan"),
                  t=int(rng.integers(0, 500)), t_anneal=288, t_max=480, eta=float(rng.uniform(0.5, 0.99)),
                  V=int(rng.choice([32000, 151936, 256000])))
        if trial % 7 == 0:
            kw.update(tau_min=0.5, tau_max=1.5)
        a, b = e3.make_sched(**kw), oracle.make_sched(**kw)
        for _ in range(5):
            H = float(rng.uniform(0.02, 1.5))
            ta = e3.e3_update_temperature_gap(a, H)
            tb = oracle.update_temperature_gap(b, H)
            assert ta == pytest.approx(tb, rel=1e-10)
            assert a.t == b.t and a.H_init == b.H_init
    s = e3.make_sched(tau=1.0, H_init=0.2, V=1000)
    for bad in (0.0, -1.0, float("nan"), float("inf"), 999.0):   # 999 > (N-1)/e: no root
        with pytest.raises(e3.E3Error):
            e3.e3_update_temperature_gap(s, bad)
    assert s.tau == 1.0 and s.t == 0


def test_difficulty_model_and_curriculum_match_the_oracle(oracle_mod):
    """Sec. 4.1: cumulative statistics, descending-average-reward ranks, bounds curriculum; then Algorithm 1 on the ranks."""
    import numpy as np
    from paper_2505_18573_b200 import binding as e3
    o = oracle_mod
    rng = np.random.default_rng(11)
    D, B = 300, 64
    n1 = np.zeros(D, np.int64); r1 = np.zeros(D, np.float64)
    n2 = np.zeros(D, np.int64); r2 = np.zeros(D, np.float64)
    p_q = rng.random(D)
    for epoch in range(3):
        g_min, g_max = e3.e3_budget_curriculum(8, 2, 2, 16, epoch)
        assert (g_min, g_max) == o.budget_curriculum(8, 2, 2, 16, epoch)
        k = e3.e3_difficulty_rank(n1, r1)
        assert np.array_equal(k, o.difficulty_rank(n2, r2))
        for start in range(0, D - B + 1, B):
            ids = np.arange(start, start + B)
            G = e3.e3_allocate_budget(k[ids], 8, g_min, g_max)
            assert sum(G) == 8 * B and G == list(o.allocate_budget(k[ids], 8, g_min, g_max))
            rewards = (rng.random(sum(G)) < np.repeat(p_q[ids], G)).astype(np.float32)
            e3.e3_difficulty_accumulate(n1, r1, ids, G, rewards)
            o.difficulty_accumulate(n2, r2, ids, G, rewards)
            assert np.array_equal(n1, n2) and np.array_equal(r1, r2)
    k = e3.e3_difficulty_rank(n1, r1)
    assert sorted(k) == [(i + 1) / D for i in range(D)]
    seen = n1 > 0
    assert np.corrcoef(k[seen], p_q[seen])[0, 1] < -0.8          # easy questions (high success rate) get small k
    for e in range(12):
        assert e3.e3_budget_curriculum(8, 3, 1, 20, e) == o.budget_curriculum(8, 3, 1, 20, e)
    L = e3.lib()
    assert L.e3_budget_curriculum(8, 2, 9, 16, 1, None, None) == 1
    n3 = np.zeros(4, np.int64); r3 = np.zeros(4, np.float64)
    with pytest.raises(e3.E3Error):
        e3.e3_difficulty_accumulate(n3, r3, [1, 4], [1, 1], [1.0, 1.0])
    assert n3.sum() == 0 and r3.sum() == 0                        # a rejected batch changes nothing
    with pytest.raises(e3.E3Error):
        e3.e3_budget_curriculum(8, 2, 9, 16, 1)
