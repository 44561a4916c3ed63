"""ctypes binding of the fp64 CPU oracle (``e3_oracle.c``).

TEST INFRASTRUCTURE, NOT PRODUCT CODE: only ``tests/``, the smoke check and the
benchmark's CPU-baseline leg may import this package.  It imports nothing from
the CUDA package and the CUDA package imports nothing from here.

``build()`` compiles the C file with gcc into ``oracle/libe3_oracle.so``; the
library is rebuilt when the source is newer than the binary.  Every wrapper
takes numpy arrays (bf16 logits as ``uint16`` bit patterns) and returns fp64.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_DIR, "e3_oracle.c")
_LIB = os.path.join(_DIR, "libe3_oracle.so")

F32, BF16 = 0, 1
SAMPLER_TOKEN, SAMPLER_BLOCK = 0, 1
SAMPLE_BLOCK = 256


def build(force: bool = False) -> str:
    """Compile the oracle (gcc, IEEE semantics, OpenMP over rows only)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-shared",
               "-fPIC", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.e3o_token_uniform.restype = C.c_double
        _lib.e3o_block_uniform.restype = C.c_double
        _lib.e3o_inblock_uniform.restype = C.c_double
        _lib.e3o_anneal_target.restype = C.c_double
        _lib.e3o_entropy_gap.restype = C.c_double
    return _lib


def num_threads() -> int:
    return int(lib().e3o_num_threads())


def _p(a, ty=C.c_void_p):
    return None if a is None else a.ctypes.data_as(ty)


def _logits_args(logits: np.ndarray):
    """(pointer, dtype code, rows, V, row stride in elements) of a 2-D logits array."""
    assert logits.ndim == 2
    if logits.dtype == np.float32:
        dt = F32
    elif logits.dtype == np.uint16:
        dt = BF16
    else:
        raise TypeError("logits must be float32, or uint16 holding bf16 bit patterns")
    assert logits.strides[1] == logits.itemsize, "innermost dimension must be contiguous"
    stride = logits.strides[0] // logits.itemsize if logits.shape[0] > 1 else logits.shape[1]
    return _p(logits), dt, logits.shape[0], logits.shape[1], stride


def philox4x32_10(key_lo: int, key_hi: int, ctr) -> np.ndarray:
    c = np.ascontiguousarray(ctr, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().e3o_philox4x32_10(C.c_uint32(key_lo), C.c_uint32(key_hi), _p(c), _p(out))
    return out


def token_uniform(seed: int, counter: int, grow: int, i: int) -> float:
    return float(lib().e3o_token_uniform(C.c_uint64(seed), C.c_uint64(counter), C.c_uint32(grow), C.c_int64(i)))


def block_uniform(seed: int, counter: int, grow: int, b: int) -> float:
    return float(lib().e3o_block_uniform(C.c_uint64(seed), C.c_uint64(counter), C.c_uint32(grow), C.c_int64(b)))


def inblock_uniform(seed: int, counter: int, grow: int) -> float:
    return float(lib().e3o_inblock_uniform(C.c_uint64(seed), C.c_uint64(counter), C.c_uint32(grow)))


@dataclass
class SampleResult:
    tok: np.ndarray         # int32 [rows]; -1 = invalid row
    logp: np.ndarray        # float64 [rows]
    ent: np.ndarray         # float64 [rows], -sum p ln p
    ent_dec: np.ndarray     # float64 [rows], beta sum p Delta + ln Z
    y1: np.ndarray          # best perturbed score
    y2: np.ndarray          # second best perturbed score
    cdf_margin: np.ndarray  # sampler 1 only


def sample(logits: np.ndarray, temps: np.ndarray, seed: int, counter: int, row_base: int = 0,
           sampler: int = SAMPLER_TOKEN) -> SampleResult:
    ptr, dt, rows, V, stride = _logits_args(logits)
    temps = np.ascontiguousarray(temps, dtype=np.float32)
    assert temps.shape == (rows,)
    tok = np.empty(rows, np.int32)
    outs = [np.empty(rows, np.float64) for _ in range(6)]
    rc = lib().e3o_sample(ptr, dt, C.c_int64(rows), C.c_int64(V), C.c_int64(stride), _p(temps),
                          C.c_uint64(seed), C.c_uint64(counter), C.c_int64(row_base), C.c_int(sampler),
                          _p(tok), *[_p(o) for o in outs])
    if rc != 0:
        raise ValueError(f"e3o_sample: invalid argument ({rc})")
    return SampleResult(tok, *outs)


def sample_repeat(row: np.ndarray, tau: float, seed: int, counter0: int, grow: int, sampler: int,
                  n: int) -> np.ndarray:
    row = np.ascontiguousarray(row)
    ptr, dt, _, V, _ = _logits_args(row.reshape(1, -1))
    tok = np.empty(n, np.int32)
    rc = lib().e3o_sample_repeat(ptr, dt, C.c_int64(V), C.c_float(tau), C.c_uint64(seed), C.c_uint64(counter0),
                                 C.c_int64(grow), C.c_int(sampler), C.c_int64(n), _p(tok))
    if rc != 0:
        raise ValueError("e3o_sample_repeat: invalid argument")
    return tok


def token_logp_entropy(logits: np.ndarray, targets: np.ndarray, mask=None, temps=None, temp_scalar: float = 1.0):
    """Returns (logp, ent, ent_dec), each float64 [rows]."""
    ptr, dt, rows, V, stride = _logits_args(logits)
    targets = np.ascontiguousarray(targets, dtype=np.int32)
    mask = None if mask is None else np.ascontiguousarray(mask, dtype=np.uint8)
    temps = None if temps is None else np.ascontiguousarray(temps, dtype=np.float32)
    outs = [np.empty(rows, np.float64) for _ in range(3)]
    rc = lib().e3o_token_logp_entropy(ptr, dt, C.c_int64(rows), C.c_int64(V), C.c_int64(stride), _p(targets),
                                      _p(mask), _p(temps), C.c_float(temp_scalar), *[_p(o) for o in outs])
    if rc != 0:
        raise ValueError("e3o_token_logp_entropy: invalid argument")
    return tuple(outs)


def row_gap(logits: np.ndarray, temps=None, temp_scalar: float = 1.0, mask=None, greedy: bool = False) -> np.ndarray:
    """Mean logit gap beta * sum_i p_i (z_max - z_i) per row, float64 [rows]."""
    ptr, dt, rows, V, stride = _logits_args(logits)
    mask = None if mask is None else np.ascontiguousarray(mask, dtype=np.uint8)
    temps = None if temps is None else np.ascontiguousarray(temps, dtype=np.float32)
    out = np.empty(rows, np.float64)
    rc = lib().e3o_row_gap(ptr, dt, C.c_int64(rows), C.c_int64(V), C.c_int64(stride), _p(mask), _p(temps),
                           C.c_float(temp_scalar), C.c_int(int(greedy)), _p(out))
    if rc != 0:
        raise ValueError("e3o_row_gap: invalid argument")
    return out


def token_logp_entropy_backward(logits: np.ndarray, targets: np.ndarray, g_logp=None, g_ent=None, mask=None, temps=None,
                                temp_scalar: float = 1.0) -> np.ndarray:
    """Gradient with respect to the logits, float64 [rows, V]."""
    ptr, dt, rows, V, stride = _logits_args(logits)
    targets = np.ascontiguousarray(targets, dtype=np.int32)
    mask = None if mask is None else np.ascontiguousarray(mask, dtype=np.uint8)
    temps = None if temps is None else np.ascontiguousarray(temps, dtype=np.float32)
    g_logp = None if g_logp is None else np.ascontiguousarray(g_logp, dtype=np.float32)
    g_ent = None if g_ent is None else np.ascontiguousarray(g_ent, dtype=np.float32)
    out = np.empty((rows, V), np.float64)
    rc = lib().e3o_token_logp_entropy_backward(ptr, dt, C.c_int64(rows), C.c_int64(V), C.c_int64(stride), _p(targets),
                                               _p(mask), _p(temps), C.c_float(temp_scalar), _p(g_logp), _p(g_ent),
                                               _p(out))
    if rc != 0:
        raise ValueError("e3o_token_logp_entropy_backward: invalid argument")
    return out


def masked_mean_entropy(ent: np.ndarray, mask=None):
    """Returns (mean, count) as Python floats."""
    ent = np.ascontiguousarray(ent, dtype=np.float32)
    mask = None if mask is None else np.ascontiguousarray(mask, dtype=np.uint8)
    mean, cnt = C.c_double(), C.c_double()
    rc = lib().e3o_masked_mean_entropy(_p(ent), _p(mask), C.c_int64(ent.size), C.byref(mean), C.byref(cnt))
    if rc != 0:
        raise ValueError("e3o_masked_mean_entropy: invalid argument")
    return mean.value, cnt.value


def sequence_mean_entropy(ent: np.ndarray, mask=None):
    """Mean over sequences of the per-sequence mean entropy; ent [n_seq, seq_len].  Returns (mean, sequences used)."""
    ent = np.ascontiguousarray(ent, dtype=np.float32)
    assert ent.ndim == 2
    mask = None if mask is None else np.ascontiguousarray(mask, dtype=np.uint8)
    mean, cnt = C.c_double(), C.c_double()
    rc = lib().e3o_sequence_mean_entropy(_p(ent), _p(mask), C.c_int64(ent.shape[0]), C.c_int64(ent.shape[1]),
                                         C.byref(mean), C.byref(cnt))
    if rc != 0:
        raise ValueError("e3o_sequence_mean_entropy: invalid argument")
    return mean.value, cnt.value


def group_advantage(rewards: np.ndarray, group_offsets: np.ndarray, eps: float = 1e-6, unbiased: bool = True):
    """Returns (adv float64 [n], flags uint8 [n_groups])."""
    rewards = np.ascontiguousarray(rewards, dtype=np.float32)
    off = np.ascontiguousarray(group_offsets, dtype=np.int64)
    ng = off.size - 1
    adv = np.zeros(rewards.size, np.float64)
    flags = np.zeros(max(ng, 0), np.uint8)
    rc = lib().e3o_group_advantage(_p(rewards), _p(off), C.c_int64(ng), C.c_float(eps), C.c_int(int(unbiased)),
                                   _p(adv), _p(flags))
    if rc != 0:
        raise ValueError(f"e3o_group_advantage: invalid argument ({rc})")
    return adv, flags


def allocate_budget(k, G: int, G_min: int, G_max: int, greedy_mode: int = 0) -> np.ndarray:
    k = np.ascontiguousarray(k, dtype=np.float64)
    out = np.zeros(k.size, np.int32)
    rc = lib().e3o_allocate_budget(_p(k), C.c_int64(k.size), C.c_int32(G), C.c_int32(G_min), C.c_int32(G_max),
                                   C.c_int(greedy_mode), _p(out))
    if rc == 1:
        raise ValueError("e3o_allocate_budget: invalid argument")
    if rc == 2:
        raise ArithmeticError("e3o_allocate_budget: infeasible")
    return out


def grpo_objective(logp, logp_old, mask, adv, group_offsets, clip_eps: float = 0.2):
    """Returns (J, grad float64 [n_seq, seq_len], clipped fraction).  logp arrays are [n_seq, seq_len]."""
    logp = np.ascontiguousarray(logp, dtype=np.float32)
    logp_old = np.ascontiguousarray(logp_old, dtype=np.float32)
    n_seq, seq_len = logp.shape
    mask = None if mask is None else np.ascontiguousarray(mask, dtype=np.uint8).reshape(n_seq, seq_len)
    adv = np.ascontiguousarray(adv, dtype=np.float32)
    off = np.ascontiguousarray(group_offsets, dtype=np.int64)
    grad = np.empty((n_seq, seq_len), np.float64)
    J, frac = C.c_double(), C.c_double()
    rc = lib().e3o_grpo_objective(_p(logp), _p(logp_old), _p(mask), C.c_int64(n_seq), C.c_int64(seq_len), _p(adv),
                                  _p(off), C.c_int64(off.size - 1), C.c_float(clip_eps), _p(grad), C.byref(J),
                                  C.byref(frac))
    if rc != 0:
        raise ValueError("e3o_grpo_objective: invalid argument")
    return J.value, grad, frac.value


def difficulty_accumulate(n_c: np.ndarray, r_c: np.ndarray, question_ids, G, rewards) -> None:
    """Adds one batch to the cumulative counts (int64) and rewards (float64), in place."""
    assert n_c.dtype == np.int64 and r_c.dtype == np.float64 and n_c.size == r_c.size
    q = np.ascontiguousarray(question_ids, dtype=np.int64)
    g = np.ascontiguousarray(G, dtype=np.int32)
    r = np.ascontiguousarray(rewards, dtype=np.float32)
    assert r.size == int(g.sum())
    rc = lib().e3o_difficulty_accumulate(C.c_int64(n_c.size), _p(n_c), _p(r_c), _p(q), _p(g), _p(r), C.c_int64(q.size))
    if rc != 0:
        raise ValueError("e3o_difficulty_accumulate: invalid argument")


def difficulty_rank(n_c: np.ndarray, r_c: np.ndarray) -> np.ndarray:
    n_c = np.ascontiguousarray(n_c, dtype=np.int64)
    r_c = np.ascontiguousarray(r_c, dtype=np.float64)
    out = np.empty(n_c.size, np.float64)
    rc = lib().e3o_difficulty_rank(C.c_int64(n_c.size), _p(n_c), _p(r_c), _p(out))
    if rc != 0:
        raise ValueError("e3o_difficulty_rank: invalid argument")
    return out


def budget_curriculum(G: int, step: int, G_min_limit: int, G_max_limit: int, epochs_done: int):
    lo, hi = C.c_int32(), C.c_int32()
    rc = lib().e3o_budget_curriculum(C.c_int32(G), C.c_int32(step), C.c_int32(G_min_limit), C.c_int32(G_max_limit),
                                     C.c_int64(epochs_done), C.byref(lo), C.byref(hi))
    if rc != 0:
        raise ValueError("e3o_budget_curriculum: invalid argument")
    return lo.value, hi.value


class Sched(C.Structure):
    _fields_ = [("tau", C.c_double), ("H_init", C.c_double), ("t", C.c_int64), ("t_anneal", C.c_int64),
                ("t_max", C.c_int64), ("eta", C.c_double), ("V", C.c_int64), ("tau_min", C.c_double),
                ("tau_max", C.c_double)]


def make_sched(tau=1.0, H_init=float("nan"), t=0, t_anneal=1 << 62, t_max=1 << 62, eta=0.9, V=151936,
               tau_min=0.0, tau_max=0.0) -> Sched:
    return Sched(tau, H_init, t, t_anneal, t_max, eta, V, tau_min, tau_max)


def anneal_target(s: Sched) -> float:
    return float(lib().e3o_anneal_target(C.byref(s)))


def update_temperature(s: Sched, H_t: float) -> float:
    out = C.c_double()
    rc = lib().e3o_update_temperature(C.byref(s), C.c_double(H_t), C.byref(out))
    if rc != 0:
        raise ValueError("e3o_update_temperature: invalid argument")
    return out.value


def entropy_gap(H: float, N: int) -> float:
    """x = beta * Delta of the two-level model that has entropy H over N entries (root x >= 1)."""
    return float(lib().e3o_entropy_gap(C.c_double(H), C.c_int64(N)))


def update_temperature_gap(s: Sched, H_t: float) -> float:
    out = C.c_double()
    rc = lib().e3o_update_temperature_gap(C.byref(s), C.c_double(H_t), C.byref(out))
    if rc != 0:
        raise ValueError("e3o_update_temperature_gap: invalid argument")
    return out.value

