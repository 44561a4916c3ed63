"""Thin ctypes binding of ``libe3.so`` (declared in ``include/e3.h``).

Argument marshalling only: every step of the path runs in the CUDA library.  Device calls take
``torch`` CUDA tensors (used for their memory and stream, nothing else), pass raw pointers and
sizes through the C ABI and return the output tensors.  There is no CPU fallback: if the library
has not been built, or a tensor is not on a CUDA device, the call raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libe3.so")

E3_OK = 0
E3_ERR_INVALID_ARG, E3_ERR_DTYPE, E3_ERR_ALIGNMENT, E3_ERR_WORKSPACE, E3_ERR_INFEASIBLE, E3_ERR_CUDA, E3_ERR_TIMEOUT = 1, 2, 3, 4, 5, 6, 7
E3_STATUS_TIMEOUT = 1
E3_F32, E3_BF16 = 0, 1
E3_SAMPLER_TOKEN, E3_SAMPLER_BLOCK, E3_SAMPLER_TOKEN_AUDIT = 0, 1, 2
E3_CALL_SAMPLE, E3_CALL_TOKEN_LOGP_ENTROPY, E3_CALL_MASKED_MEAN_ENTROPY, E3_CALL_GRPO_OBJECTIVE = 0, 1, 2, 3
E3_CALL_SEQUENCE_MEAN_ENTROPY = 4
E3_SAMPLE_BLOCK = 256

EXPORTS = ("e3_status_string", "e3_workspace_bytes", "e3_sample", "e3_token_logp_entropy",
           "e3_token_logp_entropy_backward", "e3_grpo_objective",
           "e3_masked_mean_entropy", "e3_masked_mean_entropy_static", "e3_group_advantage", "e3_allocate_budget", "e3_update_temperature",
           "e3_anneal_target", "e3_entropy_gap", "e3_update_temperature_gap", "e3_difficulty_accumulate", "e3_difficulty_rank", "e3_budget_curriculum",
           "e3_test_arm_stall", "e3_probe_read", "e3_sequence_mean_entropy")


class E3Error(RuntimeError):
    def __init__(self, call: str, status: int):
        self.status = status
        super().__init__(f"{call} failed: {status_string(status)} ({status})")


class e3_sched(C.Structure):
    """Mirror of the C struct ``e3_sched``."""
    _fields_ = [("tau", C.c_double), ("H_init", C.c_double), ("t", C.c_int64), ("t_anneal", C.c_int64),
                ("t_max", C.c_int64), ("eta", C.c_double), ("V", C.c_int64), ("tau_min", C.c_double),
                ("tau_max", C.c_double)]


_lib = None


def lib() -> C.CDLL:
    """The loaded library; raises if it has not been built (no fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2505_18573_b200.build`")
        L = C.CDLL(LIB_PATH)
        L.e3_status_string.restype = C.c_char_p
        L.e3_status_string.argtypes = [C.c_int]
        L.e3_workspace_bytes.restype = C.c_size_t
        L.e3_workspace_bytes.argtypes = [C.c_int, C.c_int64, C.c_int64, C.c_int]
        L.e3_sample.restype = C.c_int
        L.e3_sample.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_uint64,
                                C.c_uint64, C.c_int64, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.e3_token_logp_entropy.restype = C.c_int
        L.e3_token_logp_entropy.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_int64, C.c_void_p,
                                            C.c_void_p, C.c_void_p, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p,
                                            C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.e3_token_logp_entropy_backward.restype = C.c_int
        L.e3_token_logp_entropy_backward.argtypes = [C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_int64, C.c_void_p,
                                                     C.c_void_p, C.c_void_p, C.c_float, C.c_void_p, C.c_void_p,
                                                     C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]
        L.e3_masked_mean_entropy.restype = C.c_int
        L.e3_masked_mean_entropy.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p,
                                             C.c_size_t, C.c_void_p]
        L.e3_sequence_mean_entropy.restype = C.c_int
        L.e3_sequence_mean_entropy.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p,
                                               C.c_void_p, C.c_size_t, C.c_void_p]
        L.e3_masked_mean_entropy_static.restype = C.c_int
        L.e3_masked_mean_entropy_static.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p,
                                                    C.c_void_p]
        L.e3_group_advantage.restype = C.c_int
        L.e3_group_advantage.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_float, C.c_int, C.c_void_p,
                                         C.c_void_p, C.c_void_p]
        L.e3_allocate_budget.restype = C.c_int
        L.e3_allocate_budget.argtypes = [C.c_void_p, C.c_int64, C.c_int32, C.c_int32, C.c_int32, C.c_int, C.c_void_p]
        L.e3_update_temperature.restype = C.c_int
        L.e3_update_temperature.argtypes = [C.POINTER(e3_sched), C.c_double, C.POINTER(C.c_double)]
        L.e3_update_temperature_gap.restype = C.c_int
        L.e3_update_temperature_gap.argtypes = [C.POINTER(e3_sched), C.c_double, C.POINTER(C.c_double)]
        L.e3_entropy_gap.restype = C.c_double
        L.e3_entropy_gap.argtypes = [C.c_double, C.c_int64]
        L.e3_grpo_objective.restype = C.c_int
        L.e3_grpo_objective.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p,
                                        C.c_int64, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t,
                                        C.c_void_p]
        L.e3_difficulty_accumulate.restype = C.c_int
        L.e3_difficulty_accumulate.argtypes = [C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                               C.c_int64]
        L.e3_difficulty_rank.restype = C.c_int
        L.e3_difficulty_rank.argtypes = [C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p]
        L.e3_budget_curriculum.restype = C.c_int
        L.e3_budget_curriculum.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int64,
                                           C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        L.e3_anneal_target.restype = C.c_double
        L.e3_anneal_target.argtypes = [C.POINTER(e3_sched)]
        L.e3_probe_read.restype = C.c_int
        L.e3_probe_read.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p, C.c_size_t, C.c_void_p]
        L.e3_test_arm_stall.restype = None
        L.e3_test_arm_stall.argtypes = [C.c_int64, C.c_uint64]
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().e3_status_string(int(status)).decode()


def _check(call: str, status: int) -> None:
    if status != E3_OK:
        raise E3Error(call, status)


def _dev(t, name: str):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor (there is no CPU path)")
    return t


def _ptr(t) -> int | None:
    return None if t is None else t.data_ptr()


def _stream(stream) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def _logits_desc(logits: torch.Tensor):
    _dev(logits, "logits")
    if logits.dim() != 2 or (logits.shape[1] > 1 and logits.stride(1) != 1):
        raise ValueError("logits must be 2-D with a contiguous last dimension")
    if logits.dtype == torch.float32:
        dt = E3_F32
    elif logits.dtype == torch.bfloat16:
        dt = E3_BF16
    else:
        raise ValueError("logits must be float32 or bfloat16")
    rows, V = logits.shape
    stride = logits.stride(0) if rows > 1 else max(V, logits.stride(0))
    return dt, rows, V, stride


def e3_workspace_bytes(which: int, rows: int, V: int = 0, dt: int = E3_F32) -> int:
    return int(lib().e3_workspace_bytes(which, rows, V, dt))


_row_workspaces = {}


def _row_workspace(device, stream_handle: int, which: int, rows: int, V: int, dt: int):
    """Scratch for the row kernels, one buffer per (device, stream): calls that may overlap on the GPU
    must not share a workspace.  Callers that manage memory themselves pass ``workspace=`` instead."""
    key = (device.index, stream_handle)
    need = e3_workspace_bytes(which, rows, V, dt)
    ws = _row_workspaces.get(key)
    if ws is None or ws.numel() < need:
        ws = torch.empty(max(need, 16), dtype=torch.uint8, device=device)
        _row_workspaces[key] = ws
    return ws


def _status_word(status):
    if status is not None and (not status.is_cuda or status.dtype != torch.int32 or status.numel() < 1):
        raise ValueError("status must be an int32 CUDA tensor")
    return status


def e3_sample(logits, temps, seed: int, counter: int, row_base: int = 0, sampler: int = E3_SAMPLER_TOKEN,
              out_tok=None, out_logp=None, out_ent=None, want_logp: bool = True, want_ent: bool = True,
              out_gap=None, want_gap: bool = False, status=None, workspace=None, stream=None):
    """Rollout step: returns (tok int32, logp float32 | None, ent float32 | None), each [rows]; with
    ``want_gap`` or ``out_gap`` a fourth element, the mean logit gap float32 [rows].  ``status``: optional
    int32 CUDA tensor, the device status word (E3_STATUS_TIMEOUT is OR-ed in, never cleared)."""
    dt, rows, V, stride = _logits_desc(logits)
    _dev(temps, "temps")
    if temps.dtype != torch.float32 or temps.numel() != rows or not temps.is_contiguous():
        raise ValueError("temps must be a contiguous float32 tensor with one entry per row")
    dev = logits.device
    if out_tok is None:
        out_tok = torch.empty(rows, dtype=torch.int32, device=dev)
    if out_logp is None and want_logp:
        out_logp = torch.empty(rows, dtype=torch.float32, device=dev)
    if out_ent is None and want_ent:
        out_ent = torch.empty(rows, dtype=torch.float32, device=dev)
    if out_gap is None and want_gap:
        out_gap = torch.empty(rows, dtype=torch.float32, device=dev)
    sh = _stream(stream)
    if workspace is None:
        workspace = _row_workspace(dev, sh, E3_CALL_SAMPLE, rows, V, dt)
    st = lib().e3_sample(_ptr(logits), dt, rows, V, stride, _ptr(temps), seed, counter, row_base, sampler,
                         _ptr(out_tok), _ptr(out_logp), _ptr(out_ent), _ptr(out_gap), _ptr(_status_word(status)),
                         _ptr(workspace), workspace.numel() * workspace.element_size(), sh)
    _check("e3_sample", st)
    if out_gap is not None:
        return out_tok, out_logp, out_ent, out_gap
    return out_tok, out_logp, out_ent


def e3_token_logp_entropy(logits, targets, mask=None, temps=None, temp_scalar: float = 1.0, out_logp=None,
                          out_ent=None, out_gap=None, want_gap: bool = False, out_sum=None, status=None,
                          workspace=None, stream=None):
    """Training-side pass: returns (logp float32, ent float32), each [rows]; masked rows give 0.  With
    ``want_gap`` or ``out_gap`` a third element, the mean logit gap float32 [rows].  ``out_sum``: optional
    float64 CUDA tensor [2] that receives (sum of entropies over unmasked rows, their number), the fused
    batch entropy.  ``status``: optional int32 CUDA tensor, the device status word."""
    dt, rows, V, stride = _logits_desc(logits)
    _dev(targets, "targets"); _dev(mask, "mask"); _dev(temps, "temps")
    if targets.dtype != torch.int32 or targets.numel() != rows:
        raise ValueError("targets must be int32 with one entry per row")
    if mask is not None and (mask.dtype != torch.uint8 or mask.numel() != rows):
        raise ValueError("mask must be uint8 with one entry per row")
    if temps is not None and (temps.dtype != torch.float32 or temps.numel() != rows):
        raise ValueError("temps must be float32 with one entry per row")
    dev = logits.device
    if out_logp is None:
        out_logp = torch.empty(rows, dtype=torch.float32, device=dev)
    if out_ent is None:
        out_ent = torch.empty(rows, dtype=torch.float32, device=dev)
    if out_gap is None and want_gap:
        out_gap = torch.empty(rows, dtype=torch.float32, device=dev)
    if out_sum is not None and (not out_sum.is_cuda or out_sum.dtype != torch.float64 or out_sum.numel() != 2
                                or not out_sum.is_contiguous()):
        raise ValueError("out_sum must be a contiguous float64 CUDA tensor with two entries")
    sh = _stream(stream)
    if workspace is None:
        workspace = _row_workspace(dev, sh, E3_CALL_TOKEN_LOGP_ENTROPY, rows, V, dt)
    sum_ptr = None if out_sum is None else out_sum.data_ptr()
    st = lib().e3_token_logp_entropy(_ptr(logits), dt, rows, V, stride, _ptr(targets), _ptr(mask), _ptr(temps),
                                     float(temp_scalar), _ptr(out_logp), _ptr(out_ent), _ptr(out_gap), sum_ptr,
                                     None if sum_ptr is None else sum_ptr + 8, _ptr(_status_word(status)),
                                     _ptr(workspace), workspace.numel() * workspace.element_size(), sh)
    _check("e3_token_logp_entropy", st)
    if out_gap is not None:
        return out_logp, out_ent, out_gap
    return out_logp, out_ent


def e3_token_logp_entropy_backward(logits, targets, logp, ent, g_logp=None, g_ent=None, mask=None, temps=None,
                                   temp_scalar: float = 1.0, out=None, stream=None):
    """Gradient of the training-side outputs with respect to the logits: tensor like ``logits``."""
    dt, rows, V, stride = _logits_desc(logits)
    for name, t in (("targets", targets), ("logp", logp), ("ent", ent), ("g_logp", g_logp), ("g_ent", g_ent),
                    ("mask", mask), ("temps", temps)):
        _dev(t, name)
        if t is not None and (t.numel() != rows or not t.is_contiguous()):
            raise ValueError(f"{name} must be contiguous with one entry per row")
    if targets.dtype != torch.int32 or logp.dtype != torch.float32 or ent.dtype != torch.float32:
        raise ValueError("targets must be int32, logp and ent float32")
    if out is None:
        out = torch.empty((rows, V), dtype=logits.dtype, device=logits.device)
    _, orows, oV, ostride = _logits_desc(out)
    if out.dtype != logits.dtype or orows != rows or oV != V:
        raise ValueError("out must have the shape and dtype of logits")
    st = lib().e3_token_logp_entropy_backward(_ptr(logits), dt, rows, V, stride, _ptr(targets), _ptr(mask), _ptr(temps),
                                              float(temp_scalar), _ptr(logp), _ptr(ent), _ptr(g_logp), _ptr(g_ent),
                                              _ptr(out), ostride, _stream(stream))
    _check("e3_token_logp_entropy_backward", st)
    return out


def e3_masked_mean_entropy(ent, mask=None, out=None, workspace=None, stream=None):
    """Returns a float64 CUDA tensor [2] = (mean, count).  No host synchronisation."""
    _dev(ent, "ent"); _dev(mask, "mask")
    if ent.dtype != torch.float32 or not ent.is_contiguous():
        raise ValueError("ent must be a contiguous float32 tensor")
    n = ent.numel()
    if mask is not None and (mask.dtype != torch.uint8 or mask.numel() != n):
        raise ValueError("mask must be uint8 with one entry per token")
    if out is None:
        out = torch.empty(2, dtype=torch.float64, device=ent.device)
    need = e3_workspace_bytes(E3_CALL_MASKED_MEAN_ENTROPY, n)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=ent.device)
    st = lib().e3_masked_mean_entropy(_ptr(ent), _ptr(mask), n, out.data_ptr(), out.data_ptr() + 8,
                                      _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream))
    _check("e3_masked_mean_entropy", st)
    return out


def e3_sequence_mean_entropy(ent, mask=None, out=None, workspace=None, stream=None):
    """Mean over sequences of the per-sequence mean entropy; ``ent`` (and ``mask``) are [n_seq, seq_len].
    Returns a float64 CUDA tensor [2] = (mean, number of sequences with a token)."""
    _dev(ent, "ent"); _dev(mask, "mask")
    if ent.dim() != 2 or ent.dtype != torch.float32 or not ent.is_contiguous():
        raise ValueError("ent must be a contiguous float32 tensor [n_seq, seq_len]")
    n_seq, seq_len = ent.shape
    if mask is not None and (mask.dtype != torch.uint8 or mask.numel() != ent.numel() or not mask.is_contiguous()):
        raise ValueError("mask must be contiguous uint8 with one entry per token")
    if out is None:
        out = torch.empty(2, dtype=torch.float64, device=ent.device)
    if workspace is None:
        workspace = torch.empty(e3_workspace_bytes(E3_CALL_SEQUENCE_MEAN_ENTROPY, n_seq), dtype=torch.uint8,
                                device=ent.device)
    st = lib().e3_sequence_mean_entropy(_ptr(ent), _ptr(mask), n_seq, seq_len, out.data_ptr(), out.data_ptr() + 8,
                                        _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream))
    _check("e3_sequence_mean_entropy", st)
    return out


E3_STATIC_MEAN_MAX_TOKENS = 1 << 26


def e3_masked_mean_entropy_static(ent, mask=None, out=None, stream=None):
    """Mean entropy without any scratch buffer from the caller (for code that may not allocate
    device memory: plugins inside another engine's stream, fixed-pool or real-time processes).
    The partial sums use a 16 KiB array built into the library, shared by every call on the
    device, so calls must not overlap on the GPU.  ``out`` (float64 CUDA tensor [2] = mean, count)
    must be passed by callers that really cannot allocate; when omitted it is created here with
    torch for convenience.  Raises E3Error(E3_ERR_WORKSPACE) above E3_STATIC_MEAN_MAX_TOKENS."""
    _dev(ent, "ent"); _dev(mask, "mask")
    if ent.dtype != torch.float32 or not ent.is_contiguous():
        raise ValueError("ent must be a contiguous float32 tensor")
    n = ent.numel()
    if mask is not None and (mask.dtype != torch.uint8 or mask.numel() != n):
        raise ValueError("mask must be uint8 with one entry per token")
    if out is None:
        out = torch.empty(2, dtype=torch.float64, device=ent.device)
    st = lib().e3_masked_mean_entropy_static(_ptr(ent), _ptr(mask), n, out.data_ptr(), out.data_ptr() + 8,
                                             _stream(stream))
    _check("e3_masked_mean_entropy_static", st)
    return out


def e3_group_advantage(rewards, group_offsets, eps: float = 1e-6, unbiased: bool = True, out_adv=None,
                       out_flags=None, want_flags: bool = True, stream=None):
    """Returns (adv float32 [n], flags uint8 [n_groups] | None)."""
    _dev(rewards, "rewards"); _dev(group_offsets, "group_offsets")
    if rewards.dtype != torch.float32 or group_offsets.dtype != torch.int64:
        raise ValueError("rewards must be float32 and group_offsets int64")
    ng = group_offsets.numel() - 1
    if out_adv is None:
        out_adv = torch.zeros_like(rewards)
    if out_flags is None and want_flags:
        out_flags = torch.zeros(max(ng, 0), dtype=torch.uint8, device=rewards.device)
    st = lib().e3_group_advantage(_ptr(rewards), _ptr(group_offsets), ng, float(eps), int(bool(unbiased)),
                                  _ptr(out_adv), _ptr(out_flags), _stream(stream))
    _check("e3_group_advantage", st)
    return out_adv, out_flags


def e3_grpo_objective(logp, logp_old, adv, group_offsets, mask=None, clip_eps: float = 0.2, out_g_logp=None,
                      want_grad: bool = True, out=None, workspace=None, stream=None):
    """GRPO objective over tokens laid out [n_seq, seq_len].  Returns (out float64 CUDA [2] = (J, clipped
    fraction), g_logp float32 [n_seq, seq_len] | None)."""
    for name, t in (("logp", logp), ("logp_old", logp_old), ("adv", adv), ("group_offsets", group_offsets), ("mask", mask)):
        _dev(t, name)
    if logp.dim() != 2 or logp.shape != logp_old.shape or not logp.is_contiguous() or not logp_old.is_contiguous():
        raise ValueError("logp and logp_old must be contiguous [n_seq, seq_len] tensors of the same shape")
    if logp.dtype != torch.float32 or logp_old.dtype != torch.float32 or adv.dtype != torch.float32:
        raise ValueError("logp, logp_old and adv must be float32")
    n_seq, seq_len = logp.shape
    if adv.numel() != n_seq or group_offsets.dtype != torch.int64:
        raise ValueError("adv needs one entry per response, group_offsets must be int64")
    if mask is not None and (mask.dtype != torch.uint8 or mask.numel() != n_seq * seq_len or not mask.is_contiguous()):
        raise ValueError("mask must be contiguous uint8 with one entry per token")
    if out_g_logp is None and want_grad:
        out_g_logp = torch.empty((n_seq, seq_len), dtype=torch.float32, device=logp.device)
    if out is None:
        out = torch.empty(2, dtype=torch.float64, device=logp.device)
    need = e3_workspace_bytes(E3_CALL_GRPO_OBJECTIVE, n_seq)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=logp.device)
    st = lib().e3_grpo_objective(_ptr(logp), _ptr(logp_old), _ptr(mask), n_seq, seq_len, _ptr(adv), _ptr(group_offsets),
                                 group_offsets.numel() - 1, float(clip_eps), _ptr(out_g_logp), out.data_ptr(),
                                 out.data_ptr() + 8, _ptr(workspace), workspace.numel(), _stream(stream))
    _check("e3_grpo_objective", st)
    return out, out_g_logp


def e3_allocate_budget(k, G: int, G_min: int, G_max: int, greedy_mode: int = 0):
    """Algorithm 1 on the host: list of per-question rollout counts."""
    B = len(k)
    karr = (C.c_double * max(B, 1))(*[float(x) for x in k])
    out = (C.c_int32 * max(B, 1))()
    st = lib().e3_allocate_budget(karr, B, G, G_min, G_max, greedy_mode, out)
    _check("e3_allocate_budget", st)
    return [int(out[i]) for i in range(B)]


def make_sched(tau: float = 1.0, H_init: float = float("nan"), t: int = 0, t_anneal: int = 1 << 62,
               t_max: int = 1 << 62, eta: float = 0.9, V: int = 151936, tau_min: float = 0.0,
               tau_max: float = 0.0) -> e3_sched:
    return e3_sched(tau, H_init, t, t_anneal, t_max, eta, V, tau_min, tau_max)


def e3_update_temperature(s: e3_sched, H_t: float) -> float:
    out = C.c_double()
    st = lib().e3_update_temperature(C.byref(s), float(H_t), C.byref(out))
    _check("e3_update_temperature", st)
    return out.value


def e3_update_temperature_gap(s: e3_sched, H_t: float) -> float:
    out = C.c_double()
    st = lib().e3_update_temperature_gap(C.byref(s), float(H_t), C.byref(out))
    _check("e3_update_temperature_gap", st)
    return out.value


def e3_entropy_gap(H: float, N: int) -> float:
    return lib().e3_entropy_gap(float(H), int(N))


def e3_anneal_target(s: e3_sched) -> float:
    return float(lib().e3_anneal_target(C.byref(s)))


def e3_difficulty_accumulate(n_c, r_c, question_ids, G, rewards) -> None:
    """Adds one batch to the caller's cumulative counts (numpy int64) and rewards (numpy float64), in place."""
    import numpy as np
    if n_c.dtype != np.int64 or r_c.dtype != np.float64 or n_c.size != r_c.size:
        raise ValueError("n_c must be int64 and r_c float64, one entry per question")
    q = np.ascontiguousarray(question_ids, dtype=np.int64)
    g = np.ascontiguousarray(G, dtype=np.int32)
    r = np.ascontiguousarray(rewards, dtype=np.float32)
    if g.size != q.size or r.size != int(g.sum()):
        raise ValueError("one G per question id and sum(G) rewards are needed")
    st = lib().e3_difficulty_accumulate(n_c.size, n_c.ctypes.data, r_c.ctypes.data, q.ctypes.data, g.ctypes.data,
                                        r.ctypes.data, q.size)
    _check("e3_difficulty_accumulate", st)


def e3_difficulty_rank(n_c, r_c):
    """Normalised difficulty ranks k (numpy float64, one per question) from the cumulative statistics."""
    import numpy as np
    n = np.ascontiguousarray(n_c, dtype=np.int64)
    r = np.ascontiguousarray(r_c, dtype=np.float64)
    out = np.empty(n.size, np.float64)
    st = lib().e3_difficulty_rank(n.size, n.ctypes.data, r.ctypes.data, out.ctypes.data)
    _check("e3_difficulty_rank", st)
    return out


def e3_budget_curriculum(G: int, step: int, G_min_limit: int, G_max_limit: int, epochs_done: int):
    """(G_min, G_max) after ``epochs_done`` finished iterations over the dataset."""
    lo, hi = C.c_int32(), C.c_int32()
    st = lib().e3_budget_curriculum(G, step, G_min_limit, G_max_limit, epochs_done, C.byref(lo), C.byref(hi))
    _check("e3_budget_curriculum", st)
    return lo.value, hi.value



def e3_test_arm_stall(tile: int, wait_ns: int) -> None:
    """Test hook: the next row call leaves one 4 KiB tile uncopied and bounds its waits by ``wait_ns``."""
    lib().e3_test_arm_stall(int(tile), int(wait_ns))


E3_PROBE_SCRATCH_BYTES = 65536


def e3_probe_read(buf, scratch=None, stream=None):
    """Measurement aid: one read-only pass over ``buf`` (a CUDA tensor whose size is a multiple of 16 bytes)."""
    _dev(buf, "buf")
    if scratch is None:
        scratch = torch.empty(E3_PROBE_SCRATCH_BYTES, dtype=torch.uint8, device=buf.device)
    st = lib().e3_probe_read(_ptr(buf), buf.numel() * buf.element_size(), _ptr(scratch),
                             scratch.numel() * scratch.element_size(), _stream(stream))
    _check("e3_probe_read", st)
    return scratch
