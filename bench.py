#!/usr/bin/env python
"""Benchmark of the vocabulary-side hot path on B200.

One "step" is one pass of the whole path over one synthetic rollout batch shaped like the
paper's (64 prompts x 8 rollouts = 512 rows, V = 151,936, bf16 logits):

    256 decode steps of e3_sample (fused temperature softmax + entropy + log-prob + Gumbel-max
        sample; the logits rotate through a ring of 8 distinct buffers = 1.24 GB, larger than L2,
        the Philox step counter advances every launch)
  + one e3_token_logp_entropy over the ring's 4,096 rows (the training forward of those tokens) with the
    batch entropy fused into the call (sum of entropies and count)
  + e3_group_advantage over the 512 rollouts (64 groups of 8)
  + the host temperature update fed by the mean entropy (16 bytes device -> host).

`value` = logit rows per second over all ranks with the logits resident in HBM; a row counts when its
logits are read (all decode rows, the unmasked rows of the training pass).  `e2e` = the
same step with the logits in pinned HOST memory: every decode step copies its logits host ->
device and its tokens device -> host inside the timed region.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--sampler 0|1] [--impl e3|reference]

The step uses sampler 1 (blocked Gumbel-max) unless told otherwise; `kernels` in the output line
gives the device time of every row kernel alone (both samplers and the training-side pass), timed
with CUDA events over the same ring of logits, `ceiling_read_only_GBps` the rate of a plain read-only
sum kernel over that ring, `configs` the other benchmark configurations (tiny batch, full training pass,
variable budgets, stress rows) and `parity` the comparison of one decode step with the CPU oracle.

Under torchrun (N > 1) every rank runs the same per-GPU batch with its own row_base (weak
scaling; rows are independent, the only exchange is a 16-byte all-reduce of the entropy sum
and count).  `--impl reference` times the fp64 CPU oracle on a bounded sample of the same
workload on the host cores (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

ROWS, V, DECODE_STEPS, RING = 512, 151936, 256, 8
GROUP = 8
METRIC = "logit rows/s, fused sample+entropy, V=151,936"
UNIT = "rows/s"
# dram__bytes_read.sum + dram__bytes_write.sum of one e3_sample launch of this workload (ncu capture summarised in
# profiles/rows_kernel_c2_ncu_full.txt and rows_kernel_sampler0_c2_ncu_full.txt), streaming kernel only.
NCU_TRAFFIC_BYTES = {0: 161.7e6, 1: 160.0e6}
WORKLOAD = "rollout decode step: 512 rows (64 prompts x 8 rollouts) x V=151,936 bf16, 256 decode steps"


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def __exit__(self, *a):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm)}


def cpu_baseline(sampler: int, budget_s: float = 12.0):
    """The oracle as it stands, timed on the host cores on a bounded sample of the workload's rows."""
    import torch
    import oracle
    from paper_2505_18573_b200 import inputs
    oracle.build()
    probe_rows = 16
    logits = inputs.zipf_gaussian_logits(64, V, seed=10, dtype=torch.bfloat16)
    temps = inputs.uniform_temps(64, seed=2).numpy()
    arr = inputs.to_oracle_array(logits)
    t0 = time.perf_counter()
    oracle.sample(arr[:probe_rows], temps[:probe_rows], 0, 0, 0, sampler)
    per_row = (time.perf_counter() - t0) / probe_rows
    n = int(max(64, min(32768, budget_s / max(per_row, 1e-9))))
    reps = (n + 63) // 64
    t0 = time.perf_counter()
    for r in range(reps):
        oracle.sample(arr, temps, 0, r, 0, sampler)
    dt = time.perf_counter() - t0
    rows = reps * 64
    return {"value": rows / dt, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{rows} rows of the workload's logits (64 distinct rows x {reps} step counters), "
                      f"sampler {sampler}, {dt:.1f} s"}


def run_reference(args, rank: int):
    """Reference arm = the CPU oracle (there is no other implementation of the paper's path)."""
    if rank != 0:
        return
    import numpy as np
    import torch
    import oracle
    from paper_2505_18573_b200 import inputs
    oracle.build()
    rows = 256
    logits = inputs.to_oracle_array(inputs.zipf_gaussian_logits(rows, V, seed=10, dtype=torch.bfloat16))
    temps = inputs.uniform_temps(rows, seed=2).numpy()
    for w in range(args.warmup):
        oracle.sample(logits[:16], temps[:16], 0, w, 0, args.sampler)
    times = []
    for k in range(args.steps):
        t0 = time.perf_counter()
        r = oracle.sample(logits, temps, 0, 1000 + k, 0, args.sampler)
        oracle.token_logp_entropy(logits[:8], r.tok[:8], temp_scalar=1.0)
        oracle.masked_mean_entropy(r.ent.astype(np.float32), None)
        oracle.group_advantage((r.tok % 2).astype(np.float32), np.arange(0, rows + 1, GROUP))
        times.append(time.perf_counter() - t0)
    total = sum(times)
    value = (rows + 8) * args.steps / total
    sample = f"{rows} sampled rows + 8 training-side rows of the workload per step (full workload: 135,168 rows)"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "sampler": args.sampler, "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def verified_step(e3, inputs, logits, temps, tok, logp, ent, sampler):
    """One decode launch of the workload against the CPU oracle, row by row."""
    import numpy as np
    import torch
    import oracle
    oracle.build()
    e3.e3_sample(logits, temps, 0, 0, 0, sampler, out_tok=tok, out_logp=logp, out_ent=ent)
    torch.cuda.synchronize()
    ref = oracle.sample(inputs.to_oracle_array(logits), temps.cpu().numpy(), 0, 0, 0, sampler)
    got = tok.cpu().numpy()
    near = (ref.y1 - ref.y2) < 1e-6
    if sampler == 1:
        near = near | (ref.cdf_margin < 1e-6)
    diff = got != ref.tok
    same = ~diff
    return {"rows": int(got.size), "sampler": sampler,
            "mismatches": int((diff & ~near).sum()), "mismatches_on_near_tie_rows": int((diff & near).sum()),
            "near_tie_rows": int(near.sum()),
            "max_err_ent": float(np.nanmax(np.abs(ent.cpu().numpy() - ref.ent))),
            "max_err_logp": float(np.nanmax(np.abs(logp.cpu().numpy()[same] - ref.logp[same]))),
            "tolerance": 2e-3}


def other_configs(e3, inputs, dev, peak, time_alone):
    """Device times of the other configurations (inputs resident, CUDA events); generation time excluded."""
    import torch
    out = {}

    def rate(nbytes, us):
        return {"us": us, "GBps": nbytes / us / 1e3, "frac_of_measured_peak": nbytes / us / 1e3 / peak}

    # c1: 64 rows (8 prompts x 8 rollouts) x 32,000 fp32: 8.2 MB, fits L2, latency-bound
    r, v = 64, 32000
    lg = inputs.zipf_gaussian_logits(r, v, seed=1, dtype=torch.float32, device=dev)
    tp = inputs.uniform_temps(r, seed=2, device=dev)
    rew = inputs.bernoulli_rewards([8] * 8, 0.5, seed=3, device=dev)
    off = inputs.group_offsets([8] * 8, device=dev)
    tok = torch.empty(r, dtype=torch.int32, device=dev); lp = torch.empty(r, device=dev); en = torch.empty(r, device=dev)
    adv = torch.empty(r, device=dev)
    out["c1"] = {"workload": "64 x 32,000 fp32 (8.2 MB, L2-resident: latency-bound)",
                 "e3_sample[sampler 0]_us": time_alone(lambda d: e3.e3_sample(lg, tp, 0, d, 0, 0, out_tok=tok, out_logp=lp, out_ent=en)),
                 "e3_sample[sampler 1]_us": time_alone(lambda d: e3.e3_sample(lg, tp, 0, d, 0, 1, out_tok=tok, out_logp=lp, out_ent=en)),
                 "e3_group_advantage_us": time_alone(lambda d: e3.e3_group_advantage(rew, off, out_adv=adv, want_flags=False))}

    # c4: 256 prompts, budgets from Algorithm 1 (2..32 rollouts, 4,096 rows) x 151,936 bf16
    k = inputs.beta22_difficulty(256, seed=6)
    budgets = e3.e3_allocate_budget(k, 16, 2, 32)
    r, v = sum(budgets), V
    lg = inputs.zipf_gaussian_logits(r, v, seed=40, dtype=torch.bfloat16, device=dev)
    tp = inputs.uniform_temps(r, seed=41, device=dev)
    rew = inputs.bernoulli_rewards(budgets, 1.0 - k, seed=7, device=dev)
    off = inputs.group_offsets(budgets, device=dev)
    tok = torch.empty(r, dtype=torch.int32, device=dev); lp = torch.empty(r, device=dev); en = torch.empty(r, device=dev)
    adv = torch.empty(r, device=dev)
    nb = r * v * 2
    out["c4"] = {"workload": f"{r} rows (256 ragged groups) x 151,936 bf16 (1.24 GB)",
                 "e3_sample[sampler 0]": rate(nb, time_alone(lambda d: e3.e3_sample(lg, tp, 3, d, 0, 0, out_tok=tok, out_logp=lp, out_ent=en), reps=8)),
                 "e3_sample[sampler 1]": rate(nb, time_alone(lambda d: e3.e3_sample(lg, tp, 3, d, 0, 1, out_tok=tok, out_logp=lp, out_ent=en), reps=16)),
                 "e3_group_advantage_us": time_alone(lambda d: e3.e3_group_advantage(rew, off, out_adv=adv, want_flags=False))}
    del lg

    # c5: 4,096 x 256,000 fp32 (4.2 GB); even rows near one-hot, odd rows flat, timed together and apart
    r, v = 4096, 256000
    lg = inputs.onehot_flat_logits(r, v, seed=20, device=dev)
    tp = inputs.loguniform_temps(r, seed=21, device=dev)
    tg = inputs.uniform_targets(r, v, seed=22, device=dev)
    tok = torch.empty(r, dtype=torch.int32, device=dev); lp = torch.empty(r, device=dev); en = torch.empty(r, device=dev)
    c5 = {"workload": "4,096 x 256,000 fp32 (4.2 GB): even rows near one-hot, odd rows flat"}
    for name, sl in (("all_rows", slice(None)), ("one_hot_rows", slice(0, None, 2)), ("flat_rows", slice(1, None, 2))):
        lgs, tps, tgs = lg[sl], tp[sl].contiguous(), tg[sl].contiguous()
        n = lgs.shape[0]
        nb = n * v * 4
        c5[name] = {
            "rows": n,
            "e3_sample[sampler 0]": rate(nb, time_alone(lambda d: e3.e3_sample(lgs, tps, 4, d, 0, 0, out_tok=tok[:n], out_logp=lp[:n], out_ent=en[:n]), reps=4)),
            "e3_sample[sampler 1]": rate(nb, time_alone(lambda d: e3.e3_sample(lgs, tps, 4, d, 0, 1, out_tok=tok[:n], out_logp=lp[:n], out_ent=en[:n]), reps=8)),
            "e3_token_logp_entropy": rate(nb, time_alone(lambda d: e3.e3_token_logp_entropy(lgs, tgs, temps=tps, out_logp=lp[:n], out_ent=en[:n]), reps=8))}
    out["c5"] = c5
    del lg, lgs

    # c3: 64 sequences x 2,048 tokens x 151,936 bf16 (39.8 GB) in one call, response lengths in [256, 2048]
    n_seq, seq_len, v = 64, 2048, V
    r = n_seq * seq_len
    free, _ = torch.cuda.mem_get_info(dev)
    if free < 48 * 2**30:
        out["c3"] = {"skipped": "needs 48 GB of free device memory"}
        return out
    lg = torch.empty((r, v), dtype=torch.bfloat16, device=dev)
    for c in range(r // 8192):
        lg[c * 8192:(c + 1) * 8192] = inputs.zipf_gaussian_logits(8192, v, seed=100 + c, dtype=torch.bfloat16, device=dev)
    tg = inputs.uniform_targets(r, v, seed=4, device=dev)
    mk, lengths = inputs.response_mask(n_seq, seq_len, seed=5, min_len=256, device=dev)
    lp = torch.empty(r, device=dev); en = torch.empty(r, device=dev)
    sm = torch.empty(2, dtype=torch.float64, device=dev)
    us = time_alone(lambda d: e3.e3_token_logp_entropy(lg, tg, mask=mk, temp_scalar=1.0, out_logp=lp, out_ent=en, out_sum=sm), reps=3)
    un = int(lengths.sum().item())
    out["c3"] = {"workload": "131,072 rows (64 x 2,048) x 151,936 bf16 (39.8 GB), mask = first L_s tokens, L_s ~ U{256..2048}",
                 "e3_token_logp_entropy_with_fused_entropy_sum": {
                     "us": us, "rows": r, "unmasked_rows": un, "rows_per_s_all": r / us * 1e6,
                     "rows_per_s_unmasked": un / us * 1e6, "GBps_unmasked_bytes": un * v * 2 / us / 1e3,
                     "frac_of_measured_peak": un * v * 2 / us / 1e3 / peak},
                 "mean_entropy": float(sm[0] / sm[1])}
    del lg
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--sampler", type=int, default=1, choices=[0, 1],
                    help="0 = one Gumbel per vocabulary entry, 1 = one Gumbel per block of 256 entries (default)")
    ap.add_argument("--impl", default="e3", choices=["e3", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true",
                    help="skip the other configurations (c1, c3, c4, c5): a short run, e.g. for a launch list")
    ap.add_argument("--profile-launches", type=int, default=0,
                    help="run this many decode launches plus one training-side launch and exit (for ncu captures)")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist
    from paper_2505_18573_b200 import binding as e3
    from paper_2505_18573_b200 import inputs

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    e3.lib()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    # ---- synthetic batch, resident in HBM --------------------------------------------------------
    row_base = rank * ROWS
    batch = torch.empty((RING * ROWS, V), dtype=torch.bfloat16, device=dev)   # the ring, also the training batch
    ring = [batch[i * ROWS:(i + 1) * ROWS] for i in range(RING)]
    for i in range(RING):
        ring[i].copy_(inputs.zipf_gaussian_logits(ROWS, V, seed=10 + i + 1000 * rank, dtype=torch.bfloat16, device=dev))
    temps = inputs.uniform_temps(ROWS, seed=2 + 1000 * rank, device=dev)
    all_toks = torch.zeros(RING * ROWS, dtype=torch.int32, device=dev)
    toks = [all_toks[i * ROWS:(i + 1) * ROWS] for i in range(RING)]
    sizes = [GROUP] * (ROWS // GROUP)
    rewards = inputs.bernoulli_rewards(sizes, 0.5, seed=3 + rank, device=dev)
    offsets = inputs.group_offsets(sizes, device=dev)
    mask, _ = inputs.response_mask(RING, ROWS, seed=5 + rank, min_len=ROWS // 8, device=dev)
    logp = torch.empty(ROWS, dtype=torch.float32, device=dev)
    ent = torch.empty(ROWS, dtype=torch.float32, device=dev)
    t_logp = torch.empty(RING * ROWS, dtype=torch.float32, device=dev)
    t_ent = torch.empty(RING * ROWS, dtype=torch.float32, device=dev)
    adv = torch.empty(ROWS, dtype=torch.float32, device=dev)
    flags = torch.empty(ROWS // GROUP, dtype=torch.uint8, device=dev)
    mean_out = torch.empty(2, dtype=torch.float64, device=dev)
    ws = torch.empty(e3.e3_workspace_bytes(e3.E3_CALL_MASKED_MEAN_ENTROPY, RING * ROWS), dtype=torch.uint8, device=dev)
    mean_host = torch.empty(2, dtype=torch.float64).pin_memory()
    sched = e3.make_sched(tau=1.0, V=V, t_anneal=288, t_max=480, eta=0.9)
    stream = torch.cuda.current_stream()
    # kernels per step: the blocked sampler is two kernels per call; training pass 1 + 2 (fused sum); advantage 1
    launches_per_step = DECODE_STEPS * (2 if args.sampler == 1 else 1) + 1 + 2 + 1

    def decode_loop(step_index):
        for d in range(DECODE_STEPS):
            b = d % RING
            e3.e3_sample(ring[b], temps, 0, step_index * DECODE_STEPS + d, row_base, args.sampler,
                         out_tok=toks[b], out_logp=logp, out_ent=ent)

    def tail(step_index):
        # the training forward; the sum of entropies and the count come out of the same call
        e3.e3_token_logp_entropy(batch, all_toks, mask=mask, temp_scalar=float(sched.tau),
                                 out_logp=t_logp, out_ent=t_ent, out_sum=mean_out)
        e3.e3_group_advantage(rewards, offsets, out_adv=adv, out_flags=flags)
        if world > 1:
            dist.all_reduce(mean_out)     # the path's only exchange: 16 bytes (sum, count)
        mean_host.copy_(mean_out, non_blocking=True)
        stream.synchronize()
        e3.e3_update_temperature(sched, float(mean_host[0]) / float(mean_host[1]))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    if args.profile_launches > 0:
        for d in range(args.profile_launches):
            e3.e3_sample(ring[d % RING], temps, 0, d, row_base, args.sampler, out_tok=toks[d % RING],
                         out_logp=logp, out_ent=ent)
        for d in range(2):   # the training-side kernel on one ring buffer (512 rows), then on the whole batch
            e3.e3_token_logp_entropy(ring[d], all_toks[:ROWS], temps=temps, out_logp=logp, out_ent=ent)
        e3.e3_token_logp_entropy(batch, all_toks, mask=mask, temp_scalar=1.0, out_logp=t_logp, out_ent=t_ent)
        dz = torch.empty((ROWS, V), dtype=torch.bfloat16, device=dev)
        e3.e3_token_logp_entropy_backward(batch[:ROWS], all_toks[:ROWS], t_logp[:ROWS], t_ent[:ROWS], t_logp[:ROWS],
                                          t_ent[:ROWS], mask=mask[:ROWS], out=dz)
        torch.cuda.synchronize()
        print(json.dumps({"profile_launches": args.profile_launches}), flush=True)
        return

    for w in range(args.warmup):
        decode_loop(w); tail(w)

    # ---- timed region: K steps, logits resident ----------------------------------------------------
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    dec_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    tail_ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    barrier()
    with ClockSampler(local_rank) as clocks:
        ev0.record()
        for k in range(args.steps):
            dec_ev[k][0].record()
            decode_loop(args.warmup + k)
            dec_ev[k][1].record()
            tail(args.warmup + k)
            tail_ev[k].record()
        ev1.record()
        barrier()
    ms_total = ev0.elapsed_time(ev1)
    ms_decode = sum(a.elapsed_time(b) for a, b in dec_ev)
    ms_tail = sum(dec_ev[k][1].elapsed_time(tail_ev[k]) for k in range(args.steps))
    tmax = torch.tensor([ms_total], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
    ms_total_max = float(tmax[0])
    unmasked = int(mask.sum().item())
    rows_per_step = DECODE_STEPS * ROWS + unmasked          # rows whose logits are read
    rows_per_step_all = (DECODE_STEPS + RING) * ROWS        # ... counting the masked training rows too
    value = world * rows_per_step * args.steps / (ms_total_max * 1e-3)

    # ---- end to end: logits in pinned host memory --------------------------------------------------
    e2e = None
    if args.e2e_steps > 0:
        host_ring = [torch.empty((ROWS, V), dtype=torch.bfloat16).pin_memory() for _ in range(RING)]
        for h, d in zip(host_ring, ring):
            h.copy_(d)
        stage = [torch.empty((ROWS, V), dtype=torch.bfloat16, device=dev) for _ in range(2)]
        tok_host = torch.empty((DECODE_STEPS, ROWS), dtype=torch.int32).pin_memory()
        temps_host = temps.cpu().pin_memory()
        torch.cuda.synchronize()

        def e2e_step(step_index):
            tdev = temps_host.to(dev, non_blocking=True)
            for d in range(DECODE_STEPS):
                s = stage[d % 2]
                s.copy_(host_ring[d % RING], non_blocking=True)
                e3.e3_sample(s, tdev, 0, step_index * DECODE_STEPS + d, row_base, args.sampler,
                             out_tok=toks[d % RING], out_logp=logp, out_ent=ent)
                tok_host[d].copy_(toks[d % RING], non_blocking=True)
            for b in range(RING):
                sl = slice(b * ROWS, (b + 1) * ROWS)
                s = stage[b % 2]
                s.copy_(host_ring[b], non_blocking=True)
                e3.e3_token_logp_entropy(s, toks[b], mask=mask[sl], temp_scalar=float(sched.tau),
                                         out_logp=t_logp[sl], out_ent=t_ent[sl])
            e3.e3_masked_mean_entropy(t_ent, mask, out=mean_out, workspace=ws)
            e3.e3_group_advantage(rewards, offsets, out_adv=adv, out_flags=flags)
            mean_host.copy_(mean_out, non_blocking=True)
            stream.synchronize()
            e3.e3_update_temperature(sched, float(mean_host[0]))

        e2e_unmasked = unmasked
        e2e_step(10_000)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for k in range(args.e2e_steps):
            e2e_step(10_001 + k)
        e1.record()
        barrier()
        e2e_ms = torch.tensor([e0.elapsed_time(e1)], dtype=torch.float64, device=dev)
        if world > 1:
            dist.all_reduce(e2e_ms, op=dist.ReduceOp.MAX)
        e2e = {"value": world * rows_per_step * args.e2e_steps / (float(e2e_ms[0]) * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": (DECODE_STEPS + RING) * ROWS * V * 2 + ROWS * 4,
               "rows_per_step": DECODE_STEPS * ROWS + e2e_unmasked,
               "d2h_bytes_per_step": DECODE_STEPS * ROWS * 4 + 16}

    # ---- every row kernel alone (device time, CUDA events, same ring) -------------------------------
    def time_alone(fn, reps=64):
        for d in range(min(RING, max(2, reps // 2))):
            fn(d)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for d in range(reps):
            fn(d)
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) * 1e3 / reps

    targets1 = all_toks[:ROWS]
    alone = {
        "e3_sample[sampler 0]": time_alone(lambda d: e3.e3_sample(ring[d % RING], temps, 0, d, row_base, 0,
                                                                    out_tok=toks[d % RING], out_logp=logp, out_ent=ent)),
        "e3_sample[sampler 1]": time_alone(lambda d: e3.e3_sample(ring[d % RING], temps, 0, d, row_base, 1,
                                                                    out_tok=toks[d % RING], out_logp=logp, out_ent=ent)),
        "e3_token_logp_entropy": time_alone(lambda d: e3.e3_token_logp_entropy(ring[d % RING], targets1, temps=temps,
                                                                                 out_logp=logp, out_ent=ent)),
    }
    # backward of the training-side pass over one ring buffer (reads and writes 155.6 MB each)
    g1 = torch.ones(ROWS, dtype=torch.float32, device=dev)
    dz = torch.empty((ROWS, V), dtype=torch.bfloat16, device=dev)
    e3.e3_token_logp_entropy(ring[0], targets1, temps=temps, out_logp=logp, out_ent=ent)
    bwd_us = time_alone(lambda d: e3.e3_token_logp_entropy_backward(ring[d % RING], targets1, logp, ent, g1, g1,
                                                                    temps=temps, out=dz))

    # GRPO objective over 512 responses x 2,048 tokens (latency-bound: a few bytes per token)
    gl = torch.randn((ROWS, 2048), device=dev) * 0.1 - 1.0
    gmask, _ = inputs.response_mask(ROWS, 2048, seed=9, min_len=256, device=dev)
    gout = torch.empty(2, dtype=torch.float64, device=dev)
    ggrad = torch.empty((ROWS, 2048), dtype=torch.float32, device=dev)
    gws = torch.empty(e3.e3_workspace_bytes(e3.E3_CALL_GRPO_OBJECTIVE, ROWS), dtype=torch.uint8, device=dev)
    grpo_us = time_alone(lambda d: e3.e3_grpo_objective(gl, gl, adv, offsets, mask=gmask, out_g_logp=ggrad, out=gout,
                                                        workspace=gws))

    # ---- practical read-only ceiling: a plain sum kernel over the same ring (and over the whole 1.24 GB) ---------
    probe_scratch = torch.empty(e3.E3_PROBE_SCRATCH_BYTES, dtype=torch.uint8, device=dev)
    probe_us = time_alone(lambda d: e3.e3_probe_read(ring[d % RING], scratch=probe_scratch))
    probe_all_us = time_alone(lambda d: e3.e3_probe_read(batch, scratch=probe_scratch), reps=16)

    configs, parity = None, None
    if rank == 0 and world == 1:
        peak_gbs, _ = _peaks()
        if not args.no_configs:
            configs = other_configs(e3, inputs, dev, peak_gbs, time_alone)
        if not args.no_cpu_baseline:
            parity = verified_step(e3, inputs, ring[0], temps, toks[0], logp, ent, args.sampler)

    if rank == 0:
        peak, peak_kind = _peaks()
        bytes_per_launch = ROWS * V * 2 + ROWS * 4 + ROWS * 12
        launch_s = ms_decode * 1e-3 / (args.steps * DECODE_STEPS)
        achieved = bytes_per_launch / launch_s / 1e9
        train_bytes = unmasked * V * 2
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_total_max / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "logits": "bf16", "arithmetic": "fp32 streaming sums, fp64 row epilogue",
                       "sampler": args.sampler, "rows_per_gpu": ROWS, "V": V,
                       "decode_steps": DECODE_STEPS, "l2": f"ring of {RING} logits buffers (1.24 GB) larger than L2",
                       "step": "256 x e3_sample + e3_token_logp_entropy(4096 rows, fused entropy sum) + group advantage + host tau update",
                       "rows_per_step": rows_per_step, "rows_per_step_with_masked": rows_per_step_all,
                       "value_with_masked_rows": world * rows_per_step_all * args.steps / (ms_total_max * 1e-3),
                       "e2e_steps": args.e2e_steps},
            "roofline": {"bound": "hbm", "kernel": f"rows_kernel (e3_sample, sampler {args.sampler}, bf16)"
                                                   + (" + block_sample_kernel" if args.sampler == 1 else ""),
                         "achieved": achieved, "peak": peak,
                         "peak_kind": peak_kind, "unit": "GB/s", "frac": achieved / peak,
                         "frac_of_measured_peak": achieved / peak, "frac_of_8TBs": achieved / 8000.0,
                         "frac_of_read_only_ceiling": achieved / (ROWS * V * 2 / probe_us / 1e3),
                         "us_per_launch": launch_s * 1e6, "bytes_per_launch": bytes_per_launch,
                         "traffic": NCU_TRAFFIC_BYTES.get(args.sampler)},
            "ceiling_read_only_GBps": ROWS * V * 2 / probe_us / 1e3,
            "ceiling_read_only": {"kernel": "e3_probe_read (plain sum over the logits, four thread blocks per SM)",
                                  "per_ring_buffer_155.6MB": {"us": probe_us, "GBps": ROWS * V * 2 / probe_us / 1e3},
                                  "whole_ring_1.24GB": {"us": probe_all_us, "GBps": RING * ROWS * V * 2 / probe_all_us / 1e3}},
            "training_side": {"ms_per_step": ms_tail / args.steps, "unmasked_rows": unmasked,
                              "GBps_incl_small_kernels_and_sync": train_bytes / (ms_tail * 1e-3 / args.steps) / 1e9},
            "kernels": {k: {"us_per_launch": v, "GBps": bytes_per_launch / v / 1e3,
                            "frac_of_measured_peak": bytes_per_launch / v / 1e3 / peak,
                            "frac_of_8TBs": bytes_per_launch / v / 1e3 / 8000.0}
                        for k, v in alone.items()},
            "grpo_objective": {"kernel": "e3_grpo_objective, 512 responses x 2,048 tokens", "us_per_call": grpo_us},
            "backward": {"kernel": "e3_token_logp_entropy_backward (not part of the step)",
                         "us_per_launch": bwd_us, "GBps_read_plus_write": 2 * ROWS * V * 2 / bwd_us / 1e3,
                         "frac_of_measured_peak": 2 * ROWS * V * 2 / bwd_us / 1e3 / peak},
            "configs": configs,
            "parity": parity,
            "e2e": e2e,
            "gpu_launches": launches_per_step * args.steps,
            "clocks": clocks.summary(),
        }
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(args.sampler)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
