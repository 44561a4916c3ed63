"""The row-sharded (data-parallel) use of the path on two ranks, on CPU with the gloo backend.

The path shards by rows with no data-path exchange: every rank draws with the same seed and step counter
and passes the index of its first row (row_base), so the draws equal those of one process over the whole
batch; the only exchange is the 16-byte all-reduce of (entropy sum, token count) behind the batch mean.
The ranks run the oracle (there is no GPU here); the CUDA path takes the same row_base argument and is
checked against the oracle, split batches included, in the GPU tests."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out_dir):
    import sys
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import oracle
    from paper_2505_18573_b200 import inputs
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    rows, V = 24, 3000
    logits = inputs.zipf_gaussian_logits(rows, V, seed=1).numpy()      # every rank builds the whole batch ...
    temps = inputs.uniform_temps(rows, seed=2).numpy()
    mask = (np.arange(rows) % 5 != 0).astype(np.uint8)
    lo, hi = rank * rows // world, (rank + 1) * rows // world          # ... and works on its own rows
    r = oracle.sample(logits[lo:hi], temps[lo:hi], 9, 4, row_base=lo)
    ent32 = r.ent.astype(np.float32)
    mean, cnt = oracle.masked_mean_entropy(ent32, mask[lo:hi])
    red = torch.tensor([0.0 if cnt == 0 else mean * cnt, cnt], dtype=torch.float64)
    dist.all_reduce(red)
    gathered = [None] * world
    dist.all_gather_object(gathered, (r.tok, ent32))
    if rank == 0:
        whole = oracle.sample(logits, temps, 9, 4, row_base=0)
        tok = np.concatenate([g[0] for g in gathered])
        ent = np.concatenate([g[1] for g in gathered])
        gmean, gcnt = oracle.masked_mean_entropy(whole.ent.astype(np.float32), mask)
        np.save(os.path.join(out_dir, "ok.npy"),
                np.array([np.array_equal(tok, whole.tok), np.array_equal(ent, whole.ent.astype(np.float32)),
                          float(red[1]) == gcnt, abs(float(red[0] / red[1]) - gmean) < 1e-12]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_draw_the_same_tokens_as_one_and_reduce_the_batch_mean(tmp_path):
    import oracle
    oracle.build()   # before the ranks start, so that they only load the library
    port = _free_port()
    mp.spawn(_rank_main, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    ok = np.load(tmp_path / "ok.npy")
    assert ok.all(), ok
