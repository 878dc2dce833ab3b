"""The multi-rank part of the benchmark on CPU: two gloo ranks reduce their timings and counts the way bench.py
does for N GPUs (slowest rank's time, tokens and frames summed), and draw different batches."""
import os
import sys

import numpy as np
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    from paper_2503_05931_b200 import workloads as wl
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = wl.make_workload("cfg2", seed=bench.rank_seed("cfg2", rank), with_weights=False, with_enc=False)
    ms = 100.0 + 50.0 * rank
    total_ms, tok, frames = bench.reduce_over_ranks(ms, float(w.dec_lens.sum()), float(w.enc_lens.sum()), "cpu", world)
    out[rank] = (total_ms, tok, frames, int(w.dec_lens.sum()), int(w.enc_lens.sum()))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reduce_like_the_benchmark():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, 29611, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    tok_sum = res[0][3] + res[1][3]
    frame_sum = res[0][4] + res[1][4]
    assert res[0][3] != res[1][3]                       # different batches per rank
    for r in (0, 1):
        assert res[r][0] == 150.0                       # the slowest rank sets the time
        assert res[r][1] == tok_sum and res[r][2] == frame_sum


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_over_ranks(12.5, 3.0, 4.0, "cpu", 1) == (12.5, 3.0, 4.0)
    assert bench.rank_seed("cfg2", 0) != bench.rank_seed("cfg2", 1)
