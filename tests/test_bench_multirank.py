"""The benchmark's multi-rank arithmetic on CPU: two gloo ranks, timings reduced to the slowest rank, whole-job
throughput = replicas x per-replica work / slowest time.  (The op shards over batch and head with no exchange,
so ranks are independent replicas; there is no data-path collective to test.)"""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = [10.0 + 5.0 * rank, 100.0 - 30.0 * rank]          # rank 1 is slower on the first, rank 0 on the second
    got = bench.max_over_ranks(mine, dist, torch.device("cpu"))
    dist.barrier()
    dist.destroy_process_group()
    out[rank] = got


def test_two_gloo_ranks_report_the_slowest_rank():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    assert out[0] == [15.0, 100.0] and out[1] == [15.0, 100.0]


def test_single_process_and_aggregate_value():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5], None, None) == [1.5, 2.5]
    # 4 replicas, 10 units each per step, slowest step 2 ms -> 20000 units/s
    assert bench.whole_job_value(10.0, 4, 2.0) == 20000.0


def test_effective_pairs_count_what_survives_the_padding_mask():
    """bench.py's effective FLOP count against the oracle's token-level mask: a (query block, key block) pair of the
    layout counts if some valid query row of the block attends some valid key of the key block."""
    sys.path.insert(0, ROOT)
    import numpy as np
    import bench
    import paper_2007_14062_b200 as bb
    from paper_2007_14062_b200 import synth
    from oracle import bigbird_oracle as O
    wl = synth.Workload("eff", "bf16", 3, 2, 10 * 64, 64, 64, 3, 2, 3, 0, seed=5, lengths="ragged:64:640")
    L = bb.bigbird_build_layout(wl.N, wl.b, wl.w, wl.g, wl.r, wl.seed, wl.H, wl.mode)
    kpm = synth.key_padding_mask(wl)
    kpm[1, 130:] = 0                                            # a length that is not a multiple of the block size
    kpm[1, :130] = 1
    got = bench.effective_pairs(L, wl, kpm)
    gr = O.Graph(wl.N, wl.b, wl.w, wl.g, wl.r, wl.seed, wl.H, wl.mode)
    want = 0
    nb = wl.N // wl.b
    for h in range(wl.H):
        A = O.build_mask(gr, h)                                 # [N, N] 0/1, token level
        for bi in range(wl.B):
            valid = kpm[bi].numpy() != 0
            M = A.astype(bool) & valid[:, None] & valid[None, :]
            want += int(M.reshape(nb, wl.b, nb, wl.b).any(axis=(1, 3)).sum())
    assert got == want
    assert bench.effective_pairs(L, wl, None) == wl.B * bench.counted_pairs(L)
    L.close()
