"""The N > 1 path of bench.py on CPU: two gloo ranks, barrier and max-over-ranks timing, and the
head-independent sharding the path allows (no data-path collective)."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import bench
    r, w, local = bench.dist_setup()
    assert (r, w, local) == (rank, world, rank)
    bench.barrier(w)
    # every rank times its own share; the reported time is the slowest rank's, the work is the sum
    mine = 10.0 + 5.0 * rank
    slowest = bench.reduce_over_ranks(mine, w, torch.device("cpu"))
    total = bench.reduce_over_ranks(mine, w, torch.device("cpu"), "sum")
    assert total == 25.0
    # the path shards by head with no exchange: each rank's oracle result for its own heads equals
    # the single-process result for those heads
    import oracle
    from paper_2608_02504_b200 import workloads
    cfg = workloads.CONFIGS["tiny"]
    heads = list(range(cfg["heads"]))[r::w]        # what `bench.py --shard heads` gives rank r
    Q, K, V = workloads.make_qkv(cfg, "cpu", heads=heads)
    Qf, Kf, Vf = workloads.make_qkv(cfg, "cpu")
    same = all(torch.equal(a[0, i], b[0, h]) for a, b in ((Q, Qf), (K, Kf), (V, Vf)) for i, h in enumerate(heads))
    rows = np.arange(8)
    ref = oracle.attention_rows(workloads.bf16_bits(Q[0, 0]), workloads.bf16_bits(K[0, 0]),
                                workloads.bf16_bits(V[0, 0]), 0.125, rows)
    out[rank] = (slowest, same, float(ref["H_def"].sum()))
    dist.destroy_process_group()


@pytest.mark.timeout(300)
def test_two_gloo_ranks():
    world = 2
    port = 29500 + os.getpid() % 2000
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    assert out[0][0] == out[1][0] == 15.0          # max over ranks, on every rank
    assert out[0][1] and out[1][1]                 # a rank's head subset reproduces the full tensors
    assert out[0][2] != out[1][2]                  # different heads, different data


def test_reference_arm_non_zero_ranks_do_nothing(monkeypatch, capsys):
    sys.path.insert(0, ROOT)
    import bench
    monkeypatch.setenv("RANK", "1")

    class A:
        config, tau, heads, cpu_rows, warmup, steps, gpus, shard = "tiny", None, None, 128, 0, 1, 2, "replicas"
    bench.run_reference(A)
    assert capsys.readouterr().out == ""
