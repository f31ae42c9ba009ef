"""World-size-2 checks of the multi-rank bookkeeping, on CPU ranks over gloo."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import workloads as wl
from paper_2110_09195_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        info = replicas.rank_info()
        assert (info.rank, info.world, info.local_rank) == (rank, world, rank)
        # strong split: the ranks' slices of one batch tile it exactly
        lo, hi = wl.shard_batch(7, rank, world)
        (covered,) = replicas.sum_over_ranks([hi - lo], world)
        # weak scaling: every rank a batch of its own, time = slowest rank
        ms_mine = 2.0 + rank            # rank 1 is the slow one
        value, ms = replicas.job_throughput(64, ms_mine, world)
        mx = replicas.max_over_ranks([ms_mine, -float(rank)], world)
        # the ranks draw different activations for the same layer and the same weights
        shape = wl.get_workload("single16").layers[0]
        seed = wl.layer_seed(0, 0)
        a = wl.draw_activation_bits(shape, 2, seed + 7919 * rank)
        p = wl.draw_layer_params(shape, 5, seed)
        q.put((rank, covered, value, ms, mx, int(a.sum()), int(np.asarray(p.idx_packed, dtype=np.int64).sum())))
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_two_ranks_over_gloo():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=100) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, covered, value, ms, mx, _, _ in got:
        assert covered == 7
        assert ms == 3.0                                   # the slowest rank's time
        assert value == pytest.approx(128 / 3.0e-3)        # both ranks' images over it
        assert mx == [3.0, 0.0]
    assert got[0][5] != got[1][5]      # different activations per rank
    assert got[0][6] == got[1][6]      # the same weights


def test_single_rank_is_identity():
    assert replicas.max_over_ranks([1.5, 2.5], 1) == [1.5, 2.5]
    v, ms = replicas.job_throughput(64, 0.5, 1)
    assert ms == 0.5 and v == pytest.approx(128000.0)
    assert replicas.rank_info({}).world == 1
    with pytest.raises(ValueError):
        replicas.rank_info({"RANK": "2", "WORLD_SIZE": "2"})
    with pytest.raises(ValueError):
        replicas.job_throughput(1, 0.0, 1)
