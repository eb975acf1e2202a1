"""The N > 1 host path (request sharding, barrier, max-over-ranks timing) on two
CPU ranks with the gloo backend.  No GPU is involved."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2511_12280_b200 import replicas as rp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = rp.shard_requests(9, rank, world)
        dist.barrier()
        slow = rp.max_over_ranks(10.0 + rank)                 # rank 1 is the slow one
        tot = rp.sum_over_ranks(float(len(mine)))
        thr = rp.whole_job_steps_per_second([5.0], 2.0 + rank)   # 5 steps each; slowest rank took 3 s
        out[rank] = (mine, slow, tot, thr)
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_and_reduce():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    r0, r1 = out[0], out[1]
    assert r0[0] + r1[0] == list(range(9)) and abs(len(r0[0]) - len(r1[0])) <= 1
    assert r0[1] == r1[1] == 11.0
    assert r0[2] == r1[2] == 9.0
    assert r0[3] == r1[3] == pytest.approx(10.0 / 3.0)


def test_sharding_covers_every_request_once():
    for n in (0, 1, 7, 8, 9, 64):
        for w in (1, 2, 3, 8):
            parts = [rp.shard_requests(n, r, w) for r in range(w)]
            assert sum(parts, []) == list(range(n))
            assert max(map(len, parts)) - min(map(len, parts)) <= 1
    with pytest.raises(ValueError):
        rp.shard_requests(4, 2, 2)


def test_single_process_is_identity():
    assert rp.max_over_ranks(3.5) == 3.5 and rp.sum_over_ranks(2.0) == 2.0
