"""The N>1 path of the benchmark on CPU: two gloo ranks, barrier + max-over-ranks timing protocol,
disjoint replica seeds per rank."""

import os
import socket

import pytest
import torch
import torch.multiprocessing as mp

from paper_2609_36222_b200 import multi


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist = multi.init_process_group("gloo")
    assert multi.env_ranks() == (rank, world, rank)
    multi.barrier(dist)
    slowest = multi.max_over_ranks(10.0 + 5.0 * rank, dist)
    ids = multi.replica_layer_ids(rank, 3)
    gathered = [None] * world
    dist.all_gather_object(gathered, ids)
    multi.barrier(dist)
    out[rank] = (slowest, gathered)
    dist.destroy_process_group()


def test_two_rank_timing_protocol_and_disjoint_replicas():
    world, port = 2, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for rank in (0, 1):
        slowest, gathered = res[rank]
        assert slowest == 15.0                      # every rank sees the slowest rank's time
        flat = [i for ids in gathered for i in ids]
        assert len(flat) == len(set(flat)) == 6     # no weight replica is shared between ranks
    assert multi.whole_job_us_per_step(0.08, 2) == pytest.approx(40.0)


def test_single_process_defaults(monkeypatch):
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        monkeypatch.delenv(k, raising=False)
    assert multi.env_ranks() == (0, 1, 0)
    assert multi.init_process_group("gloo") is None
    assert multi.max_over_ranks(3.5, None) == 3.5
    assert multi.replica_layer_ids(2, 2) == [2000, 2001]
