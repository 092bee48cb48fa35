"""The several-GPU path on CPU: two gloo ranks shard the tokens, each runs the layer on its
rows (here with the CPU oracle standing in for the device library), and the pieces put together
equal the unsharded result bit for bit; the timing reduction returns the slowest rank's time."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2305_10727_b200 import inputs, replicas


def test_shard_rows_partition():
    for M in (1, 2, 7, 197, 12608):
        for world in (1, 2, 3, 8):
            spans = [replicas.shard_rows(M, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == M
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        replicas.shard_rows(10, 2, 2)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        d = inputs.random_layer(5, 301, 128, 64)
        prep = oracle.prepare_weight(d["W"])
        x_scale = np.float32(0.03125)                      # supplied scale: no collective on the data path
        lo, hi = replicas.shard_rows(301, world, rank)
        part = oracle.layer_forward(np.ascontiguousarray(d["X"][lo:hi]), prep, d["bias"], act=1, x_scale=x_scale)
        np.save(os.path.join(out_dir, "y%d.npy" % rank), part["Y"])
        slowest = replicas.max_over_ranks(10.0 + rank, torch.device("cpu"))
        assert slowest == 10.0 + world - 1
        assert replicas.whole_job_throughput(100.0, slowest, world) == world * 100.0 / slowest
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_tokens_without_collective(tmp_path):
    oracle.build()
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    d = inputs.random_layer(5, 301, 128, 64)
    prep = oracle.prepare_weight(d["W"])
    whole = oracle.layer_forward(d["X"], prep, d["bias"], act=1, x_scale=np.float32(0.03125))["Y"]
    parts = np.concatenate([np.load(tmp_path / ("y%d.npy" % r)) for r in range(world)])
    assert np.array_equal(parts.view(np.uint16), whole.view(np.uint16))
