"""Host logic of the multi-rank path on CPU: candidate slices and the gather of
per-candidate results over a world-size-2 gloo group."""
from __future__ import annotations

import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_1711_01912_b200 import shard


def test_slices_partition_the_candidates():
    for P in (0, 1, 7, 64, 8191, 16384):
        for world in (1, 2, 3, 8):
            sl = shard.all_slices(P, world)
            assert sl[0][0] == 0 and sl[-1][1] == P
            assert all(a[1] == b[0] for a, b in zip(sl, sl[1:]))
            sizes = [b - a for a, b in sl]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        shard.candidate_slice(10, 2, 2)


def _worker(rank, world, port, P, k, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        j0, j1 = shard.candidate_slice(P, world, rank)
        # every rank derives its slice of a deterministic global result
        cp = torch.arange(P, dtype=torch.int64) * 3 + 1
        load = torch.arange(k * P, dtype=torch.int64).reshape(k, P)
        got = shard.gather_summaries({"cp": cp[j0:j1].clone(), "load": load[:, j0:j1].clone()}, P)
        ok = torch.equal(got["cp"], cp) and torch.equal(got["load"], load)
        q.put((rank, bool(ok)))
    finally:
        dist.destroy_process_group()


def test_gather_over_gloo_world_size_2():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, 101, 3, q)) for r in range(2)]
    for p in procs:
        p.start()
    results = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert sorted(results) == [(0, True), (1, True)]
