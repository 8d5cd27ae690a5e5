"""GPU parity of the rank-driven partitioners against the oracle, through the C ABI: vertex ranks (Eq. 5, Eq. 6), the
critical path (Section 3.2.2), Batch Split (Section 3.2.1) and Critical Path partitioning (Eq. 7) -- every vertex,
bit-exact.  The tie rules (smallest id, lower device index) make every result unique, so whole arrays are compared."""
from __future__ import annotations

import numpy as np
import pytest

from paper_1711_01912_b200 import inputs as I
from helpers import graph_from_edges, load_golden, oracle_graph
from test_gpu_parity import gpu_graph

pytestmark = pytest.mark.gpu

INF = np.iinfo(np.int64).max


def _compare(g, dev, caps_list):
    """Ranks, path and both partitions of graph g under device tables dev, once per capacity vector."""
    import oracle
    og = oracle_graph(g)
    up, down, total = oracle.ranks(og)
    path = oracle.critical_path(og, down)
    for C in caps_list:
        d = I.Devices(dev.k, dev.s, np.asarray(C, np.int64), dev.B, dev.scale)
        G = gpu_graph(g, d)
        gup, gdown, gtotal = G.ranks()
        assert np.array_equal(gup.cpu().numpy(), up)
        assert np.array_equal(gdown.cpu().numpy(), down)
        assert np.array_equal(gtotal.cpu().numpy(), total)
        gpath = G.critical_path(gdown)
        assert np.array_equal(gpath.cpu().numpy(), path)
        part, bad = oracle.batch_split(total, og.mem, d.k, d.s, d.C)
        gpart, gbad = G.batch_split(gtotal)
        assert gbad == bad and np.array_equal(gpart.cpu().numpy(), part)
        part, bad = oracle.cp_partition(og, path, d.k, d.s, d.C, d.scale)
        gpart, gbad = G.cp_partition(gpath)
        assert gbad == bad and np.array_equal(gpart.cpu().numpy(), part)
        G.close()
    return og, total


def test_worked_dags():
    gold = load_golden("ranks_worked.json")["w2"]
    spec = load_golden("w2_two_sinks.json")
    g = graph_from_edges(spec["n"], spec["edges"], spec["c"])
    k = spec["k"]
    dev = I.Devices(k, np.asarray(spec["s"], np.int32), np.full(k, INF, np.int64),
                    np.asarray([[1 if a == b else 100 for b in range(k)] for a in range(k)], np.int64), spec["S"])
    caps = [np.full(k, INF, np.int64)]
    for case in gold["batch_split"] + gold["cp_partition"]:
        if case["C"] != "inf":
            caps.append(np.array([INF if x == "inf" else x for x in case["C"]], np.int64))
    _compare(g, dev, caps)


def test_configs_with_and_without_capacity_pressure():
    for w in (I.config1(), I.config2(), I.small_random(31, 700, 2500, 50, 4, with_mem=True),
              I.small_random(32, 1, 0, 3, 4), I.small_random(33, 300, 0, 5, 4, with_mem=True)):
        g, d = w.graph, w.devices
        og = oracle_graph(g)
        msum = int(og.mem.sum())
        k = d.k
        caps = [np.full(k, INF, np.int64),
                np.full(k, msum // max(1, k - 1) + 1, np.int64),          # tight: most devices fill up
                np.full(k, max(1, msum // (2 * k)), np.int64)]            # too small: some vertices fit nowhere
        rng = np.random.default_rng(k)
        caps.append(rng.integers(max(1, msum // (4 * k)), msum + 2, size=k).astype(np.int64))
        _compare(g, d, caps)


def test_equal_ranks_equal_speeds_and_many_devices():
    rng = np.random.default_rng(8)
    n = 1500
    # all costs equal and no edges: every rank equal, the id decides; 64 devices of two speeds
    g = graph_from_edges(n, [], np.full(n, 9), mem=rng.integers(1, 50, size=n))
    s = np.where(np.arange(64) % 3 == 0, 7, 2).astype(np.int32)
    dev = I.Devices(64, s, np.full(64, INF, np.int64), np.full((64, 64), 10, np.int64), 4)
    msum = int(g.mem.sum())
    _compare(g, dev, [np.full(64, INF, np.int64), np.full(64, msum // 40, np.int64), np.full(64, msum // 80, np.int64)])
    # a deep chain with a hub: long critical path, path divided among the devices when none holds it
    edges = [(v, v + 1, 5) for v in range(n - 1)] + [(v, n - 1, 3) for v in range(0, n - 2, 7)]
    g = graph_from_edges(n, edges, rng.integers(1, 100, size=n), mem=np.ones(n, np.int64))
    dev = I.Devices(5, np.array([3, 9, 9, 1, 4], np.int32), np.full(5, INF, np.int64), np.full((5, 5), 10, np.int64), 16)
    _compare(g, dev, [np.full(5, INF, np.int64), np.full(5, 400, np.int64), np.array([100, 200, 300, 2000, 50], np.int64)])


def test_full_size_config3():
    w = I.config3()
    og = oracle_graph(w.graph)
    msum = int(og.mem.sum())
    k = w.devices.k
    _compare(w.graph, w.devices, [np.full(k, INF, np.int64), np.full(k, msum // (k - 2), np.int64)])
