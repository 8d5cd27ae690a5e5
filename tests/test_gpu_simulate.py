"""GPU parity of the batched list-scheduling simulation (Section 4, criteria 1-6; FIFO, PCT and MSR) against the oracle,
through the C ABI: start time of every vertex and the makespan of every compared candidate, bit-exact."""
from __future__ import annotations

import numpy as np
import pytest

from paper_1711_01912_b200 import inputs as I
from helpers import graph_from_edges, load_golden, oracle_graph
from test_gpu_parity import gpu_graph, padded

pytestmark = pytest.mark.gpu

INF = np.iinfo(np.int64).max


def _compare(g, dev, part, cols=None, pad_fill=0, msr_weights=None):
    """Simulate all candidates on the GPU under the three policies; compare the listed columns (default all)."""
    import oracle
    import torch
    from paper_1711_01912_b200 import tfps
    og = oracle_graph(g)
    G = gpu_graph(g, dev)
    dpart, P, ldp = padded(part, fill=pad_fill)
    out = G.eval_batch(dpart, P)
    cols = list(range(P)) if cols is None else list(cols)
    res = {}
    weights = (1, 1, 1, 5) if msr_weights is None else msr_weights
    tfps.tfps_msr_weights_set(G.handle, *weights)
    for policy in (tfps.SCHED_FIFO, tfps.SCHED_PCT, tfps.SCHED_MSR):
        start, mk = G.simulate(dpart, P, policy, out["blevel"] if policy == tfps.SCHED_PCT else None)
        G.status()
        hs, hm = start.cpu().numpy(), mk.cpu().numpy()
        if ldp > P:
            assert not hs[:, P:].any()   # padding columns are not written
        for j in cols:
            r = oracle.eval_partition(og, dev.k, dev.s, dev.C, dev.B, dev.scale, part[:, j])
            ostart, omk = oracle.simulate(og, dev.k, dev.s, dev.B, dev.scale, part[:, j], policy, r.blevel, weights)
            assert hm[j] == omk, (policy, j)
            assert np.array_equal(hs[:, j], ostart), (policy, j)
        res[policy] = hm
        # no schedule beats the critical path or the busiest device, for every candidate
        cp = out["cp"][:P].cpu().numpy()
        load = out["load"][:, :P].cpu().numpy()
        assert (hm >= cp).all() and (hm >= load.max(axis=0)).all()
    G.close()
    return res


def test_hand_worked_schedule():
    g = load_golden("sim_worked.json")
    G = graph_from_edges(g["n"], g["edges"], g["c"])
    dev = I.Devices(g["k"], np.asarray(g["s"], np.int32), np.full(g["k"], INF, np.int64), np.asarray(g["B"], np.int64), g["S"])
    part = np.repeat(np.asarray(g["p"], np.uint8)[:, None], 5, axis=1)
    res = _compare(G, dev, part)
    from paper_1711_01912_b200 import tfps
    assert (res[tfps.SCHED_FIFO] == g["fifo"]["makespan"]).all() and (res[tfps.SCHED_PCT] == g["pct_policy"]["makespan"]).all()


def test_hand_worked_msr_schedule():
    from paper_1711_01912_b200 import tfps
    g = load_golden("sim_msr_worked.json")
    G = graph_from_edges(g["n"], g["edges"], g["c"])
    dev = I.Devices(g["k"], np.asarray(g["s"], np.int32), np.full(g["k"], INF, np.int64), np.asarray(g["B"], np.int64), g["S"])
    part = np.repeat(np.asarray(g["p"], np.uint8)[:, None], 3, axis=1)
    for case in g["cases"]:
        res = _compare(G, dev, part, msr_weights=tuple(case["weights"]))
        assert (res[tfps.SCHED_MSR] == case["makespan"]).all()


def test_small_configs_every_candidate():
    w = I.config1()
    _compare(w.graph, w.devices, w.part_full(), pad_fill=255)
    w = I.small_random(91, 400, 1500, 50, 37, with_mem=True)     # k = 50: two devices per lane
    _compare(w.graph, w.devices, w.part_full(), pad_fill=255)
    w = I.small_random(92, 1, 0, 2, 3)
    _compare(w.graph, w.devices, w.part_full())
    w = I.small_random(93, 200, 0, 4, 9)                          # no edges at all
    _compare(w.graph, w.devices, w.part_full())


def test_zero_cost_vertices_and_parallel_edges():
    rng = np.random.default_rng(4)
    n, k, P = 120, 3, 40
    edges = []
    for v in range(1, n):
        for u in rng.integers(max(0, v - 9), v, size=int(rng.integers(1, 4))):
            edges.append((int(u), v, int(rng.integers(0, 50))))
    edges += edges[:20]                                           # parallel edges
    c = rng.integers(0, 4, size=n)                                # many vertices of zero execution time
    g = graph_from_edges(n, edges, c)
    dev = I.Devices(k, np.array([1, 2, 5], np.int32), np.full(k, INF, np.int64), rng.integers(1, 9, size=(k, k)).astype(np.int64), 2)
    _compare(g, dev, rng.integers(0, k, size=(n, P), dtype=np.uint8), msr_weights=(3, 0, 2, 7))


def test_config2_sampled_candidates_and_more_candidates_than_warps():
    w = I.config2()
    part = w.part_full()                                          # 4,096 candidates: several per warp
    _compare(w.graph, w.devices, part, cols=[0, 1, 777, 2047, 2048, 4095], pad_fill=255)


def test_ids_out_of_range_are_reported():
    from paper_1711_01912_b200 import tfps
    w = I.config1()
    part = w.part_full().copy()
    part[5, 3] = 200
    G = gpu_graph(w.graph, w.devices)
    dpart, P, ldp = padded(part)
    start, mk = G.simulate(dpart, P, tfps.SCHED_FIFO)
    with pytest.raises(tfps.TfpsError) as ei:
        G.status()
    assert ei.value.code == tfps.ERR_BAD_PARTITION
    assert int(mk[3]) == -1 and int(mk[2]) > 0
    G.close()


def test_degenerate_calls():
    """Empty graph, zero candidates, calls before tfps_devices_set, an unknown policy, bad weights."""
    import torch
    from paper_1711_01912_b200 import tfps
    empty = graph_from_edges(0, [], [])
    dev = I.Devices(2, np.array([1, 2], np.int32), np.full(2, INF, np.int64), np.array([[1, 5], [5, 1]], np.int64), 4)
    G = gpu_graph(empty, dev)
    up, down, total = G.ranks()
    assert up.numel() == 0 and G.critical_path(down).numel() == 0
    part, bad = G.batch_split(total)
    assert part.numel() == 0 and bad == 0
    part, bad = G.cp_partition(torch.zeros(0, dtype=torch.int32, device="cuda"))
    assert part.numel() == 0 and bad == 0
    ids = torch.zeros((0, 16), dtype=torch.uint8, device="cuda")
    _, mk = G.simulate(ids, 5, want_start=False)
    assert mk.tolist() == [0] * 5
    G.close()
    w = I.config1()
    G = gpu_graph(w.graph)                                # devices not set
    dpart, P, ldp = padded(w.part_full())
    up, down, total = G.ranks()                           # ranks need no device tables
    assert int(up.max()) == int(down.max()) > 0
    for call in (lambda: G.batch_split(total), lambda: G.cp_partition(G.critical_path(down)), lambda: G.simulate(dpart, P)):
        with pytest.raises(tfps.TfpsError) as ei:
            call()
        assert ei.value.code == tfps.ERR_STATE
    G.devices_set(w.devices.k, w.devices.s, w.devices.C, w.devices.B, w.devices.scale)
    _, mk = G.simulate(dpart, 0)
    assert mk.numel() == 0
    with pytest.raises(tfps.TfpsError) as ei:
        G.simulate(dpart, P, policy=7)
    assert ei.value.code == tfps.ERR_INVALID_ARG
    with pytest.raises(tfps.TfpsError) as ei:
        G.simulate(dpart, P, policy=tfps.SCHED_PCT)       # PCT without the path computation times
    assert ei.value.code == tfps.ERR_INVALID_ARG
    with pytest.raises(tfps.TfpsError) as ei:
        tfps.tfps_msr_weights_set(G.handle, 1, -1, 1, 5)
    assert ei.value.code == tfps.ERR_INVALID_ARG
    G.close()
