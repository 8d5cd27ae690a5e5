"""Pins of the oracle's placement-constraint check (collocation constraints, Eq. 3; device constraints, Eq. 4):
a worked example, closed forms on the partition p(v) = v mod k, and invariants that a dropped term, a swapped
operand or an off-by-one in the indexing would break; and of its critical-vertex mask (Section 3.2): the critical
sets of the worked DAGs, derived by hand from their edge lists, a chain, and path properties."""
from __future__ import annotations

import numpy as np

import oracle
from helpers import graph_from_edges, load_golden, oracle_graph
from paper_1711_01912_b200 import inputs as I


def _col(p):
    return np.asarray(p, np.uint8).reshape(-1, 1)


def test_worked_example():
    # four vertices, partition [0, 1, 0, 1]
    part = _col([0, 1, 0, 1])
    pairs = [(0, 2), (1, 3), (0, 1)]          # same, same, different: one violated
    devs = [(0, 0), (1, 0), (3, 1), (2, 1)]   # holds, violated, holds, violated
    coll, dev = oracle.eval_constraints(part, pairs, devs)
    assert coll.tolist() == [1] and dev.tolist() == [2]
    # no constraints: nothing to violate
    coll, dev = oracle.eval_constraints(part, np.zeros((0, 2), np.int32), np.zeros((0, 2), np.int32))
    assert coll.tolist() == [0] and dev.tolist() == [0]


def test_closed_forms_on_the_modulo_partition():
    n, k = 60, 4
    v = np.arange(n)
    part = _col(v % k)
    same = np.stack([v[:-k], v[:-k] + k], axis=1)          # (v, v + k): always the same device
    diff = np.stack([v[:-1], v[:-1] + 1], axis=1)          # (v, v + 1): never the same device for k > 1
    coll, _ = oracle.eval_constraints(part, same, [])
    assert coll[0] == 0
    coll, _ = oracle.eval_constraints(part, diff, [])
    assert coll[0] == n - 1
    coll, _ = oracle.eval_constraints(part, np.concatenate([same, diff]), [])
    assert coll[0] == n - 1
    hold = np.stack([v, v % k], axis=1)
    miss = np.stack([v, (v + 1) % k], axis=1)
    _, dev = oracle.eval_constraints(part, [], hold)
    assert dev[0] == 0
    _, dev = oracle.eval_constraints(part, [], miss)
    assert dev[0] == n
    # a vertex listed with two different devices violates exactly one of the two requirements
    _, dev = oracle.eval_constraints(part, [], [(5, 1), (5, 2)])
    assert dev[0] == 1


def test_invariants_on_random_inputs():
    rng = np.random.default_rng(11)
    n, k, P = 200, 7, 25
    part = rng.integers(0, k, size=(n, P), dtype=np.uint8)
    pairs = rng.integers(0, n, size=(300, 2)).astype(np.int32)
    devs = np.stack([rng.integers(0, n, size=150), rng.integers(0, k, size=150)], axis=1).astype(np.int32)
    coll, dev = oracle.eval_constraints(part, pairs, devs)
    # independent count, column by column, with python sets of positions
    for j in range(P):
        p = part[:, j].tolist()
        assert coll[j] == sum(1 for a, b in pairs.tolist() if p[a] != p[b])
        assert dev[j] == sum(1 for v, d in devs.tolist() if p[v] != d)
    # the order of a pair does not matter; (v, v) is never violated; renaming the devices changes no collocation count
    coll2, _ = oracle.eval_constraints(part, pairs[:, ::-1], [])
    assert np.array_equal(coll, coll2)
    loops = np.stack([np.arange(n), np.arange(n)], axis=1)
    assert not oracle.eval_constraints(part, loops, [])[0].any()
    perm = rng.permutation(k).astype(np.uint8)
    coll3, dev3 = oracle.eval_constraints(perm[part], pairs, np.stack([devs[:, 0], perm[devs[:, 1]]], axis=1))
    assert np.array_equal(coll, coll3) and np.array_equal(dev, dev3)
    # everything on one device: no collocation pair is violated, and exactly the device constraints naming another device
    one = np.full((n, 1), 3, np.uint8)
    c1, d1 = oracle.eval_constraints(one, pairs, devs)
    assert c1[0] == 0 and d1[0] == int((devs[:, 1] != 3).sum())
    # selected columns
    c4, d4 = oracle.eval_constraints(part, pairs, devs, cols=[4, 0, 24])
    assert c4.tolist() == coll[[4, 0, 24]].tolist() and d4.tolist() == dev[[4, 0, 24]].tolist()


# ---------------------------------------------------------------------------------------- critical vertices
def test_critical_sets_of_the_worked_dags():
    """Longest paths found by hand from the edge lists and the costs of the worked examples:
    diamond 0->1, 0->2, 1->3, 2->3 with p = [0,1,0,1]: 0->2->3 (16 + 0 + 24 + 2 + 2 = 44), so {0, 2, 3};
    everything on the fast device: 0->1->3 (4 + 8 + 2 = 14), so {0, 1, 3};
    two-sink DAG: the direct edge 0->5 (30 + 75 + 12 = 117), so {0, 5}."""
    gd = load_golden("w1_diamond.json")
    og = oracle_graph(graph_from_edges(gd["n"], gd["edges"], gd["c"]))
    want = {0: {0, 2, 3}, 1: {0, 1, 3}, 2: {0, 2, 3}}
    for i, cs in enumerate(gd["cases"]):
        part = np.asarray(cs["p"], np.uint8).reshape(-1, 1)
        r = oracle.eval_batch(og, gd["k"], gd["s"], np.full(gd["k"], np.iinfo(np.int64).max), np.asarray(cs["B"]), gd["S"], part)
        mask = oracle.critical_mask(r.tlevel, r.blevel, r.cp)
        assert set(np.nonzero(mask[:, 0])[0].tolist()) == want[i], (i, mask[:, 0])
    gd = load_golden("w2_two_sinks.json")
    og = oracle_graph(graph_from_edges(gd["n"], gd["edges"], gd["c"]))
    cs = gd["cases"][0]
    part = np.asarray(cs["p"], np.uint8).reshape(-1, 1)
    r = oracle.eval_batch(og, gd["k"], gd["s"], np.full(gd["k"], np.iinfo(np.int64).max), np.asarray(cs["B"]), gd["S"], part)
    mask = oracle.critical_mask(r.tlevel, r.blevel, r.cp)
    assert set(np.nonzero(mask[:, 0])[0].tolist()) == {0, 5}


def test_critical_mask_properties():
    # a chain: every vertex is critical under every partition
    n = 30
    g = graph_from_edges(n, [(i, i + 1, 1000 + i) for i in range(n - 1)], np.arange(1, n + 1))
    rng = np.random.default_rng(3)
    part = rng.integers(0, 3, size=(n, 9), dtype=np.uint8)
    s, B = [1, 2, 5], np.array([[0, 7, 9], [3, 0, 11], [5, 2, 0]])
    r = oracle.eval_batch(oracle_graph(g), 3, s, np.full(3, np.iinfo(np.int64).max), B, 6, part)
    assert oracle.critical_mask(r.tlevel, r.blevel, r.cp).all()
    # random layered graph: the critical vertices contain a source and a sink, every critical vertex that is not a sink
    # has a critical successor, and no vertex exceeds the critical-path length
    w = I.small_random(55, 120, 400, 4, 12)
    og = oracle_graph(w.graph)
    d = w.devices
    part = w.part_full()
    r = oracle.eval_batch(og, d.k, d.s, d.C, d.B, d.scale, part)
    mask = oracle.critical_mask(r.tlevel, r.blevel, r.cp)
    assert (r.tlevel + r.blevel <= r.cp[None, :]).all()
    c = I.to_csr(w.graph)
    for j in range(part.shape[1]):
        crit = np.nonzero(mask[:, j])[0]
        assert any(c.in_ptr[v] == c.in_ptr[v + 1] for v in crit) and any(c.out_ptr[v] == c.out_ptr[v + 1] for v in crit)
        for v in crit:
            succ = c.out_dst[c.out_ptr[v]:c.out_ptr[v + 1]]
            assert len(succ) == 0 or mask[succ, j].any()
