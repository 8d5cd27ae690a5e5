"""Pins of the oracle's vertex ranks (Eq. 5, Eq. 6), critical path (Section 3.2.2, steps 1-4), Batch Split
(Section 3.2.1) and Critical Path partitioning (Section 3.2.2, Eq. 7): values derived by hand on the two worked DAGs
(tests/golden/ranks_worked.json), every path enumerated on small random DAGs, the single-device evaluation of the same
graph, closed forms (chain, unit memory, equal devices) and invariants a dropped term, a wrong sort direction, a
non-strict capacity test or a swapped operand would break."""
from __future__ import annotations

import numpy as np

import oracle
from helpers import graph_from_edges, load_golden, oracle_graph

INF = np.iinfo(np.int64).max


def _worked(name):
    g = load_golden(name)
    return graph_from_edges(g["n"], g["edges"], g["c"]), g


def _caps(C, k):
    if C == "inf":
        return np.full(k, INF, np.int64)
    return np.array([INF if x == "inf" else x for x in C], np.int64)


def test_hand_values_on_the_worked_dags():
    gold = load_golden("ranks_worked.json")
    for key, name in (("w1", "w1_diamond.json"), ("w2", "w2_two_sinks.json")):
        g, _ = _worked(name)
        og = oracle_graph(g)
        up, down, total = oracle.ranks(og)
        assert up.tolist() == gold[key]["up"]
        assert down.tolist() == gold[key]["down"]
        assert total.tolist() == gold[key]["total"]
        assert oracle.critical_path(og, down).tolist() == gold[key]["path"]


def test_partitioners_on_the_second_worked_dag():
    gold = load_golden("ranks_worked.json")["w2"]
    g, spec = _worked("w2_two_sinks.json")
    og = oracle_graph(g)
    assert og.mem.tolist() == gold["mem"]
    up, down, total = oracle.ranks(og)
    k, s, S = spec["k"], spec["s"], spec["S"]
    for case in gold["batch_split"]:
        part, bad = oracle.batch_split(total, og.mem, k, s, _caps(case["C"], k))
        assert part.tolist() == case["part"] and bad == case["unplaced"], case
    path = oracle.critical_path(og, down)
    for case in gold["cp_partition"]:
        part, bad = oracle.cp_partition(og, path, k, s, _caps(case["C"], k), S)
        assert part.tolist() == case["part"] and bad == case["unplaced"], case


def _random_dag(rng, n, m):
    edges = set()
    while len(edges) < m:
        u, v = sorted(rng.integers(0, n, size=2).tolist())
        if u != v:
            edges.add((u, v))
    perm = rng.permutation(n)    # ids in no topological order
    return [(int(perm[u]), int(perm[v]), int(rng.integers(1, 1000))) for (u, v) in sorted(edges)]


def _all_paths_ranks(n, edges, c):
    """upRank / downRank by enumerating every path (depth-first, python ints)."""
    succ = [[] for _ in range(n)]
    pred = [[] for _ in range(n)]
    for (u, v, _) in edges:
        succ[u].append(v)
        pred[v].append(u)

    def longest(v, nxt):
        best = 0
        for x in nxt[v]:
            best = max(best, longest(x, nxt))
        return best + c[v]

    return [longest(v, succ) for v in range(n)], [longest(v, pred) for v in range(n)]


def test_ranks_against_enumerated_paths_and_single_device_evaluation():
    rng = np.random.default_rng(5)
    for trial in range(12):
        n = int(rng.integers(2, 13))
        edges = _random_dag(rng, n, int(rng.integers(1, min(3 * n, n * (n - 1) // 2) + 1)))
        c = rng.integers(1, 50, size=n)
        g = graph_from_edges(n, edges, c)
        og = oracle_graph(g)
        up, down, total = oracle.ranks(og)
        bu, bd = _all_paths_ranks(n, edges, c.tolist())
        assert up.tolist() == bu and down.tolist() == bd
        assert total.tolist() == [a + b for a, b in zip(bu, bd)]
        # one device of unit speed, one tick per unit: blevel = upRank, tlevel + c = downRank (evaluation pinned elsewhere)
        r = oracle.eval_partition(og, 1, [1], [INF], [[1]], 1, np.zeros(n, np.uint8))
        assert np.array_equal(r.blevel, up) and np.array_equal(r.tlevel + c, down)
        # the critical path: a real path from a source to a sink whose cost is the largest downward rank
        path = oracle.critical_path(og, down).tolist()
        eset = {(u, v) for (u, v, _) in edges}
        assert all((a, b) in eset for a, b in zip(path, path[1:]))
        assert og.in_ptr[path[0] + 1] == og.in_ptr[path[0]] and og.out_ptr[path[-1] + 1] == og.out_ptr[path[-1]]
        assert sum(int(c[v]) for v in path) == int(down.max()) == int(up.max())


def test_chain_closed_form():
    n = 40
    c = np.arange(1, n + 1)
    g = graph_from_edges(n, [(v, v + 1, 7) for v in range(n - 1)], c)
    og = oracle_graph(g)
    up, down, total = oracle.ranks(og)
    assert np.array_equal(down, np.cumsum(c))
    assert np.array_equal(up, np.cumsum(c[::-1])[::-1])
    assert np.array_equal(total, c.sum() + c)          # c_v is in both ranks
    assert oracle.critical_path(og, down).tolist() == list(range(n))


def test_batch_split_closed_forms_and_invariants():
    rng = np.random.default_rng(9)
    n, k = 100, 4
    total = rng.permutation(n).astype(np.int64) * 3 + 5          # distinct ranks
    order = np.argsort(-total)
    s = np.array([2, 9, 4, 7], np.int32)                         # fastest first: 1, 3, 2, 0
    # unbounded capacities: everything on the fastest device
    part, bad = oracle.batch_split(total, np.ones(n, np.int64), k, s, np.full(k, INF, np.int64))
    assert bad == 0 and (part == 1).all()
    # unit memory, room for exactly 10 / 20 / 30 / 40 vertices (usage must stay BELOW capacity): batches by rank
    C = np.array([41, 11, 31, 21], np.int64)
    part, bad = oracle.batch_split(total, np.ones(n, np.int64), k, s, C)
    assert bad == 0
    assert (part[order[:10]] == 1).all() and (part[order[10:30]] == 3).all()
    assert (part[order[30:60]] == 2).all() and (part[order[60:]] == 0).all()
    # equal ranks: ascending vertex id decides
    part, bad = oracle.batch_split(np.full(n, 7, np.int64), np.ones(n, np.int64), k, s, C)
    assert (part[:10] == 1).all() and (part[10:30] == 3).all() and (part[30:60] == 2).all() and (part[60:] == 0).all()
    # equal speeds: the lower device index is the "faster" one
    part, _ = oracle.batch_split(total, np.ones(n, np.int64), 2, [5, 5], [INF, INF])
    assert (part == 0).all()
    # random memory sizes: capacities hold whenever nothing was left over, and a vertex sits on a slower device only
    # if the faster ones were too full for it when its turn came
    mem = rng.integers(1, 100, size=n).astype(np.int64)
    C = np.array([5000, 700, 900, 800], np.int64)
    part, bad = oracle.batch_split(total, mem, k, s, C)
    assert bad == 0
    used = np.zeros(k, np.int64)
    speed_order = [1, 3, 2, 0]
    for v in order:
        for d in speed_order:
            if d == part[v]:
                break
            assert used[d] + mem[v] >= C[d]
        used[part[v]] += mem[v]
        assert used[part[v]] < C[part[v]]


def test_cp_partition_closed_forms_and_invariants():
    n, k, S = 60, 3, 4
    c = np.full(n, 10, np.int32)
    g = graph_from_edges(n, [(0, 1, 1)], c, mem=np.ones(n, np.int64))    # vertices 2.. are isolated
    og = oracle_graph(g)
    _, down, _ = oracle.ranks(og)
    path = oracle.critical_path(og, down)
    assert path.tolist() == [0, 1]
    # equal devices, no capacity limit: the path on device 0 (lowest index among the fastest), the rest dealt to the least
    # loaded device: loads (2, 0, 0) -> 1, 2, 1, 2, 0, 1, 2, 0, ...
    part, bad = oracle.cp_partition(og, path, k, [6, 6, 6], np.full(k, INF, np.int64), S)
    assert bad == 0 and part[:2].tolist() == [0, 0]
    expect = [1, 2, 1, 2] + [(i % 3) for i in range(n - 6)]
    assert part[2:].tolist() == expect
    loads = np.bincount(part, minlength=k)
    assert loads.max() - loads.min() <= 1
    # one device: everything on it
    part, bad = oracle.cp_partition(og, path, 1, [3], [INF], S)
    assert bad == 0 and (part == 0).all()
    # a twice as fast device takes twice as many equal vertices (Eq. 7 balances finish times, not counts)
    g2 = graph_from_edges(n, [], c, mem=np.ones(n, np.int64))
    og2 = oracle_graph(g2)
    part, _ = oracle.cp_partition(og2, np.zeros(0, np.int32), 2, [1, 2], [INF, INF], S)
    cnt = np.bincount(part, minlength=2)
    assert abs(int(cnt[1]) - 2 * int(cnt[0])) <= 2
    # capacity: room for 9 vertices on each device except the last; nothing exceeds it, the last takes the rest
    C = np.array([10, 10, INF], np.int64)
    part, bad = oracle.cp_partition(og, path, k, [6, 6, 6], C, S)
    cnt = np.bincount(part, minlength=k)
    assert bad == 0 and cnt[0] == 9 and cnt[1] == 9 and cnt[2] == n - 18
    # the path is divided when no device holds it: chain of 6 with room for 2 per device
    chain = graph_from_edges(6, [(v, v + 1, 1) for v in range(5)], [5] * 6, mem=np.ones(6, np.int64))
    oc = oracle_graph(chain)
    _, dn, _ = oracle.ranks(oc)
    part, bad = oracle.cp_partition(oc, oracle.critical_path(oc, dn), 3, [1, 3, 2], [3, 3, 3], S)
    assert bad == 0 and part.tolist() == [1, 1, 2, 2, 0, 0]
