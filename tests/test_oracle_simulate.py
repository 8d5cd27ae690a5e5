"""Pins of the oracle's list-scheduling simulation (Section 4, criteria 1-6; FIFO and PCT policies): a schedule worked
by hand (tests/golden/sim_worked.json), a tick-by-tick simulation written independently, closed forms (one device, one
device per vertex, independent vertices) and the invariants the criteria state, checked on the produced schedule."""
from __future__ import annotations

import numpy as np

import oracle
from helpers import cdiv, graph_from_edges, load_golden, oracle_graph

INF = np.iinfo(np.int64).max


def _evaluate(og, k, s, B, S, p):
    return oracle.eval_partition(og, k, s, [INF] * k, B, S, np.asarray(p, np.uint8))


def test_hand_worked_schedule():
    g = load_golden("sim_worked.json")
    G = graph_from_edges(g["n"], g["edges"], g["c"])
    og = oracle_graph(G)
    r = _evaluate(og, g["k"], g["s"], g["B"], g["S"], g["p"])
    assert r.blevel.tolist() == g["pct"]
    start, mk = oracle.simulate(og, g["k"], g["s"], g["B"], g["S"], g["p"], 0)
    assert start.tolist() == g["fifo"]["start"] and mk == g["fifo"]["makespan"]
    start, mk = oracle.simulate(og, g["k"], g["s"], g["B"], g["S"], g["p"], 1, r.blevel)
    assert start.tolist() == g["pct_policy"]["start"] and mk == g["pct_policy"]["makespan"]


def test_hand_worked_msr_schedule():
    g = load_golden("sim_msr_worked.json")
    og = oracle_graph(graph_from_edges(g["n"], g["edges"], g["c"]))
    for case in g["cases"]:
        start, mk = oracle.simulate(og, g["k"], g["s"], g["B"], g["S"], g["p"], 2, None, case["weights"])
        assert start.tolist() == case["start"] and mk == case["makespan"], case


def _tick_simulation(n, edges, c, k, s, B, S, p, policy, prio, weights=(1, 1, 1, 5)):
    """The same rules, one tick at a time (python ints): at every tick first the executions that end are completed,
    then idle devices pick; repeated within the tick while zero-length executions keep ending."""
    rt = [cdiv(c[v] * S, s[p[v]]) for v in range(n)]
    succ = [[] for _ in range(n)]
    left = [0] * n
    for (u, v, t) in edges:
        succ[u].append((v, 0 if p[u] == p[v] else cdiv(t * S, B[p[u]][p[v]])))
        left[v] += 1
    indeg = list(left)
    out = [[] for _ in range(n)]
    for (u, v, t) in edges:
        out[u].append(v)
    ready = [0] * n
    known = [left[v] == 0 for v in range(n)]
    started = [False] * n
    start = [0] * n
    running = [None] * k
    done = 0
    T = 0
    last = 0
    while done < n:
        changed = True
        while changed:
            changed = False
            for d in range(k):
                if running[d] is not None and running[d][1] == T:
                    u = running[d][0]
                    running[d] = None
                    done += 1
                    last = max(last, T)
                    changed = True
                    for (x, w) in succ[u]:
                        ready[x] = max(ready[x], T + w)
                        left[x] -= 1
                        if left[x] == 0:
                            known[x] = True
            idle = [running[d] is None for d in range(k)]          # as the devices stand before anybody starts

            def msr(v):
                a, b, g_, dl = weights
                return sum(a + b * (p[x] != p[v]) + g_ * (indeg[x] == 1) + dl * (idle[p[x]] and indeg[x] == 1) for x in out[v])

            for d in range(k):
                if running[d] is None:
                    cand = [v for v in range(n) if p[v] == d and known[v] and not started[v] and ready[v] <= T]
                    if cand:
                        key = ((lambda v: (ready[v], v)) if policy == 0 else (lambda v: (-prio[v], v)) if policy == 1
                               else (lambda v: (-msr(v), v)))
                        v = min(cand, key=key)
                        started[v] = True
                        start[v] = T
                        running[d] = (v, T + rt[v])
                        changed = changed or rt[v] == 0
        T += 1
    return start, last


def _random_instance(rng, n, m, k, zero_cost=False):
    edges = set()
    while len(edges) < m:
        u, v = sorted(rng.integers(0, n, size=2).tolist())
        if u != v:
            edges.add((u, v))
    perm = rng.permutation(n)
    edges = [(int(perm[u]), int(perm[v]), int(rng.integers(0, 6))) for (u, v) in sorted(edges)]
    c = rng.integers(0 if zero_cost else 1, 6, size=n)
    s = rng.integers(1, 4, size=k)
    B = rng.integers(1, 4, size=(k, k))
    p = rng.integers(0, k, size=n)
    return edges, c, s, B, p


def test_against_tick_by_tick_simulation():
    rng = np.random.default_rng(17)
    for trial in range(30):
        n = int(rng.integers(1, 16))
        k = int(rng.integers(1, 5))
        m = int(rng.integers(0, min(3 * n, n * (n - 1) // 2) + 1))
        edges, c, s, B, p = _random_instance(rng, n, m, k, zero_cost=trial % 3 == 0)
        S = int(rng.integers(1, 4))
        og = oracle_graph(graph_from_edges(n, edges, c))
        r = _evaluate(og, k, s, B, S, p)
        weights = [int(x) for x in rng.integers(0, 6, size=4)]
        for policy in (0, 1, 2):
            start, mk = oracle.simulate(og, k, s, B, S, p, policy, r.blevel, weights)
            ts, tm = _tick_simulation(n, edges, c.tolist(), k, s.tolist(), B.tolist(), S, p.tolist(), policy, r.blevel.tolist(),
                                      weights)
            assert start.tolist() == ts and mk == tm, (trial, policy)


def test_closed_forms():
    rng = np.random.default_rng(3)
    # one device: never idle, makespan = sum of execution times, whatever the policy
    n = 40
    edges, c, _, _, _ = _random_instance(rng, n, 70, 1)
    og = oracle_graph(graph_from_edges(n, edges, c))
    p = np.zeros(n, np.uint8)
    r = _evaluate(og, 1, [2], [[1]], 4, p)
    for policy in (0, 1):
        start, mk = oracle.simulate(og, 1, [2], [[1]], 4, p, policy, r.blevel)
        assert mk == sum(cdiv(int(x) * 4, 2) for x in c)
        order = np.argsort(start, kind="stable")                        # back to back in the order they ran
        assert start[order].tolist() == np.concatenate([[0], np.cumsum(cdiv_vec(c, 4, 2)[order])[:-1]]).tolist()
    # one device per vertex: nothing ever waits for a device, start = earliest start of the evaluation, makespan = CP
    n, k = 30, 30
    edges, c, s, B, _ = _random_instance(rng, n, 60, k)
    og = oracle_graph(graph_from_edges(n, edges, c))
    p = np.arange(n, dtype=np.uint8)
    r = _evaluate(og, k, s, B, 3, p)
    for policy in (0, 1):
        start, mk = oracle.simulate(og, k, s, B, 3, p, policy, r.blevel)
        assert np.array_equal(start, r.tlevel) and mk == r.cp
    # independent vertices on one device: FIFO runs them by id, PCT by descending execution time (equal: by id)
    c = np.array([3, 9, 3, 7, 1, 9])
    og = oracle_graph(graph_from_edges(6, [], c))
    p = np.zeros(6, np.uint8)
    r = _evaluate(og, 1, [1], [[1]], 1, p)
    start, mk = oracle.simulate(og, 1, [1], [[1]], 1, p, 0)
    assert start.tolist() == [0, 3, 12, 15, 22, 23] and mk == 32
    start, mk = oracle.simulate(og, 1, [1], [[1]], 1, p, 1, r.blevel)
    assert start.tolist() == [25, 0, 28, 18, 31, 9] and mk == 32


def cdiv_vec(c, S, s):
    return np.array([cdiv(int(x) * S, s) for x in c])


def test_criteria_hold_on_the_schedule():
    rng = np.random.default_rng(23)
    for trial in range(8):
        n, k = 300, int(rng.integers(2, 9))
        edges, c, s, B, p = _random_instance(rng, n, 700, k)
        S = 5
        og = oracle_graph(graph_from_edges(n, edges, c))
        r = _evaluate(og, k, s, B, S, p)
        rt = np.array([cdiv(int(c[v]) * S, int(s[p[v]])) for v in range(n)])
        for policy in (0, 1, 2):
            start, mk = oracle.simulate(og, k, s, B, S, p, policy, r.blevel)
            fin = start + rt
            assert mk == fin.max()
            assert mk >= r.cp and mk >= r.load.max()                     # no schedule beats the critical path or a device's load
            ready = np.zeros(n, np.int64)
            for (u, v, t) in edges:                                      # criterion 4
                w = 0 if p[u] == p[v] else cdiv(t * S, int(B[p[u]][p[v]]))
                ready[v] = max(ready[v], fin[u] + w)
            assert (start >= ready).all()
            for d in range(k):
                on = np.nonzero(p == d)[0]
                o = on[np.argsort(start[on], kind="stable")]
                assert (start[o][1:] >= fin[o][:-1]).all()               # criteria 2 and 3: one at a time, no interruption
                # criterion 6 and its converse: while a vertex waits although executable, its device is busy
                busy = [(int(start[v]), int(fin[v])) for v in o]
                for v in on:
                    t = int(ready[v])
                    for (a, b) in busy:
                        if a <= t < b:
                            t = b
                    assert t >= start[v], (trial, policy, v)
