"""Pins for the CPU oracle against things other than itself: hand-computed
worked DAGs (tests/golden), brute-force path enumeration, library longest-path
routines, the unit-cost setting of Lemma 1, closed forms, the exact-rational
real-valued model, and invariants.  CPU only."""
from __future__ import annotations

import itertools
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_1711_01912_b200 import inputs as I
from helpers import brute_force, cdiv, graph_from_edges, load_golden, oracle_graph, real_valued

INF = np.iinfo(np.int64).max


def run(g, k, s, C, B, S, p):
    og = oracle_graph(g)
    return og, oracle.eval_partition(og, k, s, C, B, S, np.asarray(p, np.uint8))


# ---------------------------------------------------------------- worked DAGs
@pytest.mark.parametrize("fname", ["w1_diamond.json", "w2_two_sinks.json"])
def test_worked_examples(fname):
    w = load_golden(fname)
    g = graph_from_edges(w["n"], w["edges"], w["c"])
    for case in w["cases"]:
        k = w["k"]
        C = case.get("C", [INF] * k)
        og, r = run(g, k, w["s"], C, case["B"], w["S"], case["p"])
        assert og.level.tolist() == w["level"], case["name"]
        if "num_levels" in w:
            assert og.num_levels == w["num_levels"]
        assert r.tlevel.tolist() == case["tlevel"], case["name"]
        assert r.blevel.tolist() == case["blevel"], case["name"]
        assert r.cp == case["cp"], case["name"]
        assert r.load.tolist() == case["load"], case["name"]
        if "memload" in case:
            assert og.mem.tolist() == case["mem"]
            assert r.memload.tolist() == case["memload"]
            assert r.viol == case["viol"]


def test_capacity_inequality_is_strict():
    # Eq. 2 demands usage < C: exactly at capacity is a violation, one below is not
    w = load_golden("w2_two_sinks.json")
    case = w["cases"][0]
    g = graph_from_edges(w["n"], w["edges"], w["c"])
    _, r = run(g, 3, w["s"], [3101, 1700, 1251], case["B"], w["S"], case["p"])
    assert r.viol == 0b010
    _, r = run(g, 3, w["s"], [INF, INF, INF], case["B"], w["S"], case["p"])
    assert r.viol == 0


# ---------------------------------------------------------------- brute force
def _tiny_cases():
    rng = np.random.default_rng(11)
    for trial in range(60):
        n = int(rng.integers(1, 13))
        k = int(rng.integers(1, 5))
        pairs = [(u, v) for u in range(n) for v in range(u + 1, n)]
        keep = rng.random(len(pairs)) < rng.uniform(0.1, 0.6)
        edges = [(u, v, int(rng.integers(0, 5000))) for (u, v), kp in zip(pairs, keep) if kp]
        if trial % 7 == 0 and edges:
            edges.append(edges[0])  # parallel edge, max semantics
        relab = rng.permutation(n)
        edges = [(int(relab[u]), int(relab[v]), t) for (u, v, t) in edges]
        c = rng.integers(0, 50, size=n)
        s = rng.integers(1, 9, size=k)
        B = rng.integers(1, 400, size=(k, k))
        S = int(rng.integers(1, 20))
        p = rng.integers(0, k, size=n)
        yield n, k, edges, c, s, B, S, p


def test_brute_force_all_paths():
    for n, k, edges, c, s, B, S, p in _tiny_cases():
        g = graph_from_edges(n, edges, c)
        _, r = run(g, k, s, [INF] * k, B, S, p)
        tl, bl, cp = brute_force(n, edges, c.tolist(), s.tolist(), B.tolist(), S, p.tolist())
        assert r.tlevel.tolist() == tl
        assert r.blevel.tolist() == bl
        assert r.cp == cp


# ------------------------------------------------- single device vs libraries
def test_single_device_equals_library_longest_path():
    nx = pytest.importorskip("networkx")
    for seed in range(6):
        w = I.small_random(seed, 200 + 37 * seed, 500 + 90 * seed, 3, 1)
        g = w.graph
        for d in range(3):
            sd = int(w.devices.s[d])
            for S in (sd, 16):
                _, r = run(g, 3, w.devices.s, [INF] * 3, w.devices.B, S, np.full(g.n, d))
                rt = [cdiv(int(cv) * S, sd) for cv in g.c]
                G = nx.DiGraph()
                G.add_nodes_from(range(g.n))
                G.add_node("sink")
                for u, v in zip(g.src.tolist(), g.dst.tolist()):
                    G.add_edge(u, v, weight=rt[u])
                for v in range(g.n):
                    G.add_edge(v, "sink", weight=rt[v])
                assert r.cp == nx.dag_longest_path_length(G, weight="weight")
                if S == sd:  # pure computational complexity: max upRank of Eq. 5
                    assert rt == g.c.tolist()


def test_single_device_against_scipy_shortest_path_on_negated_weights():
    sp = pytest.importorskip("scipy.sparse")
    csg = pytest.importorskip("scipy.sparse.csgraph")
    w = I.small_random(3, 150, 400, 2, 1)
    g = w.graph
    S = 16
    og, r = run(g, 2, w.devices.s, [INF] * 2, w.devices.B, S, np.zeros(g.n))
    rt = [cdiv(int(cv) * S, int(w.devices.s[0])) for cv in g.c]
    # edge (u->v) weighs -(rt[u]*big + 1): the +1 keeps zero-cost edges stored in the sparse
    # matrix and is removed again by the floor division (a path has fewer than big edges)
    big = 10 ** 6
    pairs = sorted(set(zip(g.src.tolist(), g.dst.tolist())))
    rows = [u for u, _ in pairs]
    cols = [v for _, v in pairs]
    vals = [-(rt[u] * big + 1.0) for u in rows]
    A = sp.csr_matrix((vals, (rows, cols)), shape=(g.n, g.n))
    sources = [int(v) for v in np.nonzero(og.level == 0)[0]]
    D = csg.bellman_ford(A, directed=True, indices=sources)
    longest = (-D).max(axis=0)  # unreachable = -inf, own source = 0
    tl = np.floor(longest / big).astype(np.int64)
    assert tl.tolist() == r.tlevel.tolist()


# ------------------------------------------------------- Lemma 1 unit setting
def test_unit_cost_setting_ties_levels_to_paths():
    nx = pytest.importorskip("networkx")
    for seed in range(5):
        w = I.small_random(100 + seed, 300, 700, 1, 1)
        g = w.graph
        g = I.Graph(n=g.n, src=g.src, dst=g.dst, t=np.zeros_like(g.t), c=np.ones(g.n, np.int32), mem=None, layers=0)
        og, r = run(g, 1, [1], [INF], [[0]], 1, np.zeros(g.n))
        assert r.tlevel.tolist() == og.level.tolist()
        assert r.cp == og.num_levels
        G = nx.DiGraph()
        G.add_nodes_from(range(g.n))
        G.add_edges_from(zip(g.src.tolist(), g.dst.tolist()))
        gens = list(nx.topological_generations(G))
        assert len(gens) == og.num_levels
        for l, gen in enumerate(gens):
            assert sorted(gen) == og.order[og.level_ptr[l]:og.level_ptr[l + 1]].tolist()
        # height(v)+1 = number of vertices on the longest path starting at v
        Gr = G.reverse()
        for l, gen in enumerate(nx.topological_generations(Gr)):
            for v in gen:
                assert r.blevel[v] == l + 1


def test_cycle_is_reported():
    g = graph_from_edges(3, [(0, 1, 1), (1, 2, 1), (2, 0, 1)], [1, 1, 1])
    with pytest.raises(oracle.OracleError) as ei:
        oracle_graph(g)
    assert ei.value.code == oracle.CYCLE
    g = graph_from_edges(2, [(0, 0, 1)], [1, 1])
    with pytest.raises(oracle.OracleError):
        oracle_graph(g)


# ----------------------------------------------------------------- closed forms
def test_chain_closed_form():
    n, S = 9, 6
    c = np.arange(1, n + 1)
    t = [100 * (i + 1) for i in range(n - 1)]
    edges = [(i, i + 1, t[i]) for i in range(n - 1)]
    s = [2, 3]
    B = [[0, 7], [11, 0]]
    p = [i % 2 for i in range(n)]
    g = graph_from_edges(n, edges, c)
    _, r = run(g, 2, s, [INF, INF], B, S, p)
    rt = [cdiv(int(c[i]) * S, s[p[i]]) for i in range(n)]
    w = [cdiv(t[i] * S, B[p[i]][p[i + 1]]) for i in range(n - 1)]
    assert r.cp == sum(rt) + sum(w)
    assert r.tlevel.tolist() == [sum(rt[:i]) + sum(w[:i]) for i in range(n)]
    assert r.blevel.tolist() == [sum(rt[i:]) + sum(w[i:]) for i in range(n)]


def test_fork_join_closed_form():
    q, S = 5, 4
    c = [3] + [10 + i for i in range(q)] + [7]
    edges = [(0, 1 + i, 50 + i) for i in range(q)] + [(1 + i, q + 1, 80 - i) for i in range(q)]
    s = [1, 2, 4]
    B = [[0, 5, 9], [6, 0, 3], [4, 8, 0]]
    p = [0] + [i % 3 for i in range(q)] + [2]
    g = graph_from_edges(q + 2, edges, c)
    _, r = run(g, 3, s, [INF] * 3, B, S, p)
    rt = [cdiv(c[v] * S, s[p[v]]) for v in range(q + 2)]
    w = lambda u, v, t: 0 if p[u] == p[v] else cdiv(t * S, B[p[u]][p[v]])
    arms = [w(0, 1 + i, 50 + i) + rt[1 + i] + w(1 + i, q + 1, 80 - i) for i in range(q)]
    assert r.cp == rt[0] + max(arms) + rt[q + 1]
    assert r.tlevel[q + 1] == rt[0] + max(arms)
    assert r.blevel[0] == r.cp


def test_complete_layered_single_device_closed_form():
    layers, width = 5, 4
    rng = np.random.default_rng(5)
    c = rng.integers(1, 30, size=layers * width)
    edges = [(l * width + i, (l + 1) * width + j, 1) for l in range(layers - 1) for i in range(width) for j in range(width)]
    g = graph_from_edges(layers * width, edges, c)
    _, r = run(g, 1, [1], [INF], [[0]], 1, np.zeros(layers * width))
    assert r.cp == sum(int(c[l * width:(l + 1) * width].max()) for l in range(layers))


# ----------------------------------------------------- real-valued error bound
def test_integer_ticks_never_underestimate_and_stay_within_bound():
    for seed in range(8):
        w = I.small_random(40 + seed, 40, 90, 3, 1)
        g = w.graph
        d = w.devices
        p = np.random.default_rng(seed).integers(0, 3, size=g.n)
        for S in (1, 16, 1000):
            _, r = run(g, 3, d.s, [INF] * 3, d.B, S, p)
            edges = list(zip(g.src.tolist(), g.dst.tolist(), g.t.tolist()))
            T, Bl, cp = real_valued(g.n, edges, g.c.tolist(), d.s.tolist(), d.B.tolist(), p.tolist())
            # a path with q vertices has at most q + (q-1) rounded terms, each rounded up by < 1 tick
            og = oracle_graph(g)
            assert Fraction(r.cp, S) >= cp
            assert Fraction(r.cp, S) - cp < Fraction(2 * og.num_levels, S)
            for v in range(g.n):
                assert Fraction(int(r.tlevel[v]), S) >= T[v]
                assert Fraction(int(r.blevel[v]), S) >= Bl[v]
                assert Fraction(int(r.blevel[v]), S) - Bl[v] < Fraction(2 * og.num_levels, S)


# -------------------------------------------------------------------- invariants
def _rand_setup(seed, n=120, m=300, k=4):
    w = I.small_random(seed, n, m, k, 1)
    p = np.random.default_rng([seed, 1]).integers(0, k, size=n).astype(np.uint8)
    return w.graph, w.devices, p


def test_cp_identities_and_bounds():
    for seed in range(10):
        g, d, p = _rand_setup(seed)
        og, r = run(g, d.k, d.s, d.C, d.B, 16, p)
        rt = np.array([cdiv(int(g.c[v]) * 16, int(d.s[p[v]])) for v in range(g.n)])
        assert r.cp == (r.tlevel + rt).max()
        assert r.cp == r.blevel[og.level == 0].max()
        assert r.cp == (r.tlevel + r.blevel).max()
        assert ((r.tlevel + r.blevel) <= r.cp).all()
        assert rt.max() <= r.cp
        assert r.load.sum() == rt.sum()
        assert r.memload.sum() == og.mem.sum()
        for dd in range(d.k):
            assert r.load[dd] == rt[p == dd].sum()
            assert r.memload[dd] == og.mem[p == dd].sum()
            assert bool(r.viol >> dd & 1) == bool(r.memload[dd] >= d.C[dd])
        # sinks: blevel = rt; sources: tlevel = 0
        outdeg = np.diff(og.out_ptr)
        assert (r.blevel[outdeg == 0] == rt[outdeg == 0]).all()
        assert (r.tlevel[og.level == 0] == 0).all()


def test_monotone_in_bandwidth_and_speed():
    for seed in range(6):
        g, d, p = _rand_setup(20 + seed)
        _, r0 = run(g, d.k, d.s, d.C, d.B, 16, p)
        rng = np.random.default_rng(seed)
        B2 = d.B + rng.integers(0, 1000, size=d.B.shape)
        _, r1 = run(g, d.k, d.s, d.C, B2, 16, p)
        assert r1.cp <= r0.cp and (r1.tlevel <= r0.tlevel).all() and (r1.blevel <= r0.blevel).all()
        s2 = d.s + rng.integers(0, 5, size=d.k).astype(np.int32)
        _, r2 = run(g, d.k, s2, d.C, d.B, 16, p)
        assert r2.cp <= r0.cp and (r2.blevel <= r0.blevel).all()


def test_reversal_duality():
    for seed in range(6):
        g, d, p = _rand_setup(30 + seed)
        _, r = run(g, d.k, d.s, d.C, d.B, 16, p)
        gr = I.Graph(n=g.n, src=g.dst, dst=g.src, t=g.t, c=g.c, mem=g.mem, layers=0)
        _, rr = run(gr, d.k, d.s, d.C, d.B.T.copy(), 16, p)
        rt = np.array([cdiv(int(g.c[v]) * 16, int(d.s[p[v]])) for v in range(g.n)])
        assert (rr.tlevel + rt == r.blevel).all()
        assert (rr.blevel == r.tlevel + rt).all()
        assert rr.cp == r.cp


def test_relabelling_and_edge_order_invariance():
    for seed in range(6):
        g, d, p = _rand_setup(50 + seed)
        og, r = run(g, d.k, d.s, d.C, d.B, 16, p)
        g2, perm = I.relabel(g, seed)
        p2 = np.empty_like(p)
        p2[perm] = p
        og2, r2 = run(g2, d.k, d.s, d.C, d.B, 16, p2)
        assert (r2.tlevel[perm] == r.tlevel).all()
        assert (r2.blevel[perm] == r.blevel).all()
        assert r2.cp == r.cp and (r2.load == r.load).all() and (r2.memload == r.memload).all()
        assert (og2.level[perm] == og.level).all()


def test_linear_in_scale_when_quotients_are_integral():
    g, d, p = _rand_setup(77, k=3)
    s = np.array([1, 2, 4], np.int32)
    B = np.array([[0, 1, 2], [4, 0, 1], [2, 2, 0]], np.int64)
    g = I.Graph(n=g.n, src=g.src, dst=g.dst, t=g.t * 4, c=g.c * 4, mem=g.mem, layers=0)
    p = (p % 3).astype(np.uint8)
    _, r1 = run(g, 3, s, [INF] * 3, B, 1, p)
    _, r7 = run(g, 3, s, [INF] * 3, B, 7, p)
    assert (r7.tlevel == 7 * r1.tlevel).all() and (r7.blevel == 7 * r1.blevel).all() and r7.cp == 7 * r1.cp


def test_same_device_ignores_diagonal_and_zero_size_costs_nothing():
    g = graph_from_edges(3, [(0, 1, 500), (1, 2, 0)], [2, 3, 4])
    _, a = run(g, 2, [1, 1], [INF, INF], [[0, 10], [10, 0]], 1, [0, 0, 1])
    _, b = run(g, 2, [1, 1], [INF, INF], [[-5, 10], [10, 123456]], 1, [0, 0, 1])
    assert a.tlevel.tolist() == b.tlevel.tolist() == [0, 2, 5]
    assert a.cp == b.cp == 9


def test_isolated_vertices_and_empty_graph():
    g = graph_from_edges(3, [], [5, 0, 9])
    og, r = run(g, 2, [1, 3], [INF, INF], [[0, 1], [1, 0]], 3, [0, 1, 1])
    assert og.num_levels == 1 and og.order.tolist() == [0, 1, 2]
    assert r.tlevel.tolist() == [0, 0, 0] and r.blevel.tolist() == [15, 0, 9] and r.cp == 15
    g0 = graph_from_edges(0, [], [])
    og0 = oracle_graph(g0)
    assert og0.num_levels == 0


def test_bad_partition_and_overflow_are_reported():
    g = graph_from_edges(2, [(0, 1, 2 ** 40)], [2 ** 31 - 1, 1])
    og = oracle_graph(g)
    with pytest.raises(oracle.OracleError) as ei:
        oracle.eval_partition(og, 2, [1, 1], [INF, INF], [[0, 1], [1, 0]], 1, np.array([0, 2], np.uint8))
    assert ei.value.code == oracle.BAD_PARTITION
    with pytest.raises(oracle.OracleError) as ei:
        oracle.eval_partition(og, 2, [1, 1], [INF, INF], [[0, 1], [1, 0]], 2 ** 40, np.array([0, 1], np.uint8))
    assert ei.value.code == oracle.OVERFLOW


def test_batch_layout_matches_single_calls():
    w = I.config1()
    og = oracle_graph(w.graph)
    part = w.part_full()
    d = w.devices
    b = oracle.eval_batch(og, d.k, d.s, d.C, d.B, d.scale, part, cols=[3, 0, 63])
    for i, j in enumerate([3, 0, 63]):
        r = oracle.eval_partition(og, d.k, d.s, d.C, d.B, d.scale, np.ascontiguousarray(part[:, j]))
        assert (b.tlevel[:, i] == r.tlevel).all() and (b.blevel[:, i] == r.blevel).all() and b.cp[i] == r.cp
