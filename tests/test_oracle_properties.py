"""Property-based checks of the oracle on hypothesis-generated DAGs (CPU only):
the exact invariants every evaluation must satisfy, whatever the graph."""
from __future__ import annotations

import numpy as np
from hypothesis import HealthCheck, given, settings, strategies as st

import oracle
from paper_1711_01912_b200 import inputs as I
from helpers import brute_force, cdiv, graph_from_edges, oracle_graph

INF = np.iinfo(np.int64).max


@st.composite
def dags(draw, max_n=10):
    n = draw(st.integers(1, max_n))
    k = draw(st.integers(1, 4))
    perm = draw(st.permutations(list(range(n))))
    edges = []
    for u in range(n):
        for v in range(u + 1, n):
            if draw(st.integers(0, 3)) == 0:
                edges.append((perm[u], perm[v], draw(st.integers(0, 10 ** 6))))
    c = draw(st.lists(st.integers(0, 10 ** 4), min_size=n, max_size=n))
    s = draw(st.lists(st.integers(1, 64), min_size=k, max_size=k))
    B = [[draw(st.integers(1, 10 ** 5)) for _ in range(k)] for _ in range(k)]
    S = draw(st.integers(1, 64))
    p = draw(st.lists(st.integers(0, k - 1), min_size=n, max_size=n))
    return n, k, edges, c, s, B, S, p


@settings(max_examples=120, deadline=None, suppress_health_check=[HealthCheck.too_slow])
@given(dags())
def test_oracle_equals_path_enumeration_and_identities(case):
    n, k, edges, c, s, B, S, p = case
    g = graph_from_edges(n, edges, c)
    og = oracle_graph(g)
    r = oracle.eval_partition(og, k, s, [INF] * k, B, S, np.asarray(p, np.uint8))
    tl, bl, cp = brute_force(n, edges, c, s, B, S, p)
    assert r.tlevel.tolist() == tl and r.blevel.tolist() == bl and r.cp == cp
    rt = np.array([cdiv(c[v] * S, s[p[v]]) for v in range(n)])
    assert r.cp == (r.tlevel + rt).max() == (r.tlevel + r.blevel).max() == r.blevel[og.level == 0].max()
    assert r.load.sum() == rt.sum() and r.memload.sum() == og.mem.sum()
    # levels: every edge goes to a strictly higher level, and each non-source has a predecessor one level below
    for (u, v, _) in edges:
        assert og.level[u] < og.level[v]
    for v in range(n):
        preds = [u for (u, x, _) in edges if x == v]
        assert og.level[v] == (0 if not preds else 1 + max(og.level[u] for u in preds))


@settings(max_examples=60, deadline=None, suppress_health_check=[HealthCheck.too_slow])
@given(dags(max_n=9), st.integers(1, 5000))
def test_more_bandwidth_or_speed_never_lengthens_paths(case, bump):
    n, k, edges, c, s, B, S, p = case
    g = graph_from_edges(n, edges, c)
    og = oracle_graph(g)
    pa = np.asarray(p, np.uint8)
    r0 = oracle.eval_partition(og, k, s, [INF] * k, B, S, pa)
    B2 = [[b + bump for b in row] for row in B]
    r1 = oracle.eval_partition(og, k, s, [INF] * k, B2, S, pa)
    s2 = [x + 1 for x in s]
    r2 = oracle.eval_partition(og, k, s2, [INF] * k, B, S, pa)
    assert r1.cp <= r0.cp and (r1.tlevel <= r0.tlevel).all() and (r1.blevel <= r0.blevel).all()
    assert r2.cp <= r0.cp and (r2.blevel <= r0.blevel).all()
