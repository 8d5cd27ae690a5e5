"""Test helpers: graph plumbing and slow independent referees used to pin the
oracle.  Nothing here is imported by the oracle or by the CUDA package."""
from __future__ import annotations

import json
import os
from fractions import Fraction

import numpy as np

from paper_1711_01912_b200 import inputs as I

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def load_golden(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return json.load(f)


def graph_from_edges(n, edges, c, mem=None, t_dtype=np.int64):
    e = np.asarray(edges, np.int64).reshape(-1, 3)
    return I.Graph(n=n, src=e[:, 0].astype(np.int32), dst=e[:, 1].astype(np.int32), t=e[:, 2].astype(t_dtype),
                   c=np.asarray(c, np.int32), mem=None if mem is None else np.asarray(mem, np.int64), layers=0)


def oracle_graph(g):
    import oracle
    c = I.to_csr(g)
    return oracle.OracleGraph(g.n, c.in_ptr, c.in_src, c.in_t, c.out_ptr, c.out_dst, c.out_t, g.c, g.mem)


def cdiv(a, b):
    return -((-a) // b)


def brute_force(n, edges, c, s, B, S, p):
    """Enumerate every path of the DAG by depth-first search (python ints).
    Returns (tlevel, blevel, cp): tlevel[v] = longest cost of a path ending
    just before v starts, blevel[v] = longest cost of a path starting with v's
    own execution, cp = longest source-to-sink path."""
    succ = [[] for _ in range(n)]
    pred_count = [0] * n
    for (u, v, t) in edges:
        succ[u].append((v, t))
        pred_count[v] += 1
    rt = [cdiv(c[v] * S, s[p[v]]) for v in range(n)]

    def w(u, v, t):
        return 0 if p[u] == p[v] else cdiv(t * S, B[p[u]][p[v]])

    tl = [0] * n
    bl = [0] * n
    best = [0]

    def walk(v, start, origin_costs):
        # start = start time of v along this path; origin_costs = list of
        # (vertex, start time of that vertex on this path) for the prefix
        fin = start + rt[v]
        tl[v] = max(tl[v], start)
        for (x, sx) in origin_costs:
            bl[x] = max(bl[x], fin - sx)
        bl[v] = max(bl[v], rt[v])
        best[0] = max(best[0], fin)
        origin_costs.append((v, start))
        for (x, t) in succ[v]:
            walk(x, fin + w(v, x, t), origin_costs)
        origin_costs.pop()

    for v in range(n):
        # start from every vertex so that blevel sees every suffix; only
        # source starts define tlevel, so restore tl for non-sources
        if pred_count[v] == 0:
            walk(v, 0, [])
    return tl, bl, best[0]


def real_valued(n, edges, c, s, B, p):
    """The paper's real-valued model evaluated with exact rationals by
    memoised recursion (no rounding): returns (tlevel, blevel, cp)."""
    from functools import lru_cache
    import sys
    sys.setrecursionlimit(10000)
    succ = [[] for _ in range(n)]
    pred = [[] for _ in range(n)]
    for (u, v, t) in edges:
        succ[u].append((v, t))
        pred[v].append((u, t))
    rt = [Fraction(int(c[v]), int(s[p[v]])) for v in range(n)]

    def tr(u, v, t):
        return Fraction(0) if p[u] == p[v] else Fraction(int(t), int(B[p[u]][p[v]]))

    @lru_cache(None)
    def bl(v):
        return rt[v] + max([bl(x) + tr(v, x, t) for (x, t) in succ[v]], default=Fraction(0))

    @lru_cache(None)
    def tl(v):
        return max([tl(u) + rt[u] + tr(u, v, t) for (u, t) in pred[v]], default=Fraction(0))

    T = [tl(v) for v in range(n)]
    Bv = [bl(v) for v in range(n)]
    return T, Bv, max(T[v] + rt[v] for v in range(n))
