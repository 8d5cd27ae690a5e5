"""Pins of the oracle's placement-constraint check (collocation constraints, Eq. 3; device constraints, Eq. 4):
a worked example, closed forms on the partition p(v) = v mod k, and invariants that a dropped term, a swapped
operand or an off-by-one in the indexing would break."""
from __future__ import annotations

import numpy as np

import oracle


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
