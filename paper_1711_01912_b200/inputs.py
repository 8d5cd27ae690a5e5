"""Seeded synthetic inputs: layered DAGs shaped like TensorFlow training graphs,
device tables and candidate partitions.

This module only *draws* inputs.  It contains none of the method's arithmetic
(no runtimes, no transfer costs, no levels, no loads) and is the single piece of
code that both the CUDA path's tests/benchmark and the CPU oracle's tests are
allowed to share.  Everything is produced with ``numpy.random.default_rng``
(PCG64) in a fixed draw order: structure, c, t, mem, B, partitions.

Vertex ids are issued layer by layer; ``relabel`` applies a seeded permutation
for the relabelling-invariance tests.  Candidate partitions are drawn in row
blocks with one child generator per block, so any block of rows of the
``[n][P]`` id matrix can be regenerated without materialising the rest.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Iterator, Optional, Tuple

import numpy as np

INT64_MAX = np.iinfo(np.int64).max
SCALE = 16  # ticks per paper time unit; a multiple of every speed used below

#: rows of the id matrix drawn from one child generator
PART_ROW_BLOCK = 4096


@dataclasses.dataclass
class Graph:
    """Edge-list form of G=(V,E) with vertex costs c, edge sizes t and
    optional per-vertex memory (problem tuple of Section 2)."""

    n: int
    src: np.ndarray  # int32[m]
    dst: np.ndarray  # int32[m]
    t: np.ndarray  # int32[m] or int64[m]
    c: np.ndarray  # int32[n]
    mem: Optional[np.ndarray]  # int32/int64[n] or None
    layers: int  # generator layers (not necessarily the longest-path levels)

    @property
    def m(self) -> int:
        return int(self.src.shape[0])


@dataclasses.dataclass
class Devices:
    """k devices: speeds s, capacities C, bandwidth matrix B[src][dst]."""

    k: int
    s: np.ndarray  # int32[k]
    C: np.ndarray  # int64[k]
    B: np.ndarray  # int64[k][k]
    scale: int = SCALE


@dataclasses.dataclass
class Csr:
    """Both adjacency directions of a Graph in CSR form."""

    n: int
    m: int
    in_ptr: np.ndarray  # int64[n+1]
    in_src: np.ndarray  # int32[m]
    in_t: np.ndarray  # t dtype [m]
    out_ptr: np.ndarray  # int64[n+1]
    out_dst: np.ndarray  # int32[m]
    out_t: np.ndarray  # t dtype [m]


def to_csr(g: Graph) -> Csr:
    """Group the edge list by destination (in-CSR) and by source (out-CSR).
    Inside a row edges keep their edge-list order (stable)."""
    n, m = g.n, g.m
    oi = np.argsort(g.dst, kind="stable")
    oo = np.argsort(g.src, kind="stable")
    in_ptr = np.zeros(n + 1, np.int64)
    out_ptr = np.zeros(n + 1, np.int64)
    np.cumsum(np.bincount(g.dst, minlength=n), out=in_ptr[1:])
    np.cumsum(np.bincount(g.src, minlength=n), out=out_ptr[1:])
    return Csr(
        n=n,
        m=m,
        in_ptr=in_ptr,
        in_src=np.ascontiguousarray(g.src[oi], np.int32),
        in_t=np.ascontiguousarray(g.t[oi]),
        out_ptr=out_ptr,
        out_dst=np.ascontiguousarray(g.dst[oo], np.int32),
        out_t=np.ascontiguousarray(g.t[oo]),
    )


def relabel(g: Graph, seed: int) -> Tuple[Graph, np.ndarray]:
    """Rename vertex v to perm[v] and shuffle the edge list.  Returns the new
    graph and perm (old id -> new id)."""
    rng = np.random.default_rng([seed, 0x5EED])
    perm = rng.permutation(g.n).astype(np.int32)
    eperm = rng.permutation(g.m)
    inv = np.empty_like(perm)
    inv[perm] = np.arange(g.n, dtype=np.int32)
    g2 = Graph(
        n=g.n,
        src=perm[g.src][eperm],
        dst=perm[g.dst][eperm],
        t=g.t[eperm],
        c=g.c[inv],
        mem=None if g.mem is None else g.mem[inv],
        layers=g.layers,
    )
    return g2, perm


# --------------------------------------------------------------------------
# draws
# --------------------------------------------------------------------------

def _clip_round(x: np.ndarray, lo: float, hi: float, dtype) -> np.ndarray:
    return np.clip(np.rint(x), lo, hi).astype(dtype)


def _lognormal(rng, mu, sigma, size, hi, dtype):
    return _clip_round(rng.lognormal(mu, sigma, size), 1, hi, dtype)


def _loguniform(rng, lo, hi, size, dtype):
    return _clip_round(np.exp(rng.uniform(math.log(lo), math.log(hi), size)), lo, hi, dtype)


def _distinct_from_pool(rng, rows: int, pool: int, want: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """For each of `rows` rows pick want[r] distinct numbers of range(pool)
    (random keys, smallest first).  Returns (row index, pick) flattened."""
    keys = rng.random((rows, pool))
    rank = np.argsort(keys, axis=1)
    take = np.arange(pool)[None, :] < want[:, None]
    r, j = np.nonzero(take)
    return r, rank[r, j]


def _dedupe(src, dst):
    key = dst.astype(np.int64) * (1 << 32) + src.astype(np.int64)
    _, first = np.unique(key, return_index=True)
    first.sort()
    return src[first], dst[first]


# --------------------------------------------------------------------------
# graph structures
# --------------------------------------------------------------------------

def _layered_prev2(rng, layers: int, width: int):
    """Tiny layered DAG: 1-3 in-edges from distinct vertices of the previous
    two layers (layer 1: the previous one)."""
    srcs, dsts = [], []
    for l in range(1, layers):
        lo_layer = max(0, l - 2)
        pool = (l - lo_layer) * width
        want = rng.integers(1, 4, size=width)
        r, pick = _distinct_from_pool(rng, width, pool, want)
        srcs.append(lo_layer * width + pick)
        dsts.append(l * width + r)
    return np.concatenate(srcs).astype(np.int32), np.concatenate(dsts).astype(np.int32)


def _resnet_like(layers: int, width: int):
    """Backbone chain in slot 0 with a skip edge into every third layer;
    slots 1..width-1 are side branches hanging between consecutive backbone
    vertices (parameter/gradient style).  Deterministic structure."""
    srcs, dsts = [], []
    b = np.arange(layers, dtype=np.int64) * width
    srcs.append(b[:-1]); dsts.append(b[1:])
    l3 = np.arange(3, layers, 3)
    srcs.append(b[l3 - 3]); dsts.append(b[l3])
    side = (np.arange(layers, dtype=np.int64)[:, None] * width + np.arange(1, width)[None, :])
    # in-edge from b_{l-1}
    srcs.append(np.repeat(b[:-1], width - 1)); dsts.append(side[1:].ravel())
    # out-edge to b_{l+1}
    srcs.append(side[:-1].ravel()); dsts.append(np.repeat(b[1:], width - 1))
    return np.concatenate(srcs).astype(np.int32), np.concatenate(dsts).astype(np.int32)


def _inception_like(rng, layers: int, modules: int, slots: int, avg_in_degree: float):
    """Wide DAG of `modules` modules x `slots` slots per layer.  Every 4th
    layer is a concat layer: slot 0 of a module merges the module's live
    branches (4..slots of them) of the previous layer, the other slots pass
    one live branch through.  In the layer after a concat the live branches fan
    out of the concat vertex.  Extra edges from the previous two layers bring
    the average in-degree to `avg_in_degree`."""
    width = modules * slots
    n = layers * width
    vid = lambda l, mo, sl: (l * modules + mo) * slots + sl
    srcs, dsts = [], []
    mo = np.arange(modules)
    live = rng.integers(4, slots + 1, size=modules)  # live branches feeding the next concat
    for l in range(1, layers):
        if l % 4 == 0:
            # concat: fan-in = live branches of the module
            for sl in range(slots):
                sel = mo[live > sl]
                srcs.append(vid(l - 1, sel, sl)); dsts.append(vid(l, sel, 0))
            # pass-through slots take one random live branch of their module
            for sl in range(1, slots):
                pick = (rng.random(modules) * live).astype(np.int64)
                srcs.append(vid(l - 1, mo, pick)); dsts.append(vid(l, mo, sl))
            live = rng.integers(4, slots + 1, size=modules)
        elif l % 4 == 1:
            # fan-out: live branches start at the concat vertex, the rest carry on
            for sl in range(slots):
                is_live = live > sl
                srcs.append(np.where(is_live, vid(l - 1, mo, 0), vid(l - 1, mo, sl)))
                dsts.append(vid(l, mo, sl))
        else:
            for sl in range(slots):
                srcs.append(vid(l - 1, mo, sl)); dsts.append(vid(l, mo, sl))
    src = np.concatenate(srcs).astype(np.int64)
    dst = np.concatenate(dsts).astype(np.int64)
    target = int(round(avg_in_degree * n))
    extra = target - src.shape[0]
    # extras: destination uniform over layers >= 1, source uniform over the previous 2 layers
    over = int(extra * 1.02) + 16
    d = rng.integers(width, n, size=over)
    dl = d // width
    lo = np.maximum(dl - 2, 0) * width
    s = lo + (rng.random(over) * (dl * width - lo)).astype(np.int64)
    src = np.concatenate([src, s]); dst = np.concatenate([dst, d])
    src, dst = _dedupe(src, dst)
    src, dst = src[:target], dst[:target]
    return src.astype(np.int32), dst.astype(np.int32)


def _rnn_like(rng, layers: int, width: int):
    """Deep narrow DAG: cell (l,i) takes (l-1,i) plus 1-2 distinct other cells
    of layer l-1."""
    rows = (layers - 1) * width
    want = rng.integers(1, 3, size=rows)
    r, pick = _distinct_from_pool(rng, rows, width - 1, want)
    l = r // width + 1
    i = r % width
    other = pick + (pick >= i)  # skip the own cell
    base = np.arange(rows, dtype=np.int64)
    src = np.concatenate([base, (l - 1) * width + other])
    dst = np.concatenate([base + width, l * width + i])
    return src.astype(np.int32), dst.astype(np.int32)


def _powerlaw_fanin(rng, layers: int, width: int, alpha: float, dmax: int, back: int):
    """Fan-in d with P(d) ~ d^-alpha on 1..dmax, sources drawn from the
    previous `back` layers; repeated picks of the same source are dropped."""
    n = layers * width
    rows = n - width
    pd = np.arange(1, dmax + 1, dtype=np.float64) ** (-alpha)
    pd /= pd.sum()
    deg = rng.choice(np.arange(1, dmax + 1), size=rows, p=pd)
    dst = np.repeat(np.arange(width, n, dtype=np.int64), deg)
    dl = dst // width
    lo = np.maximum(dl - back, 0) * width
    src = lo + (rng.random(dst.shape[0]) * (dl * width - lo)).astype(np.int64)
    src, dst = _dedupe(src, dst)
    return src.astype(np.int32), dst.astype(np.int32)


def _random_layered(rng, n: int, m: int, layers: int):
    """Paper-shaped sparse DAG (Table 1 sizes): vertices spread over layers,
    every non-first-layer vertex gets one in-edge from an earlier layer and
    the remaining edges connect random earlier -> later layer pairs."""
    layer_of = np.sort(rng.integers(0, layers, size=n))
    layer_of[0] = 0
    if n >= 2 and layer_of[-1] == 0:
        layer_of[-1] = 1
    first_of = np.searchsorted(layer_of, np.arange(layers + 1))
    non_src = np.nonzero(layer_of > 0)[0]
    hi = first_of[layer_of[non_src]]  # vertices of earlier layers are [0, hi)
    non_src = non_src[hi > 0]; hi = hi[hi > 0]
    src = (rng.random(non_src.shape[0]) * hi).astype(np.int64)
    dst = non_src.astype(np.int64)
    for _attempt in range(64):  # dense requests may not be satisfiable: give up and return fewer edges
        if src.shape[0] >= m:
            break
        need = (m - src.shape[0]) * 2 + 8
        d = rng.integers(0, n, size=need)
        h = first_of[layer_of[d]]
        ok = h > 0
        d = d[ok]; h = h[ok]
        s = (rng.random(d.shape[0]) * h).astype(np.int64)
        src = np.concatenate([src, s]); dst = np.concatenate([dst, d])
        src, dst = _dedupe(src, dst)
    return src[:m].astype(np.int32), dst[:m].astype(np.int32)


# --------------------------------------------------------------------------
# configs
# --------------------------------------------------------------------------

@dataclasses.dataclass
class Workload:
    name: str
    seed: int
    graph: Graph
    devices: Devices
    P: int
    part_kind: str  # "uniform" | "half_hash"

    def part_rows(self, r0: int, r1: int, cols: Optional[np.ndarray] = None) -> np.ndarray:
        """Rows [r0, r1) of the uint8 id matrix ``[n][P]`` (optionally only the
        listed candidate columns)."""
        return partition_rows(self, r0, r1, cols)

    def part_blocks(self, cols: Optional[np.ndarray] = None) -> Iterator[Tuple[int, np.ndarray]]:
        for r0 in range(0, self.graph.n, PART_ROW_BLOCK):
            r1 = min(self.graph.n, r0 + PART_ROW_BLOCK)
            yield r0, partition_rows(self, r0, r1, cols)

    def part_full(self) -> np.ndarray:
        out = np.empty((self.graph.n, self.P), np.uint8)
        for r0, blk in self.part_blocks():
            out[r0:r0 + blk.shape[0]] = blk
        return out

    def part_columns(self, cols) -> np.ndarray:
        cols = np.asarray(cols, np.int64)
        out = np.empty((self.graph.n, cols.shape[0]), np.uint8)
        for r0, blk in self.part_blocks(cols):
            out[r0:r0 + blk.shape[0]] = blk
        return out


def _uniform_block(seed: int, block: int, rows: int, P: int, k: int) -> np.ndarray:
    rng = np.random.default_rng([seed, 0x9A27, block])
    return rng.integers(0, k, size=(rows, P), dtype=np.uint8)


def partition_rows(w: Workload, r0: int, r1: int, cols=None) -> np.ndarray:
    k, P, n = w.devices.k, w.P, w.graph.n
    assert 0 <= r0 <= r1 <= n
    out = np.empty((r1 - r0, P if cols is None else len(cols)), np.uint8)
    b0 = r0 // PART_ROW_BLOCK
    b1 = (r1 + PART_ROW_BLOCK - 1) // PART_ROW_BLOCK
    for b in range(b0, b1):
        lo = b * PART_ROW_BLOCK
        hi = min(n, lo + PART_ROW_BLOCK)
        blk = _uniform_block(w.seed, b, hi - lo, P, k)
        if w.part_kind == "half_hash":
            # candidate 0 is exactly v mod k; candidates 1..P/2-1 use a
            # multiplicative hash of v with a per-candidate odd multiplier
            half = P // 2
            v = np.arange(lo, hi, dtype=np.uint64)[:, None]
            j = np.arange(half, dtype=np.uint64)[None, :]
            mult = (np.uint64(0x9E3779B97F4A7C15) * (np.uint64(2) * j + np.uint64(w.seed * 2 + 1))) | np.uint64(1)
            h = (v + np.uint64(1)) * mult
            h ^= h >> np.uint64(29)
            h *= np.uint64(0xBF58476D1CE4E5B9)
            h ^= h >> np.uint64(32)
            hashed = (h % np.uint64(k)).astype(np.uint8)
            hashed[:, 0] = (np.arange(lo, hi) % k).astype(np.uint8)
            blk[:, :half] = hashed
        a = max(r0, lo); e = min(r1, hi)
        sub = blk[a - lo:e - lo]
        out[a - r0:e - r0] = sub if cols is None else sub[:, cols]
    return out


def _finish(name, seed, rng, src, dst, n, layers, c_draw, t_draw, mem_draw, dev_draw, P, part_kind):
    m = src.shape[0]
    c = c_draw(rng, n)
    t = t_draw(rng, m)
    mem = mem_draw(rng, n) if mem_draw is not None else None
    dev = dev_draw(rng)
    g = Graph(n=n, src=src, dst=dst, t=t, c=c, mem=mem, layers=layers)
    return Workload(name=name, seed=seed, graph=g, devices=dev, P=P, part_kind=part_kind)


def _offdiag_uniform(rng, k, lo, hi):
    B = rng.integers(lo, hi + 1, size=(k, k)).astype(np.int64)
    B[np.arange(k), np.arange(k)] = 0
    return B


def _grouped_B(k, group, inside, across):
    g = np.arange(k) // group
    B = np.where(g[:, None] == g[None, :], inside, across).astype(np.int64)
    B[np.arange(k), np.arange(k)] = 0
    return B


def config1(seed: int = 0) -> Workload:
    """Tiny layered DAG: n=256, 16 layers x 16, k=2, P=64."""
    rng = np.random.default_rng(seed)
    src, dst = _layered_prev2(rng, 16, 16)
    return _finish(
        "cfg1_tiny_layered", seed, rng, src, dst, 256, 16,
        lambda r, n: r.integers(1, 1001, size=n).astype(np.int32),
        lambda r, m: _loguniform(r, 1e3, 1e6, m, np.int32),
        None,
        lambda r: Devices(2, np.array([1, 4], np.int32), np.full(2, INT64_MAX, np.int64),
                          np.array([[0, 1000], [1000, 0]], np.int64)),
        64, "uniform")


def config2(seed: int = 1) -> Workload:
    """Communication-intensive ResNet-like DAG: n=4096, 256 layers x 16, k=4, P=4096."""
    rng = np.random.default_rng(seed)
    src, dst = _resnet_like(256, 16)
    return _finish(
        "cfg2_resnet_like", seed, rng, src, dst, 4096, 256,
        lambda r, n: _lognormal(r, 5, 1.5, n, 2**31 - 1, np.int32),
        lambda r, m: _lognormal(r, 13, 2, m, 2**31 - 1, np.int32),
        lambda r, n: r.integers(10**4, 10**7 + 1, size=n).astype(np.int32),
        lambda r: Devices(4, np.array([1, 1, 8, 8], np.int32), np.full(4, 2**31, np.int64),
                          _offdiag_uniform(r, 4, 10**3, 10**5)),
        4096, "half_hash")


def config3(seed: int = 2) -> Workload:
    """Inception-like wide DAG: n=65,536, 512 layers x 128, k=8, P=16,384."""
    rng = np.random.default_rng(seed)
    src, dst = _inception_like(rng, 512, 16, 8, 2.5)
    n = 65536
    assert abs(src.shape[0] / n - 2.5) <= 0.05
    return _finish(
        "cfg3_inception_like", seed, rng, src, dst, n, 512,
        lambda r, n_: _lognormal(r, 6, 2, n_, 2**31 - 1, np.int32),
        lambda r, m: _lognormal(r, 14, 2, m, 2**40, np.int64),
        None,
        lambda r: Devices(8, np.array([1, 1, 2, 2, 4, 4, 16, 16], np.int32), np.full(8, INT64_MAX, np.int64),
                          _grouped_B(8, 2, 10**5, 10**4)),
        16384, "uniform")


def config4(seed: int = 3) -> Workload:
    """Deep narrow RNN-unrolled DAG: n=262,144, 16,384 layers x 16, k=4, P=1024."""
    rng = np.random.default_rng(seed)
    src, dst = _rnn_like(rng, 16384, 16)
    return _finish(
        "cfg4_rnn_unrolled", seed, rng, src, dst, 262144, 16384,
        lambda r, n: r.integers(10, 501, size=n).astype(np.int32),
        lambda r, m: r.integers(10**4, 10**5 + 1, size=m).astype(np.int32),
        None,
        lambda r: Devices(4, np.array([1, 2, 4, 8], np.int32), np.full(4, INT64_MAX, np.int64),
                          _offdiag_uniform(r, 4, 10**3, 10**4)),
        1024, "uniform")


def config5(seed: int = 4, layers: int = 2048, width: int = 512, P: int = 8192) -> Workload:
    """Large data-parallel training DAG: n=1,048,576, 2048 layers x 512,
    power-law fan-in, k=16, P=8192.  The capacity is one value for all devices,
    placed from the mean and spread of a sum of n/k uniform memory draws so
    that roughly a tenth of uniform random partitions exceed it on some
    device."""
    rng = np.random.default_rng(seed)
    src, dst = _powerlaw_fanin(rng, layers, width, 2.2, 64, 4)
    n = layers * width
    k = 16
    lo, hi = 10**4, 10**8
    mu = (lo + hi) / 2.0
    sd = (hi - lo) / math.sqrt(12.0)
    # a device receives Binomial(n, 1/k) vertices, each U[lo,hi]:
    # variance = n/k * (sd^2 + mu^2 (1 - 1/k))
    var = n / k * (sd * sd + mu * mu * (1.0 - 1.0 / k))
    z = 2.48  # per-device tail 1-0.9**(1/16)
    cap = int(n / k * mu + z * math.sqrt(var))
    s = np.array([16] * 4 + [1] * 12, np.int32)
    return _finish(
        "cfg5_large_dp", seed, rng, src, dst, n, layers,
        lambda r, n_: _lognormal(r, 6, 2, n_, 2**31 - 1, np.int32),
        lambda r, m: _lognormal(r, 15, 2.5, m, 2**40, np.int64),
        lambda r, n_: r.integers(lo, hi + 1, size=n_).astype(np.int64),
        lambda r: Devices(k, s, np.full(k, cap, np.int64), _grouped_B(k, 4, 10**5, 5 * 10**3)),
        P, "uniform")


def paper_shaped(which: int = 0, seed: int = 7, P: int = 32) -> Workload:
    """Sparse DAG with the node/edge counts of one of the three networks of
    Table 1 and the simulation parameters of Section 5.1: 50 devices, speeds
    U[10,100], link rates U[10,60], tensors U[1,100], vertex cost U[1,100]."""
    n, m = [(347, 531), (3069, 5533), (5271, 9214)][which]
    rng = np.random.default_rng([seed, which])
    src, dst = _random_layered(rng, n, m, max(8, n // 12))
    k = 50
    return _finish(
        f"paper_table1_{which}", seed * 16 + which, rng, src, dst, n, max(8, n // 12),
        lambda r, n_: r.integers(1, 101, size=n_).astype(np.int32),
        lambda r, m_: r.integers(1, 101, size=m_).astype(np.int32),
        None,
        lambda r: Devices(k, r.integers(10, 101, size=k).astype(np.int32), np.full(k, INT64_MAX, np.int64),
                          _offdiag_uniform(r, k, 10, 60), scale=SCALE),
        P, "uniform")


def small_random(seed: int, n: int, m: int, k: int, P: int, t_dtype=np.int64, with_mem=True,
                 layers: Optional[int] = None) -> Workload:
    """Small random DAG for property tests (arbitrary shape, awkward sizes)."""
    rng = np.random.default_rng([seed, n, m, k])
    layers = layers or max(2, int(math.sqrt(n)))
    if n >= 2 and m > 0:
        src, dst = _random_layered(rng, n, m, layers)
    else:
        src = np.zeros(0, np.int32); dst = np.zeros(0, np.int32)
    tmax = 2**30 if t_dtype == np.int32 else 2**36
    return _finish(
        f"rand_n{n}_m{m}_k{k}", seed, rng, src, dst, n, layers,
        lambda r, n_: r.integers(0, 2000, size=n_).astype(np.int32),
        lambda r, m_: _clip_round(np.exp(r.uniform(0, math.log(tmax), m_)) - 1, 0, tmax, t_dtype),
        (lambda r, n_: r.integers(0, 10**6, size=n_).astype(np.int64)) if with_mem else None,
        lambda r: Devices(k, r.integers(1, 17, size=k).astype(np.int32),
                          r.integers(10**5, 10**8, size=k).astype(np.int64),
                          _offdiag_uniform(r, k, 1, 10**5)),
        P, "uniform")


CONFIGS = {1: config1, 2: config2, 3: config3, 4: config4, 5: config5}


def make_config(i: int) -> Workload:
    return CONFIGS[i]()
