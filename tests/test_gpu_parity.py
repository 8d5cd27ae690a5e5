"""GPU parity: the CUDA library, called through its C ABI, against the CPU
oracle on the same seeded inputs.  Everything is integer, so the bar is
bit-exact equality of every output."""
from __future__ import annotations

import numpy as np
import pytest

from paper_1711_01912_b200 import inputs as I
from helpers import graph_from_edges, load_golden, oracle_graph

pytestmark = pytest.mark.gpu

INF = np.iinfo(np.int64).max
SENTINEL = -0x0123456789ABCDEF


def _torch():
    import torch
    return torch


def gpu_graph(g, dev=None):
    from paper_1711_01912_b200 import tfps
    c = I.to_csr(g)
    G = tfps.Graph(g.n, c.in_ptr, c.in_src, c.in_t, g.c, c.out_ptr, c.out_dst, c.out_t, g.mem)
    if dev is not None:
        G.devices_set(dev.k, dev.s, dev.C, dev.B, dev.scale)
    return G


def padded(part: np.ndarray, ldp=None, fill=0):
    torch = _torch()
    n, P = part.shape
    ldp = max(16, (P + 15) // 16 * 16) if ldp is None else ldp
    buf = np.full((n, ldp), fill, np.uint8)
    buf[:, :P] = part
    return torch.from_numpy(buf).cuda(), P, ldp


def run_and_compare(g, dev, part, flags, cols=None, pad_fill=0, check_padding=True):
    """Evaluate all P candidates on the GPU, compare the listed columns (default
    all) with the oracle, and check that padding columns keep their sentinel."""
    import oracle
    from paper_1711_01912_b200 import tfps
    torch = _torch()
    G = gpu_graph(g, dev)
    dpart, P, ldp = padded(part, fill=pad_fill)
    n, k = g.n, dev.k
    out = {
        "tlevel": torch.full((n, ldp), SENTINEL, dtype=torch.int64, device="cuda"),
        "blevel": torch.full((n, ldp), SENTINEL, dtype=torch.int64, device="cuda"),
        "cp": torch.full((max(P, 1),), SENTINEL, dtype=torch.int64, device="cuda"),
        "load": torch.full((k, ldp), SENTINEL, dtype=torch.int64, device="cuda"),
        "memload": torch.full((k, ldp), SENTINEL, dtype=torch.int64, device="cuda"),
        "viol": torch.full((max(P, 1),), SENTINEL, dtype=torch.int64, device="cuda"),
    }
    G.eval_batch(dpart, P, flags=flags, out=out)
    og = oracle_graph(g)
    cols = list(range(P)) if cols is None else list(cols)
    ref = oracle.eval_batch(og, k, dev.s, dev.C, dev.B, dev.scale, part, cols)
    tl = out["tlevel"].cpu().numpy(); bl = out["blevel"].cpu().numpy()
    assert np.array_equal(tl[:, cols], ref.tlevel)
    assert np.array_equal(bl[:, cols], ref.blevel)
    assert np.array_equal(out["cp"].cpu().numpy()[cols], ref.cp)
    assert np.array_equal(out["load"].cpu().numpy()[:, cols], ref.load)
    assert np.array_equal(out["memload"].cpu().numpy()[:, cols], ref.memload)
    assert np.array_equal(out["viol"].cpu().numpy().view(np.uint64)[cols], ref.viol)
    if check_padding and ldp > P:
        for name in ("tlevel", "blevel", "load", "memload"):
            assert (out[name][:, P:] == SENTINEL).all(), f"{name}: padding columns were written"
    G.close()
    return out


VARIANTS = [1, 2]  # TFPS_EVAL_LEVEL_SYNC, TFPS_EVAL_SLICED


# -------------------------------------------------------------------- worked DAGs
@pytest.mark.parametrize("flags", VARIANTS)
@pytest.mark.parametrize("fname", ["w1_diamond.json", "w2_two_sinks.json"])
def test_worked_examples_on_gpu(fname, flags):
    from paper_1711_01912_b200 import tfps
    w = load_golden(fname)
    g = graph_from_edges(w["n"], w["edges"], w["c"])
    for case in w["cases"]:
        k = w["k"]
        dev = I.Devices(k, np.array(w["s"], np.int32), np.array(case.get("C", [INF] * k), np.int64),
                        np.array(case["B"], np.int64), scale=w["S"])
        G = gpu_graph(g, dev)
        part, P, ldp = padded(np.array(case["p"], np.uint8)[:, None])
        out = G.eval_batch(part, P, flags=flags)
        assert out["tlevel"][:, 0].tolist() == case["tlevel"]
        assert out["blevel"][:, 0].tolist() == case["blevel"]
        assert out["cp"][0].item() == case["cp"]
        assert out["load"][:, 0].tolist() == case["load"]
        if "memload" in case:
            assert out["memload"][:, 0].tolist() == case["memload"]
            assert out["viol"][0].item() == case["viol"]
        level, order, lp, L = G.topo_levels()
        assert level.tolist() == w["level"]
        G.close()


# ------------------------------------------------------------------ configs 1 and 2
@pytest.mark.parametrize("flags", VARIANTS + [0])
def test_config1_every_candidate(flags):
    w = I.config1()
    run_and_compare(w.graph, w.devices, w.part_full(), flags)


@pytest.mark.parametrize("flags", VARIANTS)
def test_config2_every_candidate(flags):
    w = I.config2()
    run_and_compare(w.graph, w.devices, w.part_full(), flags)


@pytest.mark.parametrize("device_arrays", [False, True])
@pytest.mark.parametrize("give_out_edges", [False, True])
def test_graph_create_spaces_and_transposed_out_edges(device_arrays, give_out_edges):
    """tfps_graph_create from host arrays and from device arrays (ptr_space = TFPS_DEVICE), with the out-edge CSR
    given and with all three out-edge arrays NULL (built by transposing the in-edges): same results as the oracle,
    with and without per-vertex memory, int32 and int64 edge sizes."""
    from paper_1711_01912_b200 import tfps
    import oracle
    torch = _torch()
    for w in (I.config1(), I.small_random(321, 400, 1500, 5, 70, t_dtype=np.int32, with_mem=False),
              I.small_random(322, 300, 900, 3, 40, with_mem=True)):
        g, d = w.graph, w.devices
        c = I.to_csr(g)
        outs = (c.out_ptr, c.out_dst, c.out_t) if give_out_edges else (None, None, None)
        G = tfps.Graph(g.n, c.in_ptr, c.in_src, c.in_t, g.c, outs[0], outs[1], outs[2], g.mem, device_arrays=device_arrays)
        G.devices_set(d.k, d.s, d.C, d.B, d.scale)
        part = w.part_full()
        dpart, P, ldp = padded(part)
        ref = oracle.eval_batch(oracle_graph(g), d.k, d.s, d.C, d.B, d.scale, part)
        for flags in VARIANTS:
            out = G.eval_batch(dpart, P, flags=flags, out={})
            assert np.array_equal(out["tlevel"].cpu().numpy()[:, :P], ref.tlevel)
            assert np.array_equal(out["blevel"].cpu().numpy()[:, :P], ref.blevel)
            assert np.array_equal(out["cp"].cpu().numpy()[:P], ref.cp)
            assert np.array_equal(out["load"].cpu().numpy()[:, :P], ref.load)
            assert np.array_equal(out["memload"].cpu().numpy()[:, :P], ref.memload)
            assert np.array_equal(out["viol"].cpu().numpy().view(np.uint64)[:P], ref.viol)
        G.close()


def test_config1_relabelled():
    w = I.config1()
    g2, perm = I.relabel(w.graph, 5)
    part = w.part_full()
    part2 = np.empty_like(part)
    part2[perm] = part
    run_and_compare(g2, w.devices, part2, 2)
    run_and_compare(g2, w.devices, part2, 1)


# ----------------------------------------------------------------- topological levels
@pytest.mark.parametrize("maker", [I.config1, I.config2, I.config3, I.config4])
def test_topo_levels_match_oracle(maker):
    w = maker()
    g, _ = I.relabel(w.graph, 9)
    og = oracle_graph(g)
    G = gpu_graph(g)
    level, order, lp, L = G.topo_levels()
    assert L == og.num_levels
    assert np.array_equal(lp, og.level_ptr)
    assert np.array_equal(level.cpu().numpy(), og.level)
    assert np.array_equal(order.cpu().numpy(), og.order)
    G.close()


# ------------------------------------------------------------------- awkward shapes
@pytest.mark.parametrize("flags", VARIANTS)
@pytest.mark.parametrize("n,m,k,P,tdt", [
    (1, 0, 1, 1, np.int64), (2, 1, 2, 3, np.int32), (37, 90, 3, 17, np.int64), (300, 900, 5, 33, np.int32),
    (513, 2000, 8, 70, np.int64), (1000, 2500, 64, 48, np.int64), (257, 700, 16, 129, np.int32),
    (64, 0, 4, 40, np.int64), (700, 3000, 2, 1000, np.int64),
])
def test_random_small_graphs(n, m, k, P, tdt, flags):
    w = I.small_random(1000 + n + P, n, m, k, P, t_dtype=tdt, with_mem=(n % 2 == 1))
    part = w.part_full()
    # garbage in the padding columns must be ignored (and must not be validated)
    run_and_compare(w.graph, w.devices, part, flags, pad_fill=255)


@pytest.mark.parametrize("which", [0, 1])
def test_paper_shaped_graphs_k50(which):
    w = I.paper_shaped(which)
    run_and_compare(w.graph, w.devices, w.part_full(), 2)
    run_and_compare(w.graph, w.devices, w.part_full(), 1)


def test_parallel_edges_zero_costs_isolated_vertices():
    edges = [(0, 1, 10), (0, 1, 5000), (1, 2, 0), (0, 2, 7)]
    g = graph_from_edges(5, edges, [3, 0, 4, 9, 0])
    dev = I.Devices(3, np.array([1, 2, 5], np.int32), np.array([10, 5000, INF], np.int64),
                    np.array([[0, 3, 1], [7, 0, 2], [1, 1, 0]], np.int64), scale=5)
    rng = np.random.default_rng(3)
    part = rng.integers(0, 3, size=(5, 27), dtype=np.uint8)
    for flags in VARIANTS:
        run_and_compare(g, dev, part, flags)


def test_extreme_magnitudes_exact_division():
    # large t, large and tiny bandwidths, large scale: exercises the division constants at the domain's edge
    rng = np.random.default_rng(17)
    n = 64
    w = I.small_random(5, n, 200, 6, 40)
    g = w.graph
    t = rng.integers(0, 2 ** 40, size=g.m).astype(np.int64)
    t[:8] = [0, 1, 2, 2 ** 40, 2 ** 40 - 1, 3, 2 ** 39, 2 ** 20 + 1]
    g = I.Graph(n=n, src=g.src, dst=g.dst, t=t, c=rng.integers(0, 2 ** 31 - 1, size=n).astype(np.int32), mem=None, layers=0)
    B = rng.integers(1, 2 ** 40, size=(6, 6)).astype(np.int64)
    B[0, 1] = 1; B[1, 0] = 2; B[2, 3] = 3; B[3, 2] = 2 ** 40; B[4, 5] = 2 ** 31 - 1; B[5, 4] = 2 ** 31 + 1
    dev = I.Devices(6, np.array([1, 2, 3, 7, 2 ** 31 - 1, 65536], np.int32), np.full(6, INF, np.int64), B, scale=2 ** 12 - 1)
    for flags in VARIANTS:
        run_and_compare(g, dev, w.part_full(), flags)


# -------------------------------------------------------------------- option handling
def test_cp_only_uses_workspace_and_matches():
    import oracle
    from paper_1711_01912_b200 import tfps
    w = I.config2()
    part = w.part_full()[:, :100]
    G = gpu_graph(w.graph, w.devices)
    dpart, P, ldp = padded(part)
    og = oracle_graph(w.graph)
    d = w.devices
    ref = oracle.eval_batch(og, d.k, d.s, d.C, d.B, d.scale, part, want_levels=False)
    for flags in VARIANTS:
        out = G.eval_batch(dpart, P, want=("cp",), flags=flags)
        assert np.array_equal(out["cp"].cpu().numpy(), ref.cp)
        out = G.eval_batch(dpart, P, want=("cp", "blevel"), flags=flags)  # CP from the backward pass alone
        assert np.array_equal(out["cp"].cpu().numpy(), ref.cp)
        out = G.eval_batch(dpart, P, want=("viol",), flags=flags)
        assert np.array_equal(out["viol"].cpu().numpy().view(np.uint64), ref.viol)
    G.close()


def test_host_entry_point_matches():
    import oracle
    w = I.config2()
    part = w.part_full()[:, :200]
    G = gpu_graph(w.graph, w.devices)
    n, P = part.shape
    ldp = 208
    buf = np.zeros((n, ldp), np.uint8); buf[:, :P] = part
    res = G.eval_batch_host(buf, P, want=("tlevel", "blevel", "cp", "load", "memload", "viol"))
    og = oracle_graph(w.graph)
    d = w.devices
    ref = oracle.eval_batch(og, d.k, d.s, d.C, d.B, d.scale, part)
    assert np.array_equal(res["tlevel"][:, :P], ref.tlevel)
    assert np.array_equal(res["blevel"][:, :P], ref.blevel)
    assert np.array_equal(res["cp"], ref.cp)
    assert np.array_equal(res["load"][:, :P], ref.load)
    assert np.array_equal(res["memload"][:, :P], ref.memload)
    assert np.array_equal(res["viol"], ref.viol)
    G.close()


def test_host_entry_point_pipelined_in_two_column_chunks():
    """Enough candidates for the host entry point to upload and evaluate in two column chunks."""
    import oracle
    w = I.config1()
    n = w.graph.n
    P = 15000
    ldp = 15008
    rng = np.random.default_rng(9)
    buf = rng.integers(0, w.devices.k, size=(n, ldp), dtype=np.uint8)
    G = gpu_graph(w.graph, w.devices)
    res = G.eval_batch_host(buf, P, want=("tlevel", "blevel", "cp", "load", "memload", "viol"))
    og = oracle_graph(w.graph)
    d = w.devices
    cols = [0, 1, 7423, 7424, 7551, 7552, 7553, 14999]   # both sides of the chunk boundary
    ref = oracle.eval_batch(og, d.k, d.s, d.C, d.B, d.scale, buf, cols)
    assert np.array_equal(res["tlevel"][:, cols], ref.tlevel)
    assert np.array_equal(res["blevel"][:, cols], ref.blevel)
    assert np.array_equal(res["cp"][cols], ref.cp)
    assert np.array_equal(res["load"][:, cols], ref.load)
    assert np.array_equal(res["memload"][:, cols], ref.memload)
    assert np.array_equal(res["viol"][cols], ref.viol)
    # every candidate: CP = max_v(tlevel + blevel)
    assert np.array_equal((res["tlevel"][:, :P] + res["blevel"][:, :P]).max(axis=0), res["cp"][:P])
    G.close()


def test_transpose_u8():
    from paper_1711_01912_b200 import tfps
    torch = _torch()
    rng = np.random.default_rng(0)
    for P, n in [(1, 1), (70, 130), (64, 64), (333, 1000)]:
        src = rng.integers(0, 255, size=(P, n), dtype=np.uint8)
        dst = tfps.transpose_u8(torch.from_numpy(src).cuda())
        assert np.array_equal(dst.cpu().numpy()[:, :P], src.T)
        assert (dst[:, P:] == 0).all()


def test_deterministic_repeat():
    torch = _torch()
    w = I.config2()
    G = gpu_graph(w.graph, w.devices)
    dpart, P, ldp = padded(w.part_full())
    a = G.eval_batch(dpart, P, flags=2)
    b = G.eval_batch(dpart, P, flags=2, out={})
    for kname in ("tlevel", "blevel", "cp", "load", "memload", "viol"):
        assert torch.equal(a[kname], b[kname])
    G.close()


# ------------------------------------------------------------------------- errors
def test_error_codes():
    from paper_1711_01912_b200 import tfps
    torch = _torch()
    # cycle
    g = graph_from_edges(3, [(0, 1, 1), (1, 2, 1), (2, 0, 1)], [1, 1, 1])
    G = gpu_graph(g)
    with pytest.raises(tfps.TfpsError) as ei:
        G.topo_levels()
    assert ei.value.code == tfps.ERR_CYCLE
    with pytest.raises(tfps.TfpsError) as ei:
        G.devices_set(1, [1], [INF], [[0]], 1)
    assert ei.value.code == tfps.ERR_CYCLE
    G.close()
    # self loop
    c = I.to_csr(graph_from_edges(2, [(0, 1, 1)], [1, 1]))
    bad_src = c.in_src.copy(); bad_src[0] = 1
    with pytest.raises(tfps.TfpsError) as ei:
        tfps.Graph(2, c.in_ptr, bad_src, c.in_t, [1, 1])
    assert ei.value.code == tfps.ERR_CYCLE
    # malformed CSR
    w = I.config1()
    c = I.to_csr(w.graph)
    p2 = c.in_ptr.copy(); p2[5] = p2[4] - 1
    with pytest.raises(tfps.TfpsError) as ei:
        tfps.Graph(w.graph.n, p2, c.in_src, c.in_t, w.graph.c)
    assert ei.value.code == tfps.ERR_BAD_CSR
    s2 = c.in_src.copy(); s2[3] = w.graph.n
    with pytest.raises(tfps.TfpsError) as ei:
        tfps.Graph(w.graph.n, c.in_ptr, s2, c.in_t, w.graph.c)
    assert ei.value.code == tfps.ERR_BAD_CSR
    t2 = c.out_t.copy(); t2[7] += 1  # in/out multisets differ
    with pytest.raises(tfps.TfpsError) as ei:
        tfps.Graph(w.graph.n, c.in_ptr, c.in_src, c.in_t, w.graph.c, c.out_ptr, c.out_dst, t2)
    assert ei.value.code == tfps.ERR_BAD_CSR
    # devices
    G = gpu_graph(w.graph)
    d = w.devices
    with pytest.raises(tfps.TfpsError) as ei:
        G.eval_batch(torch.zeros((w.graph.n, 16), dtype=torch.uint8, device="cuda"), 4)
    assert ei.value.code == tfps.ERR_STATE
    with pytest.raises(tfps.TfpsError) as ei:
        G.devices_set(65, np.ones(65), np.ones(65), np.ones((65, 65)), 1)
    assert ei.value.code == tfps.ERR_BAD_DEVICES
    with pytest.raises(tfps.TfpsError) as ei:
        G.devices_set(2, [1, 0], d.C, d.B, 16)
    assert ei.value.code == tfps.ERR_BAD_DEVICES
    with pytest.raises(tfps.TfpsError) as ei:
        G.devices_set(2, d.s, d.C, [[0, 0], [5, 0]], 16)
    assert ei.value.code == tfps.ERR_BAD_DEVICES
    with pytest.raises(tfps.TfpsError) as ei:
        G.devices_set(2, d.s, d.C, d.B, 2 ** 45)
    assert ei.value.code == tfps.ERR_OVERFLOW
    G.devices_set(d.k, d.s, d.C, d.B, d.scale)
    # bad ldp, missing workspace
    part = torch.zeros((w.graph.n, 16), dtype=torch.uint8, device="cuda")
    with pytest.raises(tfps.TfpsError) as ei:
        tfps.tfps_eval_batch(G.handle, 20, 16, part.data_ptr(), None, None, None, None, None, None, None, 0, 0, 0)
    assert ei.value.code == tfps.ERR_INVALID_ARG
    cp = torch.zeros(16, dtype=torch.int64, device="cuda")
    with pytest.raises(tfps.TfpsError) as ei:
        tfps.tfps_eval_batch(G.handle, 16, 16, part.data_ptr(), None, None, cp.data_ptr(), None, None, None, None, 0, 0, 0)
    assert ei.value.code == tfps.ERR_WORKSPACE
    # pointers the 16-byte vector accesses of the kernels cannot take are refused before anything is launched
    lev = torch.zeros((5 * 16 + 2,), dtype=torch.int64, device="cuda")
    for bad in (dict(part=part.data_ptr() + 1), dict(tlevel=lev.data_ptr() + 8), dict(blevel=lev.data_ptr() + 8), dict(cp=cp.data_ptr() + 8)):
        a = dict(part=part.data_ptr(), tlevel=lev.data_ptr(), blevel=None, cp=cp.data_ptr())
        a.update(bad)
        with pytest.raises(tfps.TfpsError) as ei:
            tfps.tfps_eval_batch(G.handle, 16, 16, a["part"], a["tlevel"], a["blevel"], a["cp"], None, None, None, None, 0, 0, 0)
        assert ei.value.code == tfps.ERR_INVALID_ARG, bad
    # P == 0: nothing happens
    tfps.tfps_eval_batch(G.handle, 0, 16, part.data_ptr(), None, None, None, None, None, None, None, 0, 0, 0)
    # id >= k is reported through the status word and the context stays usable
    part[5, 3] = 2
    for flags in VARIANTS:
        with pytest.raises(tfps.TfpsError) as ei:
            G.eval_batch(part, 16, flags=flags)
        assert ei.value.code == tfps.ERR_BAD_PARTITION
        with pytest.raises(tfps.TfpsError) as ei:
            G.eval_batch(part, 16, want=("cp",), flags=flags)
        assert ei.value.code == tfps.ERR_BAD_PARTITION
    part[5, 3] = 1
    out = G.eval_batch(part, 16)
    assert (out["cp"] > 0).all()
    G.close()


# ------------------------------------------------------ kernel shapes of the sliced pass
@pytest.mark.parametrize("table", [0, 1])
@pytest.mark.parametrize("cpt", [1, 2, 4, 8])
def test_sliced_kernel_shapes(cpt, table, monkeypatch):
    """Every candidates-per-lane width, with the per-edge cost table on and off,
    on device tables that exercise each table-building path: few distinct values
    (classes), many distinct values with k*k <= 64 (per-entry division), k = 16
    grouped (8 table passes) and k = 50 (no table: direct division)."""
    monkeypatch.setenv("TFPS_SLICED_CPT", str(cpt))
    monkeypatch.setenv("TFPS_SLICED_TABLE", str(table))
    monkeypatch.setenv("TFPS_SLICED_WARPS", "4")
    monkeypatch.setenv("TFPS_LEAN", "0")
    for g, dev, part in _shape_cases(cpt * 2 + table):
        run_and_compare(g, dev, part, 2, pad_fill=255)


def _shape_cases(seed):
    rng = np.random.default_rng(seed)
    cpt = seed // 2
    cases = []
    w = I.small_random(70 + cpt, 300, 900, 3, 77)          # classes, one pass
    cases.append((w.graph, w.devices, w.part_full()))
    w = I.small_random(80 + cpt, 400, 1300, 8, 300)        # 56 distinct bandwidths: per-entry division, two passes
    cases.append((w.graph, w.devices, w.part_full()))
    w = I.config5(layers=12, width=64, P=100)               # k = 16 grouped: classes, eight passes, fan-in up to 64
    cases.append((w.graph, w.devices, w.part_full()))
    w = I.paper_shaped(0)                                   # k = 50
    cases.append((w.graph, w.devices, w.part_full()))
    # a vertex with more in-edges than a staged chunk holds
    n = 700
    edges = [(u, n - 1, int(rng.integers(0, 10 ** 6))) for u in range(n - 1)] + [(0, u, 5) for u in range(1, 40)]
    g = graph_from_edges(n, edges, rng.integers(0, 100, size=n))
    dev = I.Devices(4, np.array([1, 2, 2, 4], np.int32), np.full(4, INF, np.int64),
                    np.array([[0, 10, 10, 7], [10, 0, 7, 7], [3, 3, 0, 10], [7, 10, 3, 0]], np.int64), scale=3)
    cases.append((g, dev, rng.integers(0, 4, size=(n, 45), dtype=np.uint8)))
    return cases


def _small_costs(g):
    """Same graph with edge sizes below 50,000, so that every path length fits 32 bits."""
    return I.Graph(n=g.n, src=g.src, dst=g.dst, t=(g.t % 50000).astype(g.t.dtype), c=g.c, mem=g.mem, layers=g.layers)


def _grouped_devices(k, rng):
    """Two speeds and three bandwidths in groups of two: few distinct values, asymmetric."""
    s = np.where(np.arange(k) % 2 == 0, 3, 11).astype(np.int32)
    grp = np.arange(k) // 2
    B = np.where(grp[:, None] == grp[None, :], 900, 70).astype(np.int64)
    B[np.triu_indices(k, 1)] += 13
    return I.Devices(k, s, np.full(k, INF, np.int64), B, scale=int(rng.integers(1, 40)))


@pytest.mark.parametrize("slice_,cpt", [(16, 1), (16, 2), (16, 4), (32, 1), (32, 2), (64, 2)])
def test_lean_kernel_candidates_per_lane(slice_, cpt, monkeypatch):
    """The lean windowed pass with 1, 2 or 4 candidates per lane (a vertex is served by slice / cpt lanes): the deep
    narrow graph, the wide graph, a random graph with k = 8 and ragged candidate counts."""
    from paper_1711_01912_b200 import tfps
    monkeypatch.setenv("TFPS_LEAN_SLICE", str(slice_))
    monkeypatch.setenv("TFPS_LEAN_CPT", str(cpt))
    rng = np.random.default_rng(slice_ * 10 + cpt)
    w = I.config4()
    g = w.graph
    keep = g.dst < 16 * 120
    g4 = I.Graph(n=16 * 120, src=g.src[keep], dst=g.dst[keep], t=g.t[keep], c=g.c[:16 * 120], mem=None, layers=120)
    cases = [(g4, w.devices, w.part_rows(0, 16 * 120)[:, :83])]
    w = I.config3()
    g = w.graph
    keep = g.dst < 128 * 8
    g3 = I.Graph(n=128 * 8, src=g.src[keep], dst=g.dst[keep], t=g.t[keep], c=g.c[:128 * 8], mem=None, layers=8)
    cases.append((g3, w.devices, w.part_rows(0, 128 * 8)[:, :130]))
    w = I.small_random(9300 + slice_ + cpt, 700, 2500, 8, 77)
    cases.append((_small_costs(w.graph), _grouped_devices(8, rng), w.part_full()))
    for g, dev, part in cases:
        run_and_compare(g, dev, part, 2, pad_fill=255)
    G = gpu_graph(cases[0][0], cases[0][1])
    dpart, P, ldp = padded(cases[0][2])
    G.eval_batch(dpart, P, flags=2)
    assert tfps.tfps_last_pass_kernel(G.handle) == "pass_lean_kernel"
    G.close()


@pytest.mark.parametrize("depth", [1, 3])
@pytest.mark.parametrize("slice_,warps", [(16, 1), (16, 8), (32, 4), (64, 2), (64, 32), (128, 16)])
def test_lean_kernel_shapes(slice_, warps, depth, monkeypatch):
    """The lean windowed pass for every block shape (candidates per block, warps, stage depth): graphs with
    wide and narrow levels, ragged candidate counts, k up to 8 with few and with many distinct bandwidths,
    zero costs, vertices of high degree; device tables it does not take (k > 8, more than 30 distinct
    bandwidths) fall back to the older kernels and must agree as well."""
    from paper_1711_01912_b200 import tfps
    monkeypatch.setenv("TFPS_LEAN", "1")
    monkeypatch.setenv("TFPS_LEAN_SLICE", str(slice_))
    monkeypatch.setenv("TFPS_SLICED_WARPS", str(warps))
    monkeypatch.setenv("TFPS_LEAN_DEPTH", str(depth))
    rng = np.random.default_rng(slice_ * 100 + warps)
    took = []
    cases = []
    for (n, m, k, P) in [(1, 0, 1, 1), (50, 120, 2, 16), (700, 2500, 8, 77), (1500, 9000, 5, 150), (400, 0, 3, 33)]:
        w = I.small_random(9000 + n + slice_, n, m, k, P, t_dtype=np.int64 if n % 2 else np.int32, with_mem=bool(n % 3))
        dev = w.devices if k < 4 else _grouped_devices(k, rng)
        cases.append((_small_costs(w.graph), dev, w.part_full()))
    w = I.small_random(9100 + slice_, 600, 2000, 6, 90)       # 30 distinct bandwidths: the most the lean pass takes
    cases.append((_small_costs(w.graph), w.devices, w.part_full()))
    w = I.small_random(9200 + slice_, 500, 1500, 7, 40)       # 42 distinct bandwidths: falls back
    cases.append((_small_costs(w.graph), w.devices, w.part_full()))
    w = I.config3()
    g = w.graph
    keep = g.dst < 128 * 12   # first 12 layers of the wide graph (levels of 128 vertices)
    g3 = I.Graph(n=128 * 12, src=g.src[keep], dst=g.dst[keep], t=g.t[keep], c=g.c[:128 * 12], mem=None, layers=12)
    cases.append((g3, w.devices, w.part_rows(0, 128 * 12)[:, :200]))
    w = I.config4()
    g = w.graph
    keep = g.dst < 16 * 200
    g4 = I.Graph(n=16 * 200, src=g.src[keep], dst=g.dst[keep], t=g.t[keep], c=g.c[:16 * 200], mem=None, layers=200)
    cases.append((g4, w.devices, w.part_rows(0, 16 * 200)[:, :97]))
    n = 900   # one vertex with 899 in-edges, a level of 860 vertices
    edges = [(u, n - 1, int(rng.integers(0, 10 ** 6))) for u in range(n - 1)] + [(0, u, 5) for u in range(1, 40)]
    gh = graph_from_edges(n, edges, rng.integers(0, 100, size=n))
    cases.append((gh, _grouped_devices(4, rng), rng.integers(0, 4, size=(n, 45), dtype=np.uint8)))
    for g, dev, part in cases:
        run_and_compare(g, dev, part, 2, pad_fill=255)
        G = gpu_graph(g, dev)
        dpart, P, ldp = padded(part)
        G.eval_batch(dpart, P, flags=2)
        took.append(tfps.tfps_last_pass_kernel(G.handle) == "pass_lean_kernel")
        G.close()
    # which cases the lean pass takes depends on the block shape (the window of a graph with long edges does not
    # fit beside wide slices); the deep narrow graph always fits, the table with 42 bandwidths never does
    assert took[8] and sum(took) >= 3 and not took[6], f"kernel choice per case: {took}"


@pytest.mark.parametrize("depth", [1, 3])
@pytest.mark.parametrize("slice_,warps", [(8, 1), (8, 8), (16, 2), (32, 4), (64, 16), (128, 8)])
def test_lean64_kernel_shapes(slice_, warps, depth, monkeypatch):
    """The wide lean pass (int64 levels, up to 16 devices) for every block shape: path lengths beyond 32 bits,
    k = 9..16 with grouped tables, the cases of the narrow pass forced onto the wide kernel, zero costs, a vertex
    of high degree, ragged candidate counts; k = 17 and tables with more than 30 bandwidths fall back."""
    from paper_1711_01912_b200 import tfps
    monkeypatch.setenv("TFPS_LEAN", "1")
    monkeypatch.setenv("TFPS_LEAN_FORCE_WIDE", "1")
    monkeypatch.setenv("TFPS_LEAN_SLICE", str(slice_))
    monkeypatch.setenv("TFPS_SLICED_WARPS", str(warps))
    monkeypatch.setenv("TFPS_LEAN_DEPTH", str(depth))
    rng = np.random.default_rng(slice_ * 1000 + warps)
    cases = []
    for (n, m, k, P) in [(1, 0, 1, 1), (60, 150, 2, 9), (700, 2500, 16, 77), (900, 5000, 12, 130), (300, 0, 9, 33)]:
        w = I.small_random(9500 + n + slice_, n, m, k, P, t_dtype=np.int64, with_mem=bool(n % 3))   # t up to 2^36
        dev = w.devices if k < 4 else _grouped_devices(k, rng)
        cases.append((w.graph, dev, w.part_full()))
    w = I.small_random(9600 + slice_, 400, 1200, 17, 40)        # k = 17: not taken
    cases.append((w.graph, _grouped_devices(17, rng), w.part_full()))
    w = I.config4()
    g = w.graph
    keep = g.dst < 16 * 200
    g4 = I.Graph(n=16 * 200, src=g.src[keep], dst=g.dst[keep], t=g.t[keep], c=g.c[:16 * 200], mem=None, layers=200)
    cases.append((g4, w.devices, w.part_rows(0, 16 * 200)[:, :97]))
    w = I.config5(layers=12, width=64, P=100)                    # k = 16, int64 path lengths, fan-in up to 64
    cases.append((w.graph, w.devices, w.part_full()))
    took = []
    for g, dev, part in cases:
        run_and_compare(g, dev, part, 2, pad_fill=255)
        G = gpu_graph(g, dev)
        dpart, P, ldp = padded(part)
        G.eval_batch(dpart, P, flags=2)
        took.append(tfps.tfps_last_pass_kernel(G.handle) == "pass_lean64_kernel")
        G.close()
    # the deep narrow graph always fits; k = 17 never does
    assert took[6] and sum(took) >= 3 and not took[5], f"kernel choice per case: {took}"


@pytest.mark.parametrize("wide", [0, 1])
def test_lean_plan_in_callers_vertex_order(wide, monkeypatch):
    """The lean plan walked in the caller's vertex numbering (TFPS_LEAN_ORDER=2) instead of level order: graphs
    numbered layer by layer take it, a randomly relabelled graph is not topologically numbered and keeps the level
    order; results are the same either way."""
    from paper_1711_01912_b200 import tfps
    monkeypatch.setenv("TFPS_LEAN_ORDER", "2")
    monkeypatch.setenv("TFPS_LEAN_FORCE_WIDE", str(wide))
    w = I.config3()
    g = w.graph
    keep = g.dst < 128 * 10
    g3 = I.Graph(n=128 * 10, src=g.src[keep], dst=g.dst[keep], t=g.t[keep], c=g.c[:128 * 10], mem=None, layers=10)
    part3 = w.part_rows(0, 128 * 10)[:, :150]
    run_and_compare(g3, w.devices, part3, 2, pad_fill=255)
    g3r, perm = I.relabel(g3, 5)
    part3r = np.empty_like(part3)
    part3r[perm] = part3
    run_and_compare(g3r, w.devices, part3r, 2, pad_fill=255)
    w5 = I.config5(layers=40, width=64, P=70)   # edges reach four layers back: the numbering has the shorter edges
    dev5 = w5.devices
    run_and_compare(w5.graph, dev5, w5.part_full(), 2, pad_fill=255)
    w4 = I.config4()
    g = w4.graph
    keep = g.dst < 16 * 150
    g4 = I.Graph(n=16 * 150, src=g.src[keep], dst=g.dst[keep], t=g.t[keep], c=g.c[:16 * 150], mem=None, layers=150)
    run_and_compare(g4, w4.devices, w4.part_rows(0, 16 * 150)[:, :50], 2, pad_fill=255)


@pytest.mark.parametrize("levrec", [0, 1, 2])
@pytest.mark.parametrize("split", [1, 3, 8])
def test_level_kernels_with_partial_items(split, levrec, monkeypatch):
    """The step-synchronous kernels (0: per-relaxation division kernel, 1: record pass with one launch per step,
    2: persistent record pass) with vertices of many edges cut into partial work items of at most `split` edges: a
    hub with hundreds of in-edges next to vertices of degree one, the power-law fan-in graph with k = 16, a graph
    with k = 17 (record pass with the 64-device tables)."""
    from paper_1711_01912_b200 import tfps
    monkeypatch.setenv("TFPS_TILE_SPLIT", str(split))
    monkeypatch.setenv("TFPS_LEVREC", "1" if levrec else "0")
    monkeypatch.setenv("TFPS_STEP_PERSISTENT", "1" if levrec == 2 else "0")
    rng = np.random.default_rng(77 + split)
    n = 700
    edges = [(u, n - 1, int(rng.integers(0, 10 ** 6))) for u in range(n - 1)] + [(0, u, 5) for u in range(1, 60)]
    gh = graph_from_edges(n, edges, rng.integers(0, 100, size=n))
    run_and_compare(gh, _grouped_devices(4, rng), rng.integers(0, 4, size=(n, 45), dtype=np.uint8), 1, pad_fill=255)
    w = I.config5(layers=14, width=64, P=130)
    out = run_and_compare(w.graph, w.devices, w.part_full(), 1, pad_fill=255)
    G = gpu_graph(w.graph, w.devices)
    dpart, P, ldp = padded(w.part_full())
    G.eval_batch(dpart, P, flags=1)
    assert tfps.tfps_last_pass_kernel(G.handle) == ["pass_level_kernel", "pass_stepchain_kernel", "pass_steprec_kernel"][levrec]
    G.close()
    w = I.small_random(4242 + split, 500, 3000, 17, 40)
    run_and_compare(w.graph, w.devices, w.part_full(), 1, pad_fill=255)


@pytest.mark.parametrize("split", [1, 3, 8])
def test_dataflow_record_pass(split, monkeypatch):
    """The dataflow form of the record pass (ready bits per vertex and candidate tile instead of grid-wide steps): a
    ragged pair of tiles, exactly one tile, nine tiles with a ragged last one, sixteen tiles, a hub of hundreds
    of in-edges cut into partial items next to vertices without edges, a chain (every item waits for the one before);
    batches beyond 32 tiles take the chained launches."""
    from paper_1711_01912_b200 import tfps
    monkeypatch.setenv("TFPS_TILE_SPLIT", str(split))
    monkeypatch.setenv("TFPS_STEP_FLOW", "1")
    rng = np.random.default_rng(177 + split)
    for P in (300, 256, 2100, 4096):
        w = I.config5(layers=14, width=64, P=P)
        run_and_compare(w.graph, w.devices, w.part_full(), 1, pad_fill=255)
    G = gpu_graph(w.graph, w.devices)
    dpart, P, ldp = padded(w.part_full())
    G.eval_batch(dpart, P, flags=1)
    assert tfps.tfps_last_pass_kernel(G.handle) == "pass_flow_kernel"
    G.close()
    n = 700
    edges = [(u, n - 1, int(rng.integers(0, 10 ** 6))) for u in range(n - 1)] + [(0, u, 5) for u in range(1, 60)]
    gh = graph_from_edges(n, edges, rng.integers(0, 100, size=n))
    run_and_compare(gh, _grouped_devices(4, rng), rng.integers(0, 4, size=(n, 270), dtype=np.uint8), 1, pad_fill=255)
    n = 3000
    chain = graph_from_edges(n, [(u, u + 1, int(rng.integers(0, 10 ** 5))) for u in range(n - 1)], rng.integers(0, 100, size=n))
    run_and_compare(chain, _grouped_devices(4, rng), rng.integers(0, 4, size=(n, 200), dtype=np.uint8), 1, pad_fill=255)
    w = I.config5(layers=9, width=32, P=8300)
    run_and_compare(w.graph, w.devices, w.part_full(), 1, pad_fill=255)


def test_loads_kernel_table_widths():
    """Loads, memory loads and violation flags for every width of the runtime table (k = 1 .. 32) and beyond
    it (k = 33, 64: the shuffle-based kernel), with bounded capacities so that some flags are set."""
    for k in (1, 2, 3, 5, 8, 9, 16, 17, 32, 33, 64):
        w = I.small_random(7000 + k, 300, 700, k, 130, with_mem=bool(k % 2))
        d = w.devices
        memsum = int(np.sum(w.graph.mem)) if w.graph.mem is not None else int(np.sum(w.graph.t))
        dev = I.Devices(k, d.s, np.full(k, max(1, memsum // max(1, k - 1)), np.int64), d.B, d.scale)
        run_and_compare(w.graph, dev, w.part_full(), 0, pad_fill=255)


def test_loads_kernel_value_ranges():
    """Loads and memory loads over the value ranges an accumulator has to hold: all-small costs, all-huge costs and
    memory sizes (sums far beyond 2^32), huge values in the first rows only, per-block sums just below / exactly at
    2^32, with candidates that put every vertex on one device."""
    rng = np.random.default_rng(99)
    w = I.small_random(4242, 1500, 3000, 4, 130, with_mem=True)
    g0 = w.graph
    n = g0.n
    dev = I.Devices(4, np.ones(4, np.int32), np.full(4, INF, np.int64), w.devices.B, scale=1)
    part = w.part_full().copy()
    part[:, 0] = 0          # every vertex on device 0
    part[:, 1] = 3
    cases = []
    cases.append((rng.integers(0, 1000, size=n).astype(np.int32), rng.integers(0, 1000, size=n).astype(np.int64)))
    cases.append((np.full(n, 2 ** 31 - 1, np.int32), rng.integers(2 ** 33, 2 ** 40, size=n).astype(np.int64)))
    c = rng.integers(0, 1000, size=n).astype(np.int32)
    mem = rng.integers(0, 1000, size=n).astype(np.int64)
    c[:40] = 2 ** 31 - 1
    mem[5:90] = 2 ** 36 + 17
    cases.append((c, mem))
    cases.append((np.full(n, 2 ** 24 - 1, np.int32), np.full(n, 2 ** 24 - 1, np.int64)))   # 256 rows: 2^32 - 256
    cases.append((np.full(n, 2 ** 24, np.int32), np.full(n, 2 ** 24, np.int64)))           # 256 rows: exactly 2^32
    cases.append((np.full(n, 5, np.int32), np.full(n, 2 ** 32 - 1, np.int64)))
    for c, mem in cases:
        g = I.Graph(n=n, src=g0.src, dst=g0.dst, t=g0.t, c=c, mem=mem, layers=g0.layers)
        run_and_compare(g, dev, part, 0, pad_fill=255)


# ------------------------------------------------------------- randomized sweep
def test_randomized_shapes_all_variants():
    """Forty seeded random workloads (sizes, device counts, candidate counts, dtypes, device-table structure
    drawn at random), each evaluated by the automatic choice and by both forced kernel families."""
    rng = np.random.default_rng(2024)
    for trial in range(40):
        n = int(rng.integers(1, 900))
        m = int(rng.integers(0, 4 * n))
        k = int(rng.choice([1, 2, 3, 4, 5, 8, 12, 16, 17, 33, 64]))
        P = int(rng.choice([1, 7, 31, 32, 33, 64, 100, 257]))
        tdt = np.int32 if trial % 2 else np.int64
        w = I.small_random(5000 + trial, n, m, k, P, t_dtype=tdt, with_mem=bool(trial % 3))
        dev = w.devices
        if trial % 4 == 0 and k > 1:   # structured tables: two speeds, two bandwidths (value classes)
            s = np.where(np.arange(k) % 2 == 0, 3, 11).astype(np.int32)
            grp = np.arange(k) // 2
            B = np.where(grp[:, None] == grp[None, :], 900, 70).astype(np.int64)
            dev = I.Devices(k, s, dev.C, B, scale=int(rng.integers(1, 40)))
        part = w.part_full()
        for flags in (0, 1, 2):
            run_and_compare(w.graph, dev, part, flags, pad_fill=255)


@pytest.mark.parametrize("warps,wide,rec_v", [(16, 8, 64), (1, 4, 4), (5, 8, 16), (31, 6, 64)])
def test_ring_pass(warps, wide, rec_v, monkeypatch):
    """The ring pass (blocks of eight candidates, finish times of the last R vertices in shared memory): ragged and
    single slices, records of a few vertices (every stage slot is reused many times), wide rounds for vertices with many
    edges next to vertices without any, a hub of hundreds of in-edges, a chain (one vertex per step), more than 16
    devices, a relabelled graph (steps are the topological levels) and a caller's order (steps cut from the numbering)."""
    from paper_1711_01912_b200 import tfps
    monkeypatch.setenv("TFPS_RING", "2")
    monkeypatch.setenv("TFPS_LEAN", "0")
    monkeypatch.setenv("TFPS_RING_WARPS", str(warps))
    monkeypatch.setenv("TFPS_RING_WIDE", str(wide))
    monkeypatch.setenv("TFPS_RING_REC_V", str(rec_v))
    rng = np.random.default_rng(977 + warps)
    for P in (300, 8, 13, 1000):
        w = I.config5(layers=14, width=64, P=P)
        run_and_compare(w.graph, w.devices, w.part_full(), 0, pad_fill=255)
    G = gpu_graph(w.graph, w.devices)
    dpart, P, ldp = padded(w.part_full())
    G.eval_batch(dpart, P, flags=0)
    assert tfps.tfps_last_pass_kernel(G.handle) == "pass_ring_kernel"
    G.close()
    n = 700
    edges = [(u, n - 1, int(rng.integers(0, 10 ** 6))) for u in range(n - 1)] + [(0, u, 5) for u in range(1, 60)]
    gh = graph_from_edges(n, edges, rng.integers(0, 100, size=n))
    run_and_compare(gh, _grouped_devices(4, rng), rng.integers(0, 4, size=(n, 270), dtype=np.uint8), 0, pad_fill=255)
    n = 3000
    chain = graph_from_edges(n, [(u, u + 1, int(rng.integers(0, 10 ** 5))) for u in range(n - 1)], rng.integers(0, 100, size=n))
    run_and_compare(chain, _grouped_devices(4, rng), rng.integers(0, 4, size=(n, 40), dtype=np.uint8), 0, pad_fill=255)
    w = I.small_random(5151 + warps, 500, 3000, 17, 40)
    run_and_compare(w.graph, w.devices, w.part_full(), 0, pad_fill=255)
    w = I.config5(layers=14, width=64, P=24)
    g2, _ = I.relabel(w.graph, 5)
    run_and_compare(g2, w.devices, w.part_full(), 0, pad_fill=255)


@pytest.mark.parametrize("family", ["lean", "lean64", "steprec", "flow", "ring"])
def test_bounded_waits_run_out(family, monkeypatch):
    """The bounded device-side waits, made to run out on the host's terms: with a limit of zero polls every wait of
    the windowed kernels (for a staged record) and of the persistent record pass (for the other blocks' signal) gives
    up at once; the kernels vote, let their few copies in flight land, and return.  The call reports
    TFPS_ERR_TIMEOUT through the status word, nothing hangs or faults, and the next call on the same handle is
    bit-exact again."""
    from paper_1711_01912_b200 import tfps
    if family in ("steprec", "flow"):
        w = I.config5(layers=14, width=64, P=300)
        flags = tfps.EVAL_LEVEL_SYNC
        monkeypatch.setenv("TFPS_STEP_PERSISTENT" if family == "steprec" else "TFPS_STEP_FLOW", "1")
    elif family == "ring":
        w = I.config5(layers=14, width=64, P=300)
        flags = tfps.EVAL_AUTO
        monkeypatch.setenv("TFPS_RING", "2")
        monkeypatch.setenv("TFPS_LEAN", "0")
    else:
        w = I.config2()
        w.P = 200
        flags = tfps.EVAL_SLICED
        if family == "lean64":
            monkeypatch.setenv("TFPS_LEAN_FORCE_WIDE", "1")
    G = gpu_graph(w.graph, w.devices)
    dpart, P, ldp = padded(w.part_full()[:, :w.P])
    monkeypatch.setenv("TFPS_WAIT_LIMIT", "0")
    out = G.eval_batch(dpart, P, flags=flags, check=False)
    kernel = tfps.tfps_last_pass_kernel(G.handle)
    assert kernel == {"lean": "pass_lean_kernel", "lean64": "pass_lean64_kernel", "steprec": "pass_steprec_kernel",
                      "flow": "pass_flow_kernel", "ring": "pass_ring_kernel"}[family]
    with pytest.raises(tfps.TfpsError) as ei:
        G.status()
    assert ei.value.code == tfps.ERR_TIMEOUT
    monkeypatch.delenv("TFPS_WAIT_LIMIT")
    G.close()
    run_and_compare(w.graph, w.devices, w.part_full()[:, :w.P], {"lean": 2, "lean64": 2, "ring": 0}.get(family, 1), pad_fill=255)
