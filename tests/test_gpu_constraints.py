"""GPU parity of the placement-constraint check (collocation constraints, Eq. 3; device constraints, Eq. 4) against
the oracle: counts per candidate, bit-exact, through the C ABI."""
from __future__ import annotations

import numpy as np
import pytest

from paper_1711_01912_b200 import inputs as I
from test_gpu_parity import gpu_graph, padded

pytestmark = pytest.mark.gpu


def _check(w, pairs, devs, P=None, pad_fill=0):
    import oracle
    part = w.part_full() if P is None else w.part_full()[:, :P]
    G = gpu_graph(w.graph)
    G.constraints_set(pairs, devs)
    dpart, P, ldp = padded(part, fill=pad_fill)
    coll, dev = G.eval_constraints(dpart, P)
    rc, rd = oracle.eval_constraints(part, pairs, devs)
    assert np.array_equal(coll.cpu().numpy().astype(np.int64), rc)
    assert np.array_equal(dev.cpu().numpy().astype(np.int64), rd)
    G.close()
    return rc, rd


def test_constraints_match_oracle_on_configs():
    rng = np.random.default_rng(5)
    for w, P in ((I.config1(), None), (I.config2(), 1000), (I.small_random(77, 900, 3000, 50, 333), None)):
        n, k = w.graph.n, w.devices.k
        for npairs, ndev in ((0, 0), (1, 1), (255, 257), (2000, 700)):
            pairs = rng.integers(0, n, size=(npairs, 2))
            devs = np.stack([rng.integers(0, n, size=ndev), rng.integers(0, k, size=ndev)], axis=1)
            rc, rd = _check(w, pairs, devs, P, pad_fill=255)
            if npairs >= 255:
                assert rc.max() > 0 and rd.max() > 0   # the case is not vacuous


def test_constraints_closed_forms_and_lists_replaced():
    """Edges of the graph as collocation pairs: a candidate violates exactly its cross-device edges; a second
    tfps_constraints_set replaces the first; ragged candidate counts; only one of the two outputs requested."""
    import torch
    from paper_1711_01912_b200 import tfps
    w = I.config2()
    g = w.graph
    part = w.part_full()[:, :77]
    G = gpu_graph(g)
    G.constraints_set(np.stack([g.src, g.dst], axis=1), np.zeros((0, 2), np.int32))
    dpart, P, ldp = padded(part, fill=200)
    coll, dev = G.eval_constraints(dpart, P)
    cross = (part[g.src] != part[g.dst]).sum(axis=0)
    assert np.array_equal(coll.cpu().numpy(), cross) and not dev.any()
    v = np.arange(g.n)
    G.constraints_set(np.zeros((0, 2), np.int32), np.stack([v, v % w.devices.k], axis=1))
    coll, dev = G.eval_constraints(dpart, P)
    assert not coll.any()
    assert np.array_equal(dev.cpu().numpy(), (part != (v % w.devices.k)[:, None].astype(np.uint8)).sum(axis=0))
    assert dev[0] == 0   # candidate 0 of this configuration is exactly v mod k
    only = torch.full((P,), -1, dtype=torch.int32, device="cuda")
    tfps.tfps_eval_constraints(G.handle, P, ldp, dpart.data_ptr(), None, only.data_ptr(), 0)
    torch.cuda.synchronize()
    assert torch.equal(only, dev)
    with pytest.raises(tfps.TfpsError) as ei:
        G.constraints_set([(0, g.n)], [])
    assert ei.value.code == tfps.ERR_INVALID_ARG
    G.close()


def test_critical_mask_matches_oracle():
    """tfps_critical_mask on the outputs of tfps_eval_batch against the oracle's mask of the oracle's levels: worked
    DAG shapes, ragged candidate counts (odd P, padding columns untouched), a wide and a deep graph."""
    import oracle
    import torch
    from paper_1711_01912_b200 import tfps
    from helpers import oracle_graph
    for w, P in ((I.config1(), 63), (I.config2(), 301), (I.small_random(91, 500, 1700, 6, 130), None)):
        part = w.part_full() if P is None else w.part_full()[:, :P]
        d = w.devices
        G = gpu_graph(w.graph, d)
        dpart, P, ldp = padded(part)
        out = G.eval_batch(dpart, P)
        mask = tfps.critical_mask(out, P)
        ref = oracle.eval_batch(oracle_graph(w.graph), d.k, d.s, d.C, d.B, d.scale, part)
        want = oracle.critical_mask(ref.tlevel, ref.blevel, ref.cp)
        got = mask.cpu().numpy()
        assert np.array_equal(got[:, :P], want)
        assert not got[:, P:].any()
        assert want.any(axis=0).all()   # every candidate has a critical path
        G.close()
    with pytest.raises(tfps.TfpsError):
        tfps.tfps_critical_mask(4, 4, 16, out["tlevel"].data_ptr() + 8, out["blevel"].data_ptr(), out["cp"].data_ptr(), mask.data_ptr(), 0)
