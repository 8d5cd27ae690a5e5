"""The allocation-free entry point tfps_eval_cp_noalloc.

Some users of the library cannot allocate device memory at the moment they
evaluate candidates (they run inside somebody else's memory plan, or in a loop
that must not hit a device-wide synchronising cudaMalloc).  For them the library
carries its own fixed scratch array.  This test drives the entry point through
the C ABI twice in a row -- the second call finds the first call's leftovers in
the shared array -- and requires the critical-path lengths to equal, bit for
bit, those of the ordinary entry point with a caller workspace.  The device's
free memory as the driver reports it (cudaMemGetInfo, which sees every
allocation of the process, the library's own included) must not shrink across
the calls.  It also checks that a problem too large for the built-in array is
refused with TFPS_ERR_WORKSPACE instead of being run.

This file is named so that pytest collects it last.
"""
from __future__ import annotations

import numpy as np
import pytest

from paper_1711_01912_b200 import inputs as I

pytestmark = pytest.mark.gpu


def test_noalloc_matches_workspace_entry_point_twice():
    import torch
    from paper_1711_01912_b200 import tfps

    w = I.config2()
    g = tfps.graph_from_workload(w)
    n = w.graph.n
    stream = torch.cuda.current_stream().cuda_stream
    full = w.part_full()
    for call, (c0, P) in enumerate([(0, 777), (2048, 1000)]):   # two different candidate sets, back to back
        ldp = tfps.round_up_ldp(P)
        assert n * ldp * 8 <= tfps.NOALLOC_SCRATCH_BYTES
        host = np.zeros((n, ldp), np.uint8)
        host[:, :P] = full[:, c0:c0 + P]
        part = torch.from_numpy(host).cuda()
        ref = g.eval_batch(part, P, want=("cp",), out={})["cp"]          # existing entry point, caller workspace
        cp = torch.full((P,), -1, dtype=torch.int64, device="cuda")
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        tfps.tfps_eval_cp_noalloc(g.handle, P, ldp, part.data_ptr(), cp.data_ptr(), 0, stream)
        g.status()
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after >= free_before, f"call {call}: {free_before - free_after} bytes of device memory went away"
        assert torch.equal(cp, ref[:P]), f"call {call}: cp differs from tfps_eval_batch"
    # too large for the built-in scratch: refused, nothing launched
    big_ldp = (tfps.NOALLOC_SCRATCH_BYTES // (8 * n) // 16 + 2) * 16
    part = torch.zeros((n, big_ldp), dtype=torch.uint8, device="cuda")
    cp = torch.zeros(big_ldp, dtype=torch.int64, device="cuda")
    with pytest.raises(tfps.TfpsError) as ei:
        tfps.tfps_eval_cp_noalloc(g.handle, big_ldp, big_ldp, part.data_ptr(), cp.data_ptr(), 0, stream)
    assert ei.value.code == tfps.ERR_WORKSPACE
    g.close()
