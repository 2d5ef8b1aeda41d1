"""gnnpre_hop_static, the hop that allocates nothing, against the oracle.

Some callers may not allocate device memory (a framework's pool owns the device, or the process
has frozen its footprint), so they cannot build a plan; gnnpre_hop_static serves them with a
scratch array that is part of the library image.  This file is collected last on purpose: the
static array is shared by every call in the process, and a failure here must not hide the other
tests from a run that stops at the first failure.
"""
import numpy as np
import pytest
import torch

import gnnpre_inputs as gi
import oracle as orc
from parity_util import TOL, hop_error, to_np

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2207_12000_b200 import binding
    return binding


@pytest.mark.parametrize("op", (0, 1, 2))
def test_static_hop_matches_planned_hop_twice_in_a_row(B, op):
    """Two calls back to back with different inputs: the second must not see anything the first left
    in the shared scratch array.  Each result is compared with the hop that the planned entry point
    (gnnpre_build_plan + gnnpre_propagate) gives for the same inputs, and with the fp64 oracle, both at
    the tolerance of the parity tests; the graph has isolated nodes and hubs far longer than a segment."""
    g = gi.rmat(20000, 300000, 21, directed_candidates=True)
    drp, dci = g.rowptr.cuda(), g.colidx.cuda()
    rp, ci = g.rowptr.numpy(), g.colidx.numpy()
    for F in (100, 16):
        plan = B.gnnpre_build_plan(drp, dci, op, F, gin_eps=0.1)
        for seed in (1, 2):
            X = gi.normal_matrix(g.n, F, seed, device="cuda")
            want = orc.propagate(op, 0.1, rp, ci, to_np(X), 1)[0]
            planned, _ = B.gnnpre_propagate(plan, X, 1)
            buf = torch.full((g.n, F + 4), -5.0, device="cuda")
            got = B.gnnpre_hop_static(drp, dci, op, X, buf[:, :F], gin_eps=0.1)
            torch.cuda.synchronize()
            assert hop_error(to_np(got), to_np(planned[0]).astype(np.float64)) <= TOL
            assert hop_error(to_np(got), want) <= TOL
            assert bool((buf[:, F:] == -5.0).all())
        plan.close()


def test_static_hop_wide_rows_longer_segments_and_no_allocation(B):
    """Rows of 256 and 512 columns (two and four 128-bit pieces per lane) on a graph large enough that the
    segments must grow beyond 64 edges for their partial sums to fit the fixed array (3.2 M edges at F = 256:
    segments of 128 edges).  After the first call the device's free memory is read before and after each call:
    the entry point must not change it."""
    import ctypes
    g = gi.rmat(100000, 1600000, 22, directed_candidates=False)
    assert 2 * ((g.nnz + 63) // 64) * 256 * 4 > 64 << 20  # 64-edge segments would not fit
    drp, dci = g.rowptr.cuda(), g.colidx.cuda()
    rp, ci = g.rowptr.numpy(), g.colidx.numpy()
    for F, op in ((256, 0), (512, 1), (132, 2)):
        X = gi.normal_matrix(g.n, F, 5, device="cuda")
        out = torch.empty_like(X)
        want = orc.propagate(op, 0.1, rp, ci, to_np(X), 1)[0]
        B.gnnpre_hop_static(drp, dci, op, X, out, gin_eps=0.1)  # may be the first call on this device: set-up
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        for _ in range(2):
            out.fill_(7.0)
            B.gnnpre_hop_static(drp, dci, op, X, out, gin_eps=0.1)
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] == free_before
            assert hop_error(to_np(out), want) <= TOL
    # a problem whose partial sums cannot fit whatever the segment length: refused before anything is launched
    # (the edge count is only read, never followed, so a made-up one is safe to pass)
    csr = B.gnnpre_csr_t(g.n, 1 << 35, drp.data_ptr(), dci.data_ptr(), B.GNNPRE_MEM_DEVICE)
    X = torch.zeros((g.n, 512), device="cuda")
    rc = B._lib.gnnpre_hop_static(ctypes.byref(csr), 0, 0.0, 512, X.data_ptr(), 512, torch.empty_like(X).data_ptr(), 512,
                                  torch.cuda.current_stream().cuda_stream)
    assert rc == -11


def test_static_hop_edge_cases_and_limits(B):
    g = gi.from_edge_list(6, [])  # no edges: only self-loop terms
    X = gi.normal_matrix(6, 8, 3, device="cuda")
    out = torch.empty_like(X)
    B.gnnpre_hop_static(g.rowptr.cuda(), g.colidx.cuda(), 0, X, out)
    torch.cuda.synchronize()
    assert torch.equal(out, X)
    B.gnnpre_hop_static(g.rowptr.cuda(), g.colidx.cuda(), 1, X, out)
    torch.cuda.synchronize()
    assert bool((out == 0).all())
    wide = torch.zeros((6, 516), device="cuda")
    with pytest.raises(B.GnnpreError) as ei:
        B.gnnpre_hop_static(g.rowptr.cuda(), g.colidx.cuda(), 0, wide, torch.empty_like(wide))
    assert ei.value.status == -11  # beyond the fixed array's reach: a clear refusal, nothing launched
