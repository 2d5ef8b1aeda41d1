"""GPU parity: the CUDA library, called through its C ABI, against the fp64 CPU oracle.

Integer outputs (degrees, the support's edge list, block tables, Eq. 12) must match bit for bit;
scale factors are fp64-computed and rounded once, so they match bit for bit too; propagated
features must stay within 1e-5 relative error per hop.
"""
import itertools

import numpy as np
import pytest
import torch

import gnnpre_inputs as gi
import oracle as orc
from parity_util import TOL, backward_error, check_all_hops, hop_error, single_hop_of, to_np

pytestmark = pytest.mark.gpu

OPS = (0, 1, 2)
EPS = 0.1


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2207_12000_b200 import binding
    return binding


def dev(g):
    return g.rowptr.cuda(), g.colidx.cuda()


def small_graphs():
    yield "er33", gi.erdos_renyi(33, 70, 5)
    yield "er1000", gi.erdos_renyi(1000, 6000, 6)
    yield "rmat3000", gi.rmat(3000, 20000, 7, directed_candidates=True)
    yield "star", gi.from_edge_list(700, [(0, j) for j in range(1, 650)])  # hub + isolated tail nodes
    yield "path2", gi.from_edge_list(2, [(0, 1)])
    yield "lonely", gi.from_edge_list(5, [])  # no edges at all


# ------------------------------------------------------------------ plan parity (bit-exact)

@pytest.mark.parametrize("name,g", list(small_graphs()) + [("c1", None)])
@pytest.mark.parametrize("op", OPS)
def test_plan_matches_oracle_bit_for_bit(B, name, g, op):
    if g is None:
        g = gi.make_graph(gi.WORKLOADS["c1"])
    rp, ci = g.rowptr.numpy(), g.colidx.numpy()
    drp, dci = dev(g)
    deg = orc.degrees(rp)
    np.testing.assert_array_equal(to_np(B.gnnpre_degrees(drp, dci)), deg)
    rp_t, ci_t = orc.support(op, rp, ci)
    m = int(rp_t[-1])
    for b in sorted({1, 2, 3, 7, 64, m} - {0}):
        if b > m:
            continue
        plan = B.gnnpre_build_plan(drp, dci, op, 16, gin_eps=EPS, force_blocks=b, force_col_slabs=1, segment_edges=8)
        info = plan.info()
        assert (info["n"], info["nnz"], info["nnz_tilde"], info["b"], info["c"]) == (g.n, g.nnz, m, b, 1)
        assert info["B_S"] == 4 * m + 8 * (g.n + 1) and info["B_X"] == 4 * g.n * 16
        pdeg, r, c = B.gnnpre_plan_scales(plan)
        np.testing.assert_array_equal(pdeg.numpy(), deg)
        wr, wc = orc.scales_f32(op, deg)
        np.testing.assert_array_equal(r.numpy().view(np.uint32), wr.view(np.uint32))
        np.testing.assert_array_equal(c.numpy().view(np.uint32), wc.view(np.uint32))
        srp, sci = B.gnnpre_plan_support(plan)
        np.testing.assert_array_equal(srp.numpy(), rp_t)
        np.testing.assert_array_equal(sci.numpy(), ci_t)
        e_off = orc.block_offsets(m, b)
        row_lo, row_hi, fp, lp = orc.block_rows(rp_t, e_off)
        for l in range(b):
            blk = B.gnnpre_plan_block(plan, l)
            assert (blk["e_lo"], blk["e_hi"]) == (e_off[l], e_off[l + 1])
            assert (blk["row_lo"], blk["row_hi"]) == (row_lo[l], row_hi[l])
            assert (blk["first_row_partial"], blk["last_row_partial"]) == (fp[l], lp[l])
        plan.close()


def test_plan_with_caller_degrees_and_budget_search(B):
    g = gi.erdos_renyi(500, 3000, 8)
    drp, dci = dev(g)
    deg = B.gnnpre_degrees(drp, dci)
    F = 64
    m = g.nnz + g.n
    B_S, B_X, B_fixed = 4 * m + 8 * (g.n + 1), 4 * g.n * F, 16 * g.n
    for budget in (B_fixed + B_S + 2 * B_X, B_fixed + B_S // 3 + B_X, B_fixed + 2000 + B_X // 2):
        want = orc.solve_budget(B_S, B_X, B_fixed, 1, 2, budget, min(m, 1 << 20), F // 4)
        plan = B.gnnpre_build_plan(drp, dci, 0, F, degrees=deg, budget_bytes=budget)
        info = plan.info()
        assert (info["b"], info["c"]) == want
        assert info["slab_width"] == orc.slab_width(F, info["c"])
        plan.close()
    with pytest.raises(B.GnnpreError) as ei:
        B.gnnpre_build_plan(drp, dci, 0, F, budget_bytes=B_fixed + 100)
    assert ei.value.status == -6


# ------------------------------------------------------------------ propagation parity

def run_case(B, g, op, F, K, *, b=1, c=1, seg=0, flags=0, ldx=None, ldo=None, seed=1):
    rp, ci = g.rowptr.numpy(), g.colidx.numpy()
    drp, dci = dev(g)
    ldx = ldx or F
    ldo = ldo or F
    Xbuf = torch.full((g.n, ldx), float("nan"), device="cuda")
    X = Xbuf[:, :F]
    X.copy_(gi.normal_matrix(g.n, F, seed, device="cuda"))
    obufs = [torch.full((g.n, ldo), -7.0, device="cuda") for _ in range(K)]
    outs = [o[:, :F] for o in obufs]
    plan = B.gnnpre_build_plan(drp, dci, op, F, gin_eps=EPS, force_blocks=b, force_col_slabs=c, segment_edges=seg,
                               flags=flags)
    B.gnnpre_propagate(plan, X, K, outs)
    torch.cuda.synchronize()
    for o in obufs:
        assert bool((o[:, F:] == -7.0).all()), "padding columns were written"
    worst = check_all_hops(op, EPS, rp, ci, to_np(X), outs, single_hop=single_hop_of(B, plan))
    plan.close()
    return worst, outs


def test_config1_erdos_renyi_gcn(B):
    """Configuration 1: 4,096 nodes, 32,768 edges, F=64, K=2, GCN, a single edge block."""
    w = gi.WORKLOADS["c1"]
    g = gi.make_graph(w)
    assert (g.n, g.nnz) == (4096, 65536)
    run_case(B, g, w.op, w.feat_dim, w.hops, b=w.blocks, seed=w.seed)


@pytest.mark.parametrize("name,g", list(small_graphs()))
@pytest.mark.parametrize("op", OPS)
def test_small_graphs_all_shapes(B, name, g, op):
    m = orc.support_nnz(op, g.n, g.nnz)
    for F, seg in ((4, 8), (16, 4), (20, 32), (64, 8), (100, 16), (128, 0), (256, 8), (516, 32), (640, 16), (1040, 8)):
        for b in (1, 3):
            if b > m:
                continue
            run_case(B, g, op, F, 2, b=b, seg=seg)


@pytest.mark.parametrize("op", OPS)
def test_blocks_slabs_and_launch_modes_agree(B, op):
    """Different (b, c), segment sizes and launch groupings change only the rounding order."""
    g = gi.rmat(5000, 40000, 9, directed_candidates=True)
    F, K = 72, 3
    ref = None
    for b, c, seg, flags in ((1, 1, 0, 0), (4, 1, 64, 0), (64, 1, 16, 1), (7, 3, 32, 1), (1, 18, 1, 0), (5, 2, 0, 0)):
        _, outs = run_case(B, g, op, F, K, b=b, c=c, seg=seg, flags=flags, ldx=F + 4, ldo=F + 8)
        cur = [to_np(o).astype(np.float64) for o in outs]
        if ref is None:
            ref = cur
        else:
            for k in range(K):
                assert hop_error(cur[k], ref[k]) <= TOL


def test_hub_longer_than_many_segments_and_blocks(B):
    """A row far longer than a segment and a block: its parts are summed by the fix-up pass."""
    n = 40000
    edges = [(0, j) for j in range(1, n)] + [(j, j + 1) for j in range(1, 2000)]
    g = gi.from_edge_list(n, edges)
    for op in OPS:
        run_case(B, g, op, 32, 2, b=9, seg=32)
        run_case(B, g, op, 128, 2, b=1, seg=0)


def test_runs_are_bitwise_reproducible(B):
    g = gi.rmat(20000, 200000, 10, directed_candidates=True)
    drp, dci = dev(g)
    X = gi.normal_matrix(g.n, 128, 3, device="cuda")
    plan = B.gnnpre_build_plan(drp, dci, 0, 128, force_blocks=4)
    a, _ = B.gnnpre_propagate(plan, X, 3)
    b, _ = B.gnnpre_propagate(plan, X, 3)
    torch.cuda.synchronize()
    for x, y in zip(a, b):
        assert torch.equal(x, y)
    plan.close()


def test_config2_rmat_gcn_four_blocks(B):
    """Configuration 2: 169,343 nodes, 1,166,243 directed R-MAT edges symmetrised, F=128, K=3, GCN, b=4."""
    w = gi.WORKLOADS["c2"]
    g = gi.make_graph(w, device="cuda").to("cpu")
    assert g.n == 169343
    run_case(B, g, w.op, w.feat_dim, w.hops, b=w.blocks, seed=w.seed)


@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("F", [16, 64, 128, 256, 512])
def test_config3_operator_width_block_sweep(B, op, F):
    """Configuration 3: ops x widths x block counts {1, 8, 64} on the 169,343-node graph, K=3."""
    w = gi.WORKLOADS["c3"]
    g = gi.make_graph(w, device="cuda").to("cpu")
    rp, ci = g.rowptr.numpy(), g.colidx.numpy()
    drp, dci = dev(g)
    X = gi.normal_matrix(g.n, F, w.seed, device="cuda")
    Xn = to_np(X)
    want = orc.propagate(op, w.gin_eps, rp, ci, Xn, w.hops)
    for b in w.sweep["blocks"]:
        plan = B.gnnpre_build_plan(drp, dci, op, F, gin_eps=w.gin_eps, force_blocks=b)
        outs, _ = B.gnnpre_propagate(plan, X, w.hops)
        torch.cuda.synchronize()
        one_hop = single_hop_of(B, plan)
        for k in range(w.hops):
            gk = to_np(outs[k])
            assert hop_error(gk, want[k]) <= TOL
            rows = np.random.default_rng(k).integers(0, g.n, 4096)
            # floor-free check of one hop on an input both sides share: X_0, then the oracle's hops in fp32
            prev = Xn if k == 0 else np.ascontiguousarray(want[k - 1].astype(np.float32))
            assert backward_error(op, w.gin_eps, rp, ci, prev, gk if k == 0 else one_hop(prev), rows) <= TOL
        plan.close()


# ------------------------------------------------------------------ errors and edge cases

def test_invalid_inputs_are_rejected(B):
    g = gi.erdos_renyi(100, 300, 11)
    drp, dci = dev(g)

    def status(fn):
        with pytest.raises(B.GnnpreError) as ei:
            fn()
        return ei.value.status

    assert status(lambda: B.gnnpre_build_plan(drp, dci, 0, 0)) == -1           # F < 1
    assert status(lambda: B.gnnpre_build_plan(drp, dci, 5, 16)) == -1          # bad op
    assert status(lambda: B.gnnpre_build_plan(drp, dci, 1, 16, force_blocks=g.nnz + 1)) == -1  # empty block
    assert status(lambda: B.gnnpre_build_plan(drp, dci, 0, 16, force_col_slabs=5)) == -1
    bad = dci.clone()
    bad[3] = 10 ** 6
    assert status(lambda: B.gnnpre_build_plan(drp, bad, 0, 16)) == -2          # column out of range
    bad = dci.clone()
    bad[int(g.rowptr[5])] = 5
    assert status(lambda: B.gnnpre_build_plan(drp, bad, 0, 16)) == -2          # a diagonal entry or broken order
    bad = dci.clone()
    lo = int(g.rowptr[7])
    bad[lo + 1] = bad[lo]
    assert status(lambda: B.gnnpre_build_plan(drp, bad, 0, 16)) == -2          # duplicate column
    badrp = drp.clone()
    badrp[10] = badrp[11] + 1
    assert status(lambda: B.gnnpre_build_plan(badrp, dci, 0, 16)) == -2        # rowptr not monotone
    plan = B.gnnpre_build_plan(drp, dci, 0, 16)
    X = torch.zeros((100, 18), device="cuda")[:, :16]
    assert status(lambda: B.gnnpre_propagate(plan, X, 1)) == -3               # ldx % 4
    X = torch.zeros((100, 16), device="cuda")
    assert status(lambda: B.gnnpre_propagate(plan, X, 0, [])) == -1
    assert status(lambda: B.gnnpre_propagate(plan, X, 2, [X.clone(), X])) == -1  # out aliases X
    plan.close()


def test_graph_without_edges(B):
    g = gi.from_edge_list(6, [])
    drp, dci = dev(g)
    X = gi.normal_matrix(6, 8, 1, device="cuda")
    for op, want in ((0, X), (1, torch.zeros_like(X)), (2, (1 + np.float32(EPS)) * X)):
        plan = B.gnnpre_build_plan(drp, dci, op, 8, gin_eps=EPS)
        outs, _ = B.gnnpre_propagate(plan, X, 2)
        torch.cuda.synchronize()
        torch.testing.assert_close(outs[0], want, rtol=1e-6, atol=0)
        plan.close()


# ------------------------------------------------------------------ streamed operands

@pytest.mark.parametrize("csr_on_host,x_on_host,out_on_host", [(False, True, True), (True, True, True),
                                                               (False, False, True), (True, True, False)])
@pytest.mark.parametrize("op", OPS)
def test_streamed_equals_resident_bitwise(B, op, csr_on_host, x_on_host, out_on_host):
    """Host-resident operands travel through the same kernels in the same order, so for the same
    (b, c) and segment size the result is bit-identical to the device-resident run."""
    g = gi.rmat(30000, 250000, 13, directed_candidates=True)
    F, K = 48, 3
    drp, dci = dev(g)
    X = gi.normal_matrix(g.n, F, 5, device="cuda")
    for b, c in ((1, 1), (5, 1), (3, 3), (2, 12)):
        ref_plan = B.gnnpre_build_plan(drp, dci, op, F, gin_eps=EPS, force_blocks=b, force_col_slabs=c,
                                       segment_edges=64)
        ref, _ = B.gnnpre_propagate(ref_plan, X, K)
        torch.cuda.synchronize()
        pb_plan = B.gnnpre_build_plan(drp, dci, op, F, gin_eps=EPS, force_blocks=b, force_col_slabs=c,
                                      segment_edges=64, flags=B.GNNPRE_FLAG_LAUNCH_PER_BLOCK)
        pb, _ = B.gnnpre_propagate(pb_plan, X, K)  # one launch per block: same bits as one launch per hop
        torch.cuda.synchronize()
        for k in range(K):
            assert torch.equal(pb[k], ref[k])
        pb_plan.close()
        rp, ci = (g.rowptr.pin_memory(), g.colidx.pin_memory()) if csr_on_host else (drp, dci)
        plan = B.gnnpre_build_plan(rp, ci, op, F, gin_eps=EPS, force_blocks=b, force_col_slabs=c, segment_edges=64,
                                   operands_mem=B.GNNPRE_MEM_HOST)
        assert plan.info()["structure_mem"] == (1 if csr_on_host else 0)
        Xin = X.cpu().pin_memory() if x_on_host else X
        ldo = F + 4
        if out_on_host:
            obuf = [torch.full((g.n, ldo), -3.0).pin_memory() for _ in range(K)]
        else:
            obuf = [torch.full((g.n, ldo), -3.0, device="cuda") for _ in range(K)]
        for rep in range(2):  # the second call reuses the plan's staging buffers
            outs, st = B.gnnpre_propagate(plan, Xin, K, [o[:, :F] for o in obuf], want_stats=True)
            torch.cuda.synchronize()
            for k in range(K):
                assert torch.equal(outs[k].cpu(), ref[k].cpu()), (b, c, k, rep)
                assert bool((obuf[k][:, F:] == -3.0).all())
            assert st.d2h_bytes == (4 * g.n * F * K if out_on_host else 0)
            assert st.h2d_bytes >= (4 * g.n * F if x_on_host else 0)
        plan.close()
        ref_plan.close()


def test_streamed_pageable_host_memory_and_check_against_oracle(B):
    g = gi.erdos_renyi(2000, 9000, 14)
    rp, ci = g.rowptr.numpy(), g.colidx.numpy()
    X = gi.normal_matrix(g.n, 32, 6)  # ordinary pageable host tensors
    plan = B.gnnpre_build_plan(g.rowptr, g.colidx, 0, 32, force_blocks=3, force_col_slabs=2,
                               operands_mem=B.GNNPRE_MEM_HOST)
    outs = [torch.empty(g.n, 32) for _ in range(2)]
    B.gnnpre_propagate(plan, X, 2, outs)
    check_all_hops(0, 0.0, rp, ci, X.numpy(), outs)
    plan.close()


@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("F", [68, 100, 128, 300, 516])
def test_bulk_copy_kernel_matches_register_kernel_bitwise(B, op, F):
    """Rows of 68..128 columns are staged through shared memory by the copy engine; the summation order is that
    of the register kernel for such rows (plain sums over steps of 8 edges), so the two agree bit for bit (and both
    agree with the oracle).  Rows wider than 256 columns are cut into 128-column tiles for the copy engine
    (300 = 128 + 128 + a 44-column tile left to the register kernel; 516 = four tiles + 4 columns); the register
    kernel for rows that wide sums over steps of 2 edges, so there the two paths agree to rounding only and each
    is checked against the oracle."""
    g = gi.rmat(30000, 400000, 17, directed_candidates=True)
    drp, dci = dev(g)
    X = gi.normal_matrix(g.n, F, 9, device="cuda")
    for b, seg in ((1, 256), (3, 64), (2, 1000)):  # same segment length for both: same summation order
        res = []
        for flags in (0, B.GNNPRE_FLAG_NO_BULK_COPY):
            plan = B.gnnpre_build_plan(drp, dci, op, F, gin_eps=EPS, force_blocks=b, segment_edges=seg, flags=flags)
            outs, st = B.gnnpre_propagate(plan, X, 2, want_stats=True)
            res.append(outs)
            plan.close()
        for k in range(2):
            if F <= 128:
                assert torch.equal(res[0][k], res[1][k]), (b, seg, k)
        if F > 128:
            check_all_hops(op, EPS, g.rowptr.numpy(), g.colidx.numpy(), to_np(X), res[1])
            check_all_hops(op, EPS, g.rowptr.numpy(), g.colidx.numpy(), to_np(X), res[0])
    check_all_hops(op, EPS, g.rowptr.numpy(), g.colidx.numpy(), to_np(X), res[0])


def test_two_tile_rows_on_a_graph_larger_than_the_cache(B):
    """Rows of 132..256 columns are cut into two equal tiles for the copy engine once a 128-column tile of X no
    longer fits the L2 (here 400,000 nodes: 205 MB per tile; F = 200 gives two tiles of 100 columns, F = 252 two of
    128 and 124).  Checked against the oracle, and against the register kernel to rounding."""
    g = gi.rmat(400000, 3000000, 23, directed_candidates=True)
    drp, dci = dev(g)
    rp, ci = g.rowptr.numpy(), g.colidx.numpy()
    for op, F in ((1, 200), (0, 252)):
        X = gi.normal_matrix(g.n, F, 12, device="cuda")
        res = []
        for flags in (0, B.GNNPRE_FLAG_NO_BULK_COPY):
            plan = B.gnnpre_build_plan(drp, dci, op, F, gin_eps=EPS, flags=flags)
            outs, st = B.gnnpre_propagate(plan, X, 2, want_stats=True)
            torch.cuda.synchronize()
            res.append((outs, st.kernel_launches, plan.info()["segment_edges"]))
            plan.close()
        assert res[0][2] >= 256 and res[0][1] > res[1][1]  # long segments, two segment launches per hop
        check_all_hops(op, EPS, rp, ci, to_np(X), res[0][0])
        for k in range(2):
            assert hop_error(to_np(res[0][0][k]), to_np(res[1][0][k]).astype(np.float64)) <= TOL


# ------------------------------------------------------------------ the normalised adjacency itself

@pytest.mark.parametrize("op", OPS)
def test_normalized_adjacency_values_bit_exact(B, op):
    """gnnpre_normalize against the oracle: fp64 evaluation from integer degrees, one rounding to fp32, so
    the comparison is bitwise; resident and block-streamed (host CSR, host output) runs give the same array."""
    for name, g in list(small_graphs()) + [("c1", gi.make_graph(gi.WORKLOADS["c1"]))]:
        rp, ci = g.rowptr.numpy(), g.colidx.numpy()
        want = orc.normalized_values(op, EPS, rp, ci).astype(np.float32)
        if want.size == 0:
            continue
        for b in (1, 3):
            if b > want.size:
                continue
            plan = B.gnnpre_build_plan(*dev(g), op, 16, gin_eps=EPS, force_blocks=b)
            got = B.gnnpre_normalize(plan)
            torch.cuda.synchronize()
            np.testing.assert_array_equal(to_np(got).view(np.uint32), want.view(np.uint32), err_msg=f"{name} b={b}")
            plan.close()
            hplan = B.gnnpre_build_plan(g.rowptr.pin_memory(), g.colidx.pin_memory(), op, 16, gin_eps=EPS,
                                        force_blocks=b)
            assert hplan.info()["structure_mem"] == 1
            for host_out in (True, False):
                got = B.gnnpre_normalize(hplan, host=host_out)
                torch.cuda.synchronize()
                np.testing.assert_array_equal(to_np(got).view(np.uint32), want.view(np.uint32))
            hplan.close()


def test_a_device_wait_that_runs_out_is_reported_and_leaves_the_plan_usable(B):
    """Failure detection without a fault: a warp polls a barrier that nothing completes, gives up after its
    limit and sets the plan's error word; the host reads GNNPRE_ERR_TIMEOUT once, and the same plan then
    propagates correctly."""
    g = gi.erdos_renyi(3000, 20000, 23)
    rp, ci = g.rowptr.numpy(), g.colidx.numpy()
    plan = B.gnnpre_build_plan(*dev(g), 0, 128)
    assert B.gnnpre_selftest_wait_timeout(plan, 200) == -8
    assert B.gnnpre_status_string(-8) == "timed out"
    X = gi.normal_matrix(g.n, 128, 2, device="cuda")
    outs, st = B.gnnpre_propagate(plan, X, 2, want_stats=True)  # the error word was cleared: no stale timeout
    check_all_hops(0, 0.0, rp, ci, to_np(X), outs)
    plan.close()


# ------------------------------------------------------------------ teleport (personalised PageRank) filter

@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("alpha", [0.15, 1.0])
def test_teleport_filter_matches_oracle(B, op, alpha):
    """X_k = (1 - alpha) A^ X_{k-1} + alpha X_0 for every kernel shape, with blocks and slabs, resident and
    streamed (bitwise equal to each other), against the fp64 oracle."""
    g = gi.rmat(6000, 60000, 27, directed_candidates=True)
    rp, ci = g.rowptr.numpy(), g.colidx.numpy()
    drp, dci = dev(g)
    K = 3
    for F, b, c in ((16, 1, 1), (100, 3, 1), (128, 2, 2), (256, 1, 1), (72, 4, 3)):
        X = gi.normal_matrix(g.n, F, 7, device="cuda")
        want = orc.propagate_teleport(op, EPS, alpha, rp, ci, to_np(X), K)
        plan = B.gnnpre_build_plan(drp, dci, op, F, gin_eps=EPS, force_blocks=b, force_col_slabs=c, segment_edges=64,
                                   teleport_alpha=alpha)
        outs, _ = B.gnnpre_propagate(plan, X, K)
        torch.cuda.synchronize()
        for k in range(K):
            assert hop_error(to_np(outs[k]), want[k]) <= TOL, (F, b, c, k)
        hplan = B.gnnpre_build_plan(g.rowptr.pin_memory(), g.colidx.pin_memory(), op, F, gin_eps=EPS, force_blocks=b,
                                    force_col_slabs=c, segment_edges=64, teleport_alpha=alpha,
                                    operands_mem=B.GNNPRE_MEM_HOST)
        houts = [torch.empty(g.n, F).pin_memory() for _ in range(K)]
        B.gnnpre_propagate(hplan, X.cpu().pin_memory(), K, houts)
        for k in range(K):
            assert torch.equal(houts[k], outs[k].cpu()), (F, b, c, k)
        plan.close()
        hplan.close()
    with pytest.raises(B.GnnpreError):
        B.gnnpre_build_plan(drp, dci, op, 16, teleport_alpha=1.5)


@pytest.mark.parametrize("op", OPS)
def test_weighted_hop_sum_matches_oracle(B, op):
    """Z = gamma_0 X_0 + sum_k gamma_k X_k accumulated in the kernels' epilogues: every kernel shape, blocks and
    slabs, a strided Z with untouched padding, hops kept or rotated through two buffers; then on top of the
    teleport recurrence.  The hops themselves must equal those of gnnpre_propagate bit for bit."""
    g = gi.rmat(6000, 60000, 33, directed_candidates=True)  # has isolated nodes: SAGE's empty rows are covered
    rp, ci = g.rowptr.numpy(), g.colidx.numpy()
    drp, dci = dev(g)
    gamma = [0.4, -1.5, 0.75, 2.0, -0.6]
    K = len(gamma) - 1
    for F, b, c in ((16, 1, 1), (100, 3, 1), (128, 2, 2), (256, 1, 1), (72, 4, 3), (600, 2, 1)):
        X = gi.normal_matrix(g.n, F, 9, device="cuda")
        want = orc.weighted_hop_sum(op, EPS, rp, ci, to_np(X), gamma)
        plan = B.gnnpre_build_plan(drp, dci, op, F, gin_eps=EPS, force_blocks=b, force_col_slabs=c, segment_edges=64)
        ref, _ = B.gnnpre_propagate(plan, X, K)
        zbuf = torch.full((g.n, F + 4), -3.0, device="cuda")
        hops, Z = B.gnnpre_propagate_weighted(plan, X, gamma, Z=zbuf[:, :F])
        torch.cuda.synchronize()
        assert hop_error(to_np(Z), want) <= TOL, (F, b, c)
        assert bool((zbuf[:, F:] == -3.0).all())
        for k in range(K):
            assert torch.equal(hops[k], ref[k]), (F, b, c, k)
        last2, Z2 = B.gnnpre_propagate_weighted(plan, X, gamma, keep_hops=False)
        torch.cuda.synchronize()
        assert torch.equal(Z2, Z) and torch.equal(last2[K - 1], ref[K - 1])
        plan.close()
    # with a teleport term the summed hops are those of the recurrence
    F, alpha = 100, 0.2
    X = gi.normal_matrix(g.n, F, 10, device="cuda")
    tele = orc.propagate_teleport(op, EPS, alpha, rp, ci, to_np(X), K)
    want = gamma[0] * to_np(X).astype(np.float64) + sum(gamma[k + 1] * tele[k] for k in range(K))
    plan = B.gnnpre_build_plan(drp, dci, op, F, gin_eps=EPS, force_blocks=2, teleport_alpha=alpha)
    _, Z = B.gnnpre_propagate_weighted(plan, X, gamma)
    torch.cuda.synchronize()
    assert hop_error(to_np(Z), want) <= TOL
    # refusals: Z aliasing an input or a hop, a hop written over the one it reads, a plan with host structure
    with pytest.raises(B.GnnpreError):
        B.gnnpre_propagate_weighted(plan, X, gamma, Z=X)
    o = [torch.empty_like(X) for _ in range(2)]
    with pytest.raises(B.GnnpreError):
        B.gnnpre_propagate_weighted(plan, X, gamma, out=[o[0], o[0], o[1], o[0]])
    plan.close()
    hplan = B.gnnpre_build_plan(g.rowptr.pin_memory(), g.colidx.pin_memory(), op, F, operands_mem=B.GNNPRE_MEM_HOST,
                                force_blocks=2)
    if hplan.info()["structure_mem"] == B.GNNPRE_MEM_HOST:
        with pytest.raises(B.GnnpreError):
            B.gnnpre_propagate_weighted(hplan, X, gamma)
    hplan.close()


@pytest.mark.parametrize("world", [2, 3, 8])
def test_column_shards_assemble_to_the_full_result(B, world):
    """Column sharding over `world` ranks, run here one rank after another on the one GPU (the ranks are
    independent: nothing waits on anything): every rank's slab against the oracle's columns, slabs side by side
    cover every column once."""
    from paper_2207_12000_b200.shard import propagate_column_shard
    g = gi.rmat(8000, 90000, 35, directed_candidates=True)
    rp, ci = g.rowptr.numpy(), g.colidx.numpy()
    drp, dci = dev(g)
    F, K, op = 100, 3, 0
    X = gi.normal_matrix(g.n, F, 3, device="cuda")
    want = orc.propagate(op, 0.0, rp, ci, to_np(X), K)
    covered = np.zeros(F, dtype=np.int32)
    for rank in range(world):
        lo, outs = propagate_column_shard(B, drp, dci, op, X, K, world, rank)
        torch.cuda.synchronize()
        if not outs:
            continue
        width = outs[0].shape[1]
        covered[lo:lo + width] += 1
        for k in range(K):
            assert hop_error(to_np(outs[k]), want[k][:, lo:lo + width]) <= TOL, (rank, k)
    assert (covered == 1).all()


def test_propagate_and_first_layer_inside_a_cuda_graph(B):
    """The device-resident calls only enqueue work, so a CUDA graph can capture them: K hops of configuration 1 and
    the first dense stage over them, replayed twice on fresh outputs, equal the direct calls bit for bit."""
    w = gi.WORKLOADS["c1"]
    g = gi.make_graph(w, device="cuda")
    X = gi.make_features(w, device="cuda")
    plan = B.gnnpre_build_plan(g.rowptr, g.colidx, w.op, w.feat_dim)
    ref, _ = B.gnnpre_propagate(plan, X, w.hops)
    Wt = gi.normal_matrix(64, w.feat_dim, 3, device="cuda")
    batch = torch.arange(0, g.n, 3, dtype=torch.int32, device="cuda")
    ref_y = B.gnnpre_lc_first_layer(ref, batch, Wt, relu_mask=1)
    outs = [torch.zeros_like(X) for _ in range(w.hops)]
    y = torch.zeros_like(ref_y)
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):  # one call outside the capture: one-time set-up of the kernels
        B.gnnpre_propagate(plan, X, w.hops, outs)
        B.gnnpre_lc_first_layer(outs, batch, Wt, relu_mask=1, out=y, check=False)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        B.gnnpre_propagate(plan, X, w.hops, outs)
        B.gnnpre_lc_first_layer(outs, batch, Wt, relu_mask=1, out=y, check=False)
    for _ in range(2):
        for o in outs:
            o.zero_()
        y.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert all(torch.equal(o, r) for o, r in zip(outs, ref)) and torch.equal(y, ref_y)
    assert int(flag.item()) == 0
    plan.close()


def test_resuming_from_a_finished_hop_gives_the_same_bits(B):
    """Checkpoint/resume: hops 1..2, then hop 3 started from hop 2's output, equal the uninterrupted run."""
    g = gi.rmat(20000, 200000, 29, directed_candidates=True)
    plan = B.gnnpre_build_plan(*dev(g), 1, 100, force_blocks=3)
    X = gi.normal_matrix(g.n, 100, 4, device="cuda")
    full, _ = B.gnnpre_propagate(plan, X, 3)
    first, _ = B.gnnpre_propagate(plan, X, 2)
    rest, _ = B.gnnpre_propagate(plan, first[1], 1)
    torch.cuda.synchronize()
    assert torch.equal(first[0], full[0]) and torch.equal(first[1], full[1]) and torch.equal(rest[0], full[2])
    plan.close()


@pytest.mark.parametrize("op", OPS)
def test_streamed_slabs_through_the_bulk_copy_kernel(B, op):
    """Column slabs of 100 columns (F = 200, c = 2) and a 128-column tail tile (F = 640): the tensor map of the
    bulk-copy kernel starts at a column offset, in dense slab buffers and in the caller's strided matrix."""
    g = gi.rmat(12000, 150000, 31, directed_candidates=True)
    rp, ci = g.rowptr.numpy(), g.colidx.numpy()
    for F, c in ((200, 2), (640, 1)):
        X = gi.normal_matrix(g.n, F, 8, device="cuda")
        plan = B.gnnpre_build_plan(*dev(g), op, F, gin_eps=EPS, force_blocks=3, force_col_slabs=c,
                                   operands_mem=B.GNNPRE_MEM_HOST)
        houts = [torch.empty(g.n, F).pin_memory() for _ in range(2)]
        B.gnnpre_propagate(plan, X.cpu().pin_memory(), 2, houts)
        check_all_hops(op, EPS, rp, ci, to_np(X), houts)
        plan.close()


def test_feature_width_that_is_not_a_multiple_of_four(B):
    """F = 602 (Reddit's width in the paper's dataset table): the matrices carry a leading dimension of 604; the
    two pad columns may hold anything (NaN here) without touching the 602 real ones."""
    g = gi.erdos_renyi(3000, 30000, 33)
    rp, ci = g.rowptr.numpy(), g.colidx.numpy()
    F, ld = 602, 604
    Xbuf = torch.full((g.n, ld), float("nan"), device="cuda")
    Xbuf[:, :F] = gi.normal_matrix(g.n, F, 3, device="cuda")
    obuf = [torch.zeros((g.n, ld), device="cuda") for _ in range(2)]
    plan = B.gnnpre_build_plan(*dev(g), 0, F, force_blocks=2)
    assert plan.info()["feat_dim"] == 604
    B.gnnpre_propagate(plan, Xbuf[:, :F], 2, [o[:, :F] for o in obuf])
    torch.cuda.synchronize()
    check_all_hops(0, 0.0, rp, ci, to_np(Xbuf[:, :F]).copy(), [o[:, :F] for o in obuf])
    with pytest.raises(B.GnnpreError):  # no room for the pad columns
        B.gnnpre_propagate(plan, torch.zeros((g.n, F), device="cuda")[:, :F], 1)
    plan.close()
