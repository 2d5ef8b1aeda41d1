"""Full-size GPU parity: configuration 4 as bench.py times it, and a scaled configuration 5 streamed
from pinned host memory with edge blocks and column slabs chosen by the budget solver."""
import numpy as np
import pytest
import torch

import gnnpre_inputs as gi
import oracle as orc
from parity_util import TOL, backward_error, hop_error, single_hop_of, to_np

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2207_12000_b200 import binding
    return binding


def test_config4_full_size_as_benchmarked(B):
    """2,449,029 nodes, 123.7M nnz, F=100, K=3, SAGE, 32 blocks, one launch per hop (bench.py's set-up).
    Integer plan outputs bit-exact; every hop against the full fp64 chain; sampled rows (random, the
    highest degrees, every block-boundary row) against the exact one-hop result on a shared input (X_0, then
    the oracle's previous hop in fp32); the degree-weighted column sums SAGE conserves on a symmetric graph."""
    w = gi.WORKLOADS["c4"]
    g = gi.make_graph(w, device="cuda")
    X = gi.make_features(w, device="cuda")
    assert (g.n, g.nnz) == (2449029, 123718280)
    plan = B.gnnpre_build_plan(g.rowptr, g.colidx, w.op, w.feat_dim, force_blocks=w.blocks, force_col_slabs=1)
    outs, _ = B.gnnpre_propagate(plan, X, w.hops)
    torch.cuda.synchronize()
    rp, ci = to_np(g.rowptr), to_np(g.colidx)
    deg, _, _ = B.gnnpre_plan_scales(plan)
    np.testing.assert_array_equal(deg.numpy(), orc.degrees(rp))
    e_off = orc.block_offsets(g.nnz, w.blocks)
    boundary = []
    for l in range(w.blocks):
        blk = B.gnnpre_plan_block(plan, l)
        assert (blk["e_lo"], blk["e_hi"]) == (e_off[l], e_off[l + 1])
        assert blk["row_lo"] == np.searchsorted(rp, e_off[l], side="right") - 1
        boundary += [blk["row_lo"], blk["row_hi"]]
    d = torch.from_numpy(deg.numpy()).cuda().double()
    rng = np.random.default_rng(4)
    rows = np.unique(np.concatenate([rng.integers(0, g.n, 4096), np.argsort(deg.numpy())[-64:], boundary]))
    want = orc.propagate(w.op, 0.0, rp, ci, to_np(X), w.hops)
    prev = X
    one_hop = single_hop_of(B, plan)
    for k in range(w.hops):
        got = to_np(outs[k])
        assert hop_error(got, want[k]) <= TOL
        # one hop on an input both sides share: X_0, then the oracle's previous hop rounded to fp32
        shared = to_np(X) if k == 0 else np.ascontiguousarray(want[k - 1].astype(np.float32))
        assert backward_error(w.op, 0.0, rp, ci, shared, got if k == 0 else one_hop(shared), rows) <= TOL
        a, b_ = d @ outs[k].double(), d @ prev.double()
        scale = d @ prev.double().abs()
        assert float(((a - b_).abs() / scale).max()) <= 1e-6
        prev = outs[k]
    plan.close()


def test_config5_scaled_streamed_with_budget(B):
    """Configuration 5 at 1/64 scale (1.7M nodes, 25M nnz, F=128, K=2, GCN): graph, features and outputs in
    pinned host memory, a budget small enough to force several edge blocks and column slabs."""
    w = gi.scaled(gi.WORKLOADS["c5"], 64)
    g = gi.make_graph(w, device="cuda")
    X = gi.make_features(w, device="cuda")
    F, K = w.feat_dim, w.hops
    rp_h, ci_h = g.rowptr.cpu().pin_memory(), g.colidx.cpu().pin_memory()
    m = g.nnz + g.n
    B_S, B_X, B_fixed = 4 * m + 8 * (g.n + 1), 4 * g.n * F, 16 * g.n
    budget = B_fixed + B_S // 2 + B_X // 8  # far too small for X or E whole: several blocks and many slabs
    plan = B.gnnpre_build_plan(rp_h, ci_h, w.op, F, budget_bytes=budget, operands_mem=B.GNNPRE_MEM_HOST)
    info = plan.info()
    assert (info["b"], info["c"]) == orc.solve_budget(B_S, B_X, B_fixed, 2, 4, budget, 1 << 20, F // 4)
    assert info["b"] > 1 and info["c"] > 1 and info["structure_mem"] == 1
    Xh = X.cpu().pin_memory()
    outs = [torch.empty((g.n, F), dtype=torch.float32).pin_memory() for _ in range(K)]
    _, st = B.gnnpre_propagate(plan, Xh, K, outs, want_stats=True)
    assert st.d2h_bytes == 4 * g.n * F * K
    assert st.h2d_bytes >= 4 * g.n * F + 4 * m  # X once, and E at least once
    # Eq. 12 is a model: what the plan really holds on the device after a streamed call (edge-block staging
    # buffers, four slab buffers, per-node arrays, row pointers, segment tables) stays within 10 % of the budget
    used = plan.info()["device_bytes"]
    assert used <= 1.10 * budget, (used, budget)
    ref_plan = B.gnnpre_build_plan(g.rowptr, g.colidx, w.op, F, force_blocks=info["b"], force_col_slabs=info["c"],
                                   segment_edges=info["segment_edges"])
    ref, _ = B.gnnpre_propagate(ref_plan, X, K)
    torch.cuda.synchronize()
    for k in range(K):
        assert torch.equal(ref[k].cpu(), outs[k])
    want = orc.propagate(w.op, 0.0, rp_h.numpy(), ci_h.numpy(), Xh.numpy(), K)
    for k in range(K):
        assert hop_error(outs[k].numpy(), want[k]) <= TOL
    plan.close()
    ref_plan.close()


def test_first_dense_stage_at_config4_size_sampled(B):
    """gnnpre_lc_first_layer in the launch bench.py --stage lc times: three [2,449,029 x 100] matrices, hidden 256,
    every row once in a seeded random order (19,134 tiles per matrix, the last one ragged).  The matrices are seeded
    synthetic stand-ins for the hops (the layer does not care where they came from); the oracle computes sampled
    output rows one by one: random positions, the first and last tile, and the rows around every 1,000th tile edge."""
    w = gi.WORKLOADS["c4"]
    n, F, H, K = w.n, w.feat_dim, 256, w.hops
    hops = [gi.normal_matrix(n, F, w.seed + 10 + k, device="cuda") for k in range(K)]
    Wt = gi.normal_matrix(H, F, w.seed + 77, device="cuda") / float(np.sqrt(F))
    order_np = np.random.default_rng(w.seed).permutation(n)
    order = torch.from_numpy(order_np.astype(np.int32)).cuda()
    relu_mask = 0b110
    Y = B.gnnpre_lc_first_layer(hops, order, Wt, relu_mask=relu_mask)
    rng = np.random.default_rng(11)
    edges = np.arange(0, n, 128 * 1000)
    pos = np.unique(np.clip(np.concatenate([rng.integers(0, n, 3000), np.arange(256), np.arange(n - 200, n),
                                            edges - 1, edges, edges + 1]), 0, n - 1))
    Wt_np = to_np(Wt)
    for k in range(K):
        want, scale = orc.lc_first_layer(to_np(hops[k]), order_np[pos], Wt_np, relu=bool((relu_mask >> k) & 1),
                                         want_abs=True)
        got = to_np(Y[k][torch.from_numpy(pos).cuda()]).astype(np.float64)
        assert (np.abs(got - want) <= (2.0 ** -9 + F * 2.0 ** -23) * scale).all()
    # properties that hold at any size: ReLU outputs are non-negative, and a second call with the identity order
    # returns the same rows in another place, bit for bit
    assert float(Y[1].min()) >= 0.0 and float(Y[2].min()) >= 0.0 and float(Y[0].min()) < 0.0
    Z = B.gnnpre_lc_first_layer(hops[:1], None, Wt)
    assert torch.equal(Z[0][order.long()[:100000]], Y[0][:100000])


@pytest.mark.parametrize("name", ("flickr", "reddit"))
def test_wide_feature_dataset_shapes_full_size(B, name):
    """The two wide-feature rows of the paper's dataset table as seeded R-MAT stand-ins (89,250 nodes / 899,756
    edges / F=500 and 232,965 nodes / 11,606,919 edges / F=602), GCN, K=2, whole graph resident.  F=602 is not a
    multiple of 4: the matrices carry a leading dimension of 604.  Degrees bit-exact; every hop against the fp64
    chain; hop 1 floor-free on sampled rows (random and the highest degrees); the sum GCN conserves on a symmetric
    graph, sum_i sqrt(d_i + 1) X_k[i, f], unchanged from hop to hop."""
    w = gi.WORKLOADS[name]
    g = gi.make_graph(w, device="cuda")
    F, K = w.feat_dim, w.hops
    ld = (F + 3) // 4 * 4
    X = gi.make_features(w, device="cuda", ld=ld)
    assert (g.n, g.nnz) == (w.n, 2 * w.m)
    plan = B.gnnpre_build_plan(g.rowptr, g.colidx, w.op, F)
    outs = [torch.full((g.n, ld), float("nan"), device="cuda")[:, :F] for _ in range(K)]
    B.gnnpre_propagate(plan, X, K, outs)
    torch.cuda.synchronize()
    rp, ci = to_np(g.rowptr), to_np(g.colidx)
    deg, _, _ = B.gnnpre_plan_scales(plan)
    np.testing.assert_array_equal(deg.numpy(), orc.degrees(rp))
    X_np = np.ascontiguousarray(to_np(X))
    want = orc.propagate(w.op, 0.0, rp, ci, X_np, K)
    rng = np.random.default_rng(7)
    rows = np.unique(np.concatenate([rng.integers(0, g.n, 2048), np.argsort(deg.numpy())[-64:]]))
    sq = torch.sqrt(torch.from_numpy(deg.numpy()).cuda().double() + 1.0)
    prev = X
    for k in range(K):
        got = np.ascontiguousarray(to_np(outs[k]))
        assert hop_error(got, want[k]) <= TOL
        if k == 0:
            assert backward_error(w.op, 0.0, rp, ci, X_np, got, rows) <= TOL
        a, b_ = sq @ outs[k].double(), sq @ prev.double()
        assert float(((a - b_).abs() / (sq @ prev.double().abs())).max()) <= 1e-6
        prev = outs[k]
    plan.close()
    if name == "flickr":  # the same call through pinned host buffers: two column slabs of 252 and 248 columns
        hplan = B.gnnpre_build_plan(g.rowptr, g.colidx, w.op, F, operands_mem=B.GNNPRE_MEM_HOST)
        assert hplan.info()["c"] == 2
        Xh = torch.zeros((g.n, ld), dtype=torch.float32).pin_memory()[:, :F]
        Xh.copy_(X)
        outs_h = [torch.full((g.n, ld), float("nan")).pin_memory()[:, :F] for _ in range(K)]
        B.gnnpre_propagate(hplan, Xh, K, outs_h)
        for k in range(K):
            assert hop_error(np.ascontiguousarray(outs_h[k].numpy()), want[k]) <= TOL
        hplan.close()
