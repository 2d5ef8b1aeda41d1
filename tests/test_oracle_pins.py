"""Pins for the CPU oracle: closed forms, invariants, brute force and a library cross-check.

None of these tests touches the CUDA path.  Each one is chosen so that a plausible slip in
oracle/gnnpre_oracle.c (a dropped self-loop, D instead of D~, a transposed normalisation,
an off-by-one block boundary) breaks at least one of them.
"""
import itertools
import os

import numpy as np
import pytest
import scipy.sparse as sp

import gnnpre_inputs as gi
import oracle as orc

OPS = (orc.OP_GCN, orc.OP_SAGE, orc.OP_GIN)
EPS = 0.1


def csr_of(n, edges):
    g = gi.from_edge_list(n, edges)
    return g.rowptr.numpy(), g.colidx.numpy()


def dense_adjacency(rowptr, colidx):
    n = len(rowptr) - 1
    A = np.zeros((n, n))
    for i in range(n):
        A[i, colidx[rowptr[i]:rowptr[i + 1]]] = 1.0
    return A


def random_graph(n, m, seed):
    g = gi.erdos_renyi(n, m, seed)
    return g.rowptr.numpy(), g.colidx.numpy()


def features(n, F, seed):
    return gi.normal_matrix(n, F, seed).numpy()


# ------------------------------------------------------------------ worked examples / closed forms

def test_path3_hand_worked(golden_dir):
    """Eq. 1, SAGE mean and GIN sum evaluated by hand on the path 0-1-2."""
    want = {}
    for line in open(os.path.join(golden_dir, "path3_worked.txt")):
        if not line.startswith("#"):
            name, *vals = line.split()
            want[name] = np.array([float(v) for v in vals])
    rowptr, colidx = csr_of(3, [(0, 1), (1, 2)])
    X = np.array([[1.0], [2.0], [3.0]], dtype=np.float32)
    for op, name in ((orc.OP_GCN, "gcn"), (orc.OP_SAGE, "sage"), (orc.OP_GIN, "gin")):
        got = orc.propagate(op, EPS, rowptr, colidx, X, 1)[0, :, 0]
        np.testing.assert_allclose(got, want[name], rtol=1e-15, atol=0)


def test_complete_graph_gcn_is_column_mean():
    """K_n: every D~_i = n, so S = J/n and each hop replaces every row by the column mean."""
    n, F = 9, 5
    rowptr, colidx = csr_of(n, list(itertools.combinations(range(n), 2)))
    X = features(n, F, 1)
    out = orc.propagate(orc.OP_GCN, 0.0, rowptr, colidx, X, 3)
    mean = X.astype(np.float64).mean(axis=0)
    for k in range(3):
        np.testing.assert_allclose(out[k], np.tile(mean, (n, 1)), rtol=1e-14, atol=1e-15)


def test_cycle_gcn_trinomial(golden_dir):
    """C_n: S = (A+I)/3 is circulant; hop k of a unit impulse = trinomial coefficients / 3^k."""
    rows = [list(map(int, l.split())) for l in open(os.path.join(golden_dir, "trinomial.txt")) if l[0] != "#"]
    n = 17
    rowptr, colidx = csr_of(n, [(i, (i + 1) % n) for i in range(n)])
    X = np.zeros((n, 1), dtype=np.float32)
    X[0, 0] = 1.0
    K = len(rows)
    out = orc.propagate(orc.OP_GCN, 0.0, rowptr, colidx, X, K)
    for k in range(1, K + 1):
        want = np.zeros(n)
        for offset, coeff in zip(range(-k, k + 1), rows[k - 1]):
            want[offset % n] += coeff / 3.0 ** k
        np.testing.assert_allclose(out[k - 1, :, 0], want, rtol=1e-14, atol=1e-17)


def test_regular_graph_reduces_to_scaled_adjacency():
    """d-regular: GCN = (A+I)/(d+1), SAGE = A/d, GIN = A + (1+eps) I."""
    n, F = 12, 4
    edges = [(i, (i + s) % n) for i in range(n) for s in (1, 2)]  # 4-regular circulant
    rowptr, colidx = csr_of(n, edges)
    A = dense_adjacency(rowptr, colidx)
    assert (A.sum(1) == 4).all()
    X = features(n, F, 2)
    Xd = X.astype(np.float64)
    I = np.eye(n)
    np.testing.assert_allclose(orc.propagate(orc.OP_GCN, 0, rowptr, colidx, X, 1)[0], (A + I) @ Xd / 5, rtol=1e-14)
    np.testing.assert_allclose(orc.propagate(orc.OP_SAGE, 0, rowptr, colidx, X, 1)[0], A @ Xd / 4, rtol=1e-14)
    np.testing.assert_allclose(orc.propagate(orc.OP_GIN, EPS, rowptr, colidx, X, 1)[0], (A + (1 + EPS) * I) @ Xd,
                               rtol=1e-14)


def test_star_graph_by_hand():
    """Hub 0 with m leaves: D~_hub = m+1, D~_leaf = 2."""
    m = 6
    rowptr, colidx = csr_of(m + 1, [(0, l) for l in range(1, m + 1)])
    X = features(m + 1, 3, 3)
    Xd = X.astype(np.float64)
    got = orc.propagate(orc.OP_GCN, 0, rowptr, colidx, X, 1)[0]
    hub = Xd[0] / (m + 1) + Xd[1:].sum(0) / np.sqrt(2.0 * (m + 1))
    np.testing.assert_allclose(got[0], hub, rtol=1e-14)
    for l in range(1, m + 1):
        np.testing.assert_allclose(got[l], Xd[l] / 2 + Xd[0] / np.sqrt(2.0 * (m + 1)), rtol=1e-14)
    sage = orc.propagate(orc.OP_SAGE, 0, rowptr, colidx, X, 1)[0]
    np.testing.assert_allclose(sage[0], Xd[1:].mean(0), rtol=1e-14)
    for l in range(1, m + 1):
        np.testing.assert_allclose(sage[l], Xd[0], rtol=1e-15)


def test_gin_on_ones_counts_neighbours():
    rowptr, colidx = random_graph(50, 120, 4)
    deg = np.diff(rowptr)
    X = np.ones((50, 2), dtype=np.float32)
    got = orc.propagate(orc.OP_GIN, EPS, rowptr, colidx, X, 1)[0]
    np.testing.assert_allclose(got[:, 0], deg + 1 + EPS, rtol=1e-15)


def test_isolated_nodes():
    """D_i = 0: GCN keeps the row (D~ = 1), SAGE gives a zero row, GIN scales by 1+eps."""
    rowptr, colidx = csr_of(5, [(0, 1), (1, 2)])  # nodes 3, 4 isolated
    X = features(5, 3, 5)
    Xd = X.astype(np.float64)
    np.testing.assert_array_equal(orc.propagate(orc.OP_GCN, 0, rowptr, colidx, X, 2)[1][3:], Xd[3:])
    np.testing.assert_array_equal(orc.propagate(orc.OP_SAGE, 0, rowptr, colidx, X, 1)[0][3:], 0 * Xd[3:])
    np.testing.assert_allclose(orc.propagate(orc.OP_GIN, EPS, rowptr, colidx, X, 1)[0][3:], (1 + EPS) * Xd[3:],
                               rtol=1e-15)


# ------------------------------------------------------------------ invariants on random graphs

@pytest.mark.parametrize("seed", [11, 12])
def test_fixed_points(seed):
    n = 200
    rowptr, colidx = random_graph(n, 500, seed)
    deg = np.diff(rowptr).astype(np.float64)
    ones = np.ones((n, 1), dtype=np.float32)
    sage = orc.propagate(orc.OP_SAGE, 0, rowptr, colidx, ones, 2)
    np.testing.assert_allclose(sage[0][:, 0], (deg > 0).astype(float), rtol=1e-15)
    # S D~^{1/2} 1 = D~^{1/2} 1: use perfect squares so that the fp32 input is exact
    g = gi.from_edge_list(10, [(0, j) for j in range(1, 9)] + [(9, 1), (9, 2), (9, 3)])  # D~ in {9, 2, 3, 4}
    rp, ci = g.rowptr.numpy(), g.colidx.numpy()
    v = np.sqrt(np.diff(rp) + 1.0)
    out = orc.hop_f64(orc.OP_GCN, 0, rp, ci, v[:, None])
    np.testing.assert_allclose(out[:, 0], v, rtol=1e-15)
    out = orc.hop_f64(orc.OP_GCN, 0, rowptr, colidx, np.sqrt(deg + 1.0)[:, None])
    np.testing.assert_allclose(out[:, 0], np.sqrt(deg + 1.0), rtol=1e-14)


@pytest.mark.parametrize("seed", [21, 22])
def test_conservation_laws(seed):
    """Symmetric A: sum_i sqrt(D~_i) X_k[i] is constant (GCN); sum_i D_i X_k[i] is constant (SAGE);
    sum_i X_k[i] = sum_j (D_j + 1 + eps) X_{k-1}[j] (GIN)."""
    n, F, K = 300, 6, 3
    rowptr, colidx = random_graph(n, 900, seed)
    deg = np.diff(rowptr).astype(np.float64)
    X = features(n, F, seed)
    hops = {op: np.concatenate([X.astype(np.float64)[None], orc.propagate(op, EPS, rowptr, colidx, X, K)]) for op in OPS}
    for k in range(1, K + 1):
        g = hops[orc.OP_GCN]
        np.testing.assert_allclose(np.sqrt(deg + 1) @ g[k], np.sqrt(deg + 1) @ g[0], rtol=1e-12, atol=1e-12)
        s = hops[orc.OP_SAGE]
        np.testing.assert_allclose(deg @ s[k], deg @ s[k - 1], rtol=1e-12, atol=1e-12)
        q = hops[orc.OP_GIN]
        np.testing.assert_allclose(q[k].sum(0), (deg + 1 + EPS) @ q[k - 1], rtol=1e-12, atol=1e-10)


def test_contractions():
    n, F = 400, 8
    rowptr, colidx = random_graph(n, 1500, 31)
    X = features(n, F, 31)
    g = orc.propagate(orc.OP_GCN, 0, rowptr, colidx, X, 4)
    norms = [np.linalg.norm(X.astype(np.float64), axis=0)] + [np.linalg.norm(g[k], axis=0) for k in range(4)]
    for a, b in zip(norms, norms[1:]):
        assert (b <= a * (1 + 1e-14)).all()  # spectrum of S lies in [-1, 1]
    s = orc.propagate(orc.OP_SAGE, 0, rowptr, colidx, X, 2)
    assert np.abs(s[0]).max() <= np.abs(X).max() and np.abs(s[1]).max() <= np.abs(s[0]).max()


@pytest.mark.parametrize("op", OPS)
def test_linearity_and_relabelling(op):
    n, F = 120, 5
    rowptr, colidx = random_graph(n, 400, 41)
    X, Y = features(n, F, 41), features(n, F, 42)
    a = orc.propagate(op, EPS, rowptr, colidx, X, 2)
    b = orc.propagate(op, EPS, rowptr, colidx, Y, 2)
    Xd, Yd = X.astype(np.float64), Y.astype(np.float64)
    lin = orc.hop_f64(op, EPS, rowptr, colidx, orc.hop_f64(op, EPS, rowptr, colidx, 2.0 * Xd - 0.5 * Yd))
    np.testing.assert_allclose(lin, 2.0 * a[1] - 0.5 * b[1], rtol=1e-12, atol=1e-13)
    # relabel nodes by a permutation: P A P^T, P X  ->  P X_k
    rng = np.random.default_rng(7)
    perm = rng.permutation(n)  # new id of old node i is perm[i]
    A = sp.csr_matrix((np.ones(len(colidx)), colidx, rowptr), shape=(n, n)).tocoo()
    B = sp.csr_matrix((A.data, (perm[A.row], perm[A.col])), shape=(n, n))
    B.sort_indices()
    Xp = np.empty_like(X)
    Xp[perm] = X
    c = orc.propagate(op, EPS, B.indptr.astype(np.int64), B.indices.astype(np.int32), Xp, 2)
    np.testing.assert_allclose(c[1][perm], a[1], rtol=1e-12, atol=1e-13)


# ------------------------------------------------------------------ brute force and library cross-checks

@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("seed", [51, 52, 53])
def test_dense_power_brute_force(op, seed):
    """A^ built densely in this test from its definition; A^^k X via an explicit matrix power."""
    n, F, K = 24, 3, 4
    rowptr, colidx = random_graph(n, 40 + seed % 7, seed)
    A = dense_adjacency(rowptr, colidx)
    d = A.sum(1)
    if op == orc.OP_GCN:
        At = A + np.eye(n)
        dinv = 1.0 / np.sqrt(At.sum(1))
        Ahat = dinv[:, None] * At * dinv[None, :]
        assert np.allclose(Ahat, Ahat.T)
    elif op == orc.OP_SAGE:
        Ahat = np.divide(A, d[:, None], out=np.zeros_like(A), where=d[:, None] > 0)
        assert np.allclose(Ahat.sum(1)[d > 0], 1.0)
    else:
        Ahat = A + (1 + EPS) * np.eye(n)
    np.testing.assert_allclose(orc.dense_operator(op, EPS, rowptr, colidx), Ahat, rtol=1e-15, atol=0)
    X = features(n, F, seed)
    got = orc.propagate(op, EPS, rowptr, colidx, X, K)
    for k in range(1, K + 1):
        want = np.linalg.matrix_power(Ahat, k) @ X.astype(np.float64)
        np.testing.assert_allclose(got[k - 1], want, rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("op", OPS)
def test_against_scipy_sparse_product(op):
    """The c1-sized graph through scipy.sparse CSR x dense in float64 (a textbook routine)."""
    w = gi.WORKLOADS["c1"]
    g = gi.make_graph(w)
    rowptr, colidx, n = g.rowptr.numpy(), g.colidx.numpy(), g.n
    A = sp.csr_matrix((np.ones(g.nnz), colidx, rowptr), shape=(n, n))
    d = np.asarray(A.sum(1)).ravel()
    if op == orc.OP_GCN:
        Dm = sp.diags(1.0 / np.sqrt(d + 1))
        Ahat = Dm @ (A + sp.identity(n)) @ Dm
    elif op == orc.OP_SAGE:
        Ahat = sp.diags(np.where(d > 0, 1.0 / np.maximum(d, 1), 0.0)) @ A
    else:
        Ahat = A + (1 + EPS) * sp.identity(n)
    X = gi.make_features(w).numpy()
    got = orc.propagate(op, EPS, rowptr, colidx, X, 3)
    cur = X.astype(np.float64)
    for k in range(3):
        cur = Ahat @ cur
        np.testing.assert_allclose(got[k], cur, rtol=1e-11, atol=1e-12)


def test_hop_rows_matches_full_hop_and_abs_bound():
    n, F = 150, 7
    rowptr, colidx = random_graph(n, 600, 61)
    X = features(n, F, 61)
    rows = np.array([0, 3, 149, 77, 3])
    for op in OPS:
        full = orc.propagate(op, EPS, rowptr, colidx, X, 1)[0]
        y, a = orc.hop_rows_f32(op, EPS, rowptr, colidx, X, rows)
        np.testing.assert_array_equal(y, full[rows])
        absfull = orc.propagate(op, EPS, rowptr, colidx, np.abs(X), 1)[0]  # all weights are >= 0
        np.testing.assert_allclose(a, absfull[rows], rtol=1e-14)
        assert (np.abs(y) <= a * (1 + 1e-14)).all()


def test_strided_input_is_honoured():
    n, F = 40, 6
    rowptr, colidx = random_graph(n, 90, 62)
    buf = np.full((n, 8), np.nan, dtype=np.float32)
    buf[:, :F] = features(n, F, 62)
    a = orc.propagate(orc.OP_GCN, 0, rowptr, colidx, buf[:, :F], 2)
    b = orc.propagate(orc.OP_GCN, 0, rowptr, colidx, np.ascontiguousarray(buf[:, :F]), 2)
    np.testing.assert_array_equal(a, b)


# ------------------------------------------------------------------ degrees, support, scales

def test_degrees_support_and_scales():
    rowptr, colidx = random_graph(60, 150, 71)
    A = dense_adjacency(rowptr, colidx)
    deg = orc.degrees(rowptr)
    np.testing.assert_array_equal(deg, A.sum(1).astype(np.int32))
    for op in OPS:
        rp, ci = orc.support(op, rowptr, colidx)
        want = A + np.eye(60) if op != orc.OP_SAGE else A
        assert rp[-1] == orc.support_nnz(op, 60, len(colidx)) == int(want.sum())
        for i in range(60):
            row = ci[rp[i]:rp[i + 1]]
            assert (np.diff(row) > 0).all()  # ascending, no duplicates
            np.testing.assert_array_equal(row, np.nonzero(want[i])[0])
        r, c = orc.scales_f32(op, deg)
        assert r.dtype == c.dtype == np.float32
        dense = orc.dense_operator(op, 0.0, rowptr, colidx)
        prod = r.astype(np.float64)[:, None] * want * c.astype(np.float64)[None, :]
        np.testing.assert_allclose(prod, dense, rtol=2e-7)  # fp32 rounding of the two factors
    r, _ = orc.scales_f32(orc.OP_GCN, np.array([0, 3, 8, 15], dtype=np.int32))
    np.testing.assert_array_equal(r, np.array([1.0, 0.5, 1.0 / 3.0, 0.25], dtype=np.float32))
    r, c = orc.scales_f32(orc.OP_SAGE, np.array([0, 1, 4], dtype=np.int32))
    np.testing.assert_array_equal(r, np.array([0.0, 1.0, 0.25], dtype=np.float32))
    np.testing.assert_array_equal(c, np.ones(3, dtype=np.float32))


# ------------------------------------------------------------------ edge decomposition

def test_block_offsets_exhaustive():
    """Every (m, b) with b <= m <= 40: disjoint cover, sizes within one edge, monotone."""
    for m in range(1, 41):
        for b in range(1, m + 1):
            e = orc.block_offsets(m, b)
            assert e[0] == 0 and e[-1] == m
            sizes = np.diff(e)
            assert sizes.min() >= 1 and sizes.max() - sizes.min() <= 1
            np.testing.assert_array_equal(e, [(l * m) // b for l in range(b + 1)])
    with pytest.raises(ValueError):
        orc.block_offsets(5, 6)
    with pytest.raises(ValueError):
        orc.block_offsets(5, 0)
    big = orc.block_offsets(3_000_000_000_007, 64)  # beyond 32 bits: exact integer arithmetic
    np.testing.assert_array_equal(big, [(l * 3_000_000_000_007) // 64 for l in range(65)])


@pytest.mark.parametrize("op", OPS)
def test_blocks_partition_the_operator(op):
    """Eq. 10 structurally: the block matrices are disjoint and sum to A^ exactly."""
    n = 30
    rowptr, colidx = random_graph(n, 70, 81)
    rp, ci = orc.support(op, rowptr, colidx)
    m = int(rp[-1])
    dense = orc.dense_operator(op, EPS, rowptr, colidx)
    rows_of_edge = np.repeat(np.arange(n), np.diff(rp))
    for b in (1, 2, 3, 7, m):
        e = orc.block_offsets(m, b)
        total = np.zeros_like(dense)
        seen = np.zeros((n, n), dtype=int)
        for l in range(b):
            blk = np.zeros_like(dense)
            r, c = rows_of_edge[e[l]:e[l + 1]], ci[e[l]:e[l + 1]]
            blk[r, c] = dense[r, c]
            seen[r, c] += 1
            total += blk
        assert seen.max() == 1  # pairwise disjoint
        np.testing.assert_array_equal(total, dense)  # exact: every entry lives in one block
        row_lo, row_hi, fp, lp = orc.block_rows(rp, e)
        np.testing.assert_array_equal(row_lo, np.searchsorted(rp, e[:-1], side="right") - 1)
        np.testing.assert_array_equal(row_hi, np.searchsorted(rp, e[1:] - 1, side="right") - 1)
        np.testing.assert_array_equal(fp, (rp[row_lo] < e[:-1]).astype(np.int32))
        np.testing.assert_array_equal(lp, (rp[row_hi + 1] > e[1:]).astype(np.int32))


@pytest.mark.parametrize("op", OPS)
def test_algorithm1_equals_definition(op):
    n, F, K = 40, 10, 3
    rowptr, colidx = random_graph(n, 110, 91)
    X = features(n, F, 91)
    plain = orc.propagate(op, EPS, rowptr, colidx, X, K)
    m = orc.support_nnz(op, n, len(colidx))
    for b, c in ((1, 1), (3, 1), (1, 2), (5, 3), (m, 2)):
        blocked = orc.propagate_blocked(op, EPS, rowptr, colidx, X, K, b, c)
        np.testing.assert_allclose(blocked, plain, rtol=1e-12, atol=1e-13)
    with pytest.raises(ValueError):
        orc.propagate_blocked(op, EPS, rowptr, colidx, X, K, m + 1, 1)


# ------------------------------------------------------------------ Eq. 11 / Eq. 12

def test_budget_solver_against_closed_form_and_python():
    rng = np.random.default_rng(5)
    for _ in range(200):
        B_S, B_X = int(rng.integers(1, 5000)), int(rng.integers(1, 5000))
        B_fixed = int(rng.integers(0, 50))
        beta_S, beta_X = int(rng.integers(1, 4)), int(rng.integers(1, 4))
        B_GPU = int(rng.integers(1, 4000))
        max_b, max_c = 64, 12
        got = orc.solve_budget(B_S, B_X, B_fixed, beta_S, beta_X, B_GPU, max_b, max_c)
        best = None
        for c in range(1, max_c + 1):
            room = B_GPU - B_fixed - -(-beta_X * B_X // c)
            if room <= 0:
                continue
            b = -(-beta_S * B_S // room)  # closed form: least b with ceil(beta_S B_S / b) <= room
            if b > max_b:
                continue
            key = (b * c, c, b)
            if best is None or key < best:
                best = key
        assert got == (None if best is None else (best[2], best[1]))


def test_paper_block_counts_are_feasible(golden_dir):
    """The paper's own sizes: (b, c) = (10, 16) must satisfy Eq. 12 for a 32 GB device, and the
    printed volumes must match the dataset table (fp32 features; COO with two int64 + one fp32)."""
    v = {}
    for line in open(os.path.join(golden_dir, "paper_sizes.txt")):
        if not line.startswith("#"):
            k, x = line.split()
            v[k] = int(x)
    GB = 10 ** 9
    assert round(v["nodes"] * v["features"] * 4 / GB) == v["feature_matrix_GB"]
    assert round((2 * v["edges"] + v["nodes"]) * 20 / GB) == v["normalized_adjacency_GB"]
    B_S, B_X, B_GPU = v["normalized_adjacency_GB"] * GB, v["feature_matrix_GB"] * GB, v["gpu_memory_GB"] * GB
    for beta_S, beta_X in ((1, 1), (2, 2)):
        assert -(-beta_S * B_S // v["b"]) + -(-beta_X * B_X // v["c"]) <= B_GPU
        b, c = orc.solve_budget(B_S, B_X, 0, beta_S, beta_X, B_GPU, 64, 32)
        assert b * c <= v["b"] * v["c"]  # the solver can only do at least as well
    assert orc.solve_normalisation_blocks(10, 20, 3, 1, 1, 1, 13, 100) == 3  # ceil(30/a) + 3 <= 13  ->  a = 3
    assert orc.solve_normalisation_blocks(10, 20, 30, 1, 1, 1, 13, 100) == -1


def test_slab_width():
    assert orc.slab_width(128, 1) == 128 and orc.slab_width(128, 16) == 8
    assert orc.slab_width(100, 3) == 36 and orc.slab_width(10, 2) == 8


# ------------------------------------------------------------------ the normalised adjacency itself (Eq. 1 / Eq. 10)

@pytest.mark.parametrize("op", OPS)
def test_normalized_values_rebuild_the_dense_operator(op):
    """The per-edge values, scattered by the support's structure, are the dense operator built in this
    test from its definition; every block of Eq. 10 is a slice of them and the blocks sum to S."""
    n = 40
    rowptr, colidx = random_graph(n, 100, 95)
    A = dense_adjacency(rowptr, colidx)
    d = A.sum(1)
    if op == orc.OP_GCN:
        At = A + np.eye(n)
        dinv = 1.0 / np.sqrt(At.sum(1))
        want = dinv[:, None] * At * dinv[None, :]
    elif op == orc.OP_SAGE:
        want = np.divide(A, d[:, None], out=np.zeros_like(A), where=d[:, None] > 0)
    else:
        want = A + (1 + EPS) * np.eye(n)
    rp, ci = orc.support(op, rowptr, colidx)
    vals = orc.normalized_values(op, EPS, rowptr, colidx)
    assert vals.shape == (rp[-1],)
    got = sp.csr_matrix((vals, ci, rp), shape=(n, n)).toarray()
    np.testing.assert_allclose(got, want, rtol=1e-15, atol=0)
    if op == orc.OP_GCN:
        np.testing.assert_allclose(got, got.T, rtol=1e-15)
    if op == orc.OP_SAGE:
        np.testing.assert_allclose(got.sum(1)[d > 0], 1.0, rtol=1e-14)
    for b in (1, 3, 7):
        e = orc.block_offsets(int(rp[-1]), b)
        total = np.zeros((n, n))
        rows_of_edge = np.repeat(np.arange(n), np.diff(rp))
        for l in range(b):
            blk = np.zeros((n, n))
            blk[rows_of_edge[e[l]:e[l + 1]], ci[e[l]:e[l + 1]]] = vals[e[l]:e[l + 1]]
            total += blk
        np.testing.assert_array_equal(total, got)  # Eq. 10: S = sum_l D~^{-1/2} A~^(l) D~^{-1/2}
    X = features(n, 3, 96)
    np.testing.assert_allclose(got @ X.astype(np.float64), orc.propagate(op, EPS, rowptr, colidx, X, 1)[0], rtol=1e-13,
                               atol=1e-14)


# ------------------------------------------------------------------ teleport (PPR) filter

@pytest.mark.parametrize("op", OPS)
def test_teleport_propagation_pins(op):
    """X_k = (1-a) A^ X_{k-1} + a X_0: a = 0 is the plain chain, a = 1 returns X_0, and for GCN/SAGE the
    iteration converges to the dense solution a (I - (1-a) A^)^{-1} X_0 (computed here with numpy)."""
    n, F = 30, 4
    rowptr, colidx = random_graph(n, 80, 97)
    X = features(n, F, 97)
    Xd = X.astype(np.float64)
    np.testing.assert_array_equal(orc.propagate_teleport(op, EPS, 0.0, rowptr, colidx, X, 3),
                                  orc.propagate(op, EPS, rowptr, colidx, X, 3))
    np.testing.assert_array_equal(orc.propagate_teleport(op, EPS, 1.0, rowptr, colidx, X, 3), np.stack([Xd] * 3))
    a = 0.15
    got = orc.propagate_teleport(op, EPS, a, rowptr, colidx, X, 3)
    Ahat = orc.dense_operator(op, EPS, rowptr, colidx)
    cur = Xd
    for k in range(3):
        cur = (1 - a) * (Ahat @ cur) + a * Xd
        np.testing.assert_allclose(got[k], cur, rtol=1e-13, atol=1e-14)
    if op != orc.OP_GIN:  # spectral radius <= 1: the iteration contracts with factor 1-a
        far = orc.propagate_teleport(op, EPS, 0.5, rowptr, colidx, X, 60)[-1]
        fixed = 0.5 * np.linalg.solve(np.eye(n) - 0.5 * Ahat, Xd)
        np.testing.assert_allclose(far, fixed, rtol=1e-10, atol=1e-12)


def test_teleport_on_complete_graph_closed_form():
    """K_n under GCN: A^ x = column mean, and the mean is preserved, so X_k = (1-a) mean + a X_0 for every k."""
    n, F, a = 8, 3, 0.3
    rowptr, colidx = csr_of(n, list(itertools.combinations(range(n), 2)))
    X = features(n, F, 98)
    Xd = X.astype(np.float64)
    want = (1 - a) * np.tile(Xd.mean(0), (n, 1)) + a * Xd
    got = orc.propagate_teleport(orc.OP_GCN, 0.0, a, rowptr, colidx, X, 4)
    for k in range(4):
        np.testing.assert_allclose(got[k], want, rtol=1e-13, atol=1e-15)


# ------------------------------------------------------------------ first dense stage of an LC model (Eq. 9)

def test_first_layer_against_library_product_and_special_weights():
    n, F, H = 90, 13, 7  # H != F so that a transposed weight cannot pass
    X, Wt = features(n, F, 61), features(H, F, 62)
    batch = np.random.default_rng(5).integers(0, n, size=41)
    Y, A = orc.lc_first_layer(X, batch, Wt, relu=False, want_abs=True)
    ref = X[batch].astype(np.float64) @ Wt.astype(np.float64).T
    np.testing.assert_allclose(Y, ref, rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(A, np.abs(X[batch]).astype(np.float64) @ np.abs(Wt).astype(np.float64).T, rtol=1e-13)
    assert (np.abs(Y) <= A * (1 + 1e-12)).all()
    # sigma = ReLU applied after the product, element by element
    R = orc.lc_first_layer(X, batch, Wt, relu=True)
    np.testing.assert_array_equal(R, np.maximum(Y, 0.0))
    assert (R == 0).any() and (R > 0).any()
    # one-hot weights pick columns; the identity returns the gathered rows; no batch = every row in order
    sel = np.zeros((3, F), dtype=np.float32)
    sel[0, 4] = sel[1, 0] = sel[2, 12] = 1.0
    np.testing.assert_array_equal(orc.lc_first_layer(X, batch, sel, relu=False), X[batch][:, [4, 0, 12]].astype(np.float64))
    np.testing.assert_array_equal(orc.lc_first_layer(X, None, np.eye(F, dtype=np.float32), relu=False), X.astype(np.float64))
    # a strided matrix (leading dimension above F) is honoured
    Xs = np.full((n, F + 3), np.nan, dtype=np.float32)
    Xs[:, :F] = X
    np.testing.assert_array_equal(orc.lc_first_layer(Xs[:, :F], batch, Wt, relu=False), Y)
    assert orc.lc_first_layer(X, np.zeros(0, dtype=np.int64), Wt, relu=True).shape == (0, H)


def test_first_layer_commutes_with_propagation():
    """The LC transformation rests on S^k (X W) = (S^k X) W.  With the GIN sum operator (eps = 0) and
    small integer X, W every quantity is an integer that fp32 holds exactly, so both sides are equal."""
    n, F, H, K = 60, 6, 4, 3
    rowptr, colidx = random_graph(n, 150, 71)
    rng = np.random.default_rng(72)
    X = rng.integers(-3, 4, size=(n, F)).astype(np.float32)
    Wt = rng.integers(-2, 3, size=(H, F)).astype(np.float32)
    hops = orc.propagate(orc.OP_GIN, 0.0, rowptr, colidx, X, K)
    XW = (X.astype(np.float64) @ Wt.astype(np.float64).T).astype(np.float32)
    hops_of_XW = orc.propagate(orc.OP_GIN, 0.0, rowptr, colidx, XW, K)
    batch = rng.permutation(n)[:37]
    for k in range(K):
        hop32 = hops[k].astype(np.float32)
        assert (hop32.astype(np.float64) == hops[k]).all()
        np.testing.assert_array_equal(orc.lc_first_layer(hop32, batch, Wt, relu=False), hops_of_XW[k][batch])


# ------------------------------------------------------------------ fixed-weight sum of hops (GPRGNN's filter, weights fixed)

@pytest.mark.parametrize("op", OPS)
def test_weighted_hop_sum_pins(op):
    n, F, K = 90, 4, 4
    rowptr, colidx = random_graph(n, 300, 81)
    X = features(n, F, 82)
    hops = orc.propagate(op, EPS, rowptr, colidx, X, K)
    # unit weights pick single hops (k = 0 is X itself); a general gamma is the same linear combination
    for k in range(K + 1):
        e = np.zeros(K + 1)
        e[k] = 1.0
        want = X.astype(np.float64) if k == 0 else hops[k - 1]
        np.testing.assert_allclose(orc.weighted_hop_sum(op, EPS, rowptr, colidx, X, e), want, rtol=1e-13, atol=1e-14)
    gamma = np.array([0.3, -1.25, 0.5, 2.0, -0.75])
    want = gamma[0] * X.astype(np.float64) + sum(gamma[k] * hops[k - 1] for k in range(1, K + 1))
    np.testing.assert_allclose(orc.weighted_hop_sum(op, EPS, rowptr, colidx, X, gamma), want, rtol=1e-12, atol=1e-13)
    # the K-step PageRank iteration X_k = (1-a) A^ X_{k-1} + a X_0 unrolls to such a sum:
    # X_K = (1-a)^K A^^K X_0 + a sum_{k<K} (1-a)^k A^^k X_0
    a = 0.15
    g = np.array([a * (1 - a) ** k for k in range(K)] + [(1 - a) ** K])
    ppr = orc.propagate_teleport(op, EPS, a, rowptr, colidx, X, K)[K - 1]
    np.testing.assert_allclose(orc.weighted_hop_sum(op, EPS, rowptr, colidx, X, g), ppr, rtol=1e-12, atol=1e-13)


def test_weighted_hop_sum_on_complete_graph_closed_form():
    """GCN on K_n: every hop k >= 1 is the column mean, so Z = gamma_0 X + (gamma_1 + ... + gamma_K) mean(X)."""
    n, F = 7, 3
    rowptr, colidx = csr_of(n, [(i, j) for i in range(n) for j in range(i + 1, n)])
    X = features(n, F, 83)
    gamma = np.array([0.5, 0.25, -2.0, 1.5])
    mean = X.astype(np.float64).mean(axis=0, keepdims=True)
    want = gamma[0] * X.astype(np.float64) + gamma[1:].sum() * np.repeat(mean, n, axis=0)
    np.testing.assert_allclose(orc.weighted_hop_sum(orc.OP_GCN, 0.0, rowptr, colidx, X, gamma), want, rtol=1e-12, atol=1e-13)
