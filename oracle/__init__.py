"""numpy front end of the CPU oracle (oracle/gnnpre_oracle.c).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's CPU-baseline
leg are the only callers.  The CUDA library neither imports nor links any of this, and
this package imports nothing from the CUDA package.

The C file is compiled with gcc on first use (or by `build()`); every function below
only marshals numpy arrays into the C call of the same name.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

OP_GCN, OP_SAGE, OP_GIN = 0, 1, 2

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gnnpre_oracle.c")
_LIB = os.path.join(_HERE, "libgnnpre_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc -O2 (OpenMP on); returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.run(["gcc", "-O2", "-fopenmp", "-std=c99", "-Wall", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"],
                       check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _c():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i32, i64, f64 = ctypes.c_int32, ctypes.c_int64, ctypes.c_double
        p = ctypes.c_void_p
        lib.orc_num_threads.restype = ctypes.c_int
        lib.orc_set_num_threads.argtypes = [ctypes.c_int]
        lib.orc_degrees.argtypes = [i64, p, p]
        lib.orc_scales_f32.argtypes = [ctypes.c_int, i64, p, p, p]
        lib.orc_support_nnz.argtypes = [ctypes.c_int, i64, i64]
        lib.orc_support_nnz.restype = i64
        lib.orc_support.argtypes = [ctypes.c_int, i64, p, p, p, p]
        lib.orc_dense_operator.argtypes = [ctypes.c_int, f64, i64, p, p, p]
        lib.orc_hop_f64.argtypes = [ctypes.c_int, f64, i64, p, p, i64, p, p]
        lib.orc_propagate.argtypes = [ctypes.c_int, f64, i64, p, p, i64, p, i64, ctypes.c_int, p]
        lib.orc_propagate_teleport.argtypes = [ctypes.c_int, f64, f64, i64, p, p, i64, p, i64, ctypes.c_int, p]
        lib.orc_hop_rows_f32.argtypes = [ctypes.c_int, f64, i64, p, p, i64, p, i64, i64, p, p, p]
        lib.orc_block_offsets.argtypes = [i64, i32, p]
        lib.orc_block_offsets.restype = ctypes.c_int
        lib.orc_block_rows.argtypes = [i64, p, i32, p, p, p, p, p]
        lib.orc_solve_budget.argtypes = [i64] * 8 + [p, p]
        lib.orc_solve_budget.restype = ctypes.c_int
        lib.orc_solve_normalisation_blocks.argtypes = [i64] * 8
        lib.orc_solve_normalisation_blocks.restype = i64
        lib.orc_normalized_values.argtypes = [ctypes.c_int, f64, i64, p, p, p]
        lib.orc_slab_width.argtypes = [i64, i64]
        lib.orc_slab_width.restype = i64
        lib.orc_propagate_blocked.argtypes = [ctypes.c_int, f64, i64, p, p, i64, p, i64, ctypes.c_int, i32, i32, p]
        lib.orc_propagate_blocked.restype = ctypes.c_int
        lib.orc_weighted_hop_sum.argtypes = [ctypes.c_int, f64, i64, p, p, i64, p, i64, ctypes.c_int, p, p]
        lib.orc_lc_first_layer.argtypes = [i64, p, i64, p, i64, i64, p, i64, ctypes.c_int, p, p]
        _lib = lib
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _csr(rowptr, colidx):
    rowptr = np.ascontiguousarray(np.asarray(rowptr), dtype=np.int64)
    colidx = np.ascontiguousarray(np.asarray(colidx), dtype=np.int32)
    return rowptr, colidx, rowptr.shape[0] - 1


def _f32_matrix(X):
    X = np.asarray(X)
    assert X.dtype == np.float32 and X.ndim == 2 and X.strides[1] == 4 and X.strides[0] % 4 == 0
    return X, X.strides[0] // 4


def num_threads() -> int:
    return int(_c().orc_num_threads())


def set_num_threads(t: int) -> None:
    _c().orc_set_num_threads(int(t))


def degrees(rowptr) -> np.ndarray:
    rowptr = np.ascontiguousarray(np.asarray(rowptr), dtype=np.int64)
    n = rowptr.shape[0] - 1
    deg = np.empty(n, dtype=np.int32)
    _c().orc_degrees(n, _ptr(rowptr), _ptr(deg))
    return deg


def scales_f32(op: int, deg):
    deg = np.ascontiguousarray(deg, dtype=np.int32)
    r = np.empty(deg.shape[0], dtype=np.float32)
    c = np.empty(deg.shape[0], dtype=np.float32)
    _c().orc_scales_f32(op, deg.shape[0], _ptr(deg), _ptr(r), _ptr(c))
    return r, c


def support_nnz(op: int, n: int, nnz: int) -> int:
    return int(_c().orc_support_nnz(op, n, nnz))


def support(op: int, rowptr, colidx):
    rowptr, colidx, n = _csr(rowptr, colidx)
    m = support_nnz(op, n, int(rowptr[n]))
    rp = np.empty(n + 1, dtype=np.int64)
    ci = np.empty(m, dtype=np.int32)
    _c().orc_support(op, n, _ptr(rowptr), _ptr(colidx), _ptr(rp), _ptr(ci))
    return rp, ci


def dense_operator(op: int, eps: float, rowptr, colidx) -> np.ndarray:
    rowptr, colidx, n = _csr(rowptr, colidx)
    A = np.empty((n, n), dtype=np.float64)
    _c().orc_dense_operator(op, float(eps), n, _ptr(rowptr), _ptr(colidx), _ptr(A))
    return A


def hop_f64(op: int, eps: float, rowptr, colidx, xprev: np.ndarray) -> np.ndarray:
    rowptr, colidx, n = _csr(rowptr, colidx)
    xprev = np.ascontiguousarray(xprev, dtype=np.float64)
    out = np.empty_like(xprev)
    _c().orc_hop_f64(op, float(eps), n, _ptr(rowptr), _ptr(colidx), xprev.shape[1], _ptr(xprev), _ptr(out))
    return out


def propagate(op: int, eps: float, rowptr, colidx, X, K: int) -> np.ndarray:
    """[K, n, F] fp64: hop k-1 holds A^^k X."""
    rowptr, colidx, n = _csr(rowptr, colidx)
    X, ldx = _f32_matrix(X)
    F = X.shape[1]
    out = np.empty((K, n, F), dtype=np.float64)
    _c().orc_propagate(op, float(eps), n, _ptr(rowptr), _ptr(colidx), F, _ptr(X), ldx, K, _ptr(out))
    return out


def propagate_teleport(op: int, eps: float, alpha: float, rowptr, colidx, X, K: int) -> np.ndarray:
    """[K, n, F] fp64: X_k = (1 - alpha) A^ X_{k-1} + alpha X_0."""
    rowptr, colidx, n = _csr(rowptr, colidx)
    X, ldx = _f32_matrix(X)
    F = X.shape[1]
    out = np.empty((K, n, F), dtype=np.float64)
    _c().orc_propagate_teleport(op, float(eps), float(alpha), n, _ptr(rowptr), _ptr(colidx), F, _ptr(X), ldx, K, _ptr(out))
    return out


def hop_rows_f32(op: int, eps: float, rowptr, colidx, xprev, rows, want_abs: bool = True):
    """Exact fp64 (A^ xprev)[rows] and (|A^| |xprev|)[rows] from an fp32 previous hop."""
    rowptr, colidx, n = _csr(rowptr, colidx)
    xprev, ldx = _f32_matrix(xprev)
    F = xprev.shape[1]
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    y = np.empty((rows.shape[0], F), dtype=np.float64)
    a = np.empty((rows.shape[0], F), dtype=np.float64) if want_abs else None
    _c().orc_hop_rows_f32(op, float(eps), n, _ptr(rowptr), _ptr(colidx), F, _ptr(xprev), ldx, rows.shape[0],
                          _ptr(rows), _ptr(y), _ptr(a) if want_abs else None)
    return y, a


def block_offsets(m: int, b: int) -> np.ndarray:
    e = np.empty(b + 1 if b >= 0 else 1, dtype=np.int64)
    if _c().orc_block_offsets(m, b, _ptr(e)) != 0:
        raise ValueError("empty block")
    return e


def block_rows(rowptr_t, e_off):
    rowptr_t = np.ascontiguousarray(rowptr_t, dtype=np.int64)
    e_off = np.ascontiguousarray(e_off, dtype=np.int64)
    n, b = rowptr_t.shape[0] - 1, e_off.shape[0] - 1
    out = [np.empty(b, dtype=np.int32) for _ in range(4)]
    _c().orc_block_rows(n, _ptr(rowptr_t), b, _ptr(e_off), *[_ptr(a) for a in out])
    return tuple(out)  # row_lo, row_hi, first_partial, last_partial


def solve_budget(B_S, B_X, B_fixed, beta_S, beta_X, B_GPU, max_b, max_c):
    b = np.zeros(1, dtype=np.int64)
    c = np.zeros(1, dtype=np.int64)
    rc = _c().orc_solve_budget(B_S, B_X, B_fixed, beta_S, beta_X, B_GPU, max_b, max_c, _ptr(b), _ptr(c))
    return None if rc != 0 else (int(b[0]), int(c[0]))


def solve_normalisation_blocks(B_A, B_S, B_D, alpha_A, alpha_S, alpha_D, B_GPU, max_a):
    return int(_c().orc_solve_normalisation_blocks(B_A, B_S, B_D, alpha_A, alpha_S, alpha_D, B_GPU, max_a))


def normalized_values(op: int, eps: float, rowptr, colidx) -> np.ndarray:
    """fp64 value of every edge of the support, in the order of support(op, rowptr, colidx)."""
    rowptr, colidx, n = _csr(rowptr, colidx)
    vals = np.empty(support_nnz(op, n, int(rowptr[n])), dtype=np.float64)
    _c().orc_normalized_values(op, float(eps), n, _ptr(rowptr), _ptr(colidx), _ptr(vals))
    return vals


def slab_width(F: int, c: int) -> int:
    return int(_c().orc_slab_width(F, c))


def propagate_blocked(op: int, eps: float, rowptr, colidx, X, K: int, b: int, c: int) -> np.ndarray:
    rowptr, colidx, n = _csr(rowptr, colidx)
    X, ldx = _f32_matrix(X)
    F = X.shape[1]
    out = np.empty((K, n, F), dtype=np.float64)
    rc = _c().orc_propagate_blocked(op, float(eps), n, _ptr(rowptr), _ptr(colidx), F, _ptr(X), ldx, K, b, c,
                                    _ptr(out))
    if rc != 0:
        raise ValueError("impossible (b, c)")
    return out


def lc_first_layer(Xk, batch, Wt, relu: bool, want_abs: bool = False):
    """act(Xk[batch] @ Wt.T) in fp64 (Eq. 9's first dense stage); Wt is [H, F]; batch None = all rows."""
    Xk, ldx = _f32_matrix(Xk)
    Wt, ldw = _f32_matrix(Wt)
    F, H = Xk.shape[1], Wt.shape[0]
    assert Wt.shape[1] == F
    if batch is None:
        B, bp = Xk.shape[0], None
    else:
        batch = np.ascontiguousarray(batch, dtype=np.int64)
        assert batch.size == 0 or (batch.min() >= 0 and batch.max() < Xk.shape[0])
        B, bp = batch.shape[0], _ptr(batch)
    Y = np.empty((B, H), dtype=np.float64)
    A = np.empty((B, H), dtype=np.float64) if want_abs else None
    _c().orc_lc_first_layer(B, bp, F, _ptr(Xk), ldx, H, _ptr(Wt), ldw, int(bool(relu)), _ptr(Y),
                            _ptr(A) if want_abs else None)
    return (Y, A) if want_abs else Y


def weighted_hop_sum(op: int, eps: float, rowptr, colidx, X, gamma) -> np.ndarray:
    """[n, F] fp64: sum_k gamma[k] A^^k X for k = 0..len(gamma)-1 (fixed-weight generalised PageRank)."""
    rowptr, colidx, n = _csr(rowptr, colidx)
    X, ldx = _f32_matrix(X)
    gamma = np.ascontiguousarray(gamma, dtype=np.float64)
    Z = np.empty((n, X.shape[1]), dtype=np.float64)
    _c().orc_weighted_hop_sum(op, float(eps), n, _ptr(rowptr), _ptr(colidx), X.shape[1], _ptr(X), ldx,
                              gamma.shape[0] - 1, _ptr(gamma), _ptr(Z))
    return Z
