"""Helpers shared by the GPU parity tests: error measures and oracle-side expectations."""
import numpy as np
import torch

import oracle as orc

TOL = 1e-5  # max relative error per hop against the fp64 oracle


def hop_error(got: np.ndarray, want: np.ndarray) -> float:
    """max |g - o| / max(|o|, tau), tau = RMS of the oracle's hop (outputs that cancel to ~0 are
    measured against the hop's typical magnitude)."""
    want = np.asarray(want, dtype=np.float64)
    tau = float(np.sqrt(np.mean(want * want)))
    if tau == 0.0:
        return float(np.abs(got).max(initial=0.0))
    return float((np.abs(got.astype(np.float64) - want) / np.maximum(np.abs(want), tau)).max(initial=0.0))


def backward_error(op, eps, rowptr, colidx, prev_f32: np.ndarray, got: np.ndarray, rows=None) -> float:
    """Floor-free componentwise measure of one hop: |g - A^ p| / (|A^| |p|) over the given rows,
    p being the fp32 matrix the hop read (a seeded input or an oracle hop rounded to fp32, handed to both
    sides).  Entries whose scale is 0 must be exactly 0."""
    n = prev_f32.shape[0]
    rows = np.arange(n, dtype=np.int64) if rows is None else np.asarray(rows, dtype=np.int64)
    y, a = orc.hop_rows_f32(op, eps, rowptr, colidx, prev_f32, rows)
    g = got[rows].astype(np.float64)
    zero = a == 0
    assert (g[zero] == 0).all()
    return float((np.abs(g - y)[~zero] / a[~zero]).max(initial=0.0))


def to_np(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().numpy()


def check_all_hops(op, eps, rowptr_np, colidx_np, X_np, outs, tol=TOL, single_hop=None):
    """Chain parity of every hop (fp64 oracle started from X_0, RMS floor) and the floor-free backward error of
    hop 1, every row.  With `single_hop` - a callable that runs ONE hop of the CUDA path on a given fp32 matrix and
    returns the result as numpy - the backward check is repeated for the later hops on the oracle's own previous
    hop rounded to fp32, so the kernels are also measured floor-free on smoothed inputs.  Every oracle input comes
    from the seeded generators or from the oracle itself, never from the CUDA path."""
    K = len(outs)
    want = orc.propagate(op, eps, rowptr_np, colidx_np, X_np, K)
    worst = 0.0
    for k in range(K):
        g = to_np(outs[k])
        e1 = hop_error(g, want[k])
        assert e1 <= tol, f"hop {k + 1}: relative error {e1:.3e} > {tol}"
        worst = max(worst, e1)
        if k == 0:
            prev, got = np.ascontiguousarray(X_np), g
        elif single_hop is not None:
            prev = np.ascontiguousarray(want[k - 1].astype(np.float32))
            got = single_hop(prev)
        else:
            continue
        e2 = backward_error(op, eps, rowptr_np, colidx_np, prev, got)
        assert e2 <= tol, f"hop {k + 1}: backward error {e2:.3e} > {tol}"
        worst = max(worst, e2)
    return worst


def single_hop_of(B, plan):
    """One hop of the CUDA path through `plan` on a host fp32 matrix, result as numpy."""
    def run(prev_np: np.ndarray) -> np.ndarray:
        out, _ = B.gnnpre_propagate(plan, torch.from_numpy(prev_np).cuda(), 1)
        torch.cuda.synchronize()
        return to_np(out[0])
    return run
