"""Measured coefficients of the memory-budget model (Eq. 12).

The paper leaves the coefficients of its budget constraints to be found by watching memory use on small
graphs.  This module does that for the library's streamed setting (graph and operands in host memory): it
builds plans with forced block counts (b, c) on a few small graphs, runs one streamed call each so that every
buffer the library allocates on first use exists, reads the device bytes the plan then holds, and fits

    device_bytes  ~=  beta_S * B_S / b  +  beta_X * B_X / c  +  beta_fixed * B_fixed

by least squares (B_S, B_X, B_fixed as gnnpre_plan_info reports them).  The library itself keeps the fixed
coefficients beta_S = 2, beta_X = 4 (two edge-block staging buffers, four slab buffers) and charges B_fixed
once; the fit shows how far reality is from that model.  Only marshalling and a linear solve happen here; all
device work is the library's.
"""
from __future__ import annotations

import numpy as np
import torch


def measure_budget_coefficients(B, graphs, op: int, feat_dims=(32, 64), shapes=((2, 2), (4, 2), (2, 4), (8, 4), (3, 1))):
    """`graphs`: CSRGraph objects (host tensors).  Returns a dict with the fitted coefficients, the library's
    fixed ones, and the worst relative gap between the fixed model and the measured bytes."""
    rows, rhs, model = [], [], []
    for g in graphs:
        rp, ci = g.rowptr.pin_memory(), g.colidx.pin_memory()
        for F in feat_dims:
            X = torch.zeros((g.n, F), dtype=torch.float32).pin_memory()
            outs = [torch.empty((g.n, F), dtype=torch.float32).pin_memory() for _ in range(2)]
            for b, c in shapes:
                if 4 * c > F:
                    continue
                plan = B.gnnpre_build_plan(rp, ci, op, F, force_blocks=b, force_col_slabs=c,
                                           operands_mem=B.GNNPRE_MEM_HOST)
                B.gnnpre_propagate(plan, X, 2, outs)
                info = plan.info()
                plan.close()
                rows.append([info["B_S"] / b, info["B_X"] / c, info["B_fixed"]])
                rhs.append(info["device_bytes"])
                model.append(info["beta_S"] * info["B_S"] / b + info["beta_X"] * info["B_X"] / c + info["B_fixed"])
    A = np.asarray(rows, dtype=np.float64)
    y = np.asarray(rhs, dtype=np.float64)
    coef, *_ = np.linalg.lstsq(A, y, rcond=None)
    fitted = A @ coef
    return {"beta_S": float(coef[0]), "beta_X": float(coef[1]), "beta_fixed": float(coef[2]),
            "fixed": {"beta_S": 2, "beta_X": 4, "beta_fixed": 1},
            "samples": len(rhs),
            "worst_fit_residual": float(np.max(np.abs(fitted - y) / y)),
            "worst_fixed_model_gap": float(np.max(np.abs(np.asarray(model) - y) / y)),
            "fixed_model_never_below_measured_by_more_than": float(np.max((y - np.asarray(model)) / y))}
