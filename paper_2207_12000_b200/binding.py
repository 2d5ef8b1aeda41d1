"""ctypes binding of libgnnpre.so: one Python function per C entry point, same names.

Only argument marshalling happens here.  Tensors are torch tensors used as plain device (or
host) memory; every step of the computation runs inside the library's CUDA kernels.  If the
library has not been built, importing this module raises: there is no fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Sequence

import torch

from . import build as _build

GNNPRE_OP_GCN_SYM, GNNPRE_OP_SAGE_MEAN, GNNPRE_OP_GIN_SUM = 0, 1, 2
GNNPRE_MEM_DEVICE, GNNPRE_MEM_HOST = 0, 1
GNNPRE_FLAG_LAUNCH_PER_BLOCK, GNNPRE_FLAG_SKIP_VALIDATION, GNNPRE_FLAG_NO_BULK_COPY = 1, 2, 4
GNNPRE_MAX_HOPS = 64
GNNPRE_SCHEDULE_RESIDENT, GNNPRE_SCHEDULE_SLABS, GNNPRE_SCHEDULE_PANELS = 0, 1, 2


class gnnpre_csr_t(ctypes.Structure):
    _fields_ = [("n", ctypes.c_int64), ("nnz", ctypes.c_int64), ("rowptr", ctypes.c_void_p),
                ("colidx", ctypes.c_void_p), ("mem", ctypes.c_int32)]


class gnnpre_plan_opts_t(ctypes.Structure):
    _fields_ = [("op", ctypes.c_int32), ("gin_eps", ctypes.c_float), ("feat_dim", ctypes.c_int64),
                ("budget_bytes", ctypes.c_int64), ("force_blocks", ctypes.c_int32),
                ("force_col_slabs", ctypes.c_int32), ("segment_edges", ctypes.c_int32),
                ("operands_mem", ctypes.c_int32), ("flags", ctypes.c_uint32),
                ("teleport_alpha", ctypes.c_float)]


class gnnpre_plan_info_t(ctypes.Structure):
    _fields_ = [("n", ctypes.c_int64), ("nnz", ctypes.c_int64), ("nnz_tilde", ctypes.c_int64),
                ("feat_dim", ctypes.c_int64), ("op", ctypes.c_int32), ("b", ctypes.c_int32), ("c", ctypes.c_int32),
                ("slab_width", ctypes.c_int64), ("B_S", ctypes.c_int64), ("B_X", ctypes.c_int64),
                ("B_fixed", ctypes.c_int64), ("beta_S", ctypes.c_int64), ("beta_X", ctypes.c_int64),
                ("budget_bytes", ctypes.c_int64), ("device_bytes", ctypes.c_int64), ("host_bytes", ctypes.c_int64),
                ("num_segments", ctypes.c_int64), ("num_row_fixups", ctypes.c_int64),
                ("num_scratch_rows", ctypes.c_int64), ("segment_edges", ctypes.c_int32),
                ("structure_mem", ctypes.c_int32)]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


class gnnpre_block_info_t(ctypes.Structure):
    _fields_ = [("e_lo", ctypes.c_int64), ("e_hi", ctypes.c_int64), ("row_lo", ctypes.c_int32),
                ("row_hi", ctypes.c_int32), ("first_row_partial", ctypes.c_int32),
                ("last_row_partial", ctypes.c_int32)]


class gnnpre_stats_t(ctypes.Structure):
    _fields_ = [("hop_ms", ctypes.c_float * GNNPRE_MAX_HOPS), ("total_ms", ctypes.c_float),
                ("segments_ms", ctypes.c_float), ("h2d_bytes", ctypes.c_int64), ("d2h_bytes", ctypes.c_int64),
                ("kernel_launches", ctypes.c_int64), ("segments_launches", ctypes.c_int64),
                ("startup_ms", ctypes.c_float), ("drain_ms", ctypes.c_float), ("schedule", ctypes.c_int32),
                ("upload_slabs", ctypes.c_int32)]


class GnnpreError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        text = _lib.gnnpre_status_string(status).decode()
        detail = _lib.gnnpre_last_cuda_error().decode()
        super().__init__(f"{where}: {text} ({status})" + (f" [{detail}]" if detail and status == -7 else ""))


def _load() -> ctypes.CDLL:
    path = _build.LIB
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: run paper_2207_12000_b200.build.build() (needs nvcc); "
                          "there is no fallback implementation")
    lib = ctypes.CDLL(path)
    p, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    lib.gnnpre_degrees.argtypes = [ctypes.POINTER(gnnpre_csr_t), p, p]
    lib.gnnpre_build_plan.argtypes = [ctypes.POINTER(gnnpre_csr_t), p, ctypes.POINTER(gnnpre_plan_opts_t),
                                      ctypes.POINTER(p)]
    lib.gnnpre_plan_info.argtypes = [p, ctypes.POINTER(gnnpre_plan_info_t)]
    lib.gnnpre_plan_block.argtypes = [p, i32, ctypes.POINTER(gnnpre_block_info_t)]
    lib.gnnpre_plan_scales.argtypes = [p, p, p, p]
    lib.gnnpre_plan_support.argtypes = [p, p, p]
    lib.gnnpre_propagate.argtypes = [p, p, i64, i32, i32, ctypes.POINTER(p), i64, i32, p,
                                     ctypes.POINTER(gnnpre_stats_t)]
    lib.gnnpre_hop_static.argtypes = [ctypes.POINTER(gnnpre_csr_t), i32, ctypes.c_float, i64, p, i64, p, i64, p]
    lib.gnnpre_lc_selftest_wait_timeout.argtypes = [p, i64, i64, i64, p, i64, i64, p, i64, p, ctypes.c_uint32, p]
    lib.gnnpre_propagate_weighted.argtypes = [p, p, i64, i32, ctypes.POINTER(ctypes.c_void_p), i64,
                                              ctypes.POINTER(ctypes.c_float), p, i64, p]
    lib.gnnpre_lc_first_layer.argtypes = [ctypes.POINTER(ctypes.c_void_p), i32, i64, i64, i64, p, i64, p, i64, i64,
                                          ctypes.c_uint64, i32, p, i64, i64, p, p]
    lib.gnnpre_normalize.argtypes = [p, p, i32, p]
    lib.gnnpre_solve_normalisation_blocks.argtypes = [i64] * 8 + [ctypes.POINTER(i64)]
    lib.gnnpre_selftest_wait_timeout.argtypes = [p, ctypes.c_uint32, p]
    lib.gnnpre_selftest_wait_timeout_async.argtypes = [p, ctypes.c_uint32, p]
    lib.gnnpre_plan_status.argtypes = [p, p]
    lib.gnnpre_gather_ceiling.argtypes = [p, p, i64, p, p]
    lib.gnnpre_describe_panels.argtypes = [i64, i64, i32, p, i32, ctypes.POINTER(i32), ctypes.POINTER(i32)]
    lib.gnnpre_inject_alloc_failure.argtypes = [i64, i64]
    lib.gnnpre_plan_destroy.argtypes = [p]
    lib.gnnpre_plan_destroy.restype = None
    lib.gnnpre_solve_budget.argtypes = [i64] * 8 + [ctypes.POINTER(i64), ctypes.POINTER(i64)]
    lib.gnnpre_status_string.argtypes = [ctypes.c_int]
    lib.gnnpre_status_string.restype = ctypes.c_char_p
    lib.gnnpre_last_cuda_error.restype = ctypes.c_char_p
    return lib


_lib = _load()


def _check(status: int, where: str) -> None:
    if status != 0:
        raise GnnpreError(status, where)


def _mem_of(t: torch.Tensor) -> int:
    return GNNPRE_MEM_DEVICE if t.is_cuda else GNNPRE_MEM_HOST


def _csr(rowptr: torch.Tensor, colidx: torch.Tensor) -> gnnpre_csr_t:
    assert rowptr.dtype == torch.int64 and colidx.dtype == torch.int32
    assert rowptr.is_contiguous() and colidx.is_contiguous() and rowptr.device == colidx.device
    return gnnpre_csr_t(rowptr.numel() - 1, colidx.numel(), rowptr.data_ptr(), colidx.data_ptr(), _mem_of(rowptr))


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream


def gnnpre_degrees(rowptr: torch.Tensor, colidx: torch.Tensor, stream=None) -> torch.Tensor:
    csr = _csr(rowptr, colidx)
    deg = torch.empty(csr.n, dtype=torch.int32, device=rowptr.device)
    _check(_lib.gnnpre_degrees(ctypes.byref(csr), deg.data_ptr(), _stream_ptr(stream)), "gnnpre_degrees")
    return deg


class Plan:
    """Owns a gnnpre_plan_t*; destroyed with the object."""

    def __init__(self, handle: int, keepalive):
        self._h = ctypes.c_void_p(handle)
        self._keepalive = keepalive

    @property
    def handle(self):
        return self._h

    def info(self) -> dict:
        return gnnpre_plan_info(self)

    def close(self):
        if self._h:
            _lib.gnnpre_plan_destroy(self._h)
            self._h = ctypes.c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def gnnpre_build_plan(rowptr: torch.Tensor, colidx: torch.Tensor, op: int, feat_dim: int, *, degrees=None,
                      gin_eps: float = 0.0, budget_bytes: int = 0, force_blocks: int = 0, force_col_slabs: int = 0,
                      segment_edges: int = 0, operands_mem: int = GNNPRE_MEM_DEVICE, flags: int = 0,
                      teleport_alpha: float = 0.0) -> Plan:
    csr = _csr(rowptr, colidx)
    opts = gnnpre_plan_opts_t(op, gin_eps, feat_dim, budget_bytes, force_blocks, force_col_slabs, segment_edges,
                              operands_mem, flags, teleport_alpha)
    if degrees is not None:
        assert degrees.dtype == torch.int32 and degrees.device == rowptr.device and degrees.is_contiguous()
    out = ctypes.c_void_p()
    _check(_lib.gnnpre_build_plan(ctypes.byref(csr), degrees.data_ptr() if degrees is not None else None,
                                  ctypes.byref(opts), ctypes.byref(out)), "gnnpre_build_plan")
    return Plan(out.value, None)


def gnnpre_plan_info(plan: Plan) -> dict:
    info = gnnpre_plan_info_t()
    _check(_lib.gnnpre_plan_info(plan.handle, ctypes.byref(info)), "gnnpre_plan_info")
    return info.as_dict()


def gnnpre_plan_block(plan: Plan, l: int) -> dict:
    blk = gnnpre_block_info_t()
    _check(_lib.gnnpre_plan_block(plan.handle, l, ctypes.byref(blk)), "gnnpre_plan_block")
    return {k: getattr(blk, k) for k, _ in blk._fields_}


def gnnpre_plan_scales(plan: Plan):
    """(degrees int32, rscale fp32, cscale fp32) as host tensors."""
    n = gnnpre_plan_info(plan)["n"]
    deg = torch.empty(n, dtype=torch.int32)
    r = torch.empty(n, dtype=torch.float32)
    c = torch.empty(n, dtype=torch.float32)
    _check(_lib.gnnpre_plan_scales(plan.handle, deg.data_ptr(), r.data_ptr(), c.data_ptr()), "gnnpre_plan_scales")
    return deg, r, c


def gnnpre_plan_support(plan: Plan):
    """(rowptr int64 [n+1], colidx int32 [nnz_tilde]) of the operator's support, as host tensors."""
    info = gnnpre_plan_info(plan)
    rp = torch.empty(info["n"] + 1, dtype=torch.int64)
    ci = torch.empty(info["nnz_tilde"], dtype=torch.int32)
    _check(_lib.gnnpre_plan_support(plan.handle, rp.data_ptr(), ci.data_ptr()), "gnnpre_plan_support")
    return rp, ci


def gnnpre_propagate(plan: Plan, X: torch.Tensor, K: int, out: Sequence[torch.Tensor] | None = None, *,
                     stream=None, want_stats: bool = False):
    """out[k-1] = A^ applied k times to X.  X and out are fp32 row-major views (stride(1) == 1) on the
    device, or host tensors (preferably pinned) for the streamed path.  Returns (out, stats-or-None)."""
    assert X.dtype == torch.float32 and X.dim() == 2 and X.stride(1) == 1
    n, F = X.shape
    if out is None:
        Fp = (F + 3) // 4 * 4  # the library works on whole groups of 4 columns
        if X.is_cuda:
            out = [torch.empty((n, Fp), dtype=torch.float32, device=X.device)[:, :F] for _ in range(K)]
        else:
            out = [torch.empty((n, Fp), dtype=torch.float32, pin_memory=True)[:, :F] for _ in range(K)]
    assert len(out) == K
    ldo = out[0].stride(0) if K > 0 else F
    for o in out:
        assert o.dtype == torch.float32 and o.shape == (n, F) and o.stride(1) == 1 and o.stride(0) == ldo
        assert o.is_cuda == out[0].is_cuda
    ptrs = (ctypes.c_void_p * max(K, 1))(*[o.data_ptr() for o in out])
    stats = gnnpre_stats_t() if want_stats else None
    _check(_lib.gnnpre_propagate(plan.handle, X.data_ptr(), X.stride(0), _mem_of(X), K, ptrs, ldo,
                                 _mem_of(out[0]) if K > 0 else _mem_of(X),
                                 _stream_ptr(stream), ctypes.byref(stats) if want_stats else None),
           "gnnpre_propagate")
    return list(out), stats


def gnnpre_hop_static(rowptr: torch.Tensor, colidx: torch.Tensor, op: int, X: torch.Tensor, out: torch.Tensor, *,
                      gin_eps: float = 0.0, stream=None) -> torch.Tensor:
    """out = A^ X in one call that allocates nothing (the caller supplies `out`); device tensors only."""
    assert X.dtype == torch.float32 and X.dim() == 2 and X.stride(1) == 1 and X.is_cuda
    assert out.dtype == torch.float32 and out.shape == X.shape and out.stride(1) == 1 and out.is_cuda
    csr = _csr(rowptr, colidx)
    _check(_lib.gnnpre_hop_static(ctypes.byref(csr), op, gin_eps, X.shape[1], X.data_ptr(), X.stride(0),
                                  out.data_ptr(), out.stride(0), _stream_ptr(stream)), "gnnpre_hop_static")
    return out


def gnnpre_lc_selftest_wait_timeout(hop: torch.Tensor, Wt: torch.Tensor, polls: int = 200, stream=None) -> int:
    """Status of a first-layer launch whose waits are made to run out (expected: -8, GNNPRE_ERR_TIMEOUT)."""
    n, F = hop.shape
    H = Wt.shape[0]
    Y = torch.empty((min(n, 128), H), dtype=torch.float32, device=hop.device)
    flag = torch.zeros(1, dtype=torch.int32, device=hop.device)
    return int(_lib.gnnpre_lc_selftest_wait_timeout(hop.data_ptr(), n, F, hop.stride(0), Wt.data_ptr(), H, Wt.stride(0),
                                                    Y.data_ptr(), Y.stride(0), flag.data_ptr(), polls, _stream_ptr(stream)))


def gnnpre_propagate_weighted(plan: Plan, X: torch.Tensor, gamma, *, out=None, Z: torch.Tensor | None = None,
                              keep_hops: bool = True, stream=None):
    """K = len(gamma) - 1 hops and Z = gamma[0] X + sum_k gamma[k] X_k, all on the device.
    Returns (hops, Z); with keep_hops=False two buffers alternate and hops holds only the last two."""
    K = len(gamma) - 1
    assert X.is_cuda and X.dtype == torch.float32 and X.dim() == 2 and X.stride(1) == 1
    n, F = X.shape
    Fp = (F + 3) // 4 * 4
    if out is None:
        nbuf = K if keep_hops else min(K, 2)
        bufs = [torch.empty((n, Fp), dtype=torch.float32, device=X.device)[:, :F] for _ in range(nbuf)]
        out = [bufs[k % nbuf] for k in range(K)]
    if Z is None:
        Z = torch.empty((n, Fp), dtype=torch.float32, device=X.device)[:, :F]
    for o in list(out) + [Z]:
        assert o.is_cuda and o.dtype == torch.float32 and o.shape == (n, F) and o.stride(1) == 1
    assert all(o.stride(0) == out[0].stride(0) for o in out)
    ptrs = (ctypes.c_void_p * K)(*[o.data_ptr() for o in out])
    g = (ctypes.c_float * (K + 1))(*[float(v) for v in gamma])
    _check(_lib.gnnpre_propagate_weighted(plan.handle, X.data_ptr(), X.stride(0), K, ptrs, out[0].stride(0), g,
                                          Z.data_ptr(), Z.stride(0), _stream_ptr(stream)), "gnnpre_propagate_weighted")
    return list(out), Z


GNNPRE_LC_TF32, GNNPRE_LC_TF32X3 = 0, 1


def gnnpre_lc_first_layer(hops, batch, Wt: torch.Tensor, *, relu_mask: int = 0, precision: int = GNNPRE_LC_TF32,
                          out: torch.Tensor | None = None,
                          concat: bool = False, check: bool = True, stream=None) -> torch.Tensor:
    """act(hops[k][batch] @ Wt.T) for every hop on the tensor cores (Eq. 9's first dense stage).

    hops: list of device fp32 [n, F] matrices with one common row stride; batch: device int32 row indices
    or None (all rows); Wt: device fp32 [H, F].  Returns [K, B, H], or [B, K*H] with concat=True.
    precision: GNNPRE_LC_TF32 (tf32 operands) or GNNPRE_LC_TF32X3 (split operands, fp32-like accuracy).
    With check=True the call synchronises and raises if a device-side wait ran out."""
    K = len(hops)
    n, F = hops[0].shape
    for h in hops:
        assert h.is_cuda and h.dtype == torch.float32 and h.shape == (n, F) and h.stride(1) == 1
        assert h.stride(0) == hops[0].stride(0)
    assert Wt.is_cuda and Wt.dtype == torch.float32 and Wt.dim() == 2 and Wt.shape[1] == F and Wt.stride(1) == 1
    H = Wt.shape[0]
    if batch is None:
        B, bptr = n, None
    else:
        if batch.dtype == torch.int64:  # the default index type of the host framework; the library takes int32
            batch = batch.to(torch.int32)
        assert batch.is_cuda and batch.dtype == torch.int32 and batch.dim() == 1 and batch.is_contiguous()
        B, bptr = batch.numel(), batch.data_ptr()
    if out is None:
        out = torch.empty((B, K * H) if concat else (K, B, H), dtype=torch.float32, device=Wt.device)
    if concat:
        assert out.shape == (B, K * H) and out.stride(1) == 1
        ldy, hop_stride = out.stride(0), H
    else:
        assert out.shape == (K, B, H) and out.stride(2) == 1
        ldy, hop_stride = (out.stride(1), out.stride(0)) if B > 0 else (H, 0)
    flag = torch.zeros(1, dtype=torch.int32, device=Wt.device) if check else None
    ptrs = (ctypes.c_void_p * K)(*[h.data_ptr() for h in hops])
    _check(_lib.gnnpre_lc_first_layer(ptrs, K, n, F, hops[0].stride(0), bptr, B, Wt.data_ptr(), H, Wt.stride(0),
                                      relu_mask, precision, out.data_ptr(), ldy, hop_stride,
                                      flag.data_ptr() if check else None, _stream_ptr(stream)), "gnnpre_lc_first_layer")
    if check and int(flag.item()) != 0:
        raise GnnpreError(-8, "gnnpre_lc_first_layer")
    return out


def gnnpre_normalize(plan: Plan, out: torch.Tensor | None = None, *, host: bool = False, stream=None) -> torch.Tensor:
    """fp32 value of every edge of the support (order of gnnpre_plan_support), on the device or in host memory."""
    m = gnnpre_plan_info(plan)["nnz_tilde"]
    if out is None:
        out = torch.empty(m, dtype=torch.float32, pin_memory=True) if host else torch.empty(
            m, dtype=torch.float32, device="cuda")
    assert out.dtype == torch.float32 and out.numel() == m and out.is_contiguous()
    _check(_lib.gnnpre_normalize(plan.handle, out.data_ptr(), _mem_of(out), _stream_ptr(stream)), "gnnpre_normalize")
    return out


def gnnpre_solve_normalisation_blocks(B_A, B_S, B_D, alpha_A, alpha_S, alpha_D, B_GPU, max_a):
    a = ctypes.c_int64()
    rc = _lib.gnnpre_solve_normalisation_blocks(B_A, B_S, B_D, alpha_A, alpha_S, alpha_D, B_GPU, max_a, ctypes.byref(a))
    if rc == -6:
        return -1
    _check(rc, "gnnpre_solve_normalisation_blocks")
    return a.value


def gnnpre_selftest_wait_timeout(plan: Plan, polls: int = 200, stream=None) -> int:
    """Status of a device wait that is made to run out (expected: -8, GNNPRE_ERR_TIMEOUT)."""
    return int(_lib.gnnpre_selftest_wait_timeout(plan.handle, polls, _stream_ptr(stream)))


def gnnpre_selftest_wait_timeout_async(plan: Plan, polls: int = 200, stream=None) -> None:
    """Enqueues the wait that runs out; gnnpre_plan_status then reports it once."""
    _check(_lib.gnnpre_selftest_wait_timeout_async(plan.handle, polls, _stream_ptr(stream)),
           "gnnpre_selftest_wait_timeout_async")


def gnnpre_plan_status(plan: Plan, stream=None) -> int:
    """Synchronises `stream` and returns 0, or -8 (GNNPRE_ERR_TIMEOUT) once if a kernel of the plan gave up a wait."""
    return int(_lib.gnnpre_plan_status(plan.handle, _stream_ptr(stream)))


def gnnpre_gather_ceiling(plan: Plan, X: torch.Tensor, sink: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """Enqueues the fetches of one hop (rows summed plainly, nothing stored but one float per segment): the
    yardstick the segment kernels are measured against when X fits the L2.  Returns the sink buffer."""
    assert X.is_cuda and X.dtype == torch.float32 and X.dim() == 2 and X.stride(1) == 1
    nseg = gnnpre_plan_info(plan)["num_segments"]
    if sink is None:
        sink = torch.empty(max(nseg, 1), dtype=torch.float32, device=X.device)
    assert sink.is_cuda and sink.dtype == torch.float32 and sink.numel() >= nseg and sink.is_contiguous()
    _check(_lib.gnnpre_gather_ceiling(plan.handle, X.data_ptr(), X.stride(0), sink.data_ptr(), _stream_ptr(stream)),
           "gnnpre_gather_ceiling")
    return sink


def gnnpre_describe_panels(feat_dim: int, slab_width: int, K: int):
    """(number of upload slabs, list of jobs) of the narrow-first panel schedule; a job is a dict with keys
    k, lo, hi, upload, drain_lo, drain_hi.  Host only."""
    ns, nj = ctypes.c_int32(), ctypes.c_int32()
    _check(_lib.gnnpre_describe_panels(feat_dim, slab_width, K, None, 0, ctypes.byref(ns), ctypes.byref(nj)),
           "gnnpre_describe_panels")
    buf = (ctypes.c_int32 * (6 * max(nj.value, 1)))()
    _check(_lib.gnnpre_describe_panels(feat_dim, slab_width, K, buf, nj.value, ctypes.byref(ns), ctypes.byref(nj)),
           "gnnpre_describe_panels")
    keys = ("k", "lo", "hi", "upload", "drain_lo", "drain_hi")
    return ns.value, [dict(zip(keys, buf[6 * i:6 * i + 6])) for i in range(nj.value)]


def gnnpre_inject_alloc_failure(device_countdown: int = -1, host_countdown: int = -1) -> None:
    """Test hook: the library's (countdown + 1)-th next allocation of that kind is reported as failed; -1 disarms."""
    _check(_lib.gnnpre_inject_alloc_failure(device_countdown, host_countdown), "gnnpre_inject_alloc_failure")


def gnnpre_solve_budget(B_S, B_X, B_fixed, beta_S, beta_X, B_GPU, max_b, max_c):
    b, c = ctypes.c_int64(), ctypes.c_int64()
    rc = _lib.gnnpre_solve_budget(B_S, B_X, B_fixed, beta_S, beta_X, B_GPU, max_b, max_c, ctypes.byref(b),
                                  ctypes.byref(c))
    if rc == -6:
        return None
    _check(rc, "gnnpre_solve_budget")
    return b.value, c.value


def gnnpre_status_string(status: int) -> str:
    return _lib.gnnpre_status_string(status).decode()


def exported_symbols():
    return ["gnnpre_degrees", "gnnpre_build_plan", "gnnpre_plan_info", "gnnpre_plan_block", "gnnpre_plan_scales",
            "gnnpre_plan_support", "gnnpre_propagate", "gnnpre_propagate_weighted", "gnnpre_hop_static", "gnnpre_lc_first_layer", "gnnpre_lc_selftest_wait_timeout", "gnnpre_normalize",
            "gnnpre_solve_normalisation_blocks", "gnnpre_selftest_wait_timeout", "gnnpre_selftest_wait_timeout_async",
            "gnnpre_plan_status", "gnnpre_inject_alloc_failure", "gnnpre_gather_ceiling", "gnnpre_describe_panels", "gnnpre_plan_destroy", "gnnpre_solve_budget",
            "gnnpre_status_string", "gnnpre_last_cuda_error"]
