"""gnnpre_lc_first_layer (tensor-core gather + product of Eq. 9's first dense stage) against the oracle.

Two kinds of comparison:
  * integer-valued inputs small enough that tf32 holds every operand and fp32 every partial sum
    exactly: the kernel must then equal the fp64 oracle bit for bit, which checks the gather, the
    operand layouts, the accumulator read-out and the output addressing with no tolerance at all;
  * normal inputs: |Y - oracle| <= (2^-9 + F 2^-23) * sum_f |x||w|.  The tensor core reads fp32
    operands as tf32 (relative error below 2^-10 each, so below 2^-9 + 2^-20 per product) and adds in
    fp32 (at most F roundings of 2^-24 each on partial sums bounded by sum |x||w|, doubled for slack).
    With split operands (GNNPRE_LC_TF32X3) the first term drops to 2^-20.
"""
import numpy as np
import pytest
import torch

import gnnpre_inputs as gi
import oracle as orc
from parity_util import to_np

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2207_12000_b200 import binding
    return binding


def integer_matrix(rows, cols, seed, lo, hi):
    rng = np.random.default_rng(seed)
    return rng.integers(lo, hi + 1, size=(rows, cols)).astype(np.float32)


def padded_cuda(M: np.ndarray, pad: int, fill=float("nan")):
    """Device copy of M inside a wider buffer whose extra columns hold `fill`."""
    r, c = M.shape
    ld = (c + pad + 3) // 4 * 4
    buf = torch.full((r, ld), fill, dtype=torch.float32, device="cuda")
    buf[:, :c] = torch.from_numpy(M).cuda()
    return buf[:, :c]


SHAPES = [
    # n,    F,   H,   batch size (None = every row in order), hops
    (1000, 32, 16, 128, 1),     # one tile, one K-chunk
    (1000, 64, 32, 128, 2),     # two K-chunks
    (5000, 100, 256, 4096, 3),  # the paper's settings: 4096-row batches, hidden 256, ragged K-chunk
    (3000, 128, 256, 1000, 2),  # ragged last tile
    (777, 13, 48, 300, 2),      # fewer features than one chunk
    (2000, 602, 64, 517, 1),    # Reddit's width: 19 chunks, pad columns full of NaN
    (517, 40, 80, None, 2),     # no batch: every row
    (1500, 200, 256, 700, 2),   # a weight too large to stay in shared memory at full hidden width: streamed beside the rows
    (900, 300, 192, 333, 1),    # hidden = 192: two column halves of 96 in the split-operand mode
    (400, 8, 16, 1, 1),         # a single row
    (50000, 100, 256, 50000, 3),  # more tiles than SMs: persistent loop, both accumulator buffers, many phases
]


PRECISIONS = (0, 1)  # GNNPRE_LC_TF32, GNNPRE_LC_TF32X3


@pytest.mark.parametrize("precision", PRECISIONS)
@pytest.mark.parametrize("n,F,H,bs,K", SHAPES)
def test_exact_on_small_integers(B, n, F, H, bs, K, precision):
    hops_np = [integer_matrix(n, F, 100 + k, -7, 7) for k in range(K)]
    Wt_np = integer_matrix(H, F, 7, -5, 5)
    rng = np.random.default_rng(n + F)
    batch_np = None if bs is None else rng.integers(0, n, size=bs)
    hops = [padded_cuda(h, 2) for h in hops_np]
    Wt = padded_cuda(Wt_np, 5)
    batch = None if bs is None else torch.from_numpy(batch_np.astype(np.int32)).cuda()
    relu_mask = 0b101
    Y = B.gnnpre_lc_first_layer(hops, batch, Wt, relu_mask=relu_mask, precision=precision)
    assert Y.shape == (K, n if bs is None else bs, H)
    for k in range(K):
        want = orc.lc_first_layer(hops_np[k], batch_np, Wt_np, relu=bool((relu_mask >> k) & 1))
        got = to_np(Y[k]).astype(np.float64)
        assert np.array_equal(got, want), f"hop {k}: {np.argwhere(got != want)[:5]}"


@pytest.mark.parametrize("precision", PRECISIONS)
@pytest.mark.parametrize("n,F,H,bs,K", SHAPES[2:9])
def test_normal_inputs_within_the_bound_of_the_precision(B, n, F, H, bs, K, precision):
    hops_np = [gi.normal_matrix(n, F, 200 + k).numpy() for k in range(K)]
    Wt_np = gi.normal_matrix(H, F, 9).numpy() / np.float32(np.sqrt(F))
    rng = np.random.default_rng(n + H)
    batch_np = None if bs is None else rng.permutation(n)[:bs] if bs <= n else rng.integers(0, n, size=bs)
    hops = [padded_cuda(h, 2) for h in hops_np]
    Wt = padded_cuda(Wt_np, 1)
    batch = None if bs is None else torch.from_numpy(batch_np.astype(np.int32)).cuda()
    Y = B.gnnpre_lc_first_layer(hops, batch, Wt, relu_mask=0b10, precision=precision)
    for k in range(K):
        relu = k == 1
        want, scale = orc.lc_first_layer(hops_np[k], batch_np, Wt_np, relu=relu, want_abs=True)
        got = to_np(Y[k]).astype(np.float64)
        # split operands: the dropped low x low term and the cut of each low part to tf32 cost 3 * 2^-22 < 2^-20
        bound = ((2.0 ** -9 if precision == 0 else 2.0 ** -20) + F * 2.0 ** -23) * scale
        assert (np.abs(got - want) <= bound).all(), float((np.abs(got - want) / scale).max())
        # the product is really computed: the error is far below the values themselves
        assert np.abs(got - want).max() < 0.01 * np.abs(want).max()


def test_concatenated_layout_strided_output_and_untouched_padding(B):
    n, F, H, bs, K = 1500, 100, 32, 700, 3
    hops_np = [integer_matrix(n, F, 300 + k, -6, 6) for k in range(K)]
    Wt_np = integer_matrix(H, F, 11, -4, 4)
    batch_np = np.random.default_rng(3).integers(0, n, size=bs)
    hops = [padded_cuda(h, 0) for h in hops_np]
    batch = torch.from_numpy(batch_np.astype(np.int32)).cuda()
    buf = torch.full((bs + 3, K * H + 8), -9.0, device="cuda")
    out = buf[:bs, :K * H]
    got = B.gnnpre_lc_first_layer(hops, batch, torch.from_numpy(Wt_np).cuda(), out=out, concat=True)
    assert got.data_ptr() == out.data_ptr()
    want = np.concatenate([orc.lc_first_layer(h, batch_np, Wt_np, relu=False) for h in hops_np], axis=1)
    assert np.array_equal(to_np(out).astype(np.float64), want)
    assert bool((buf[:, K * H:] == -9.0).all()) and bool((buf[bs:] == -9.0).all())


def test_more_hops_than_one_launch_carries_and_an_empty_batch(B):
    n, F, H, bs, K = 300, 24, 16, 130, 11  # eleven hop matrices: two launches (8 + 3)
    hops_np = [integer_matrix(n, F, 400 + k, -3, 3) for k in range(K)]
    Wt_np = integer_matrix(H, F, 13, -3, 3)
    batch_np = np.random.default_rng(4).integers(0, n, size=bs)
    hops = [padded_cuda(h, 0) for h in hops_np]
    batch = torch.from_numpy(batch_np.astype(np.int32)).cuda()
    mask = 0b10101010101
    Y = B.gnnpre_lc_first_layer(hops, batch, torch.from_numpy(Wt_np).cuda(), relu_mask=mask)
    for k in range(K):
        want = orc.lc_first_layer(hops_np[k], batch_np, Wt_np, relu=bool((mask >> k) & 1))
        assert np.array_equal(to_np(Y[k]).astype(np.float64), want), k
    empty = B.gnnpre_lc_first_layer(hops[:2], torch.zeros(0, dtype=torch.int32, device="cuda"),
                                    torch.from_numpy(Wt_np).cuda())
    assert empty.shape == (2, 0, H)


def test_propagate_then_first_layer_end_to_end(B):
    """The two stages chained on the device, against the fp64 oracle chained on the CPU."""
    g = gi.rmat(20000, 300000, 5, directed_candidates=True)
    F, H, K, bs = 100, 256, 3, 4096
    X = gi.normal_matrix(g.n, F, 6)
    Wt_np = gi.normal_matrix(H, F, 8).numpy() / np.float32(np.sqrt(F))
    plan = B.gnnpre_build_plan(g.rowptr.cuda(), g.colidx.cuda(), 0, F)
    outs, _ = B.gnnpre_propagate(plan, X.cuda(), K)
    batch_np = np.random.default_rng(9).permutation(g.n)[:bs]
    Y = B.gnnpre_lc_first_layer(outs, torch.from_numpy(batch_np.astype(np.int32)).cuda(),
                                torch.from_numpy(Wt_np).cuda(), relu_mask=0b110)
    hops64 = orc.propagate(0, 0.0, g.rowptr.numpy(), g.colidx.numpy(), X.numpy(), K)
    for k in range(K):
        hop32 = hops64[k].astype(np.float32)
        want, scale = orc.lc_first_layer(hop32, batch_np, Wt_np, relu=k >= 1, want_abs=True)
        # 2^-9 for tf32, 2e-5 for the hop itself (parity tolerance of the aggregation plus its fp32 rounding)
        bound = (2.0 ** -9 + F * 2.0 ** -23 + 2e-5) * scale + 1e-30
        assert (np.abs(to_np(Y[k]).astype(np.float64) - want) <= bound).all()
    plan.close()


def test_bad_arguments_are_refused(B):
    h = torch.zeros((64, 32), device="cuda")
    W = torch.zeros((16, 32), device="cuda")
    for bad_W in (torch.zeros((8, 32), device="cuda"), torch.zeros((24, 32), device="cuda"),
                  torch.zeros((272, 32), device="cuda")):  # hidden < 16, not a multiple of 16, > 256
        with pytest.raises(B.GnnpreError) as ei:
            B.gnnpre_lc_first_layer([h], None, bad_W)
        assert ei.value.status == -1
    with pytest.raises(B.GnnpreError) as ei:  # split operands, two column halves: hidden must be a multiple of 64
        B.gnnpre_lc_first_layer([h], None, torch.zeros((160, 32), device="cuda"), precision=1)
    assert ei.value.status == -1
    with pytest.raises(B.GnnpreError) as ei:  # leading dimension that is not a multiple of 4
        B.gnnpre_lc_first_layer([torch.zeros((64, 30), device="cuda")], None, torch.zeros((16, 30), device="cuda"))
    assert ei.value.status == -3
    with pytest.raises(B.GnnpreError) as ei:  # misaligned output
        buf = torch.zeros(64 * 16 + 4, device="cuda")
        B.gnnpre_lc_first_layer([h], None, W, out=buf[1:1 + 64 * 16].view(1, 64, 16))
    assert ei.value.status == -3


def test_split_operands_are_far_more_accurate_than_plain_tf32(B):
    """Same inputs, both precisions: the worst error relative to sum |x||w| falls by more than two orders of
    magnitude, into the accuracy class of an fp32 dot product of this length (its bound is F 2^-24 = 6e-6)."""
    n, F, H, bs = 6000, 100, 256, 4096
    hop_np = gi.normal_matrix(n, F, 31).numpy()
    Wt_np = gi.normal_matrix(H, F, 32).numpy() / np.float32(np.sqrt(F))
    batch_np = np.random.default_rng(6).permutation(n)[:bs]
    want, scale = orc.lc_first_layer(hop_np, batch_np, Wt_np, relu=False, want_abs=True)
    errs = []
    for precision in PRECISIONS:
        Y = B.gnnpre_lc_first_layer([torch.from_numpy(hop_np).cuda()], torch.from_numpy(batch_np.astype(np.int32)).cuda(),
                                    torch.from_numpy(Wt_np).cuda(), precision=precision)
        errs.append(float((np.abs(to_np(Y[0]).astype(np.float64) - want) / scale).max()))
    assert errs[1] < 4e-6 and errs[1] * 100 < errs[0], errs


def test_waits_that_run_out_are_reported_and_the_device_stays_usable(B):
    """Failure detection without a fault: the producers announce nothing, every bounded wait of the kernel gives
    up, the call reports TIMEOUT (-8); tensor memory was freed, so the next call runs and is exact."""
    n, F, H = 500, 100, 256
    hop_np = integer_matrix(n, F, 1, -4, 4)
    Wt_np = integer_matrix(H, F, 2, -4, 4)
    hop, Wt = torch.from_numpy(hop_np).cuda(), torch.from_numpy(Wt_np).cuda()
    for _ in range(2):
        assert B.gnnpre_lc_selftest_wait_timeout(hop, Wt, polls=200) == -8
        Y = B.gnnpre_lc_first_layer([hop], None, Wt)
        assert np.array_equal(to_np(Y[0]).astype(np.float64), orc.lc_first_layer(hop_np, None, Wt_np, relu=False))
