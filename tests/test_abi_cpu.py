"""Host-side checks that need no GPU: the library loads, exports what include/gnnpre.h declares,
rejects bad arguments before touching a device, and its Eq. 12 search agrees with the oracle's
exhaustive one."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle as orc
from paper_2207_12000_b200 import build as libbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    libbuild.build()
    from paper_2207_12000_b200 import binding as b
    return b


def declared_functions():
    text = open(os.path.join(ROOT, "include", "gnnpre.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gnnpre_[a-z_]+)\s*\(", text)))


def test_header_symbols_are_exported(binding):
    names = declared_functions()
    assert "gnnpre_build_plan" in names and "gnnpre_propagate" in names
    lib = ctypes.CDLL(libbuild.LIB)
    for name in names:
        assert hasattr(lib, name), f"{name} declared in include/gnnpre.h but not exported"
    assert sorted(binding.exported_symbols()) == names


def test_struct_layouts_match_header(binding):
    # sizes implied by the header's field lists under the C ABI (natural alignment)
    assert ctypes.sizeof(binding.gnnpre_csr_t) == 40
    assert ctypes.sizeof(binding.gnnpre_plan_opts_t) == 48
    assert ctypes.sizeof(binding.gnnpre_block_info_t) == 32
    assert ctypes.sizeof(binding.gnnpre_plan_info_t) == 152
    assert ctypes.sizeof(binding.gnnpre_stats_t) == 64 * 4 + 8 + 32 + 16


def test_status_strings(binding):
    assert binding.gnnpre_status_string(0) == "ok"
    for s in range(-11, 0):
        assert binding.gnnpre_status_string(s) != "unknown status"
    assert binding.gnnpre_status_string(-99) == "unknown status"


def test_budget_solver_matches_oracle_exhaustive_search(binding):
    rng = np.random.default_rng(12)
    for _ in range(400):
        B_S, B_X = int(rng.integers(0, 6000)), int(rng.integers(1, 6000))
        B_fixed = int(rng.integers(0, 80))
        beta_S, beta_X = int(rng.integers(1, 4)), int(rng.integers(1, 5))
        B_GPU = int(rng.integers(1, 5000))
        want = orc.solve_budget(B_S, B_X, B_fixed, beta_S, beta_X, B_GPU, 48, 16)
        got = binding.gnnpre_solve_budget(B_S, B_X, B_fixed, beta_S, beta_X, B_GPU, 48, 16)
        assert got == want, (B_S, B_X, B_fixed, beta_S, beta_X, B_GPU)


def test_paper_sizes_through_library_solver(binding, golden_dir):
    v = dict(l.split() for l in open(os.path.join(golden_dir, "paper_sizes.txt")) if not l.startswith("#"))
    GB = 10 ** 9
    B_S, B_X, B_GPU = int(v["normalized_adjacency_GB"]) * GB, int(v["feature_matrix_GB"]) * GB, int(v["gpu_memory_GB"]) * GB
    got = binding.gnnpre_solve_budget(B_S, B_X, 0, 2, 2, B_GPU, 64, 32)
    assert got == orc.solve_budget(B_S, B_X, 0, 2, 2, B_GPU, 64, 32)
    assert got[0] * got[1] <= int(v["b"]) * int(v["c"])


def test_null_and_bad_arguments_fail_without_a_device(binding):
    lib = binding._lib
    assert lib.gnnpre_build_plan(None, None, None, None) == -1
    assert lib.gnnpre_plan_info(None, None) == -1
    assert lib.gnnpre_propagate(None, None, 0, 0, 1, None, 0, 0, None, None) == -1
    assert lib.gnnpre_degrees(None, None, None) == -1
    lib.gnnpre_plan_destroy(None)  # no-op


def test_normalisation_block_count_matches_oracle(binding):
    rng = np.random.default_rng(3)
    for _ in range(300):
        B_A, B_S, B_D = (int(rng.integers(0, 5000)) for _ in range(3))
        al = [int(rng.integers(0, 4)) for _ in range(3)]
        B_GPU = int(rng.integers(1, 6000))
        want = orc.solve_normalisation_blocks(B_A, B_S, B_D, al[0], al[1], al[2], B_GPU, 64)
        got = binding.gnnpre_solve_normalisation_blocks(B_A, B_S, B_D, al[0], al[1], al[2], B_GPU, 64)
        assert got == want, (B_A, B_S, B_D, al, B_GPU)


def test_panel_schedule_invariants(binding):
    """The narrow-first panel schedule of the streamed path, checked as data (no device): the upload slabs tile the
    columns in order, start 32 wide and never exceed the plan's slab width; walking the jobs in launch order, a hop-1
    job runs on exactly one upload slab that has been requested, a later hop only reads columns the previous hop has
    already computed, no job is wider than the slab width (the scratch rows' width), every (hop, column) is computed
    exactly once and drained exactly once, and nothing is drained before it has been computed."""
    for F in (128, 160, 256, 512, 1024, 96, 64):
        for cap in (64, 96, 128, 512):
            for K in (1, 2, 3, 5):
                if cap < 64:
                    continue
                ns, jobs = binding.gnnpre_describe_panels(F, cap, K)
                slabs = []
                for j in jobs:
                    if j["upload"] >= 0:
                        assert j["k"] == 1 and j["upload"] == len(slabs)  # uploads are consumed in order
                        slabs.append((j["lo"], j["hi"]))
                assert len(slabs) == ns
                assert slabs[0][0] == 0 and slabs[-1][1] == F
                assert all(a[1] == b[0] for a, b in zip(slabs, slabs[1:]))
                assert slabs[0][1] - slabs[0][0] == min(32, F)
                assert all(0 < hi - lo <= min(cap, F) and lo % 32 == 0 for lo, hi in slabs)
                computed = np.zeros((K + 1, F), dtype=np.int32)
                computed[0, :] = 1
                drained = np.zeros((K + 1, F), dtype=np.int32)
                for j in jobs:
                    k, lo, hi = j["k"], j["lo"], j["hi"]
                    assert 1 <= k <= K and 0 <= lo < hi <= F and hi - lo <= min(cap, F)
                    assert (computed[k - 1, lo:hi] == 1).all(), (F, cap, K, j)  # its input exists
                    computed[k, lo:hi] += 1
                    dl, dh = j["drain_lo"], j["drain_hi"]
                    if dh > dl:
                        assert (computed[k, dl:dh] == 1).all(), (F, cap, K, j)  # only finished columns leave
                        assert dl % 32 == 0  # host pieces start on 128-byte boundaries
                        drained[k, dl:dh] += 1
                assert (computed[1:] == 1).all() and (drained[1:] == 1).all(), (F, cap, K)
    assert binding._lib.gnnpre_describe_panels(100, 64, 2, None, 0, None, None) == -1
