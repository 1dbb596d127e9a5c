"""The bounds-checked build of the library (-DTHEMIS_CHECK_BOUNDS), which stands in for a
memory sanitizer: every index a solver kernel computes into shared or global memory is
range-checked, a violation is recorded (never trapped) and read back through
``themis_bounds_check_report``.  The shapes at the edges of the supported ranges run
through it in every kernel mode: no violation may be reported and the results must equal
the oracle's."""
import numpy as np
import pytest

from paper_2407_14843_b200 import workloads as W
from tests.test_gpu_parity import SHAPES, _assert_results_equal

pytestmark = pytest.mark.gpu

KERNEL_IDS = ["packed16", "wide32", "pruned", "sparse", "sparse_block", "packed16_block"]


@pytest.fixture(scope="module")
def S():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    from paper_2407_14843_b200 import build
    build.build_library()
    check_lib = build.build_library(check_bounds=True)
    from paper_2407_14843_b200 import solver
    solver.use_library(check_lib)
    yield solver
    solver.use_library()                      # back to the normal library for the tests that follow


def _checked_solve(S, wl, kernel_id):
    import torch
    kernel = (kernel_id + 1) << 8
    out, ws = S.solve(wl, kernel=kernel)
    torch.cuda.synchronize()
    rep = S.themis_bounds_check_report(S.Problem.of_workload(wl, kernel), wl.vertical, ws)
    assert rep["checked"], "the bounds-checked library is not the one loaded"
    assert rep["site"] == 0, f"index {rep['index']} outside [0, {rep['limit']}) at check site {rep['site']}"
    return {k: v.cpu().numpy() for k, v in out.items()}


@pytest.mark.parametrize("kernel_id", range(6), ids=KERNEL_IDS)
def test_edge_shapes_raise_no_violation(S, oracle_mod, kernel_id):
    for shape in SHAPES:
        n_stages, c_max, batches, h_max, T, bucket_us, vertical, (lo, hi) = shape
        wl = W.random_tiny_workload(9000 + T + n_stages, 7, n_stages, c_max, batches, h_max, T, bucket_us=bucket_us,
                                    vertical=vertical, rate_lo=lo, rate_hi=hi)
        _assert_results_equal(_checked_solve(S, wl, kernel_id), oracle_mod.solve_batch(wl))


@pytest.mark.parametrize("kernel_id", range(6), ids=KERNEL_IDS)
def test_budget_lengths_and_stage_counts_raise_no_violation(S, oracle_mod, kernel_id):
    for T in (1, 2, 31, 32, 33, 127, 128, 131, 135, 136, 255, 256, 257, 263, 264, 511, 512, 903, 904, 1024, 1031, 1100,
              1899, 1900, 2047, 2048, 2049, 2055, 2056):
        wl = W.random_tiny_workload(5000 + T, 6, 3, 8, (1, 2, 4), 4, T,
                                    bucket_us=max(1, 400_000 // T) if T < 400 else 1000, rate_lo=20.0, rate_hi=120.0)
        _assert_results_equal(_checked_solve(S, wl, kernel_id), oracle_mod.solve_batch(wl))
    for n_stages in (1, 2, 64):
        wl = W.random_tiny_workload(5200 + n_stages, 5, n_stages, 4, (1, 2, 4), 3, 40 * n_stages + 60,
                                    rate_lo=10.0, rate_hi=60.0)
        _assert_results_equal(_checked_solve(S, wl, kernel_id), oracle_mod.solve_batch(wl))
    wl = W.random_tiny_workload(5300, 12, 64, 4, (1, 2), 3, 700, bucket_us=2000, rate_lo=2.0, rate_hi=30.0)   # 64 stages, short budget
    _assert_results_equal(_checked_solve(S, wl, kernel_id), oracle_mod.solve_batch(wl))
    wl = W.random_tiny_workload(5100, 2, 3, 16, (1, 2, 4, 8, 16), 8, 16383, bucket_us=100, rate_lo=50.0, rate_hi=400.0)
    _assert_results_equal(_checked_solve(S, wl, kernel_id), oracle_mod.solve_batch(wl))


@pytest.mark.parametrize("kernel_id", range(6), ids=KERNEL_IDS)
def test_benchmark_shapes_raise_no_violation(S, oracle_mod, kernel_id):
    """Subsets of the benchmark configurations (the launch shapes the benchmark times)."""
    for cfg, n in ((1, 64), (2, 64), (3, 96), (4, 8), (5, 2)):
        wl = W.make_workload(cfg, n)
        _assert_results_equal(_checked_solve(S, wl, kernel_id), oracle_mod.solve_batch(wl))


def test_long_lists_raise_no_violation(S, oracle_mod):
    """The sparse kernels' hand-over of instances that outgrow their lists."""
    from tests.test_gpu_parity import _long_front_workload
    wl = _long_front_workload()
    _assert_results_equal(_checked_solve(S, wl, 3), oracle_mod.solve_batch(wl))


def test_normal_build_reports_unchecked(S):
    import torch
    S.use_library()
    try:
        wl = W.make_workload(1, 4)
        out, ws = S.solve(wl)
        torch.cuda.synchronize()
        rep = S.themis_bounds_check_report(S.Problem.of_workload(wl), False, ws)
        assert rep == {"site": 0, "index": 0, "limit": 0, "checked": False}
    finally:
        from paper_2407_14843_b200 import build
        S.use_library(build.CHECK_LIB_PATH)
