"""themis_solve_batch_static: the solver for callers that cannot allocate
device memory (its tables live in a fixed buffer inside the library).

Collected last on purpose (file name), so a run that stops at the first
failure has already run every other test.  The check: on calls in a row, with
different shapes so that each call finds the previous call's leftovers in the
shared buffer, the results equal those of the workspace entry points and those
of the CPU oracle word for word (the solver is integer-exact, so the tolerance
is zero), with every kernel choice, and the calls leave the amount of free
device memory unchanged."""
import numpy as np
import pytest

from paper_2407_14843_b200 import workloads as W

pytestmark = pytest.mark.gpu

KEYS = ("status", "total_cost", "latency_buckets", "h", "c", "b")


@pytest.fixture(scope="module")
def S():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    from paper_2407_14843_b200 import build
    build.build_library()
    from paper_2407_14843_b200 import solver
    return solver


def _both(S, wl, kernel):
    """(static entry point, workspace entry point) on the same inputs; the static call must
    not change the free device memory."""
    import torch
    prob = S.Problem.of_workload(wl, kernel)
    dev = S.workload_to_device(wl)
    ref, _ = S.solve(wl, dev=dev, kernel=kernel)        # caller-provided workspace
    got = S.alloc_result(wl.n_instances, wl.n_stages)
    for v in got.values():
        v.fill_(-7)
    unchanged = False
    for _ in range(3):          # the figure is device-wide: tolerate a neighbour's allocation, not ours
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        S.themis_solve_batch_static(prob, dev["lat_us"], dev["profile_id"], dev["lambda_mrps"], dev["replicas"], got)
        torch.cuda.synchronize()
        unchanged = unchanged or torch.cuda.mem_get_info()[0] == free_before
    assert unchanged, "the static entry point changed the free device memory"
    return ({k: v.cpu().numpy() for k, v in got.items()}, {k: v.cpu().numpy() for k, v in ref.items()})


@pytest.mark.parametrize("kernel_id", [1, 2, 3, 4, 5, 6],
                         ids=["packed16", "wide32", "pruned", "sparse", "sparse_block", "packed16_block"])
def test_static_scratch_entry_point_matches_workspace_entry_point_and_oracle(S, oracle_mod, kernel_id):
    kernel = kernel_id << 8
    # a throwaway call first, so that the buffer's address is already known when the free
    # memory is compared (the first call on a device looks it up)
    warm = W.make_workload(1, 4)
    S.themis_solve_batch_static(S.Problem.of_workload(warm, kernel), *(S.workload_to_device(warm)[k] for k in
                                ("lat_us", "profile_id", "lambda_mrps", "replicas")),
                                S.alloc_result(warm.n_instances, warm.n_stages))
    # first call: joint problem, 3 stages, T = 500
    first = W.make_workload(1)
    assert S.themis_workspace_bytes(S.Problem.of_workload(first), False) <= S.STATIC_SCRATCH_BYTES
    first_oracle = oracle_mod.solve_batch(first)
    got, ref = _both(S, first, kernel)
    for k in KEYS:
        assert np.array_equal(got[k], ref[k]), ("first call", k)
        assert np.array_equal(got[k], first_oracle[k]), ("first call, oracle", k)
    # second call right after it: vertical problem of another shape (10 stages,
    # T = 800), so every table lands on top of stale words of the first call
    second = W.make_workload(3, 256)
    assert S.themis_workspace_bytes(S.Problem.of_workload(second), True) <= S.STATIC_SCRATCH_BYTES
    second_oracle = oracle_mod.solve_batch(second)
    got, ref = _both(S, second, kernel)
    for k in KEYS:
        assert np.array_equal(got[k], ref[k]), ("second call", k)
        assert np.array_equal(got[k], second_oracle[k]), ("second call, oracle", k)
    assert (ref["status"] == 0).any()
    # and the first problem once more, now on top of the second one's leftovers
    got, ref = _both(S, first, kernel)
    for k in KEYS:
        assert np.array_equal(got[k], ref[k]), ("third call", k)
        assert np.array_equal(got[k], first_oracle[k]), ("third call, oracle", k)


def test_static_scratch_entry_point_refuses_large_problems(S):
    import torch
    wl = W.make_workload(4, 64)                          # 64 * 8 * 4032 * 8 B = 16.5 MB: fits
    prob = S.Problem.of_workload(wl)
    dev = S.workload_to_device(wl)
    out = S.alloc_result(wl.n_instances, wl.n_stages)
    S.themis_solve_batch_static(prob, dev["lat_us"], dev["profile_id"], dev["lambda_mrps"], None, out)
    torch.cuda.synchronize()
    big = W.make_workload(4, 256)                        # 66 MB: beyond the built-in buffer
    prob = S.Problem.of_workload(big)
    assert S.themis_workspace_bytes(prob, False) > S.STATIC_SCRATCH_BYTES
    dev = S.workload_to_device(big)
    out = S.alloc_result(big.n_instances, big.n_stages)
    with pytest.raises(S.ThemisError) as e:
        S.themis_solve_batch_static(prob, dev["lat_us"], dev["profile_id"], dev["lambda_mrps"], None, out)
    assert e.value.code == S.E_STATIC_SCRATCH_EXCEEDED
    assert "32 MiB" in str(e.value)
