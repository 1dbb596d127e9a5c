"""themis_solve_batch_static: the solver for callers that cannot allocate
device memory (its tables live in a fixed buffer inside the library).

Collected last on purpose (file name), so a run that stops at the first
failure has already run every other test.  The check: on calls in a row, with
different shapes so that each call finds the previous call's leftovers in the
shared buffer, the results equal those of the workspace entry points word for
word (the solver is integer-exact, so the tolerance is zero)."""
import numpy as np
import pytest

from paper_2407_14843_b200 import workloads as W

pytestmark = pytest.mark.gpu

KEYS = ("status", "total_cost", "latency_buckets", "h", "c", "b")


def _both(S, wl):
    import torch
    prob = S.Problem.of_workload(wl)
    dev = S.workload_to_device(wl)
    ref, _ = S.solve(wl, dev=dev)                       # caller-provided workspace
    got = S.alloc_result(wl.n_instances, wl.n_stages)
    for v in got.values():
        v.fill_(-7)
    S.themis_solve_batch_static(prob, dev["lat_us"], dev["profile_id"], dev["lambda_mrps"], dev["replicas"], got)
    torch.cuda.synchronize()
    return ({k: v.cpu().numpy() for k, v in got.items()}, {k: v.cpu().numpy() for k, v in ref.items()})


def test_static_scratch_entry_point_matches_workspace_entry_point():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    from paper_2407_14843_b200 import build
    build.build_library()
    from paper_2407_14843_b200 import solver as S
    # first call: joint problem, 3 stages, T = 500
    first = W.make_workload(1)
    assert S.themis_workspace_bytes(S.Problem.of_workload(first), False) <= S.STATIC_SCRATCH_BYTES
    got, ref = _both(S, first)
    for k in KEYS:
        assert np.array_equal(got[k], ref[k]), ("first call", k)
    # second call right after it: vertical problem of another shape (10 stages,
    # T = 800), so every table lands on top of stale words of the first call
    second = W.make_workload(3, 256)
    assert S.themis_workspace_bytes(S.Problem.of_workload(second), True) <= S.STATIC_SCRATCH_BYTES
    got, ref = _both(S, second)
    for k in KEYS:
        assert np.array_equal(got[k], ref[k]), ("second call", k)
    assert (ref["status"] == 0).any()
    # and the first problem once more, now on top of the second one's leftovers
    got, ref = _both(S, first)
    for k in KEYS:
        assert np.array_equal(got[k], ref[k]), ("third call", k)


def test_static_scratch_entry_point_refuses_large_problems():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    from paper_2407_14843_b200 import build
    build.build_library()
    from paper_2407_14843_b200 import solver as S
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
