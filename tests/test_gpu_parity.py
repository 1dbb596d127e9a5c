"""Parity of the CUDA path (called through the C ABI) with the CPU oracle,
element by element and bit-exact, on the same seeded inputs."""
import dataclasses

import numpy as np
import pytest

from paper_2407_14843_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def S():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    from paper_2407_14843_b200 import build
    build.build_library()                      # no-op when the library is up to date
    from paper_2407_14843_b200 import solver
    return solver


def _gpu_solve(S, wl, tables=False, horizontal=False, mode=None, tile=None):
    """Solves through the C ABI with the kernel (0 packed16, 1 wide32, 2 pruned, 3 sparse,
    4 sparse-block) and tile under test, both passed per call in the problem's flags."""
    import torch
    mode = MODE["mode"] if mode is None else mode
    tile = MODE["tile"] if tile is None else tile
    out, ws = S.solve(wl, horizontal=horizontal, kernel=(mode + 1) << 8, tile=tile)
    torch.cuda.synchronize()
    res = {k: v.cpu().numpy() for k, v in out.items()}
    if tables:
        tb = S.workspace_tables(S.Problem.of_workload(wl), wl.vertical, ws)
        W1 = wl.T + 1
        res["G"] = tb["G"][:, :, :W1].cpu().numpy()
        res["Garg"] = tb["Garg"][:, :, :W1].cpu().numpy()
        res["A"] = tb["A"][:, :, :W1].cpu().numpy()
        res["F"] = tb["F"][:, :W1].cpu().numpy()
        res["G_pad"] = tb["G"][:, :, W1:].cpu().numpy()
    return res


RESULT_KEYS = ("status", "total_cost", "latency_buckets", "h", "c", "b")


def _diagnose(gpu, ref, idx):
    """On a mismatch: is the CUDA answer at least optimal (same status and cost, so only a
    tie was broken differently), or is it a different optimum altogether?"""
    pick = (lambda a: a) if idx is None else (lambda a: a[idx])
    st, cost = pick(gpu["status"]), pick(gpu["total_cost"])
    same_opt = (st == ref["status"]) & (cost == ref["total_cost"])
    cfg_equal = np.all(pick(gpu["h"]) == ref["h"], axis=1) & np.all(pick(gpu["c"]) == ref["c"], axis=1) \
        & np.all(pick(gpu["b"]) == ref["b"], axis=1) & (pick(gpu["latency_buckets"]) == ref["latency_buckets"])
    return (f"{int((~same_opt).sum())} instances with a different status or cost (optimality), "
            f"{int((same_opt & ~cfg_equal).sum())} with the same cost but another configuration or latency (tie-break)")


def _assert_results_equal(gpu, ref, idx=None):
    for k in RESULT_KEYS:
        a = gpu[k] if idx is None else gpu[k][idx]
        assert np.array_equal(a, ref[k]), (f"{k} differs at instances {np.argwhere(a != ref[k])[:5].tolist()}: "
                                           + _diagnose(gpu, ref, idx))


# kernel under test: 0 packed 16-bit (the default: one warp per instance for short budgets, else
# a block), 1 32-bit, 2 pruned, 3 sparse (one warp per instance, block kernel for what outgrows
# its lists), 4 sparse block kernel, 5 packed 16-bit with a block per instance at any budget;
# tile: cells per thread
MODE = {"mode": 0, "tile": 0}


@pytest.fixture(params=[0, 1, 2, 3, 4, 5], ids=["packed16", "wide32", "pruned", "sparse", "sparse_block", "packed16_block"])
def mode(request, S):
    MODE["mode"] = request.param
    yield request.param
    MODE["mode"] = 0


def _assert_tables_equal(S, gpu, ref):
    """G, Garg everywhere; F (last prefix) where the instance is solved; then
    32-bit kernel: A where F_s[t] is reachable (0 elsewhere);
    packed kernel: every prefix table F_s[t], saturated at 0x7FFF, up to the budget the
    later stages can still complete."""
    if MODE["mode"] in (3, 4): # one fused kernel: the workspace holds fronts, not the dense tables
        return
    assert np.array_equal(gpu["G"], ref["G"])
    assert np.array_equal(gpu["Garg"], ref["Garg"])
    assert (gpu["G_pad"] == S.G_INF).all()
    if MODE["mode"] == 2:      # tables of the restricted problem: only the results are comparable
        return
    if MODE["mode"] in (0, 5):
        solved = ref["status"] == 0
        assert np.array_equal(gpu["F"][solved], ref["F"][solved, -1, :])
        assert (ref["F"][ref["F"] != S.G_INF] < S.INF16).all(), "use the saturation test for such inputs"
        # prefix tables relative to the running sum of the stages' cheapest entries
        cheapest = ref["G"].astype(np.int64).min(axis=2)
        cheapest[cheapest == S.G_INF] = 0
        rel = ref["F"].astype(np.int64) - np.cumsum(cheapest, axis=1)[:, :, None]
        rel[ref["F"] == S.G_INF] = S.INF16
        # budgets the later stages cannot complete any more (their fastest candidates do not
        # fit) are not computed: "unreachable" above T - sum of their first non-empty buckets
        N_, S_, W1 = ref["G"].shape
        nonempty = ref["G"] != S.G_INF
        first = np.where(nonempty.any(axis=2), nonempty.argmax(axis=2), W1)
        later = np.zeros((N_, S_), np.int64)
        for s in range(S_ - 2, -1, -1):
            later[:, s] = np.minimum(later[:, s + 1] + first[:, s + 1], W1)
        rel[np.arange(W1)[None, None, :] > (W1 - 1 - later)[:, :, None]] = S.INF16
        assert np.array_equal(gpu["A"], rel.astype(np.uint16))
        return
    assert np.array_equal(gpu["F"], ref["F"][:, -1, :])
    reach = ref["F"] != S.G_INF
    reach[:, 0, :] = False                     # A has no row for the first stage
    assert np.array_equal(gpu["A"][reach], ref["A"][reach])
    unreach = ~reach
    unreach[:, 0, :] = False
    assert not gpu["A"][unreach].any()


# ---------------------------------------------------------------- small, full tables

@pytest.mark.parametrize("tile", [4, 8, 16])
def test_config1_every_table(S, oracle_mod, tile, mode):
    """Smallest benchmark configuration: every intermediate table and result."""
    MODE["tile"] = tile
    try:
        wl = W.make_workload(1)
        ref = oracle_mod.solve_batch(wl, dumps=True)
        gpu = _gpu_solve(S, wl, tables=True)
        _assert_tables_equal(S, gpu, ref)
        _assert_results_equal(gpu, ref)
    finally:
        MODE["tile"] = 0


@pytest.mark.parametrize("cfg,n", [(2, 96), (3, 160), (4, 12), (5, 3)])
@pytest.mark.parametrize("tile", [4, 8, 16])
def test_config_subsets_every_table(S, oracle_mod, cfg, n, tile, mode):
    """Subsets of the larger configurations (several tiles, ragged tail: T+1 is
    never a multiple of the tile): every table and result."""
    if tile == 8 and cfg == 5:
        pytest.skip("8 cells per thread would need more than 1024 threads at T = 8192")
    MODE["tile"] = tile
    try:
        wl = W.make_workload(cfg, n)
        if cfg == 3:   # seconds spread over the day so that spikes are included
            full = W.make_workload(3)
            pick = np.linspace(0, full.n_instances - 1, n).astype(int)
            wl = dataclasses.replace(full, n_instances=n, profile_id=full.profile_id[pick].copy(),
                                     lambda_mrps=full.lambda_mrps[pick].copy(), replicas=full.replicas[pick].copy())
        ref = oracle_mod.solve_batch(wl, dumps=True)
        gpu = _gpu_solve(S, wl, tables=True)
        _assert_tables_equal(S, gpu, ref)
        _assert_results_equal(gpu, ref)
    finally:
        MODE["tile"] = 0


@pytest.mark.parametrize("flags", [0, W.QUEUE_PER_REPLICA])
@pytest.mark.parametrize("vertical", [False, True])
def test_random_tiny_against_enumeration(S, oracle_mod, flags, vertical, mode):
    """Random tiny instances near the feasibility edge, against the exhaustive
    Eq. 6 enumeration (not only the DP oracle)."""
    for seed in range(5):
        T = 50 + 31 * seed
        wl = W.random_tiny_workload(4000 + seed, 40, 1 + seed % 3, 6, (1, 2, 4, 8), 4, T,
                                    flags=flags, vertical=vertical, rate_lo=20.0, rate_hi=200.0)
        gpu = _gpu_solve(S, wl)
        for n in range(wl.n_instances):
            bf = oracle_mod.brute_force(wl, n)
            assert gpu["status"][n] == bf["status"]
            assert gpu["total_cost"][n] == bf["total_cost"] and gpu["latency_buckets"][n] == bf["latency_buckets"]
            for k in ("h", "c", "b"):
                assert np.array_equal(gpu[k][n], bf[k])


def test_hand_worked_cases(S, mode):
    """The hand-derived fixtures, straight against the CUDA path."""
    from tests.test_oracle_pins import _hand_workload, hand_cases
    for case in hand_cases():
        wl = _hand_workload(case)
        gpu = _gpu_solve(S, wl)
        exp = case["expect"]
        assert int(gpu["status"][0]) == exp["status"], case["name"]
        assert gpu["h"][0].tolist() == exp["h"] and gpu["c"][0].tolist() == exp["c"], case["name"]
        assert gpu["b"][0].tolist() == exp["b"], case["name"]
        assert int(gpu["total_cost"][0]) == exp["total_cost"], case["name"]
        assert int(gpu["latency_buckets"][0]) == exp["latency_buckets"], case["name"]


def test_paper_scale_vertical(S, oracle_mod, mode):
    """A pipeline of the paper's own size: 3 stages, b and c in 1..16, one
    replica per stage, SLO 2550 ms, queue delay exactly as Eq. 4."""
    wl = W.paper_scale_workload(40)
    ref = oracle_mod.solve_batch(wl, dumps=True)
    gpu = _gpu_solve(S, wl, tables=True)
    _assert_tables_equal(S, gpu, ref)
    _assert_results_equal(gpu, ref)
    assert (ref["status"] == 0).any()


@pytest.mark.parametrize("flags", [0, W.QUEUE_PER_REPLICA])
def test_horizontal_only_solver(S, oracle_mod, flags, mode):
    """Algorithm 2 (one-core replicas, replica count computed): every table and
    result against the oracle, and results against the joint entry point."""
    for seed, (nb, h_max, T) in enumerate([((1, 2, 4, 8, 16), 12, 90), ((1, 2, 4, 8), 300, 700),
                                           ((1, 2, 4, 8, 16, 32), 64, 2100)]):
        wl = W.random_tiny_workload(7300 + seed, 48, 2 + seed, 1, nb, h_max, T, flags=flags,
                                    rate_lo=20.0, rate_hi=900.0)
        ref = oracle_mod.solve_batch(wl, dumps=True, horizontal=True)
        gpu = _gpu_solve(S, wl, tables=True, horizontal=True)
        _assert_tables_equal(S, gpu, ref)
        _assert_results_equal(gpu, ref)
        _assert_results_equal(_gpu_solve(S, wl), ref)          # joint solver, c_max = 1
        assert (ref["status"] == 0).any()
    import ctypes
    bad = S.Problem.of_workload(W.make_workload(1))             # c_max = 8: refused
    res = S.Result()
    for k in ("h", "c", "b", "total_cost", "latency_buckets", "status"):
        setattr(res, k, 256)
    one = ctypes.c_void_p(256)
    assert S._lib.themis_solve_horizontal_batch(ctypes.byref(bad), one, None, one, res, one, 1 << 40, None) \
        == S.E_INVALID_ARG


@pytest.mark.parametrize("res", [1000, 25000])
def test_vertical_fallback(S, oracle_mod, res, mode):
    """Algorithm 1 with its last branch (bisection on the rate + extra replicas):
    every output against the oracle, on trace seconds around the largest spikes."""
    import torch
    from tests.test_oracle_pins import _spiky_vertical_workload
    wl = _spiky_vertical_workload(40)
    ref = oracle_mod.vertical_fallback_batch(wl, res)
    assert (ref["status"] == 2).any() and (ref["status"] == 0).any()
    prob = S.Problem.of_workload(wl, kernel=(mode + 1) << 8)
    dev = S.workload_to_device(wl)
    ws = torch.empty(S.themis_fallback_workspace_bytes(prob), dtype=torch.uint8, device="cuda")
    out = S.alloc_result(wl.n_instances, wl.n_stages)
    lam_v = torch.empty(wl.n_instances, dtype=torch.uint32, device="cuda")
    extra = torch.empty((wl.n_instances, wl.n_stages), dtype=torch.int32, device="cuda")
    S.themis_vertical_fallback_batch(prob, dev["lat_us"], dev["profile_id"], dev["lambda_mrps"], dev["replicas"],
                                     res, int(wl.lambda_mrps.max()), out, lam_v, extra, ws)
    torch.cuda.synchronize()
    gpu = {k: v.cpu().numpy() for k, v in out.items()}
    _assert_results_equal(gpu, ref)
    assert np.array_equal(lam_v.cpu().numpy(), ref["lambda_vertical"])
    assert np.array_equal(extra.cpu().numpy(), ref["extra_replicas"])
    # a bound on lambda that is too low is reported, not silently wrong
    S.themis_vertical_fallback_batch(prob, dev["lat_us"], dev["profile_id"], dev["lambda_mrps"], dev["replicas"],
                                     res, 4 * res, out, lam_v, extra, ws)
    torch.cuda.synchronize()
    st = out["status"].cpu().numpy()
    assert (st[ref["status"] == 2] == S.STATUS_BAD_INPUT).all() and (st[ref["status"] == 0] == 0).all()


def test_stability_test_of_the_transition_policy(S, oracle_mod):
    """Horizontal solves at the current and at a predicted rate, compared on the device:
    stable exactly where the oracle's two configurations coincide."""
    import torch
    wl = W.random_tiny_workload(7500, 200, 3, 1, (1, 2, 4, 8), 40, 260, rate_lo=20.0, rate_hi=300.0)
    growth = 1.0 + 0.3 * W.rand_uniform(7501, 1, np.arange(200, dtype=np.uint64))      # up to 30 % more load
    pred = dataclasses.replace(wl, lambda_mrps=(wl.lambda_mrps * growth).astype(np.uint32))
    now_out, _ = S.solve(wl, horizontal=True)
    pred_out, _ = S.solve(pred, horizontal=True)
    stable = torch.empty(200, dtype=torch.int32, device="cuda")
    S.themis_configs_equal_batch(now_out, pred_out, stable)
    torch.cuda.synchronize()
    a, b = oracle_mod.solve_batch(wl, horizontal=True), oracle_mod.solve_batch(pred, horizontal=True)
    expect = (a["status"] == 0) & (b["status"] == 0) & np.all(a["h"] == b["h"], axis=1) \
        & np.all(a["b"] == b["b"], axis=1) & np.all(a["c"] == b["c"], axis=1)
    assert np.array_equal(stable.cpu().numpy().astype(bool), expect)
    assert expect.any() and (~expect).any()


# ---------------------------------------------------------------- edge cases

@pytest.mark.parametrize("T", [1, 2, 31, 32, 33, 127, 128, 131, 135, 136, 255, 256, 257, 263, 264, 511, 512, 902, 903, 904,
                               1024, 1031, 1100, 1898, 1899, 1900,  # 903/904: 4 -> 8 cells a tile; 1899/1900: warp -> block kernel
                               2047, 2048, 2049, 2055, 2056])
def test_budget_lengths_around_tile_boundaries(S, oracle_mod, T, mode):
    wl = W.random_tiny_workload(5000 + T, 6, 3, 8, (1, 2, 4), 4, T, bucket_us=max(1, 400_000 // T) if T < 400 else 1000,
                                rate_lo=20.0, rate_hi=120.0)
    ref = oracle_mod.solve_batch(wl, dumps=True)
    gpu = _gpu_solve(S, wl, tables=True)
    _assert_tables_equal(S, gpu, ref)
    _assert_results_equal(gpu, ref)


def test_maximum_budget_length(S, oracle_mod, mode):
    """T = 16383, the largest supported budget (1024 threads x 16 cells)."""
    wl = W.random_tiny_workload(5100, 2, 3, 16, (1, 2, 4, 8, 16), 8, 16383, bucket_us=100,
                                rate_lo=50.0, rate_hi=400.0)
    ref = oracle_mod.solve_batch(wl, dumps=True)
    gpu = _gpu_solve(S, wl, tables=True)
    _assert_tables_equal(S, gpu, ref)
    _assert_results_equal(gpu, ref)
    assert (ref["status"] == 0).all()


@pytest.mark.parametrize("n_stages", [1, 2, 64])
def test_stage_counts(S, oracle_mod, n_stages, mode):
    wl = W.random_tiny_workload(5200 + n_stages, 5, n_stages, 4, (1, 2, 4), 3, 40 * n_stages + 60,
                                rate_lo=10.0, rate_hi=60.0)
    ref = oracle_mod.solve_batch(wl, dumps=True)
    gpu = _gpu_solve(S, wl, tables=True)
    _assert_tables_equal(S, gpu, ref)
    _assert_results_equal(gpu, ref)


def test_most_stages_on_a_short_budget(S, oracle_mod, mode):
    """64 stages within 700 buckets: the one-warp-per-instance packed kernel with its per-stage
    arrays at their largest, on a budget so tight that every instance spends all of it (and a
    looser one)."""
    for bucket_us in (2000, 4000):
        wl = W.random_tiny_workload(5300, 12, 64, 4, (1, 2), 3, 700, bucket_us=bucket_us, rate_lo=2.0, rate_hi=30.0)
        ref = oracle_mod.solve_batch(wl, dumps=True)
        assert (ref["status"] == 0).all()
        gpu = _gpu_solve(S, wl, tables=True)
        _assert_tables_equal(S, gpu, ref)
        _assert_results_equal(gpu, ref)
    wl = W.random_tiny_workload(5300, 12, 64, 4, (1, 2), 3, 700, bucket_us=1000, rate_lo=2.0, rate_hi=30.0)   # all infeasible
    ref = oracle_mod.solve_batch(wl, dumps=True)
    gpu = _gpu_solve(S, wl, tables=True)
    _assert_tables_equal(S, gpu, ref)
    _assert_results_equal(gpu, ref)


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_shapes_every_kernel_and_tile(S, oracle_mod, seed):
    """Seeded random problem shapes (stages, cores, batch sizes, replicas, budget lengths on both
    sides of every kernel and tile switch-over, both queue models, joint and vertical, rates from
    starved to saturated): every kernel choice with every tile size against the oracle."""
    import random
    import torch
    rng = random.Random(seed)
    done = 0
    while done < 60:
        n_stages = rng.choice([1, 2, 3, 4, 5, 7, 10, 13])
        c_max = rng.choice([1, 2, 3, 5, 8, 16, 33, 64])
        batches = tuple(sorted(rng.sample([1, 2, 3, 4, 5, 6, 8, 12, 16, 24, 32, 48, 64], rng.choice([1, 2, 3, 4, 6]))))
        h_max = rng.choice([1, 2, 3, 8, 16, 31, 33, 64])
        T = rng.choice([1, 5, 17, 63, 64, 65, 200, 500, 903, 904, 1000, 1500, 1899, 1900, 2300, 2799, 2800, 3100])
        vertical = rng.random() < 0.3
        flags = rng.choice([0, W.QUEUE_PER_REPLICA])
        bucket_us = rng.choice([250, 500, 1000, 2000]) if T >= 100 else max(1, 300_000 // T)
        lo = rng.choice([2.0, 20.0, 200.0])
        hi = lo * rng.choice([2, 10, 30])
        if c_max * len(batches) * (1 if vertical else h_max) > 65535 or n_stages * h_max * c_max > 131070:
            continue
        done += 1
        wl = W.random_tiny_workload(20_000 + 100 * seed + done, rng.choice([3, 9, 33]), n_stages, c_max, batches, h_max, T,
                                    bucket_us=bucket_us, flags=flags, vertical=vertical, rate_lo=lo, rate_hi=hi)
        ref = oracle_mod.solve_batch(wl)
        for kernel_id in range(1, 7):
            for tile in ((0, 4, 8, 16) if kernel_id in (1, 2, 6) else (0,)):
                out, _ = S.solve(wl, kernel=kernel_id << 8, tile=tile)
                torch.cuda.synchronize()
                _assert_results_equal({k: v.cpu().numpy() for k, v in out.items()}, ref)


SHAPES = [  # n_stages, c_max, batch sizes, h_max, T, bucket_us, vertical, rate range (rps)
    (2, 1, tuple(range(1, 17)), 512, 300, 1000, False, (50.0, 4000.0)),      # widest replica table
    (3, 100, (1,), 3, 77, 2000, False, (5.0, 90.0)),                         # one batch size, ragged core count
    (4, 33, (1, 2, 5), 7, 1025, 500, True, (20.0, 300.0)),                   # one cell beyond a tile group
    (2, 2, (1, 2), 2, 16383, 100, False, (5.0, 30.0)),                       # longest budget, 8 candidates
    (64, 3, (1, 4), 2, 2500, 1000, False, (5.0, 60.0)),                      # most stages
    (5, 64, (1, 2, 4, 8, 16, 32, 64, 128), 16, 4096, 250, False, (100.0, 900.0)),   # T a power of two
    (6, 16, (1, 2, 4, 8), 64, 2056, 500, False, (200.0, 3000.0)),            # eight cells beyond the tiles
    (3, 7, (2, 3), 5, 263, 1000, True, (10.0, 80.0)),
    (3, 20, (1, 2, 4), 1, 300, 1000, False, (5.0, 200.0)),                   # joint problem with one replica count
    (2, 40000, (3,), 1, 500, 1000, False, (5.0, 50.0)),                      # core counts beyond 15 bits
    (3, 9, (1, 2, 4, 8), 40, 900, 500, False, (50.0, 2500.0)),               # replica counts: a full and a ragged chunk of 32
]


@pytest.mark.parametrize("shape", SHAPES, ids=[f"S{s[0]}_C{s[1]}_B{len(s[2])}_H{s[3]}_T{s[4]}" for s in SHAPES])
def test_assorted_shapes(S, oracle_mod, shape, mode):
    """Shapes at the edges of the supported ranges, every kernel mode, every table the mode exposes."""
    n_stages, c_max, batches, h_max, T, bucket_us, vertical, (lo, hi) = shape
    wl = W.random_tiny_workload(9000 + T + n_stages, 7, n_stages, c_max, batches, h_max, T, bucket_us=bucket_us,
                                vertical=vertical, rate_lo=lo, rate_hi=hi)
    ref = oracle_mod.solve_batch(wl, dumps=True)
    gpu = _gpu_solve(S, wl, tables=True)
    _assert_tables_equal(S, gpu, ref)
    _assert_results_equal(gpu, ref)


@pytest.mark.parametrize("vertical", [False, True])
@pytest.mark.parametrize("flags", [0, W.QUEUE_PER_REPLICA])
def test_arbitrary_latency_tables(S, oracle_mod, flags, vertical, mode):
    """Latency tables that follow no model (not monotone in cores or batch size, entries
    repeated between neighbouring core counts, odd bucket widths, batch sizes that are not
    powers of two): every table the mode exposes and every result."""
    for seed, (bucket, T, batches, c_max, h_max) in enumerate([
            (777, 400, (1, 3, 5, 6), 40, 9), (1300, 1100, (2, 7), 70, 5), (333, 2600, (1, 2, 3, 4, 9, 17), 17, 33)]):
        wl = W.arbitrary_tables_workload(8100 + seed, 12, 2 + seed, c_max, batches, h_max, T, bucket, flags, vertical)
        ref = oracle_mod.solve_batch(wl, dumps=True)
        gpu = _gpu_solve(S, wl, tables=True)
        _assert_tables_equal(S, gpu, ref)
        _assert_results_equal(gpu, ref)


def test_single_instance_single_candidate(S, oracle_mod):
    wl = W.random_tiny_workload(5300, 1, 2, 1, (1,), 1, 100, rate_lo=5.0, rate_hi=6.0)
    ref = oracle_mod.solve_batch(wl)
    _assert_results_equal(_gpu_solve(S, wl), ref)


def test_all_infeasible_and_all_slack(S, oracle_mod, mode):
    tight = W.random_tiny_workload(5400, 16, 4, 4, (1, 2), 2, 20, rate_lo=300.0, rate_hi=900.0)
    ref = oracle_mod.solve_batch(tight)
    assert (ref["status"] == 1).all()
    _assert_results_equal(_gpu_solve(S, tight), ref)
    slack = W.random_tiny_workload(5401, 16, 4, 4, (1, 2), 2, 9000, rate_lo=5.0, rate_hi=20.0)
    ref = oracle_mod.solve_batch(slack)
    assert (ref["status"] == 0).all()
    _assert_results_equal(_gpu_solve(S, slack), ref)


def test_null_profile_id_means_profile_zero(S, oracle_mod):
    import torch
    wl = W.make_workload(2, 32)
    wl0 = dataclasses.replace(wl, profile_id=np.zeros(32, np.int32))
    ref = oracle_mod.solve_batch(wl0)
    dev = S.workload_to_device(wl0)
    dev["profile_id"] = None
    out, _ = S.solve(wl0, dev=dev)
    torch.cuda.synchronize()
    _assert_results_equal({k: v.cpu().numpy() for k, v in out.items()}, ref)


def test_bad_device_inputs_are_reported_per_instance(S, oracle_mod, mode):
    """lambda = 0, a non-positive latency and replicas < 1 do not fault: the
    instance gets THEMIS_STATUS_BAD_INPUT, its neighbours are solved."""
    wl = W.make_workload(2, 8)
    lam = wl.lambda_mrps.copy()
    lam[3] = 0
    bad = dataclasses.replace(wl, lambda_mrps=lam)
    gpu = _gpu_solve(S, bad)
    ref = oracle_mod.solve_batch(wl)
    assert gpu["status"][3] == S.STATUS_BAD_INPUT and gpu["total_cost"][3] == -1 and not gpu["h"][3].any()
    keep = np.arange(8) != 3
    for k in RESULT_KEYS:
        assert np.array_equal(gpu[k][keep], ref[k][keep])
    lat = wl.lat_us.copy()
    lat[int(wl.profile_id[5]), 1, 0, 0] = 0
    gpu = _gpu_solve(S, dataclasses.replace(wl, lat_us=lat))
    assert gpu["status"][5] == S.STATUS_BAD_INPUT
    v = W.make_workload(3, 8)
    rep = v.replicas.copy()
    rep[2, 4] = 0
    gpu = _gpu_solve(S, dataclasses.replace(v, replicas=rep))
    assert gpu["status"][2] == S.STATUS_BAD_INPUT and (gpu["status"][[0, 1, 3]] != S.STATUS_BAD_INPUT).all()


def test_repeatable_and_tile_independent(S, mode):
    """Same inputs, two runs and both tile sizes: identical words everywhere
    (every cross-thread hand-off is a barrier, so nothing may depend on timing)."""
    wl = W.make_workload(4, 24)
    runs = []
    for tile in (16, 16, 8, 4):
        runs.append(_gpu_solve(S, wl, tables=True, tile=tile))
    for r in runs[1:]:
        for k in RESULT_KEYS + ("G", "Garg", "A", "F"):
            assert np.array_equal(runs[0][k], r[k]), k


def test_all_kernels_agree(S):
    """Packed 16-bit, 32-bit, pruned and the two sparse kernels: the same results, word for word."""
    for wl in (W.make_workload(3, 300), W.make_workload(4, 96), W.make_workload(2, 512)):
        runs = []
        for m in (1, 0, 2, 3, 4):
            runs.append(_gpu_solve(S, wl, mode=m))
        for r in runs[1:]:
            for k in RESULT_KEYS:
                assert np.array_equal(runs[0][k], r[k]), k


def _beyond_16_bits_workload():
    """Vertical problem with thousands of replicas per stage.  The packed kernel holds, in 15
    bits, what an instance pays beyond the sum of its stages' cheapest entries.  One group of
    instances has totals of 36000 and more but pays little beyond those entries (solved by the
    packed kernel); another must take the dearer core count in all six stages, 36000 beyond
    them, and is redone by the 32-bit kernel.  Mixed with cheap and with infeasible instances."""
    base = W.random_tiny_workload(5600, 32, 6, 2, (1, 2, 4), 4, 420, vertical=True, rate_lo=10.0, rate_hi=60.0)
    rep = base.replicas.copy()
    rep[0::4] = 6000                        # 6 stages x 6000 x c: totals of 36000 .. 72000
    rep[1::4] = np.maximum(rep[1::4], 1)
    rep[3::4] = 6000
    lam = base.lambda_mrps.copy()
    lam[2::4] = 4_000_000                   # 4000 rps on a handful of replicas: infeasible
    lat = base.lat_us.copy()                # one profile per instance: [N][S][c][b]
    lat[3::4, :, 0, :] = 130_000            # one core: 130 buckets; two cores: 65; budget 420, so
    lat[3::4, :, 1, :] = 65_000             # six stages only fit with two cores everywhere
    lat[3::4, :, :, 1:] = 900_000           # larger batches never fit
    return dataclasses.replace(base, replicas=rep, lambda_mrps=lam, lat_us=lat)


def test_totals_beyond_16_bits_fall_back_to_the_wide_kernel(S, oracle_mod):
    wl = _beyond_16_bits_workload()
    ref = oracle_mod.solve_batch(wl, dumps=True)
    assert (ref["status"] == 1).any()
    assert ((ref["total_cost"] > 0) & (ref["total_cost"] < S.INF16)).any()
    beyond = ref["total_cost"] - ref["G"].astype(np.int64).min(axis=2).sum(axis=1)
    solved = ref["status"] == 0
    assert (solved & (ref["total_cost"] >= S.INF16) & (beyond < S.INF16)).any()
    assert (solved[3::4] & (beyond[3::4] >= S.INF16)).all()
    _assert_results_equal(_gpu_solve(S, wl, mode=0), ref)     # budget of 420 buckets: one warp per instance
    _assert_results_equal(_gpu_solve(S, wl, mode=5), ref)     # the same with a block per instance


def test_recurrence_step_repeats_on_a_scored_workspace(S, oracle_mod):
    """themis_minplus_batch only consumes G and Garg: called again on the same scored
    workspace, with the same or another kernel, it returns the same results.  On the
    workload whose dear instances the packed kernel hands to the 32-bit kernel (they stay
    marked in the workspace between the calls)."""
    import torch
    wl = _beyond_16_bits_workload()
    ref = oracle_mod.solve_batch(wl)
    dev = S.workload_to_device(wl)
    ws = S.alloc_workspace(S.Problem.of_workload(wl), True)
    S.themis_score_batch(S.Problem.of_workload(wl), dev["lat_us"], dev["profile_id"], dev["lambda_mrps"],
                         dev["replicas"], ws)
    for kernel in (S.KERNEL_PACKED16, S.KERNEL_PACKED16, S.KERNEL_WIDE32, S.KERNEL_PACKED16_BLOCK, S.KERNEL_PRUNED,
                   S.KERNEL_PACKED16):
        out = S.alloc_result(wl.n_instances, wl.n_stages)
        for v in out.values():
            v.fill_(-9)
        S.themis_minplus_batch(S.Problem.of_workload(wl, kernel), dev["replicas"], out, ws)
        torch.cuda.synchronize()
        _assert_results_equal({k: v.cpu().numpy() for k, v in out.items()}, ref)


def _long_front_workload():
    """Instances whose undominated lists are long.  Three stages, one batch size, replicas fixed:
    latencies fall by a whole number of buckets per core, so every core count is an undominated
    stage entry.  Instances 0 and 3: stage 0 costs 61 per core, stage 1 costs 1 per core, and
    stage 0 gains 60 buckets per core against 1 in stage 1, so all 3600 pairs of core counts
    up to 60 are undominated states of the first two stages (the third stage has 150 entries,
    which also keeps the stage fronts out of the scratch of the upper-bound search, so nothing
    is pruned).  Instances 1 and 4: 160 undominated entries in every stage.  Instances 2 and 5:
    two core counts matter."""
    N, S_, C, w = 6, 3, 160, 100
    lat = np.empty((N, S_, C, 1), np.int32)
    rep = np.ones((N, S_), np.int32)
    c = np.arange(1, C + 1)
    for n in range(N):
        kind = n % 3
        if kind == 0:
            lat[n, 0, :, 0] = (4000 - 60 * np.minimum(c, 60)) * w
            lat[n, 1, :, 0] = (100 - np.minimum(c, 60)) * w
            lat[n, 2, :, 0] = (600 - 2 * np.minimum(c, 150)) * w
            rep[n] = (61, 1, 1)
        elif kind == 1:
            lat[n, 0, :, 0] = (3000 - 7 * c) * w + 13          # not a whole number of buckets
            lat[n, 1, :, 0] = (900 - 3 * c) * w
            lat[n, 2, :, 0] = (500 - c) * w
        else:
            lat[n, 0, :, 0] = np.where(c < 40, 700, 300) * w
            lat[n, 1, :, 0] = np.where(c < 7, 900, 500) * w
            lat[n, 2, :, 0] = np.where(c < 90, 400, 350) * w
    return W.Workload(name="long_fronts", n_instances=N, n_stages=S_, n_profiles=N, c_max=C, batch_sizes=(1,),
                      h_max=1, slo_us=4700 * w, bucket_us=w, flags=W.QUEUE_PER_REPLICA, vertical=True,
                      lat_us=lat, profile_id=np.arange(N, dtype=np.int32),
                      lambda_mrps=np.full(N, 1000, np.uint32), replicas=rep)


def test_sparse_kernel_hands_long_lists_to_the_block_kernel(S, oracle_mod):
    """The warp-per-instance kernels keep fixed-size lists; instances that outgrow them (here:
    3600 prefix states against 256 slots, 160 stage entries against 128) are listed in the
    workspace and redone by the block kernel.  Results equal the oracle's either way."""
    import torch
    wl = _long_front_workload()
    ref = oracle_mod.solve_batch(wl, dumps=True)
    assert (ref["status"] == 0).all()
    front = lambda X: (X < np.concatenate([np.full(X.shape[:2] + (1,), S.G_INF, X.dtype),
                                           np.minimum.accumulate(X, axis=2)[:, :, :-1]], axis=2)).sum(axis=2)
    g, f = front(ref["G"]), front(ref["F"])
    assert (f[[0, 3], 1] == 3600).all() and (g[[0, 3], 2] == 150).all()
    assert (g[[1, 4]] == 160).all() and (g[[2, 5]] <= 2).all()
    prob = S.Problem.of_workload(wl, S.KERNEL_SPARSE)
    out, ws = S.solve(wl, kernel=S.KERNEL_SPARSE)
    torch.cuda.synchronize()
    _assert_results_equal({k: v.cpu().numpy() for k, v in out.items()}, ref)
    lay = S.themis_workspace_layout(prob, True)
    redo_at = (lay.flag_offset + 4 * wl.n_instances + 255) // 256 * 256
    redo = ws[redo_at:redo_at + 4 * (1 + wl.n_instances)].view(torch.int32).cpu().numpy()
    assert redo[0] == 4 and sorted(redo[1:5].tolist()) == [0, 1, 3, 4]


def test_two_host_threads_with_different_kernels(S, oracle_mod):
    """The kernel choice travels with the call: two host threads, each on its own stream,
    solve different batches with different kernels at the same time, repeatedly; every
    result equals the oracle's."""
    import threading
    import torch
    jobs = [(W.make_workload(2, 192), S.KERNEL_PACKED16), (W.make_workload(3, 256), S.KERNEL_SPARSE),
            (W.make_workload(4, 24), S.KERNEL_WIDE32), (W.make_workload(2, 160), S.KERNEL_SPARSE_BLOCK)]
    refs = [oracle_mod.solve_batch(wl) for wl, _ in jobs]
    errors = []

    def work(k):
        try:
            wl, kernel = jobs[k]
            torch.cuda.set_device(0)
            with torch.cuda.stream(torch.cuda.Stream()):
                dev = S.workload_to_device(wl)
                for _ in range(12):
                    out, _ws = S.solve(wl, dev=dev, kernel=kernel)
                    torch.cuda.current_stream().synchronize()
                    _assert_results_equal({key: v.cpu().numpy() for key, v in out.items()}, refs[k])
        except BaseException as e:          # reported by the main thread
            errors.append((k, e))

    threads = [threading.Thread(target=work, args=(k,)) for k in range(len(jobs))]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors


def test_sharded_solve_on_a_one_rank_group(S, oracle_mod):
    """sharding.solve_sharded with the CUDA solver as its solve function (NCCL group of one
    rank; the two-rank split is covered on CPU with gloo)."""
    import socket
    import torch
    import torch.distributed as dist
    from paper_2407_14843_b200 import sharding
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1,
                            device_id=torch.device("cuda", 0))
    try:
        wl = W.make_workload(2, 300)
        full = sharding.solve_sharded(wl, lambda block: S.solve(block)[0])
        torch.cuda.synchronize()
        _assert_results_equal({k: v.cpu().numpy() for k, v in full.items()}, oracle_mod.solve_batch(wl))
    finally:
        dist.destroy_process_group()


def test_two_step_entry_points_equal_the_solver(S, oracle_mod):
    import torch
    wl = W.make_workload(3, 64)
    prob = S.Problem.of_workload(wl)
    dev = S.workload_to_device(wl)
    ws = S.alloc_workspace(prob, True)
    out = S.alloc_result(wl.n_instances, wl.n_stages)
    S.themis_score_batch(prob, dev["lat_us"], dev["profile_id"], dev["lambda_mrps"], dev["replicas"], ws)
    S.themis_minplus_batch(prob, dev["replicas"], out, ws)
    torch.cuda.synchronize()
    ref = oracle_mod.solve_batch(wl)
    _assert_results_equal({k: v.cpu().numpy() for k, v in out.items()}, ref)


@pytest.mark.parametrize("cfg,n", [(2, 64), (3, 64)])
def test_host_buffer_entry_point(S, oracle_mod, cfg, n):
    """themis_solve_batch_host: host arrays in, host arrays out."""
    import torch
    wl = W.make_workload(cfg, n)
    prob = S.Problem.of_workload(wl)
    ws = S.alloc_workspace(prob, wl.vertical, host_variant=True)
    out = S.alloc_result(n, wl.n_stages, device="cpu", pin=True)
    pin = lambda a: None if a is None else torch.from_numpy(a).pin_memory()
    S.themis_solve_batch_host(prob, pin(wl.lat_us), pin(wl.profile_id), pin(wl.lambda_mrps),
                              pin(wl.replicas) if wl.vertical else None, out, ws)
    ref = oracle_mod.solve_batch(wl)
    _assert_results_equal({k: v.numpy() for k, v in out.items()}, ref)


# ---------------------------------------------------------------- full sizes

def _check_properties(wl, gpu):
    """Properties that hold at any size: totals are consistent, values in range."""
    ok = gpu["status"] == 0
    assert set(np.unique(gpu["status"])) <= {0, 1}
    assert np.array_equal((gpu["h"] * gpu["c"]).sum(1)[ok], gpu["total_cost"][ok])
    assert (gpu["latency_buckets"][ok] <= wl.T).all() and (gpu["latency_buckets"][ok] >= wl.n_stages).all()
    assert (gpu["c"][ok] >= 1).all() and (gpu["c"][ok] <= wl.c_max).all()
    assert np.isin(gpu["b"][ok], wl.batch_sizes).all()
    if wl.vertical:
        assert np.array_equal(gpu["h"][ok], wl.replicas[ok])
    else:
        assert (gpu["h"][ok] >= 1).all() and (gpu["h"][ok] <= wl.h_max).all()
    assert (gpu["total_cost"][~ok] == -1).all() and not gpu["h"][~ok].any()
    # every returned stage configuration sustains the arrival rate (Eq. 6)
    bi = np.searchsorted(np.asarray(wl.batch_sizes), gpu["b"].clip(min=1))
    n_i, s_i = np.meshgrid(np.arange(wl.n_instances), np.arange(wl.n_stages), indexing="ij")
    l_us = wl.lat_us[wl.profile_id[n_i], s_i, (gpu["c"] - 1).clip(min=0), bi].astype(np.int64)
    supply = gpu["h"].astype(np.int64) * gpu["b"].astype(np.int64) * 10 ** 9
    demand = wl.lambda_mrps.astype(np.int64)[:, None] * l_us
    assert (supply >= demand)[ok].all()


def test_config2_full(S, oracle_mod, mode):
    wl = W.make_workload(2)
    gpu = _gpu_solve(S, wl)
    _check_properties(wl, gpu)
    _assert_results_equal(gpu, oracle_mod.solve_batch(wl))


_ORACLE_CACHE = {}


def _oracle_cached(oracle_mod, key, wl):
    """The oracle's answer for a workload, computed once per test session (the
    same batches are checked against every kernel mode)."""
    if key not in _ORACLE_CACHE:
        _ORACLE_CACHE[key] = oracle_mod.solve_batch(wl)
    return _ORACLE_CACHE[key]


@pytest.mark.parametrize("cfg", [3, 4])
def test_full_size_configs_every_instance(S, oracle_mod, cfg, mode):
    """Configurations 3 (86400 instances) and 4 (16384 instances) in the launch
    configuration the benchmark times: every instance against the oracle."""
    wl = W.make_workload(cfg)
    gpu = _gpu_solve(S, wl)
    _check_properties(wl, gpu)
    _assert_results_equal(gpu, _oracle_cached(oracle_mod, ("full", cfg), wl))


def test_full_size_config5_every_instance(S, oracle_mod, mode):
    """Configuration 5 (4096 instances, 20 stages, T = 8192) in the benchmark's launch
    configuration: every instance against the oracle (one oracle run per session, a few
    minutes of host time, shared by all kernel modes)."""
    wl = W.make_workload(5)
    gpu = _gpu_solve(S, wl)
    _check_properties(wl, gpu)
    _assert_results_equal(gpu, _oracle_cached(oracle_mod, ("full", 5), wl))


def test_bounded_wait_gives_up_and_reports(S, oracle_mod):
    """The recurrence kernels' barrier wait, run on a transaction that nothing delivers: it
    gives up after its attempts, the kernel returns THEMIS_STATUS_TIMEOUT for that barrier and
    the copy that was issued still lands; the context stays usable (a solve right after)."""
    import torch
    src = torch.arange(11, 15, dtype=torch.int32, device="cuda").view(torch.uint32)
    dst = torch.zeros(4, dtype=torch.uint32, device="cuda")
    status = torch.full((2,), 99, dtype=torch.int32, device="cuda")
    S.themis_wait_probe(2000, src, dst, status)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [S.STATUS_OK, S.STATUS_TIMEOUT]
    assert dst.view(torch.int32).cpu().tolist() == [11, 12, 13, 14]
    wl = W.make_workload(1)
    _assert_results_equal(_gpu_solve(S, wl), oracle_mod.solve_batch(wl))
