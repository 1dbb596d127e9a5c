"""Pins for the CPU oracle: hand-worked cases, exhaustive enumeration, closed
forms and invariants.  None of these tests touches the CUDA library."""
import dataclasses
import json
import os

import numpy as np
import pytest

from paper_2407_14843_b200 import workloads as W
from tests import pyref

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_cases.json")


def _hand_workload(case):
    if "lat_us" in case:
        lat = np.asarray(case["lat_us"], dtype=np.int32)[None]                        # [1][S][C][B]
    else:
        lat = (np.asarray(case["lat_ms"], dtype=np.int64) * 1000).astype(np.int32)[None]
    S = lat.shape[1]
    rep = case["replicas"]
    return W.Workload(
        name=case["name"], n_instances=1, n_stages=S, n_profiles=1, c_max=case["c_max"],
        batch_sizes=tuple(case["batch_sizes"]), h_max=case["h_max"],
        slo_us=case["T"] * case["bucket_us"], bucket_us=case["bucket_us"], flags=case["flags"],
        vertical=rep is not None, lat_us=np.ascontiguousarray(lat),
        profile_id=np.zeros(1, np.int32), lambda_mrps=np.asarray([case["lambda_mrps"]], np.uint32),
        replicas=None if rep is None else np.asarray([rep], np.int32))


def hand_cases():
    with open(GOLDEN) as f:
        return json.load(f)["cases"]


@pytest.mark.parametrize("case", hand_cases(), ids=lambda c: c["name"])
def test_hand_worked_cases(oracle_mod, case):
    wl = _hand_workload(case)
    exp = case["expect"]
    r = oracle_mod.solve_batch(wl)
    assert int(r["status"][0]) == exp["status"]
    assert r["h"][0].tolist() == exp["h"]
    assert r["c"][0].tolist() == exp["c"]
    assert r["b"][0].tolist() == exp["b"]
    assert int(r["total_cost"][0]) == exp["total_cost"]
    assert int(r["latency_buckets"][0]) == exp["latency_buckets"]
    # the two other CPU solvers agree with the hand result too
    for alt in (oracle_mod.alg1_scatter(wl, 0), oracle_mod.brute_force(wl, 0)):
        assert alt["status"] == exp["status"]
        assert alt["h"].tolist() == exp["h"] and alt["c"].tolist() == exp["c"] and alt["b"].tolist() == exp["b"]
        assert alt["total_cost"] == exp["total_cost"] and alt["latency_buckets"] == exp["latency_buckets"]


def _assert_same(r, n, ref, what):
    if ref is None or ref.get("status", 0) == 1:
        assert int(r["status"][n]) == 1, what
        assert int(r["total_cost"][n]) == -1 and int(r["latency_buckets"][n]) == -1, what
        assert not r["h"][n].any() and not r["c"][n].any() and not r["b"][n].any(), what
        return
    assert int(r["status"][n]) == 0, what
    assert int(r["total_cost"][n]) == ref["total_cost"], what
    assert int(r["latency_buckets"][n]) == ref["latency_buckets"], what
    assert r["h"][n].tolist() == list(ref["h"]), what
    assert r["c"][n].tolist() == list(ref["c"]), what
    assert r["b"][n].tolist() == list(ref["b"]), what


@pytest.mark.parametrize("flags", [0, W.QUEUE_PER_REPLICA])
@pytest.mark.parametrize("vertical", [False, True])
def test_random_tiny_vs_rational_brute_force(oracle_mod, flags, vertical):
    """DP oracle == exhaustive search written with exact rationals in the paper's units."""
    checked = infeasible = 0
    for seed in range(12):
        S = 1 + seed % 3
        T = [60, 100, 150, 300][seed % 4]
        wl = W.random_tiny_workload(1000 + seed + 50 * flags + 7 * vertical, 24, S, 4, (1, 2, 4), 3, T,
                                    flags=flags, vertical=vertical)
        r = oracle_mod.solve_batch(wl)
        for n in range(wl.n_instances):
            ref = pyref.solve_instance(wl, n)
            _assert_same(r, n, ref, f"seed {seed} instance {n}")
            checked += 1
            infeasible += ref is None
    assert checked == 288
    assert 0 < infeasible < checked  # both branches exercised


def test_config1_exhaustive(oracle_mod):
    """Every instance of the smallest benchmark configuration against the
    128^3-tuple enumeration and against Algorithm 1 in the paper's loop order."""
    wl = W.make_workload(1)
    r = oracle_mod.solve_batch(wl)
    for n in range(wl.n_instances):
        _assert_same(r, n, oracle_mod.brute_force(wl, n), f"brute force, instance {n}")
        _assert_same(r, n, oracle_mod.alg1_scatter(wl, n), f"scatter, instance {n}")


@pytest.mark.parametrize("half_ms", [False, True])
def test_tight_budgets_exhaustive(oracle_mod, half_ms):
    """Budgets near the feasibility edge (where ties and infeasibility occur),
    against the C enumeration and the scatter form, joint and vertical."""
    n_inf = 0
    for seed in range(6):
        for vertical in (False, True):
            w = 500 if half_ms else 1000
            T = (70 + 25 * seed) * (2 if half_ms else 1)
            wl = W.random_tiny_workload(2000 + seed, 32, 3, 6, (1, 2, 4, 8), 4, T, bucket_us=w,
                                        vertical=vertical, rate_lo=20.0, rate_hi=200.0)
            r = oracle_mod.solve_batch(wl)
            for n in range(wl.n_instances):
                _assert_same(r, n, oracle_mod.brute_force(wl, n), f"bf seed {seed} n {n}")
                _assert_same(r, n, oracle_mod.alg1_scatter(wl, n), f"scatter seed {seed} n {n}")
            n_inf += int(r["status"].sum())
    assert n_inf > 0


def test_minplus_against_numpy_definition(oracle_mod):
    """oracle.minplus == the textbook (min,+) convolution written with numpy
    broadcasting; argmin = first index of the minimum."""
    rng = np.random.default_rng(7)
    for T in (0, 1, 17, 130):
        Fp = rng.integers(0, 500, T + 1).astype(np.int64)
        G = rng.integers(0, 500, T + 1).astype(np.int64)
        Fp[rng.random(T + 1) < 0.4] = -1
        G[rng.random(T + 1) < 0.6] = -1
        BIG = 10 ** 12
        fp = np.where(Fp < 0, BIG, Fp)
        g = np.where(G < 0, BIG, G)
        t = np.arange(T + 1)[:, None]
        l = np.arange(T + 1)[None, :]
        tab = np.where(l <= t, fp[np.clip(t - l, 0, T)] + g[l], 4 * BIG)
        ref_v = tab.min(axis=1)
        ref_a = tab.argmin(axis=1)
        inf = ref_v >= BIG
        F, A = oracle_mod.minplus(np.where(Fp < 0, oracle_mod.INF, Fp), np.where(G < 0, oracle_mod.INF, G))
        assert np.array_equal(F == oracle_mod.INF, inf)
        assert np.array_equal(F[~inf], ref_v[~inf])
        assert np.array_equal(A[~inf], ref_a[~inf])
        assert not A[inf].any()


def test_minplus_single_entry_is_a_shift(oracle_mod):
    """G with one finite entry (l0, k): F = shift(Fprev, l0) + k exactly."""
    rng = np.random.default_rng(3)
    T, l0, k = 200, 37, 11
    Fp = rng.integers(1, 90, T + 1).astype(np.int32)
    Fp[rng.random(T + 1) < 0.3] = oracle_mod.INF
    G = np.full(T + 1, oracle_mod.INF, np.int32)
    G[l0] = k
    F, A = oracle_mod.minplus(Fp, G)
    assert (F[:l0] == oracle_mod.INF).all()
    src = Fp[: T + 1 - l0]
    fin = src != oracle_mod.INF
    assert np.array_equal(F[l0:][fin], src[fin] + k)
    assert (F[l0:][~fin] == oracle_mod.INF).all()
    assert (A[l0:][fin] == l0).all()


def test_score_stage_against_rational_candidates(oracle_mod):
    """G/Garg of one stage == per-bucket minimum over the rational candidate list."""
    wl = W.make_workload(2, 8)
    T = wl.T
    for n in range(4):
        for s in (0, wl.n_stages - 1):
            lam = int(wl.lambda_mrps[n])
            lat = wl.lat_us[wl.profile_id[n]][s]
            for h_fixed in (0, 3):
                G, Garg = oracle_mod.score_stage(wl.c_max, wl.batch_sizes, wl.h_max, wl.bucket_us,
                                                 wl.flags, lat, lam, h_fixed, T)
                hv = [h_fixed] if h_fixed else range(1, wl.h_max + 1)
                ref_g = np.full(T + 1, oracle_mod.INF, np.int64)
                ref_a = np.zeros(T + 1, np.int64)
                for idx, h, c, b, ell, cost in pyref.stage_candidates(
                        lat, wl.c_max, wl.batch_sizes, hv, lam, wl.bucket_us, wl.flags):
                    if ell <= T and cost < ref_g[ell]:
                        ref_g[ell], ref_a[ell] = cost, idx
                assert np.array_equal(G, ref_g)
                assert np.array_equal(Garg, ref_a)
                assert (G != oracle_mod.INF).sum() > 3


def _stage_ell(wl, n, s, h, c, b):
    """Latency in buckets of the returned configuration (rational form)."""
    bi = wl.batch_sizes.index(b)
    cands = pyref.stage_candidates(wl.lat_us[wl.profile_id[n]][s], wl.c_max, wl.batch_sizes, [h],
                                   int(wl.lambda_mrps[n]), wl.bucket_us, wl.flags)
    for idx, hh, cc, bb, ell, cost in cands:
        if cc == c and bb == b:
            return ell
    return None  # infeasible


@pytest.mark.parametrize("cfg,n", [(2, 48), (3, 64), (4, 6)])
def test_returned_configurations_satisfy_the_constraints(oracle_mod, cfg, n):
    """Every returned stage config sustains lambda; stage latencies sum to the
    reported latency <= T; h*c sums to the reported cost (Eq. 5, Eq. 6)."""
    wl = W.make_workload(cfg, n)
    if cfg == 3:  # pick seconds spread over the day, including spikes
        full = W.make_workload(cfg)
        pick = np.linspace(0, full.n_instances - 1, n).astype(int)
        wl = dataclasses.replace(full, n_instances=n, profile_id=full.profile_id[pick].copy(),
                                 lambda_mrps=full.lambda_mrps[pick].copy(), replicas=full.replicas[pick].copy())
    r = oracle_mod.solve_batch(wl)
    solved = 0
    for i in range(wl.n_instances):
        if r["status"][i]:
            continue
        solved += 1
        ells = []
        for s in range(wl.n_stages):
            h, c, b = int(r["h"][i][s]), int(r["c"][i][s]), int(r["b"][i][s])
            assert 1 <= c <= wl.c_max and b in wl.batch_sizes
            if wl.vertical:
                assert h == wl.replicas[i][s]
            else:
                assert 1 <= h <= wl.h_max
            ell = _stage_ell(wl, i, s, h, c, b)
            assert ell is not None, "returned configuration cannot sustain the arrival rate"
            ells.append(ell)
        assert sum(ells) == r["latency_buckets"][i] <= wl.T
        assert int((r["h"][i] * r["c"][i]).sum()) == r["total_cost"][i]
    assert solved > 0


def test_slack_budget_is_separable(oracle_mod):
    """With a budget no stage can exhaust, the optimum is the sum of the
    per-stage cheapest feasible configurations."""
    wl = W.random_tiny_workload(31, 16, 3, 5, (1, 2, 4), 3, 8000)
    r = oracle_mod.solve_batch(wl)
    for n in range(wl.n_instances):
        total = worst = 0
        for s in range(wl.n_stages):
            cands = pyref.stage_candidates(wl.lat_us[n][s], wl.c_max, wl.batch_sizes,
                                           range(1, wl.h_max + 1), int(wl.lambda_mrps[n]), wl.bucket_us, wl.flags)
            worst += max(x[4] for x in cands)
            total += min(x[5] for x in cands)
        assert worst <= wl.T
        assert int(r["total_cost"][n]) == total


def test_budget_below_fastest_path_is_infeasible(oracle_mod):
    wl = W.random_tiny_workload(32, 16, 3, 5, (1, 2, 4), 3, 400)
    for n in range(wl.n_instances):
        fastest = 0
        for s in range(wl.n_stages):
            cands = pyref.stage_candidates(wl.lat_us[n][s], wl.c_max, wl.batch_sizes,
                                           range(1, wl.h_max + 1), int(wl.lambda_mrps[n]), wl.bucket_us, wl.flags)
            fastest += min(x[4] for x in cands)
        one = wl.take(1, n)
        tight = dataclasses.replace(one, slo_us=fastest * wl.bucket_us)
        short = dataclasses.replace(one, slo_us=(fastest - 1) * wl.bucket_us)
        assert oracle_mod.solve_batch(tight)["status"][0] == 0
        assert oracle_mod.solve_batch(tight)["latency_buckets"][0] == fastest
        assert oracle_mod.solve_batch(short)["status"][0] == 1


def test_horizontal_restriction_closed_form(oracle_mod):
    """c_max = 1, slack budget: per stage the optimum is min over b of the
    least replica count ceil(lambda * l / b) (Algorithm 2's instance count,
    rounded up so that the throughput constraint holds)."""
    from fractions import Fraction
    import math
    wl = W.random_tiny_workload(33, 16, 2, 1, (1, 2, 4, 8), 64, 6000, rate_lo=20.0, rate_hi=300.0)
    r = oracle_mod.solve_batch(wl)
    for n in range(wl.n_instances):
        lam = Fraction(int(wl.lambda_mrps[n]), 1000)
        total = 0
        for s in range(wl.n_stages):
            need = []
            for bi, b in enumerate(wl.batch_sizes):
                l = Fraction(int(wl.lat_us[n][s][0][bi]), 1_000_000)
                need.append(math.ceil(lam * l / b))
            assert min(need) <= wl.h_max
            total += min(need)
        assert r["status"][n] == 0 and int(r["total_cost"][n]) == total


def test_stage_order_does_not_change_the_optimum(oracle_mod):
    """(min,+) is commutative and associative: permuting the stages leaves the
    optimal cost and its total latency unchanged."""
    wl = W.random_tiny_workload(34, 24, 4, 6, (1, 2, 4), 3, 260, rate_lo=20.0, rate_hi=120.0)
    r0 = oracle_mod.solve_batch(wl)
    for perm in ([3, 2, 1, 0], [1, 3, 0, 2]):
        wl2 = dataclasses.replace(wl, lat_us=np.ascontiguousarray(wl.lat_us[:, perm]))
        r1 = oracle_mod.solve_batch(wl2)
        assert np.array_equal(r0["total_cost"], r1["total_cost"])
        assert np.array_equal(r0["latency_buckets"], r1["latency_buckets"])
        assert np.array_equal(r0["h"][:, perm], r1["h"])
        ok = r0["status"] == 0
        assert np.array_equal((r0["h"] * r0["c"])[ok].sum(1), r0["total_cost"][ok])


def test_monotonicity_invariants(oracle_mod):
    """Cost never rises with a longer SLO or finer buckets; the vertical
    variant (h fixed within 1..h_max) is never cheaper than the joint one;
    with batch size 1 only (no queuing term) cost never falls as lambda grows."""
    base = W.random_tiny_workload(35, 48, 3, 6, (1, 2, 4, 8), 4, 150, rate_lo=20.0, rate_hi=200.0)
    BIG = 1 << 30
    cost = lambda r: np.where(r["status"] == 0, r["total_cost"], BIG)
    r = oracle_mod.solve_batch(base)
    longer = oracle_mod.solve_batch(dataclasses.replace(base, slo_us=base.slo_us + 23_000))
    assert (cost(longer) <= cost(r)).all()
    finer = oracle_mod.solve_batch(dataclasses.replace(base, bucket_us=500))
    assert (cost(finer) <= cost(r)).all()
    rep = W.rand_int(5, 8, np.arange(48 * 3, dtype=np.uint64), 1, 4).reshape(48, 3).astype(np.int32)
    vert = oracle_mod.solve_batch(dataclasses.replace(base, vertical=True, replicas=rep))
    assert (cost(vert) >= cost(r)).all()
    assert (cost(vert) > cost(r)).any()
    b1 = dataclasses.replace(base, batch_sizes=(1,), lat_us=np.ascontiguousarray(base.lat_us[..., :1]))
    lo = oracle_mod.solve_batch(b1)
    hi = oracle_mod.solve_batch(dataclasses.replace(b1, lambda_mrps=(b1.lambda_mrps * 1.37).astype(np.uint32)))
    assert (cost(hi) >= cost(lo)).all()
    assert (cost(hi) > cost(lo)).any()


def test_one_replica_vertical_matches_algorithm1_cost(oracle_mod):
    """With one replica per stage the objective h*c is Algorithm 1's sum of cores."""
    wl = W.paper_scale_workload(12)
    r = oracle_mod.solve_batch(wl)
    ok = r["status"] == 0
    assert ok.any()
    assert np.array_equal(r["c"][ok].sum(1), r["total_cost"][ok])
    for n in range(0, wl.n_instances, 3):
        _assert_same(r, n, oracle_mod.alg1_scatter(wl, n), f"paper-scale instance {n}")


def test_pins_catch_planted_mistakes(oracle_mod):
    """Sensitivity of the pins: feeding the oracle a wrong problem (cores and
    batch axes swapped, or the queue flag dropped) changes results that the
    rational brute force of the right problem fixes."""
    wl = W.random_tiny_workload(36, 24, 2, 4, (1, 2, 4, 8), 3, 120, rate_lo=20.0, rate_hi=150.0)
    ref = [pyref.solve_instance(wl, n) for n in range(wl.n_instances)]

    def differs(r):
        bad = 0
        for n, x in enumerate(ref):
            got = None if r["status"][n] else (int(r["total_cost"][n]), int(r["latency_buckets"][n]))
            want = None if x is None else (x["total_cost"], x["latency_buckets"])
            bad += got != want
        return bad

    assert differs(oracle_mod.solve_batch(wl)) == 0
    swapped = dataclasses.replace(wl, lat_us=np.ascontiguousarray(wl.lat_us.transpose(0, 1, 3, 2)))
    assert differs(oracle_mod.solve_batch(swapped)) > 0
    assert differs(oracle_mod.solve_batch(dataclasses.replace(wl, flags=0))) > 0


# ---------------------------------------------------------------- horizontal-only solver (Algorithm 2)

@pytest.mark.parametrize("flags", [0, W.QUEUE_PER_REPLICA])
def test_horizontal_against_rational_brute_force_and_algorithm2(oracle_mod, flags):
    """One-core replicas, replica count computed per batch size: the DP oracle
    equals exhaustive search over batch-size tuples in exact rationals, and
    Algorithm 2 run in the paper's loop order."""
    n_inf = 0
    for seed in range(8):
        T = [60, 90, 140, 400][seed % 4]
        wl = W.random_tiny_workload(7000 + seed, 24, 1 + seed % 4, 1, (1, 2, 4, 8, 16), 12, T, flags=flags,
                                    rate_lo=20.0, rate_hi=400.0)
        r = oracle_mod.solve_batch(wl, horizontal=True)
        for n in range(wl.n_instances):
            _assert_same(r, n, pyref.solve_instance_horizontal(wl, n), f"seed {seed} instance {n}")
            _assert_same(r, n, oracle_mod.alg2_scatter(wl, n), f"scatter, seed {seed} instance {n}")
        n_inf += int(r["status"].sum())
        assert (r["c"][r["status"] == 0] == 1).all()
    assert n_inf > 0


def test_horizontal_equals_joint_restricted_to_one_core(oracle_mod):
    """Extra replicas beyond the fewest that sustain lambda only add cost and
    queuing delay, so enumerating h (joint solver, c_max = 1) changes nothing."""
    wl = W.random_tiny_workload(7100, 48, 3, 1, (1, 2, 4, 8), 20, 110, rate_lo=20.0, rate_hi=300.0)
    a = oracle_mod.solve_batch(wl, horizontal=True)
    b = oracle_mod.solve_batch(wl)
    for k in ("status", "total_cost", "latency_buckets", "h", "c", "b"):
        assert np.array_equal(a[k], b[k]), k
    assert (a["status"] == 0).any() and (a["status"] == 1).any()


def test_horizontal_replica_counts_are_tight(oracle_mod):
    """Every returned replica count sustains lambda and one replica fewer would not (Eq. 6)."""
    wl = W.random_tiny_workload(7200, 32, 3, 1, (1, 2, 4, 8), 64, 3000, rate_lo=50.0, rate_hi=900.0)
    r = oracle_mod.solve_batch(wl, horizontal=True)
    for n in range(wl.n_instances):
        if r["status"][n]:
            continue
        for s in range(wl.n_stages):
            h, b = int(r["h"][n][s]), int(r["b"][n][s])
            l_us = int(wl.lat_us[n][s][0][wl.batch_sizes.index(b)])
            lam = int(wl.lambda_mrps[n])
            assert h * b * 10 ** 9 >= lam * l_us
            assert h == 1 or (h - 1) * b * 10 ** 9 < lam * l_us


# ---------------------------------------------------------------- Algorithm 1's last branch

def _spiky_vertical_workload(n_hot=24):
    """Seconds of the day-long trace around its largest spikes plus quiet ones."""
    full = W.make_workload(3)
    hot = np.argsort(full.lambda_mrps)[-n_hot:]
    pick = np.unique(np.concatenate([hot, np.arange(0, full.n_instances, 7200)]))
    return dataclasses.replace(full, n_instances=len(pick), profile_id=full.profile_id[pick].copy(),
                               lambda_mrps=full.lambda_mrps[pick].copy(), replicas=full.replicas[pick].copy())


def test_vertical_fallback_invariants(oracle_mod):
    """Where the replicas in place cannot serve the load: the rate found is
    served, the next search point is not, the extra replicas carry exactly the
    rest (one fewer would not), and feasible instances are left alone."""
    wl = _spiky_vertical_workload()
    res = 1000
    r = oracle_mod.vertical_fallback_batch(wl, res)
    plain = oracle_mod.solve_batch(wl)
    split = r["status"] == 2
    assert split.any() and (r["status"] == 0).any()
    assert np.array_equal(r["status"] == 0, plain["status"] == 0)
    keep = plain["status"] == 0
    for k in ("h", "c", "b", "total_cost", "latency_buckets"):
        assert np.array_equal(r[k][keep], plain[k][keep])
    assert np.array_equal(r["lambda_vertical"][keep], wl.lambda_mrps[keep]) and not r["extra_replicas"][keep].any()
    lv = r["lambda_vertical"]
    assert (lv[split] % res == 0).all() and (lv[split] > 0).all() and (lv[split] < wl.lambda_mrps[split]).all()
    at = oracle_mod.solve_batch(dataclasses.replace(wl, lambda_mrps=np.where(split, lv, wl.lambda_mrps).astype(np.uint32)))
    above = oracle_mod.solve_batch(dataclasses.replace(
        wl, lambda_mrps=np.where(split, np.minimum(lv + res, wl.lambda_mrps), wl.lambda_mrps).astype(np.uint32)))
    assert (at["status"][split] == 0).all() and (above["status"][split] == 1).all()
    for k in ("h", "c", "b", "total_cost", "latency_buckets"):
        assert np.array_equal(r[k][split], at[k][split])
    for n in np.flatnonzero(split):
        rest = int(wl.lambda_mrps[n]) - int(lv[n])
        for s in range(wl.n_stages):
            c, b, e = int(r["c"][n][s]), int(r["b"][n][s]), int(r["extra_replicas"][n][s])
            l_us = int(wl.lat_us[0][s][c - 1][wl.batch_sizes.index(b)])
            assert e * b * 10 ** 9 >= rest * l_us and (e - 1) * b * 10 ** 9 < rest * l_us


def test_vertical_fallback_finds_the_maximum_when_feasibility_is_monotone(oracle_mod):
    """Batch size 1 only (no queuing term): feasibility is monotone in the rate, so
    the bisection result is the largest served multiple of the resolution, which a
    linear scan over every search point confirms."""
    base = W.random_tiny_workload(7400, 10, 2, 4, (1,), 3, 60, vertical=True, rate_lo=150.0, rate_hi=400.0)
    res = 5000
    r = oracle_mod.vertical_fallback_batch(base, res)
    assert (r["status"] == 2).any()
    for n in np.flatnonzero(r["status"] != 0):
        one = base.take(1, int(n))
        served = [k for k in range(1, int(base.lambda_mrps[n]) // res + 1)
                  if oracle_mod.solve_batch(dataclasses.replace(one, lambda_mrps=np.asarray([k * res], np.uint32)))["status"][0] == 0]
        assert int(r["lambda_vertical"][n]) == (max(served) * res if served else 0)
        assert (r["status"][n] == 2) == bool(served)


def test_full_queue_model_reduces_to_the_simplified_one():
    """Eq. 3, q = max((b-1)/lambda, l(b,c) - (n*b+1)/lambda): for every candidate
    that satisfies the throughput constraint of Eq. 6 the second term is negative,
    so the solver's queue model (Eq. 4) is Eq. 3 on the feasible set."""
    from fractions import Fraction
    wl = W.make_workload(2, 16)
    checked = 0
    for n in range(0, 16, 5):
        lam = Fraction(int(wl.lambda_mrps[n]), 1000)
        for s in range(wl.n_stages):
            for h in range(1, wl.h_max + 1, 3):
                for c in range(1, wl.c_max + 1, 5):
                    for bi, b in enumerate(wl.batch_sizes):
                        l = Fraction(int(wl.lat_us[wl.profile_id[n]][s][c - 1][bi]), 1_000_000)
                        if h * Fraction(b) / l >= lam:
                            second = l - Fraction(h * b + 1) / lam
                            assert second < 0
                            assert max(Fraction(b - 1) / lam, second) == Fraction(b - 1) / lam
                            checked += 1
    assert checked > 500


# ---------------------------------------------------------------- tables that follow no model

@pytest.mark.parametrize("vertical", [False, True])
@pytest.mark.parametrize("flags", [0, W.QUEUE_PER_REPLICA])
def test_arbitrary_tables_vs_rational_brute_force(oracle_mod, flags, vertical):
    """Latency entries drawn independently (not monotone in cores or batch size, odd
    bucket widths, batch sizes that are not powers of two): DP oracle, exact-rational
    brute force and the paper's scatter order agree."""
    solved = 0
    for seed, (bucket, T, batches) in enumerate([(777, 150, (1, 3, 5)), (1300, 90, (2, 7)), (250, 500, (1, 2, 3, 4))]):
        wl = W.arbitrary_tables_workload(8000 + seed, 20, 1 + seed, 5, batches, 3, T, bucket, flags, vertical)
        r = oracle_mod.solve_batch(wl)
        for n in range(wl.n_instances):
            _assert_same(r, n, pyref.solve_instance(wl, n), f"seed {seed} instance {n}")
            _assert_same(r, n, oracle_mod.alg1_scatter(wl, n), f"scatter seed {seed} instance {n}")
        solved += int((r["status"] == 0).sum())
    assert solved > 10
