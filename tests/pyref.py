"""Pure-Python, exact-rational restatement of the paper's formulas, used only
to pin the C oracle on tiny instances.  Quantities are kept in the paper's
real-valued form (seconds, requests per second) as ``fractions.Fraction`` and
only rounded to buckets at the end, so a unit slip in the oracle's integer
restatement shows up here.
"""
import itertools
import math
from fractions import Fraction


def stage_candidates(lat_us_stage, c_max, batch_sizes, h_values, lambda_mrps, bucket_us, flags):
    """Feasible candidates of one stage as (idx, h, c, b, ell, cost).

    thr = b / l per replica, feasible iff h * thr >= lambda (Eq. 6);
    q = (b - 1) / lambda (Eq. 4), times h when flag bit 0 is set;
    ell = ceil(l / w) + ceil(q / w)."""
    lam = Fraction(int(lambda_mrps), 1000)            # requests per second
    w = Fraction(int(bucket_us), 1_000_000)           # seconds
    out, idx = [], 0
    for h in h_values:
        for c in range(1, c_max + 1):
            for bi, b in enumerate(batch_sizes):
                l = Fraction(int(lat_us_stage[c - 1][bi]), 1_000_000)
                thr = Fraction(b) / l
                if h * thr >= lam:
                    q = Fraction(b - 1) / lam * (h if flags & 1 else 1)
                    ell = math.ceil(l / w) + math.ceil(q / w)
                    out.append((idx, h, c, b, ell, h * c))
                idx += 1
    return out


def stage_candidates_horizontal(lat_us_stage, batch_sizes, h_max, lambda_mrps, bucket_us, flags):
    """Algorithm 2's candidates: one-core replicas, h = ceil(lambda / thr(b, 1))
    (the fewest replicas with thr * h >= lambda), dropped when h > h_max."""
    lam = Fraction(int(lambda_mrps), 1000)
    w = Fraction(int(bucket_us), 1_000_000)
    out = []
    for bi, b in enumerate(batch_sizes):
        l = Fraction(int(lat_us_stage[0][bi]), 1_000_000)
        h = max(1, math.ceil(lam / (Fraction(b) / l)))
        if h > h_max:
            continue
        q = Fraction(b - 1) / lam * (h if flags & 1 else 1)
        out.append((bi, h, 1, b, math.ceil(l / w) + math.ceil(q / w), h))
    return out


def solve_instance_horizontal(wl, n):
    pid = int(wl.profile_id[n])
    stages = [stage_candidates_horizontal(wl.lat_us[pid][s], wl.batch_sizes, wl.h_max,
                                          int(wl.lambda_mrps[n]), wl.bucket_us, wl.flags)
              for s in range(wl.n_stages)]
    return brute_force(stages, wl.T)


def brute_force(stages, T):
    """Eq. 6 by enumeration with the lexicographic tie-break key
    (cost, total latency, ell_{S-1}, ..., ell_1, idx_0, ..., idx_{S-1})."""
    best = None
    for tup in itertools.product(*stages):
        lat = sum(x[4] for x in tup)
        if lat > T:
            continue
        cost = sum(x[5] for x in tup)
        key = (cost, lat, tuple(x[4] for x in reversed(tup[1:])), tuple(x[0] for x in tup))
        if best is None or key < best[0]:
            best = (key, tup)
    if best is None:
        return None
    key, tup = best
    return {"total_cost": key[0], "latency_buckets": key[1],
            "h": [x[1] for x in tup], "c": [x[2] for x in tup], "b": [x[3] for x in tup],
            "ell": [x[4] for x in tup]}


def solve_instance(wl, n):
    pid = int(wl.profile_id[n])
    stages = []
    for s in range(wl.n_stages):
        hv = [int(wl.replicas[n][s])] if wl.vertical else range(1, wl.h_max + 1)
        stages.append(stage_candidates(wl.lat_us[pid][s], wl.c_max, wl.batch_sizes, hv,
                                       int(wl.lambda_mrps[n]), wl.bucket_us, wl.flags))
    return brute_force(stages, wl.T)
