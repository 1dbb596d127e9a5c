"""Seeded synthetic workloads for the batched pipeline-scaling solver.

This module only draws inputs: profiled-latency tables, arrival rates and
current replica counts.  It holds none of the solver's arithmetic (no queuing
delay, no feasibility test, no bucketing), so that both the CUDA path and the
CPU oracle can be fed the very same integer arrays.

The paper evaluates on a production request trace and on latency profiles
measured from seven DL models (Section "Experimental Evaluation"); neither is
available, so the processes below stand in for them.  The latency tables
follow the shape of the paper's profile model (Eq. 1: latency falls with the
core count and grows with the batch size) in the concrete form
``L(b, c) = ceil(alpha + beta * b / c**gamma)`` milliseconds.

Every random number is a pure function of (seed, stream, index) through the
splitmix64 output function, so instance ``i`` of a workload is the same no
matter how many instances are generated.
"""
from __future__ import annotations

import dataclasses
from typing import Optional, Sequence

import numpy as np

BASE_SEED = 0x7E4D15

# Flag bit understood by the solver entry points (mirrors include/themis.h).
QUEUE_PER_REPLICA = 1

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def _mix(z: np.ndarray) -> np.ndarray:
    """splitmix64 output function on an array of uint64 (wrap-around)."""
    with np.errstate(over="ignore"):
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        return z ^ (z >> np.uint64(31))


def rand_u64(seed: int, stream: int, index) -> np.ndarray:
    """Counter-based 64-bit draw: a pure function of (seed, stream, index)."""
    idx = np.asarray(index, dtype=np.uint64)
    with np.errstate(over="ignore"):
        key = _mix(np.asarray([seed & 0xFFFFFFFFFFFFFFFF], dtype=np.uint64)
                   + _GOLDEN * np.uint64(stream + 1))
        return _mix(key + _GOLDEN * (idx + np.uint64(1)))


def rand_uniform(seed: int, stream: int, index, lo: float = 0.0, hi: float = 1.0) -> np.ndarray:
    """Uniform double in [lo, hi) from the top 53 bits of the draw."""
    u = (rand_u64(seed, stream, index) >> np.uint64(11)).astype(np.float64) * (2.0 ** -53)
    return lo + (hi - lo) * u


def rand_normal(seed: int, stream: int, index) -> np.ndarray:
    """Standard normal by Box-Muller from two counter-based uniforms."""
    idx = np.asarray(index, dtype=np.uint64)
    u1 = ((rand_u64(seed, stream, 2 * idx) >> np.uint64(11)).astype(np.float64) + 1.0) * (2.0 ** -53)
    u2 = rand_uniform(seed, stream, 2 * idx + np.uint64(1))
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def rand_int(seed: int, stream: int, index, lo: int, hi: int) -> np.ndarray:
    """Uniform integer in [lo, hi] (inclusive)."""
    u = rand_uniform(seed, stream, index)
    return (lo + np.floor(u * (hi - lo + 1))).astype(np.int64).clip(lo, hi)


@dataclasses.dataclass
class Workload:
    """One batch of independent solver instances (all arrays on the host)."""

    name: str
    n_instances: int
    n_stages: int
    n_profiles: int
    c_max: int
    batch_sizes: tuple
    h_max: int
    slo_us: int
    bucket_us: int
    flags: int
    vertical: bool
    lat_us: np.ndarray        # int32 [P][S][c_max][n_batch], batch index fastest
    profile_id: np.ndarray    # int32 [N]
    lambda_mrps: np.ndarray   # uint32 [N], milli-requests per second
    replicas: Optional[np.ndarray] = None  # int32 [N][S], vertical variant only
    seed: int = 0

    @property
    def T(self) -> int:
        return self.slo_us // self.bucket_us

    @property
    def n_batch(self) -> int:
        return len(self.batch_sizes)

    @property
    def n_candidates(self) -> int:
        """Candidate configurations per stage."""
        k = self.c_max * self.n_batch
        return k if self.vertical else k * self.h_max

    @property
    def minplus_cells(self) -> int:
        """Triangular count of min-plus cell updates per instance."""
        T = self.T
        return (self.n_stages - 1) * (T + 1) * (T + 2) // 2

    def take(self, n: int, start: int = 0) -> "Workload":
        """A contiguous sub-batch of instances sharing the same tables."""
        sl = slice(start, start + n)
        return dataclasses.replace(
            self,
            n_instances=int(min(n, self.n_instances - start)),
            profile_id=np.ascontiguousarray(self.profile_id[sl]),
            lambda_mrps=np.ascontiguousarray(self.lambda_mrps[sl]),
            replicas=None if self.replicas is None else np.ascontiguousarray(self.replicas[sl]),
        )

    def checksums(self) -> dict:
        """Order-sensitive 64-bit checksum of every input array (for logs)."""
        def digest(a: np.ndarray) -> str:
            data = np.ascontiguousarray(a).reshape(-1).view(np.uint8)
            pad = (-data.size) % 8
            if pad:
                data = np.concatenate([data, np.zeros(pad, np.uint8)])
            words = data.view(np.uint64)
            with np.errstate(over="ignore"):
                pos = _GOLDEN * np.arange(1, words.size + 1, dtype=np.uint64)
                acc = np.bitwise_xor.reduce(_mix(words + pos))
            return f"{int(acc):016x}"
        out = {"lat_us": digest(self.lat_us), "profile_id": digest(self.profile_id),
               "lambda_mrps": digest(self.lambda_mrps)}
        if self.replicas is not None:
            out["replicas"] = digest(self.replicas)
        return out


def latency_tables(seed: int, n_profiles: int, n_stages: int, c_max: int,
                   batch_sizes: Sequence[int], beta_lo: float = 5.0, beta_hi: float = 40.0) -> np.ndarray:
    """Profiled latency tables ``L_us[p][s][c-1][bi]`` in microseconds.

    alpha ~ U[5, 20] ms, beta ~ U[beta_lo, beta_hi] ms, gamma ~ U[0.6, 1.0] per
    (profile, stage); ``L = 1000 * ceil(alpha + beta * b / c**gamma)``.
    """
    ps = np.arange(n_profiles * n_stages, dtype=np.uint64)
    alpha = rand_uniform(seed, 1, ps, 5.0, 20.0).reshape(n_profiles, n_stages, 1, 1)
    beta = rand_uniform(seed, 2, ps, beta_lo, beta_hi).reshape(n_profiles, n_stages, 1, 1)
    gamma = rand_uniform(seed, 3, ps, 0.6, 1.0).reshape(n_profiles, n_stages, 1, 1)
    c = np.arange(1, c_max + 1, dtype=np.float64).reshape(1, 1, c_max, 1)
    b = np.asarray(batch_sizes, dtype=np.float64).reshape(1, 1, 1, -1)
    lat_ms = np.ceil(alpha + beta * b / np.power(c, gamma))
    return np.ascontiguousarray((1000.0 * lat_ms).astype(np.int32))


def _to_mrps(rate_rps: np.ndarray) -> np.ndarray:
    return np.maximum(1000, np.rint(1000.0 * rate_rps)).astype(np.uint32)


def _lognormal_rates(seed: int, n: int, median: float, sigma: float, lo: float, hi: float,
                     rho: float = 0.0) -> np.ndarray:
    eps = rand_normal(seed, 4, np.arange(n, dtype=np.uint64))
    if rho > 0.0:
        z = np.empty(n)
        z[0] = eps[0]
        k = np.sqrt(1.0 - rho * rho)
        for i in range(1, n):
            z[i] = rho * z[i - 1] + k * eps[i]
    else:
        z = eps
    return np.clip(median * np.exp(sigma * z), lo, hi)


def _diurnal_trace(seed: int, n: int) -> np.ndarray:
    """One rate per second of a day: sinusoid 20..400 rps plus Poisson spikes.

    Spikes arrive as a Poisson process (mean 48 per day); each multiplies the
    base rate by U[3, 10] for U{30..120} seconds; overlapping spikes take the
    largest multiplier.
    """
    day = 86400
    i = np.arange(n, dtype=np.float64)
    base = 210.0 - 190.0 * np.cos(2.0 * np.pi * i / day)
    mult = np.ones(n)
    k = np.arange(256, dtype=np.uint64)
    gaps = -np.log1p(-rand_uniform(seed, 5, k)) * (day / 48.0)
    starts = np.floor(np.cumsum(gaps)).astype(np.int64)
    factor = rand_uniform(seed, 6, k, 3.0, 10.0)
    dur = rand_int(seed, 7, k, 30, 120)
    for s0, f, d in zip(starts, factor, dur):
        if s0 >= n:
            break
        e = min(n, s0 + int(d))
        mult[s0:e] = np.maximum(mult[s0:e], f)
    return base * mult


_CONFIGS = {
    # name, N, S, P, C, B, H, slo_us, w_us, vertical, beta range
    1: dict(name="tiny_joint", N=64, S=3, P=64, C=8, B=(1, 2, 4, 8), H=4,
            slo_us=500_000, w_us=1000, vertical=False, beta=(5.0, 40.0)),
    2: dict(name="joint", N=4096, S=5, P=64, C=16, B=(1, 2, 4, 8, 16, 32), H=16,
            slo_us=1_000_000, w_us=1000, vertical=False, beta=(5.0, 40.0)),
    3: dict(name="vertical_day_trace", N=86400, S=10, P=1, C=32, B=(1, 2, 4, 8, 16, 32), H=8,
            slo_us=800_000, w_us=1000, vertical=True, beta=(5.0, 40.0)),
    4: dict(name="large_joint", N=16384, S=8, P=64, C=64, B=(1, 2, 4, 8, 16, 32, 64), H=32,
            slo_us=2_000_000, w_us=500, vertical=False, beta=(2.0, 60.0)),
    5: dict(name="stress_joint", N=4096, S=20, P=16, C=64, B=(1, 2, 4, 8, 16, 32, 64, 128), H=64,
            slo_us=4_096_000, w_us=500, vertical=False, beta=(2.0, 60.0)),
}


def config_names() -> dict:
    return {k: v["name"] for k, v in _CONFIGS.items()}


def make_workload(cfg: int, n_instances: Optional[int] = None, seed_offset: int = 0) -> Workload:
    """Build benchmark configuration ``cfg`` (1..5).

    ``n_instances`` overrides the batch size (the first instances of the same
    random streams).  ``seed_offset`` selects an independent replica of the
    workload (used to give every rank of a multi-GPU run its own batch).
    """
    spec = _CONFIGS[cfg]
    seed = BASE_SEED + cfg + 1000003 * seed_offset
    N = spec["N"] if n_instances is None else int(n_instances)
    S, P, C, B, H = spec["S"], spec["P"], spec["C"], spec["B"], spec["H"]
    lat = latency_tables(seed, P, S, C, B, *spec["beta"])
    if cfg == 1:
        rate = rand_uniform(seed, 4, np.arange(N, dtype=np.uint64), 5.0, 50.0)
    elif cfg == 2:
        rate = _lognormal_rates(seed, N, 100.0, 0.8, 1.0, 2000.0, rho=0.9)
    elif cfg == 3:
        rate = _diurnal_trace(seed, N)
    elif cfg == 4:
        rate = _lognormal_rates(seed, N, 300.0, 0.8, 1.0, 6000.0)
    else:
        rate = _lognormal_rates(seed, N, 1000.0, 1.0, 1.0, 20000.0)
    replicas = None
    if spec["vertical"]:
        per_stage = rand_int(seed, 8, np.arange(S, dtype=np.uint64), 1, H).astype(np.int32)
        replicas = np.ascontiguousarray(np.broadcast_to(per_stage, (N, S)))
    return Workload(
        name=spec["name"], n_instances=N, n_stages=S, n_profiles=P, c_max=C,
        batch_sizes=tuple(B), h_max=H, slo_us=spec["slo_us"], bucket_us=spec["w_us"],
        flags=QUEUE_PER_REPLICA, vertical=spec["vertical"], lat_us=lat,
        profile_id=(np.arange(N, dtype=np.int64) % P).astype(np.int32),
        lambda_mrps=_to_mrps(rate), replicas=replicas, seed=seed)


def paper_scale_workload(n_instances: int = 32) -> Workload:
    """A pipeline of the size the paper has in mind (Section "Optimizer":
    batch sizes 1..16, cores 1..16, SLO of a few thousand ms; Table
    "Applications": three stages, SLO 2550 ms; arrival rates 2..12 rps),
    vertical-only with one replica per stage, queue delay as in Eq. 4."""
    seed = BASE_SEED + 99
    S, C = 3, 16
    B = tuple(range(1, 17))
    lat = latency_tables(seed, 1, S, C, B, 20.0, 120.0)
    rate = rand_uniform(seed, 4, np.arange(n_instances, dtype=np.uint64), 2.0, 12.0)
    return Workload(
        name="paper_scale_vertical", n_instances=n_instances, n_stages=S, n_profiles=1, c_max=C,
        batch_sizes=B, h_max=1, slo_us=2_550_000, bucket_us=1000, flags=0, vertical=True,
        lat_us=lat, profile_id=np.zeros(n_instances, np.int32), lambda_mrps=_to_mrps(rate),
        replicas=np.ones((n_instances, S), np.int32), seed=seed)


def random_tiny_workload(seed: int, n_instances: int, n_stages: int, c_max: int,
                         batch_sizes: Sequence[int], h_max: int, T: int, bucket_us: int = 1000,
                         flags: int = QUEUE_PER_REPLICA, vertical: bool = False,
                         rate_lo: float = 5.0, rate_hi: float = 50.0) -> Workload:
    """Small random instances (one profile per instance) for exhaustive checks."""
    lat = latency_tables(seed, n_instances, n_stages, c_max, batch_sizes)
    rate = rand_uniform(seed, 4, np.arange(n_instances, dtype=np.uint64), rate_lo, rate_hi)
    replicas = None
    if vertical:
        replicas = rand_int(seed, 8, np.arange(n_instances * n_stages, dtype=np.uint64), 1, h_max)
        replicas = replicas.reshape(n_instances, n_stages).astype(np.int32)
    return Workload(
        name=f"tiny_random_{seed}", n_instances=n_instances, n_stages=n_stages,
        n_profiles=n_instances, c_max=c_max, batch_sizes=tuple(batch_sizes), h_max=h_max,
        slo_us=T * bucket_us, bucket_us=bucket_us, flags=flags, vertical=vertical, lat_us=lat,
        profile_id=np.arange(n_instances, dtype=np.int32), lambda_mrps=_to_mrps(rate),
        replicas=replicas, seed=seed)


def profile_samples(seed: int, n_models: int, noise: float = 0.02):
    """Synthetic profiling runs for the Eq. 1 fit: every model is "measured" on the
    grid b in {1,2,4,8,16} x c in {1,2,4,8,16}; its true coefficients are drawn
    gamma~U[5,40], epsilon~U[2,20], delta~U[0.1,2], eta~U[1,10] (milliseconds) and
    each measurement carries multiplicative log-normal noise.  Returns
    (sample_b int32 [25], sample_c int32 [25], latency_ms float64 [M][25], true coeffs [M][4])."""
    grid = (1, 2, 4, 8, 16)
    sample_b = np.repeat(np.asarray(grid, np.int32), len(grid))
    sample_c = np.tile(np.asarray(grid, np.int32), len(grid))
    m = np.arange(n_models, dtype=np.uint64)
    true = np.stack([rand_uniform(seed, 11, m, 5.0, 40.0), rand_uniform(seed, 12, m, 2.0, 20.0),
                     rand_uniform(seed, 13, m, 0.1, 2.0), rand_uniform(seed, 14, m, 1.0, 10.0)], axis=1)
    b, c = sample_b.astype(np.float64), sample_c.astype(np.float64)
    clean = (true[:, 0:1] * b / c + true[:, 1:2] / c + true[:, 2:3] * b + true[:, 3:4])
    z = rand_normal(seed, 15, np.arange(n_models * b.size, dtype=np.uint64)).reshape(n_models, b.size)
    return sample_b, sample_c, clean * np.exp(noise * z), true


def arbitrary_tables_workload(seed: int, n_instances: int, n_stages: int, c_max: int,
                              batch_sizes: Sequence[int], h_max: int, T: int, bucket_us: int,
                              flags: int, vertical: bool, lat_lo_us: int = 700, lat_hi_us: int = 90_000,
                              rate_lo: float = 3.0, rate_hi: float = 400.0, repeat_prob: float = 0.3) -> Workload:
    """Instances whose latency tables follow no model at all: every entry is an
    independent draw in [lat_lo_us, lat_hi_us] microseconds (not monotone in cores or
    batch size, not multiples of the bucket), with a share of entries copied from the
    neighbouring core count so that equal latencies occur.  For robustness checks."""
    shape = (n_instances, n_stages, c_max, len(batch_sizes))
    idx = np.arange(int(np.prod(shape)), dtype=np.uint64)
    lat = rand_int(seed, 21, idx, lat_lo_us, lat_hi_us).reshape(shape)
    copy = rand_uniform(seed, 22, idx).reshape(shape) < repeat_prob
    for c in range(1, c_max):
        lat[:, :, c, :] = np.where(copy[:, :, c, :], lat[:, :, c - 1, :], lat[:, :, c, :])
    rate = rand_uniform(seed, 4, np.arange(n_instances, dtype=np.uint64), rate_lo, rate_hi)
    replicas = None
    if vertical:
        replicas = rand_int(seed, 8, np.arange(n_instances * n_stages, dtype=np.uint64), 1, h_max)
        replicas = replicas.reshape(n_instances, n_stages).astype(np.int32)
    return Workload(
        name=f"arbitrary_{seed}", n_instances=n_instances, n_stages=n_stages, n_profiles=n_instances,
        c_max=c_max, batch_sizes=tuple(batch_sizes), h_max=h_max, slo_us=T * bucket_us, bucket_us=bucket_us,
        flags=flags, vertical=vertical, lat_us=np.ascontiguousarray(lat.astype(np.int32)),
        profile_id=np.arange(n_instances, dtype=np.int32), lambda_mrps=_to_mrps(rate), replicas=replicas, seed=seed)
