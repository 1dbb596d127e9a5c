"""CPU oracle for the batched pipeline-scaling solver: ctypes access to the C files here.

TEST INFRASTRUCTURE ONLY.  Nothing in the product package may import this
module; it exists so that tests, the smoke check and the benchmark's CPU
baseline can compare the CUDA path against a plain restatement of the
method (Themis, arXiv 2407.14843: Eq. 4-6 and Algorithm 1).  It imports
nothing from the CUDA package.

``build()`` compiles ``themis_oracle.c`` and ``brute_force.c`` with gcc into
``oracle/_build/liboracle.so`` (rebuilt when a source is newer).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SOURCES = [os.path.join(_HERE, "themis_oracle.c"), os.path.join(_HERE, "brute_force.c")]
_LIB_PATH = os.path.join(_HERE, "_build", "liboracle.so")
_lib = None

INF = np.iinfo(np.int32).max
QUEUE_PER_REPLICA = 1


class _Problem(ctypes.Structure):
    _fields_ = [("n_instances", ctypes.c_int32), ("n_stages", ctypes.c_int32),
                ("n_profiles", ctypes.c_int32), ("c_max", ctypes.c_int32),
                ("n_batch", ctypes.c_int32), ("batch_sizes", ctypes.c_int32 * 16),
                ("h_max", ctypes.c_int32), ("slo_us", ctypes.c_int32),
                ("bucket_us", ctypes.c_int32), ("flags", ctypes.c_uint32)]


def build(force: bool = False) -> str:
    """Compile the C oracle if needed and return the library path."""
    os.makedirs(os.path.dirname(_LIB_PATH), exist_ok=True)
    stale = force or not os.path.exists(_LIB_PATH) or any(
        os.path.getmtime(s) > os.path.getmtime(_LIB_PATH) for s in _SOURCES)
    if stale:
        tmp = _LIB_PATH + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
                               "-Wall", "-Wextra", "-o", tmp] + _SOURCES)
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        P = ctypes.POINTER(_Problem)
        vp = ctypes.c_void_p
        lib.oracle_solve_batch.restype = ctypes.c_int
        lib.oracle_solve_batch.argtypes = [P] + [vp] * 14 + [ctypes.c_int]
        lib.oracle_score_stage.restype = None
        lib.oracle_score_stage.argtypes = [P, vp, ctypes.c_uint32, ctypes.c_int32, ctypes.c_int32, vp, vp]
        lib.oracle_minplus.restype = None
        lib.oracle_minplus.argtypes = [ctypes.c_int32, vp, vp, vp, vp]
        lib.oracle_solve_horizontal_batch.restype = ctypes.c_int
        lib.oracle_solve_horizontal_batch.argtypes = [P] + [vp] * 13 + [ctypes.c_int]
        lib.oracle_vertical_fallback_batch.restype = ctypes.c_int
        lib.oracle_vertical_fallback_batch.argtypes = [P, vp, vp, vp, vp, ctypes.c_uint32] + [vp] * 8 + [ctypes.c_int]
        for fn in (lib.oracle_alg1_scatter, lib.oracle_alg2_scatter, lib.brute_force_instance):
            fn.restype = ctypes.c_int
            fn.argtypes = [P, vp, ctypes.c_uint32, vp, vp, vp, vp, vp, vp]
        _lib = lib
    return _lib


def _problem(n_instances, n_stages, n_profiles, c_max, batch_sizes, h_max, slo_us, bucket_us, flags):
    p = _Problem()
    p.n_instances, p.n_stages, p.n_profiles = int(n_instances), int(n_stages), int(n_profiles)
    p.c_max, p.n_batch, p.h_max = int(c_max), len(batch_sizes), int(h_max)
    for i, b in enumerate(batch_sizes):
        p.batch_sizes[i] = int(b)
    p.slo_us, p.bucket_us, p.flags = int(slo_us), int(bucket_us), int(flags)
    return p


def _problem_of(wl, n_instances=None):
    return _problem(wl.n_instances if n_instances is None else n_instances, wl.n_stages,
                    wl.n_profiles, wl.c_max, wl.batch_sizes, wl.h_max, wl.slo_us, wl.bucket_us, wl.flags)


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    return None if a is None else np.ascontiguousarray(a, dtype=dtype)


def solve_batch(wl, dumps: bool = False, n_threads: int = 0, horizontal: bool = False) -> dict:
    """Solve every instance of a workload (any object with the attributes of
    ``workloads.Workload``) with the dynamic-programming oracle.
    ``horizontal`` selects Algorithm 2 (one-core replicas, replica count
    computed per batch size, at most ``h_max``); the workload must have c_max 1.

    Returns numpy arrays ``h, c, b`` [N][S], ``total_cost, latency_buckets,
    status`` [N] and ``threads``; with ``dumps`` also ``G, Garg, F, A``
    [N][S][T+1] (memory: 12 * N * S * (T+1) bytes).
    """
    lib = _load()
    N, S, W = wl.n_instances, wl.n_stages, wl.slo_us // wl.bucket_us + 1
    p = _problem_of(wl)
    lat = _c(wl.lat_us, np.int32)
    pid = _c(wl.profile_id, np.int32)
    lam = _c(wl.lambda_mrps, np.uint32)
    rep = _c(wl.replicas, np.int32) if wl.vertical else None
    out = {k: np.zeros((N, S), np.int32) for k in ("h", "c", "b")}
    out.update({k: np.zeros(N, np.int32) for k in ("total_cost", "latency_buckets", "status")})
    if dumps:
        out["G"] = np.empty((N, S, W), np.int32)
        out["Garg"] = np.empty((N, S, W), np.uint16)
        out["F"] = np.empty((N, S, W), np.int32)
        out["A"] = np.empty((N, S, W), np.uint16)
    tail = (_ptr(out["h"]), _ptr(out["c"]), _ptr(out["b"]),
            _ptr(out["total_cost"]), _ptr(out["latency_buckets"]), _ptr(out["status"]),
            _ptr(out.get("G")), _ptr(out.get("Garg")), _ptr(out.get("F")), _ptr(out.get("A")),
            int(n_threads))
    if horizontal:
        rc = lib.oracle_solve_horizontal_batch(ctypes.byref(p), _ptr(lat), _ptr(pid), _ptr(lam), *tail)
    else:
        rc = lib.oracle_solve_batch(ctypes.byref(p), _ptr(lat), _ptr(pid), _ptr(lam), _ptr(rep), *tail)
    if rc < 0:
        raise MemoryError("oracle_solve_batch: allocation failed or unsupported problem")
    out["threads"] = rc
    return out


def vertical_fallback_batch(wl, resolution_mrps: int = 1000, n_threads: int = 0) -> dict:
    """Algorithm 1 with its last branch: instances the replicas in place cannot
    serve are split into the largest rate found by bisection that vertical
    scaling serves plus extra replicas for the rest.  Returns the arrays of
    ``solve_batch`` (status 2 = split) plus ``lambda_vertical`` [N] and
    ``extra_replicas`` [N][S]."""
    lib = _load()
    N, S = wl.n_instances, wl.n_stages
    p = _problem_of(wl)
    lat, pid = _c(wl.lat_us, np.int32), _c(wl.profile_id, np.int32)
    lam, rep = _c(wl.lambda_mrps, np.uint32), _c(wl.replicas, np.int32)
    out = {k: np.zeros((N, S), np.int32) for k in ("h", "c", "b", "extra_replicas")}
    out.update({k: np.zeros(N, np.int32) for k in ("total_cost", "latency_buckets", "status")})
    out["lambda_vertical"] = np.zeros(N, np.uint32)
    rc = lib.oracle_vertical_fallback_batch(
        ctypes.byref(p), _ptr(lat), _ptr(pid), _ptr(lam), _ptr(rep), int(resolution_mrps),
        _ptr(out["h"]), _ptr(out["c"]), _ptr(out["b"]), _ptr(out["total_cost"]),
        _ptr(out["latency_buckets"]), _ptr(out["status"]), _ptr(out["lambda_vertical"]),
        _ptr(out["extra_replicas"]), int(n_threads))
    if rc < 0:
        raise RuntimeError("oracle_vertical_fallback_batch failed")
    out["threads"] = rc
    return out


def _per_instance(fn, wl, n: int) -> dict:
    S = wl.n_stages
    p = _problem_of(wl, 1)
    pid = int(wl.profile_id[n])
    lat = np.ascontiguousarray(wl.lat_us[pid], dtype=np.int32)
    rep = np.ascontiguousarray(wl.replicas[n], dtype=np.int32) if wl.vertical else None
    h, c, b = (np.zeros(S, np.int32) for _ in range(3))
    cost, lat_b = np.zeros(1, np.int32), np.zeros(1, np.int32)
    rc = fn(ctypes.byref(p), _ptr(lat), int(wl.lambda_mrps[n]), _ptr(rep),
            _ptr(h), _ptr(c), _ptr(b), _ptr(cost), _ptr(lat_b))
    if rc < 0:
        raise RuntimeError("oracle: unsupported size or allocation failure")
    return {"h": h, "c": c, "b": b, "total_cost": int(cost[0]),
            "latency_buckets": int(lat_b[0]), "status": rc}


def alg1_scatter(wl, n: int) -> dict:
    """Instance ``n`` solved by forward relaxation over reachable (stage, budget) states in
    Algorithm 1's visiting order (no per-bucket minimum, no (min,+) combine)."""
    return _per_instance(_load().oracle_alg1_scatter, wl, n)


def alg2_scatter(wl, n: int) -> dict:
    """Instance ``n`` of Algorithm 2's problem (c_max = 1) solved by the same forward relaxation."""
    return _per_instance(_load().oracle_alg2_scatter, wl, n)


def brute_force(wl, n: int) -> dict:
    """Instance ``n`` solved by exhaustive enumeration of Eq. 6 (S <= 8)."""
    return _per_instance(_load().brute_force_instance, wl, n)


def score_stage(c_max: int, batch_sizes: Sequence[int], h_max: int, bucket_us: int, flags: int,
                lat_stage: np.ndarray, lambda_m: int, h_fixed: int, T: int):
    """Per-bucket candidate minimum of one stage: returns (G, Garg)."""
    p = _problem(1, 1, 1, c_max, batch_sizes, h_max, T * bucket_us, bucket_us, flags)
    lat = np.ascontiguousarray(lat_stage, dtype=np.int32)
    G = np.empty(T + 1, np.int32)
    Garg = np.empty(T + 1, np.uint16)
    _load().oracle_score_stage(ctypes.byref(p), _ptr(lat), int(lambda_m), int(h_fixed), int(T),
                               _ptr(G), _ptr(Garg))
    return G, Garg


def minplus(Fprev: np.ndarray, G: np.ndarray):
    """One min-plus combine: returns (F, A) with the lowest index winning ties."""
    Fp = np.ascontiguousarray(Fprev, dtype=np.int32)
    Gc = np.ascontiguousarray(G, dtype=np.int32)
    T = Fp.size - 1
    F = np.empty(T + 1, np.int32)
    A = np.empty(T + 1, np.uint16)
    _load().oracle_minplus(T, _ptr(Fp), _ptr(Gc), _ptr(F), _ptr(A))
    return F, A
