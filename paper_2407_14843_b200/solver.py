"""Python binding of ``libthemis.so``: argument marshalling only.

Every function here has the name of the C entry point it forwards to
(``include/themis.h``); tensors are passed as raw device (or host) pointers
and the current torch CUDA stream as the stream handle.  PyTorch is used for
device memory and streams, nothing else: every step of the solver runs in the
library's CUDA kernels.  There is no CPU fallback: if the library has not been
built, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libthemis.so")

QUEUE_PER_REPLICA = 1
# themis_problem_t.flags: kernel choice of a call (bits 8..11) and cells per thread (bits 12..13)
(KERNEL_DEFAULT, KERNEL_PACKED16, KERNEL_WIDE32, KERNEL_PRUNED, KERNEL_SPARSE, KERNEL_SPARSE_BLOCK,
 KERNEL_PACKED16_BLOCK) = (k << 8 for k in range(7))
KERNEL_MASK = 15 << 8
TILE_FLAGS = {0: 0 << 12, 4: 1 << 12, 8: 2 << 12, 16: 3 << 12}
OK, E_INVALID_ARG, E_UNSUPPORTED_SIZE, E_WORKSPACE_TOO_SMALL, E_CUDA = 0, -1, -2, -3, -4
E_STATIC_SCRATCH_EXCEEDED = -5
STATIC_SCRATCH_BYTES = 32 << 20
STATUS_OK, STATUS_INFEASIBLE, STATUS_BAD_INPUT, STATUS_TIMEOUT = 0, 1, -1, -2
STATUS_SPLIT = 2
G_INF = 2 ** 31 - 1
MAX_T = 16383
INF16 = 0x7FFF

EXPORTS = (
    "themis_version", "themis_strerror", "themis_workspace_bytes", "themis_workspace_layout",
    "themis_solve_batch", "themis_solve_vertical_batch", "themis_score_batch", "themis_minplus_batch",
    "themis_host_workspace_bytes", "themis_solve_batch_host", "themis_solve_batch_static",
    "themis_solve_horizontal_batch", "themis_fallback_workspace_bytes", "themis_vertical_fallback_batch",
    "themis_fit_profiles_batch", "themis_configs_equal_batch",
)
# include/themis_probe.h: measurement probes, not part of the solver
PROBE_EXPORTS = ("themis_alu_probe", "themis_wait_probe", "themis_bounds_check_report")


class ThemisError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {themis_strerror(code)} ({code})")


class Problem(ctypes.Structure):
    """Mirror of ``themis_problem_t``."""
    _fields_ = [("n_instances", ctypes.c_int32), ("n_stages", ctypes.c_int32),
                ("n_profiles", ctypes.c_int32), ("c_max", ctypes.c_int32),
                ("n_batch", ctypes.c_int32), ("batch_sizes", ctypes.c_int32 * 16),
                ("h_max", ctypes.c_int32), ("slo_us", ctypes.c_int32),
                ("bucket_us", ctypes.c_int32), ("flags", ctypes.c_uint32)]

    @classmethod
    def make(cls, n_instances: int, n_stages: int, n_profiles: int, c_max: int,
             batch_sizes: Sequence[int], h_max: int, slo_us: int, bucket_us: int, flags: int = 0) -> "Problem":
        p = cls()
        p.n_instances, p.n_stages, p.n_profiles = n_instances, n_stages, n_profiles
        p.c_max, p.h_max, p.slo_us, p.bucket_us, p.flags = c_max, h_max, slo_us, bucket_us, flags
        p.n_batch = len(batch_sizes)
        for i, b in enumerate(list(batch_sizes)[:16]):
            p.batch_sizes[i] = int(b)
        return p

    @classmethod
    def of_workload(cls, wl, kernel: int = KERNEL_DEFAULT, tile: int = 0) -> "Problem":
        """``kernel``: one of the ``KERNEL_*`` flag values; ``tile``: 0, 4, 8 or 16 cells per thread."""
        return cls.make(wl.n_instances, wl.n_stages, wl.n_profiles, wl.c_max, wl.batch_sizes,
                        wl.h_max, wl.slo_us, wl.bucket_us, wl.flags | kernel | TILE_FLAGS[tile])


class Result(ctypes.Structure):
    """Mirror of ``themis_result_t`` (raw pointers)."""
    _fields_ = [(k, ctypes.c_void_p) for k in ("h", "c", "b", "total_cost", "latency_buckets", "status")]


class WorkspaceLayout(ctypes.Structure):
    """Mirror of ``themis_workspace_layout_t``."""
    _fields_ = [("g_offset", ctypes.c_size_t), ("garg_offset", ctypes.c_size_t),
                ("a_offset", ctypes.c_size_t), ("f_offset", ctypes.c_size_t),
                ("flag_offset", ctypes.c_size_t), ("total_bytes", ctypes.c_size_t),
                ("row_pitch", ctypes.c_int32), ("T", ctypes.c_int32)]


def _load(path: str = LIB_PATH) -> ctypes.CDLL:
    if not os.path.exists(path):
        raise ImportError(
            f"{path} is missing: build it with `python -m paper_2407_14843_b200.build` "
            "(there is no fallback implementation)")
    lib = ctypes.CDLL(path)
    PP, vp, sz = ctypes.POINTER(Problem), ctypes.c_void_p, ctypes.c_size_t
    lib.themis_version.restype = ctypes.c_int
    lib.themis_version.argtypes = []
    lib.themis_strerror.restype = ctypes.c_char_p
    lib.themis_strerror.argtypes = [ctypes.c_int]
    lib.themis_workspace_bytes.argtypes = [PP, ctypes.c_int, ctypes.POINTER(sz)]
    lib.themis_host_workspace_bytes.argtypes = [PP, ctypes.c_int, ctypes.POINTER(sz)]
    lib.themis_workspace_layout.argtypes = [PP, ctypes.c_int, ctypes.POINTER(WorkspaceLayout)]
    lib.themis_solve_batch.argtypes = [PP, vp, vp, vp, Result, vp, sz, vp]
    lib.themis_solve_vertical_batch.argtypes = [PP, vp, vp, vp, vp, Result, vp, sz, vp]
    lib.themis_fallback_workspace_bytes.argtypes = [PP, ctypes.POINTER(sz)]
    lib.themis_vertical_fallback_batch.argtypes = [PP, vp, vp, vp, vp, ctypes.c_uint32, ctypes.c_uint32, Result,
                                                   vp, vp, vp, sz, vp]
    lib.themis_solve_horizontal_batch.argtypes = [PP, vp, vp, vp, Result, vp, sz, vp]
    lib.themis_score_batch.argtypes = [PP, vp, vp, vp, vp, vp, sz, vp]
    lib.themis_minplus_batch.argtypes = [PP, vp, Result, vp, sz, vp]
    lib.themis_solve_batch_host.argtypes = [PP, vp, vp, vp, vp, Result, vp, sz, vp]
    lib.themis_solve_batch_static.argtypes = [PP, vp, vp, vp, vp, Result, vp]
    lib.themis_configs_equal_batch.argtypes = [ctypes.c_int32, ctypes.c_int32, Result, Result, vp, vp]
    lib.themis_fit_profiles_batch.argtypes = [ctypes.c_int32, ctypes.c_int32, vp, vp, vp, ctypes.c_int32,
                                              ctypes.c_int32, vp, vp, vp, vp, vp]
    lib.themis_alu_probe.argtypes = [ctypes.c_int] * 4 + [vp, vp]
    lib.themis_wait_probe.argtypes = [ctypes.c_int32, vp, vp, vp, vp]
    lib.themis_bounds_check_report.argtypes = [PP, ctypes.c_int, vp, sz, ctypes.POINTER(ctypes.c_int32 * 4), vp]
    for name in EXPORTS + PROBE_EXPORTS:
        if name != "themis_strerror":
            getattr(lib, name).restype = ctypes.c_int
    return lib


_lib = _load()


def _check(rc: int, where: str) -> None:
    if rc != OK:
        raise ThemisError(rc, where)


def _dptr(t: Optional[torch.Tensor], dtype: torch.dtype, what: str, cuda: bool = True):
    if t is None:
        return None
    if t.dtype != dtype or not t.is_contiguous() or t.is_cuda != cuda:
        raise TypeError(f"{what}: expected a contiguous {'cuda' if cuda else 'cpu'} tensor of {dtype}")
    return ctypes.c_void_p(t.data_ptr())


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _result(out: dict, cuda: bool = True) -> Result:
    r = Result()
    for k in ("h", "c", "b", "total_cost", "latency_buckets", "status"):
        setattr(r, k, _dptr(out[k], torch.int32, f"out[{k!r}]", cuda).value)
    return r


def themis_version() -> int:
    return _lib.themis_version()


def themis_strerror(code: int) -> str:
    return _lib.themis_strerror(code).decode()


def themis_workspace_bytes(problem: Problem, vertical: bool) -> int:
    n = ctypes.c_size_t()
    _check(_lib.themis_workspace_bytes(ctypes.byref(problem), int(vertical), ctypes.byref(n)),
           "themis_workspace_bytes")
    return n.value


def themis_host_workspace_bytes(problem: Problem, vertical: bool) -> int:
    n = ctypes.c_size_t()
    _check(_lib.themis_host_workspace_bytes(ctypes.byref(problem), int(vertical), ctypes.byref(n)),
           "themis_host_workspace_bytes")
    return n.value


def themis_workspace_layout(problem: Problem, vertical: bool) -> WorkspaceLayout:
    lay = WorkspaceLayout()
    _check(_lib.themis_workspace_layout(ctypes.byref(problem), int(vertical), ctypes.byref(lay)),
           "themis_workspace_layout")
    return lay


def themis_solve_batch(problem: Problem, lat_us, profile_id, lambda_mrps, out: dict, workspace) -> None:
    _check(_lib.themis_solve_batch(
        ctypes.byref(problem), _dptr(lat_us, torch.int32, "lat_us"), _dptr(profile_id, torch.int32, "profile_id"),
        _dptr(lambda_mrps, torch.uint32, "lambda_mrps"), _result(out),
        _dptr(workspace, torch.uint8, "workspace"), workspace.numel(), _stream()), "themis_solve_batch")


def themis_solve_vertical_batch(problem: Problem, lat_us, profile_id, lambda_mrps, replicas, out: dict,
                                workspace) -> None:
    _check(_lib.themis_solve_vertical_batch(
        ctypes.byref(problem), _dptr(lat_us, torch.int32, "lat_us"), _dptr(profile_id, torch.int32, "profile_id"),
        _dptr(lambda_mrps, torch.uint32, "lambda_mrps"), _dptr(replicas, torch.int32, "replicas"), _result(out),
        _dptr(workspace, torch.uint8, "workspace"), workspace.numel(), _stream()), "themis_solve_vertical_batch")


def themis_fallback_workspace_bytes(problem: Problem) -> int:
    n = ctypes.c_size_t()
    _check(_lib.themis_fallback_workspace_bytes(ctypes.byref(problem), ctypes.byref(n)),
           "themis_fallback_workspace_bytes")
    return n.value


def themis_vertical_fallback_batch(problem: Problem, lat_us, profile_id, lambda_mrps, replicas,
                                   resolution_mrps: int, lambda_max_mrps: int, out: dict,
                                   lambda_vertical, extra_replicas, workspace) -> None:
    _check(_lib.themis_vertical_fallback_batch(
        ctypes.byref(problem), _dptr(lat_us, torch.int32, "lat_us"), _dptr(profile_id, torch.int32, "profile_id"),
        _dptr(lambda_mrps, torch.uint32, "lambda_mrps"), _dptr(replicas, torch.int32, "replicas"),
        int(resolution_mrps), int(lambda_max_mrps), _result(out),
        _dptr(lambda_vertical, torch.uint32, "lambda_vertical"), _dptr(extra_replicas, torch.int32, "extra_replicas"),
        _dptr(workspace, torch.uint8, "workspace"), workspace.numel(), _stream()), "themis_vertical_fallback_batch")


def themis_solve_horizontal_batch(problem: Problem, lat_us, profile_id, lambda_mrps, out: dict, workspace) -> None:
    _check(_lib.themis_solve_horizontal_batch(
        ctypes.byref(problem), _dptr(lat_us, torch.int32, "lat_us"), _dptr(profile_id, torch.int32, "profile_id"),
        _dptr(lambda_mrps, torch.uint32, "lambda_mrps"), _result(out),
        _dptr(workspace, torch.uint8, "workspace"), workspace.numel(), _stream()), "themis_solve_horizontal_batch")


def themis_score_batch(problem: Problem, lat_us, profile_id, lambda_mrps, replicas, workspace) -> None:
    _check(_lib.themis_score_batch(
        ctypes.byref(problem), _dptr(lat_us, torch.int32, "lat_us"), _dptr(profile_id, torch.int32, "profile_id"),
        _dptr(lambda_mrps, torch.uint32, "lambda_mrps"), _dptr(replicas, torch.int32, "replicas"),
        _dptr(workspace, torch.uint8, "workspace"), workspace.numel(), _stream()), "themis_score_batch")


def themis_minplus_batch(problem: Problem, replicas, out: dict, workspace) -> None:
    _check(_lib.themis_minplus_batch(
        ctypes.byref(problem), _dptr(replicas, torch.int32, "replicas"), _result(out),
        _dptr(workspace, torch.uint8, "workspace"), workspace.numel(), _stream()), "themis_minplus_batch")


def themis_solve_batch_host(problem: Problem, lat_us, profile_id, lambda_mrps, replicas, out: dict,
                            workspace) -> None:
    """Inputs and ``out`` are CPU tensors (pinned for asynchronous copies)."""
    _check(_lib.themis_solve_batch_host(
        ctypes.byref(problem), _dptr(lat_us, torch.int32, "lat_us", False),
        _dptr(profile_id, torch.int32, "profile_id", False),
        _dptr(lambda_mrps, torch.uint32, "lambda_mrps", False), _dptr(replicas, torch.int32, "replicas", False),
        _result(out, cuda=False), _dptr(workspace, torch.uint8, "workspace"), workspace.numel(), _stream()),
        "themis_solve_batch_host")


def themis_solve_batch_static(problem: Problem, lat_us, profile_id, lambda_mrps, replicas, out: dict) -> None:
    """Solver variant that needs no workspace from the caller: the tables live
    in a 32 MiB buffer inside the library (for callers that cannot allocate
    device memory).  Problems whose ``themis_workspace_bytes`` exceeds
    ``STATIC_SCRATCH_BYTES`` raise ``ThemisError`` with
    ``E_STATIC_SCRATCH_EXCEEDED``.  All calls share that buffer, so keep them
    on one stream; make the first call on a device outside stream capture."""
    _check(_lib.themis_solve_batch_static(
        ctypes.byref(problem), _dptr(lat_us, torch.int32, "lat_us"), _dptr(profile_id, torch.int32, "profile_id"),
        _dptr(lambda_mrps, torch.uint32, "lambda_mrps"), _dptr(replicas, torch.int32, "replicas"), _result(out),
        _stream()), "themis_solve_batch_static")


def themis_configs_equal_batch(current: dict, predicted: dict, stable) -> None:
    """``stable[n] = 1`` iff both result sets are solved and equal at every stage."""
    n, s = current["h"].shape
    _check(_lib.themis_configs_equal_batch(n, s, _result(current), _result(predicted),
                                           _dptr(stable, torch.int32, "stable"), _stream()),
           "themis_configs_equal_batch")


def themis_fit_profiles_batch(sample_b, sample_c, latency_ms, c_max: int, batch_sizes, coeffs, lat_us, status) -> None:
    """Eq. 1 fit for ``latency_ms.shape[0]`` models; all arguments are CUDA tensors
    (``batch_sizes`` int32 on the device)."""
    n_models, n_samples = latency_ms.shape
    _check(_lib.themis_fit_profiles_batch(
        n_models, n_samples, _dptr(sample_b, torch.int32, "sample_b"), _dptr(sample_c, torch.int32, "sample_c"),
        _dptr(latency_ms, torch.float64, "latency_ms"), int(c_max), batch_sizes.numel(),
        _dptr(batch_sizes, torch.int32, "batch_sizes"), _dptr(coeffs, torch.float64, "coeffs"),
        _dptr(lat_us, torch.int32, "lat_us"), _dptr(status, torch.int32, "status"), _stream()),
        "themis_fit_profiles_batch")


def themis_alu_probe(mode: int, blocks: int, threads: int, iters: int, sink) -> None:
    if sink.numel() < blocks * threads:
        raise ValueError("sink too small")
    _check(_lib.themis_alu_probe(mode, blocks, threads, iters, _dptr(sink, torch.uint32, "sink"), _stream()),
           "themis_alu_probe")


def themis_bounds_check_report(problem: Problem, vertical: bool, workspace) -> dict:
    """Record of the bounds-checked build for the last solve on ``workspace`` (waits for the
    stream): ``{"site", "index", "limit", "checked"}``; all zero with the normal library."""
    rep = (ctypes.c_int32 * 4)()
    _check(_lib.themis_bounds_check_report(ctypes.byref(problem), int(vertical),
                                           _dptr(workspace, torch.uint8, "workspace"), workspace.numel(),
                                           ctypes.byref(rep), _stream()), "themis_bounds_check_report")
    return {"site": rep[0], "index": rep[1], "limit": rep[2], "checked": bool(rep[3])}


def use_library(path: str = LIB_PATH) -> None:
    """Routes every call of this module to the library at ``path`` (the normal one by default;
    ``build.CHECK_LIB_PATH`` for the bounds-checked build)."""
    global _lib
    _lib = _load(path)


def themis_wait_probe(max_polls: int, src16, dst16, status) -> None:
    _check(_lib.themis_wait_probe(max_polls, _dptr(src16, torch.uint32, "src16"), _dptr(dst16, torch.uint32, "dst16"),
                                  _dptr(status, torch.int32, "status"), _stream()), "themis_wait_probe")


# --- plumbing helpers (allocation and copies only) ---------------------------

def alloc_result(n_instances: int, n_stages: int, device="cuda", pin: bool = False) -> dict:
    """Result tensors of the shapes ``themis_result_t`` expects."""
    kw = dict(dtype=torch.int32, device=device)
    if pin and device == "cpu":
        kw["pin_memory"] = True
    out = {k: torch.empty((n_instances, n_stages), **kw) for k in ("h", "c", "b")}
    out.update({k: torch.empty(n_instances, **kw) for k in ("total_cost", "latency_buckets", "status")})
    return out


def alloc_workspace(problem: Problem, vertical: bool, host_variant: bool = False) -> torch.Tensor:
    n = themis_host_workspace_bytes(problem, vertical) if host_variant else themis_workspace_bytes(problem, vertical)
    return torch.empty(n, dtype=torch.uint8, device="cuda")


def workload_to_device(wl, device="cuda") -> dict:
    """Copies a ``workloads.Workload``'s arrays to the device."""
    d = {"lat_us": torch.from_numpy(wl.lat_us).to(device),
         "profile_id": torch.from_numpy(wl.profile_id).to(device),
         "lambda_mrps": torch.from_numpy(wl.lambda_mrps).to(device),
         "replicas": torch.from_numpy(wl.replicas).to(device) if wl.vertical else None}
    return d


def workspace_tables(problem: Problem, vertical: bool, workspace: torch.Tensor) -> dict:
    """Views of the intermediate tables G, Garg, A, F inside a workspace."""
    lay = themis_workspace_layout(problem, vertical)
    N, S, P = problem.n_instances, problem.n_stages, lay.row_pitch
    def view(off, dtype, shape):
        n = 1
        for s in shape:
            n *= s
        nbytes = n * torch.empty((), dtype=dtype).element_size()
        return workspace[off:off + nbytes].view(dtype).view(*shape)
    return {"G": view(lay.g_offset, torch.int32, (N, S, P)),
            "Garg": view(lay.garg_offset, torch.uint16, (N, S, P)),
            "A": view(lay.a_offset, torch.uint16, (N, S, P)),
            "F": view(lay.f_offset, torch.int32, (N, P)),
            "T": lay.T, "row_pitch": P}


def solve(wl, dev: Optional[dict] = None, workspace: Optional[torch.Tensor] = None,
          out: Optional[dict] = None, horizontal: bool = False, kernel: int = KERNEL_DEFAULT, tile: int = 0):
    """Solve a workload on the current device: allocates what is not given,
    then calls ``themis_solve_batch`` / ``themis_solve_vertical_batch`` (or
    ``themis_solve_horizontal_batch`` when ``horizontal``).  ``kernel`` and ``tile``
    go into the problem's flags (``KERNEL_*``; 0, 4, 8 or 16 cells per thread)."""
    problem = Problem.of_workload(wl, kernel, tile)
    dev = dev if dev is not None else workload_to_device(wl)
    workspace = workspace if workspace is not None else alloc_workspace(problem, wl.vertical)
    out = out if out is not None else alloc_result(wl.n_instances, wl.n_stages)
    if horizontal:
        themis_solve_horizontal_batch(problem, dev["lat_us"], dev["profile_id"], dev["lambda_mrps"], out, workspace)
    elif wl.vertical:
        themis_solve_vertical_batch(problem, dev["lat_us"], dev["profile_id"], dev["lambda_mrps"],
                                    dev["replicas"], out, workspace)
    else:
        themis_solve_batch(problem, dev["lat_us"], dev["profile_id"], dev["lambda_mrps"], out, workspace)
    return out, workspace
