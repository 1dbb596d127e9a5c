"""Host-side checks of the C ABI that need no GPU: the library loads, exports
every function the header declares, and rejects bad scalar arguments before
anything is launched."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def S():
    from paper_2407_14843_b200 import build
    build.build_library()
    from paper_2407_14843_b200 import solver
    return solver


def _good(S, **kw):
    args = dict(n_instances=4, n_stages=3, n_profiles=2, c_max=8, batch_sizes=(1, 2, 4, 8), h_max=4,
                slo_us=500_000, bucket_us=1000, flags=1)
    args.update(kw)
    return S.Problem.make(**args)


def _declared(header_name):
    header = open(os.path.join(ROOT, "include", header_name)).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    return set(re.findall(r"\b(themis_[a-z0-9_]+)\s*\(", header))


def test_every_declared_function_is_exported(S):
    """Both headers: the solver's (themis.h) and the measurement probes' (themis_probe.h)."""
    assert _declared("themis.h") == set(S.EXPORTS)
    assert _declared("themis_probe.h") == set(S.PROBE_EXPORTS)
    lib = ctypes.CDLL(S.LIB_PATH)
    for name in S.EXPORTS + S.PROBE_EXPORTS:
        assert hasattr(lib, name), name
    assert S.themis_version() == 100


def test_struct_mirrors_match_the_header(S):
    assert ctypes.sizeof(S.Problem) == 4 * (5 + 16 + 4)
    assert ctypes.sizeof(S.Result) == 6 * ctypes.sizeof(ctypes.c_void_p)
    assert ctypes.sizeof(S.WorkspaceLayout) == 6 * ctypes.sizeof(ctypes.c_size_t) + 8


def test_workspace_layout(S):
    p = _good(S, n_instances=10, n_stages=5, slo_us=1_000_000)
    lay = S.themis_workspace_layout(p, False)
    assert lay.T == 1000 and lay.row_pitch == 1024
    rows = 10 * 5 * 1024
    assert lay.g_offset == 0 and lay.garg_offset >= rows * 4
    assert lay.a_offset >= lay.garg_offset + rows * 2 and lay.f_offset >= lay.a_offset + rows * 2
    assert lay.total_bytes == S.themis_workspace_bytes(p, False)
    assert all(o % 256 == 0 for o in (lay.garg_offset, lay.a_offset, lay.f_offset, lay.flag_offset, lay.total_bytes))
    assert S.themis_host_workspace_bytes(p, False) > lay.total_bytes
    assert S.themis_host_workspace_bytes(p, True) > S.themis_host_workspace_bytes(p, False)


@pytest.mark.parametrize("kw,code", [
    (dict(n_instances=0), -1), (dict(n_stages=0), -1), (dict(n_profiles=0), -1), (dict(c_max=0), -1),
    (dict(batch_sizes=()), -1), (dict(batch_sizes=(1, 1)), -1), (dict(batch_sizes=(2, 1)), -1),
    (dict(batch_sizes=(0, 1)), -1), (dict(batch_sizes=(1, 70000)), -1), (dict(h_max=0), -1),
    (dict(slo_us=0), -1), (dict(bucket_us=0), -1), (dict(flags=2), -1),
    (dict(slo_us=999, bucket_us=1000), -1),                      # T = 0
    (dict(slo_us=16_384_000), -2),                                 # T > 16383
    (dict(n_stages=65), -2),
    (dict(c_max=64, h_max=64, batch_sizes=tuple(2 ** i for i in range(16))), -2),  # K > 65535
    (dict(n_stages=64, c_max=64, h_max=64, batch_sizes=(1,)), -2),                 # total cost bound
])
def test_invalid_problems_are_rejected_on_the_host(S, kw, code):
    p = _good(S, **kw)
    with pytest.raises(S.ThemisError) as e:
        S.themis_workspace_bytes(p, False)
    assert e.value.code == code
    # the solvers run the same validation before touching the device
    res = S.Result()
    rc = S._lib.themis_solve_batch(ctypes.byref(p), None, None, None, res, None, 0, None)
    assert rc == code


def test_max_sizes_are_accepted(S):
    p = _good(S, slo_us=16_383_000, n_stages=20, c_max=64, h_max=64, batch_sizes=tuple(2 ** i for i in range(8)))
    lay = S.themis_workspace_layout(p, False)
    assert lay.T == 16383 and lay.row_pitch == 16384
    assert S.themis_workspace_bytes(_good(S, h_max=0), True) > 0    # h_max is ignored by the vertical variant


def test_pointer_and_workspace_checks(S):
    p = _good(S)
    need = S.themis_workspace_bytes(p, False)
    res = S.Result()
    one = ctypes.c_void_p(256)
    for k in ("h", "c", "b", "total_cost", "latency_buckets", "status"):
        setattr(res, k, 256)
    lib = S._lib
    assert lib.themis_solve_batch(ctypes.byref(p), one, None, one, res, None, need, None) == S.E_INVALID_ARG
    assert lib.themis_solve_batch(ctypes.byref(p), one, None, one, res, ctypes.c_void_p(264), need, None) == S.E_INVALID_ARG
    assert lib.themis_solve_batch(ctypes.byref(p), one, None, one, res, one, need - 1, None) == S.E_WORKSPACE_TOO_SMALL
    assert lib.themis_solve_batch(ctypes.byref(p), one, None, one, S.Result(), one, need, None) == S.E_INVALID_ARG
    assert lib.themis_solve_vertical_batch(ctypes.byref(p), one, None, one, None, res, one, need, None) == S.E_INVALID_ARG
    assert lib.themis_solve_batch_host(ctypes.byref(p), one, None, one, None, res, one, need, None) == S.E_WORKSPACE_TOO_SMALL
    assert lib.themis_alu_probe(9, 1, 32, 1, one, None) == S.E_INVALID_ARG
    assert lib.themis_wait_probe(0, one, one, one, None) == S.E_INVALID_ARG
    assert lib.themis_wait_probe(100, ctypes.c_void_p(260), one, one, None) == S.E_INVALID_ARG
    assert lib.themis_wait_probe(100, one, None, one, None) == S.E_INVALID_ARG


def test_kernel_choice_is_part_of_the_problem_flags(S):
    """Kernel and tile are bits of themis_problem_t.flags; unknown values are refused and the
    choice does not change the workspace a problem needs."""
    n = ctypes.c_size_t()
    base = S.themis_workspace_bytes(_good(S), False)
    for kernel in (S.KERNEL_DEFAULT, S.KERNEL_PACKED16, S.KERNEL_WIDE32, S.KERNEL_PRUNED, S.KERNEL_SPARSE,
                   S.KERNEL_SPARSE_BLOCK, S.KERNEL_PACKED16_BLOCK):
        for tile in (0, 4, 8, 16):
            assert S.themis_workspace_bytes(_good(S, flags=1 | kernel | S.TILE_FLAGS[tile]), False) == base
    for flags in (7 << 8, 15 << 8, 1 << 14, 2, 1 << 31):
        assert S._lib.themis_workspace_bytes(ctypes.byref(_good(S, flags=flags)), 0, ctypes.byref(n)) == S.E_INVALID_ARG


def test_strerror(S):
    assert S.themis_strerror(0) == "ok"
    assert "workspace" in S.themis_strerror(-3)
    assert "CUDA" in S.themis_strerror(-4)
    assert "unknown" in S.themis_strerror(-99)


def test_header_is_plain_c_and_links_from_c(S, tmp_path):
    """include/themis.h compiles as strict C99 and a C program linked against the
    library can call the host-side entry points (nothing is launched)."""
    import subprocess
    src = tmp_path / "use_themis.c"
    src.write_text(r'''
#include <stdio.h>
#include <string.h>
#include "themis.h"
#include "themis_probe.h"
int main(void) {
    themis_problem_t p;
    themis_workspace_layout_t lay;
    size_t bytes = 0;
    memset(&p, 0, sizeof p);
    p.n_instances = 10; p.n_stages = 5; p.n_profiles = 1; p.c_max = 16; p.n_batch = 3;
    p.batch_sizes[0] = 1; p.batch_sizes[1] = 2; p.batch_sizes[2] = 4;
    p.h_max = 8; p.slo_us = 1000000; p.bucket_us = 1000; p.flags = THEMIS_QUEUE_PER_REPLICA | THEMIS_KERNEL_SPARSE | THEMIS_TILE_8;
    if (themis_version() != THEMIS_VERSION) return 1;
    if (themis_workspace_bytes(&p, 0, &bytes) != THEMIS_OK || bytes == 0) return 2;
    if (themis_workspace_layout(&p, 0, &lay) != THEMIS_OK || lay.T != 1000 || lay.row_pitch != 1024) return 3;
    p.bucket_us = 0;
    if (themis_workspace_bytes(&p, 0, &bytes) != THEMIS_E_INVALID_ARG) return 4;
    if (strcmp(themis_strerror(THEMIS_OK), "ok") != 0) return 5;
    printf("%lu\n", (unsigned long)lay.total_bytes);
    return 0;
}
''')
    exe = tmp_path / "use_themis"
    lib_dir = os.path.dirname(S.LIB_PATH)
    subprocess.check_call(["gcc", "-std=c99", "-pedantic", "-Wall", "-Wextra", "-Werror",
                           "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe),
                           "-L", lib_dir, "-l:libthemis.so", f"-Wl,-rpath,{lib_dir}"])
    out = subprocess.check_output([str(exe)]).decode().strip()
    assert int(out) == S.themis_workspace_bytes(_good(S, n_instances=10, n_stages=5, n_profiles=1, c_max=16,
                                                      batch_sizes=(1, 2, 4), h_max=8, slo_us=1_000_000), False)
