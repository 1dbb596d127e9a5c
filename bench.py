#!/usr/bin/env python
"""Benchmark of the batched pipeline-scaling solver.

A "step" is one pass of the whole hot path (candidate scoring, min-plus
recurrence, final scan, backtrack) over one batch of synthetic instances.
Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1..5] [--scaling weak|strong]
                    [--impl reference]

With N > 1 launch under ``python -m torch.distributed.run`` (one rank per GPU).
Weak scaling (default): every rank solves its own batch (independent seeds);
strong scaling: one batch is split over the ranks and the gathered answer is
checked against the one-GPU answer.  Either way there is no collective on the
solve path.  ``--impl reference`` times the CPU oracle instead (rank 0 only).

Beside the headline step the line carries: the recurrence kernel's roofline
against the integer-ALU rate measured in the same run (nominal, useful and
executed cell updates), the other dense kernel on the same batch, the sparse
solver, the end-to-end figure through the host-buffer entry point, the CPU
oracle, and the other benchmark configurations at full size.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "dp_instances_per_s"
UNIT = "instances/s"

# Integer ALU peak of one B200 for the recurrence's operation pair: 148 SMs x 64
# integer lanes per SM per clock x 1.965 GHz boost clock, one fused add-min (two
# integer operations) per lane per clock on 32-bit words; the packed 16-bit form
# of the same instruction does two half-word cells per lane per clock.
N_SMS, INT_LANES_PER_SM, SM_GHZ = 148, 64, 1.965
ALU_PEAK_TOPS_INT32 = N_SMS * INT_LANES_PER_SM * 2 * SM_GHZ / 1e3
ALU_PEAK_TOPS_INT16X2 = 2 * ALU_PEAK_TOPS_INT32
HBM_FALLBACK_GBS = 6650.0

# DRAM bytes (read + write) per launch from the ncu captures summarised under profiles/, per
# instance of the captured workload.  Traffic is proportional to the instance count (one block
# per instance, no reuse across blocks).  A figure is only reported while the kernel's sources
# still have the recorded hash.
NCU_TRAFFIC = {
    "minplus16": {"config": 4, "bytes_per_instance": (316.776448e6 + 158.014720e6) / 2368,
                  "sources": ("paper_2407_14843_b200/csrc/themis_minplus16.cu",
                              "paper_2407_14843_b200/csrc/themis_minplus16_step.cuh"),
                  "sha256_16": "0377121c1eba7f0a"},
    # score_kernel 2.259 MB read + 401.336 MB written, score_lists_kernel 0.943 MB read, per 2368 instances
    "score": {"config": 4, "bytes_per_instance": (2.258944e6 + 401.336064e6 + 0.942592e6) / 2368,
              "sources": ("paper_2407_14843_b200/csrc/themis_score.cu",), "sha256_16": "9d3d4a6e2f9c8f3b"},
}

# Warp instructions the sparse solver executes per instance (ncu smsp__inst_executed.sum of
# stage_fronts_kernel + prefix_fronts_kernel on the first instances of a configuration, see
# profiles/): what its roofline is counted in.  It does no dense table work and moves a few MB,
# so neither the cell-update rate nor HBM bounds it; instruction issue does (one warp
# instruction per scheduler and cycle: 148 SMs x 4 schedulers x the SM clock).
NCU_SPARSE_INSTRUCTIONS = {
    "sources": ("paper_2407_14843_b200/csrc/themis_front.cu",), "sha256_16": "eb8fa0ae6db90b34",
    "per_instance": {4: (55839185 + 19486326) / 2368, 3: (117619149 + 44170020) / 9472},
}


def sparse_issue_roofline(cfg: int, instances_per_s: float, sm_mhz: float, sms: int):
    """Issue-slot roofline of the sparse solver: executed warp instructions per second against
    one instruction per scheduler and cycle."""
    import hashlib
    try:
        h = hashlib.sha256()
        for src in NCU_SPARSE_INSTRUCTIONS["sources"]:
            with open(os.path.join(ROOT, src), "rb") as f:
                h.update(f.read())
        if h.hexdigest()[:16] != NCU_SPARSE_INSTRUCTIONS["sha256_16"] or cfg not in NCU_SPARSE_INSTRUCTIONS["per_instance"]:
            return None
    except OSError:
        return None
    per_instance = NCU_SPARSE_INSTRUCTIONS["per_instance"][cfg]
    peak = sms * 4 * sm_mhz * 1e6
    achieved = per_instance * instances_per_s
    return {"bound": "issue", "achieved": achieved / 1e12, "peak": peak / 1e12, "unit": "T warp instructions/s",
            "frac": achieved / peak, "warp_instructions_per_instance": per_instance,
            "peak_kind": f"derived: {sms} SMs x 4 schedulers x {sm_mhz:.0f} MHz (the clock sampled in this run)",
            "traffic": None}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=4, help="benchmark configuration 1..5 (default 4: large joint DP)")
    ap.add_argument("--instances", type=int, default=None, help="override the batch size (debugging)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=20)
    ap.add_argument("--scaling", default="weak", choices=["weak", "strong"],
                    help="weak: every rank solves its own batch; strong: one batch split over the ranks "
                         "(sharding.shard_range), the gathered answer checked against the one-GPU answer")
    ap.add_argument("--other-kernel-steps", type=int, default=3,
                    help="steps of the other dense recurrence kernel (32-bit when the packed one is timed) on the "
                         "same batch (0: skip)")
    ap.add_argument("--other-configs", type=int, nargs="*", default=[1, 2, 3, 5],
                    help="further benchmark configurations timed at full size after the headline one, one GPU only "
                         "(empty: none)")
    ap.add_argument("--other-config-steps", type=int, default=5)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--alu-probe", action="store_true",
                    help="only run the integer-ALU probe in its five instruction forms and print the rates")
    ap.add_argument("--minplus-mode", type=int, default=0, choices=[0, 1],
                    help="0: packed 16-bit min-plus kernel (default); 1: 32-bit kernel")
    ap.add_argument("--minplus-tile", type=int, default=0, choices=[0, 4, 8, 16],
                    help="cells per thread tile of the recurrence kernels (0: the library's choice)")
    ap.add_argument("--entry", default="solve", choices=["solve", "fallback", "horizontal", "fit"],
                    help="solve: the headline step (default).  The others time one of the further entry points "
                         "on one GPU with the CPU oracle beside it: fallback = themis_vertical_fallback_batch on the "
                         "day-long trace; horizontal = Algorithm 2 at the current and a predicted rate plus the "
                         "stability test; fit = themis_fit_profiles_batch")
    ap.add_argument("--pruned-steps", type=int, default=5,
                    help="extra steps with the recurrence restricted to undominated entries (0: skip)")
    return ap.parse_args()


def ncu_traffic_bytes(kernel: str, cfg: int, n_instances: int):
    import hashlib
    rec = NCU_TRAFFIC[kernel]
    try:
        h = hashlib.sha256()
        for src in rec["sources"]:
            with open(os.path.join(ROOT, src), "rb") as f:
                h.update(f.read())
        if h.hexdigest()[:16] != rec["sha256_16"]:
            return None
    except OSError:
        return None
    return rec["bytes_per_instance"] * n_instances if cfg == rec["config"] else None


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return HBM_FALLBACK_GBS, "fallback"


# --------------------------------------------------------------------------- CPU oracle legs

def oracle_sample_size(oracle, wl_full, target_s: float):
    """Times a small probe of the oracle and returns (n, probe_rate) so that n
    instances take about target_s seconds."""
    cores = os.cpu_count() or 1
    n0 = min(wl_full.n_instances, max(2, 2 * cores if wl_full.minplus_cells > 2e7 else 16 * cores))
    t = time.perf_counter()
    r = oracle.solve_batch(wl_full.take(n0))
    dt = max(time.perf_counter() - t, 1e-4)
    n = int(max(n0, min(wl_full.n_instances, target_s * n0 / dt)))
    return n, r["threads"]


def cpu_baseline(wl_full, target_s: float = 15.0):
    import oracle
    n, threads = oracle_sample_size(oracle, wl_full, target_s)
    sub = wl_full.take(n)
    t = time.perf_counter()
    oracle.solve_batch(sub)
    dt = time.perf_counter() - t
    # one thread, on a smaller prefix of the same sample (about 2 s)
    n1 = max(1, min(n, int(2.0 * n / (dt * max(1, threads)))))
    t = time.perf_counter()
    oracle.solve_batch(wl_full.take(n1), n_threads=1)
    dt1 = time.perf_counter() - t
    return {"value": n / dt, "unit": UNIT, "cores": int(threads), "kind": "oracle",
            "sample": f"first {n} of {wl_full.n_instances} instances of {wl_full.name}, {dt:.1f} s",
            "cell_updates_per_s": n * wl_full.minplus_cells / dt,
            "single_thread": {"value": n1 / dt1, "unit": UNIT, "sample": f"first {n1} instances, {dt1:.1f} s"}}


def run_reference(args):
    """The CPU oracle as the reference arm: rank 0 only, bounded sample per step."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from paper_2407_14843_b200 import workloads
    import oracle
    oracle.build()
    wl_full = workloads.make_workload(args.config, args.instances)
    total_steps = args.steps + args.warmup
    per_step_s = max(1.0, min(6.0, 120.0 / max(1, total_steps)))
    n, threads = oracle_sample_size(oracle, wl_full, per_step_s)
    sub = wl_full.take(n)
    for _ in range(args.warmup):
        oracle.solve_batch(sub)
    t = time.perf_counter()
    for _ in range(args.steps):
        oracle.solve_batch(sub)
    dt = time.perf_counter() - t
    value = n * args.steps / dt
    sample = f"first {n} of {wl_full.n_instances} instances of {wl_full.name} per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int32",
        "data": "synthetic", "config": workload_config(wl_full, args, 1),
        "cell_updates_per_s": n * wl_full.minplus_cells * args.steps / dt,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": int(threads), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- helpers

def workload_config(wl, args, world):
    return {
        "workload": f"config {args.config}: {wl.name}",
        "instances_per_gpu": wl.n_instances, "stages": wl.n_stages, "c_max": wl.c_max,
        "batch_sizes": list(wl.batch_sizes), "h_max": wl.h_max, "candidates_per_stage": wl.n_candidates,
        "T": wl.T, "bucket_us": wl.bucket_us, "slo_us": wl.slo_us, "vertical": wl.vertical,
        "queue_per_replica": bool(wl.flags & 1), "parallelism": f"instances sharded over {world} gpu(s)",
        "minplus_cells_per_instance": wl.minplus_cells,
        "cache": "per-step tables (G, Garg, A) are far larger than the 126 MB L2",
    }


class ClockSampler:
    """nvidia-smi in a child process, sampling SM clocks and throttle reasons."""
    FIELDS = ("uuid,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid: str):
        self.uuid = uuid
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=self.file, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for row in self.file.read().splitlines():
            cols = [c.strip() for c in row.split(",")]
            if len(cols) < 8 or (self.uuid and self.uuid not in cols[0]):
                continue
            try:
                sm.append(float(cols[1])); mx.append(float(cols[2])); power.append(float(cols[3]))
            except ValueError:
                continue
            for name, val in zip(names, cols[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.file.close()
        try:
            os.unlink(self.file.name)
        except OSError:
            pass
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(power)}


def probe_alu_peak(solver, torch, mode):
    """Add-min throughput sustained by themis_alu_probe in TOP/s (two operations
    per cell update): mode 1 = fused 32-bit add-min, mode 3 = packed 2 x 16-bit."""
    blocks, threads, iters = N_SMS * 8, 256, 20000          # about 20 ms per form
    cells_per_update = 2 if mode == 3 else 1
    sink = torch.empty(blocks * threads, dtype=torch.uint32, device="cuda")
    solver.themis_alu_probe(mode, blocks, threads, 50, sink)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    solver.themis_alu_probe(mode, blocks, threads, iters, sink)
    b.record()
    torch.cuda.synchronize()
    return 2.0 * cells_per_update * blocks * threads * iters * 64 / (a.elapsed_time(b) * 1e-3) / 1e12


# --------------------------------------------------------------------------- the CUDA arm

def packed_launch_shape(cells: int, tile: int = 0):
    """Tiling of the packed recurrence kernel for a budget of `cells` = T + 1 cells, as its
    launcher chooses it: cells per tile R, half-groups of 16 tiles, cells left to the
    block-wide reduction (budgets of up to 1900 cells run with one warp per instance: tiles
    of 4 or 8 cells, every cell in a tile)."""
    if cells <= 1900 and tile != 16:
        R = tile if tile in (4, 8) else (4 if cells <= 904 else 8)
        return R, ((cells + R - 1) // R + 15) // 16, False
    R = tile if tile in (4, 8, 16) else (4 if cells <= 896 + 8 else 8)
    while True:
        tiles = (cells + R - 1) // R
        half_groups = (tiles + 15) // 16
        extra = False
        if half_groups > 1 and cells - (half_groups - 1) * 16 * R <= 8:
            half_groups -= 1
            extra = True
        threads = ((half_groups + 1) // 2 + 1) // 2 * 32
        if threads <= 1024 or R == 16:
            break
        R *= 2
    return R, half_groups, extra


def cell_update_counts(torch, wl, tables, tile: int = 0):
    """Cell updates of the recurrence per batch, three ways, from the scored tables G:
    nominal   (S-1)(T+1)(T+2)/2 per instance;
    useful    cells (t, l) of stage s that are not unreachable by construction:
              l >= first reachable entry of G_s and t - l >= sum of the earlier stages' first
              reachable entries (the bounds the packed kernel skips by);
    needed    useful cells whose budget t the later stages can still complete:
              t <= T - sum of the later stages' first reachable entries (the packed kernel
              computes no budget above that limit);
    executed  what the packed kernel actually performs: per stage and tile in use its chunk
              steps (the same skip rules, in whole chunk pairs and half-groups of 16 tiles, every
              lane of a half-group running to the half-group's longest column) times R x R cells,
              plus the cells of the block-wide reduction."""
    G, T = tables["G"], wl.T
    N, S, W = wl.n_instances, wl.n_stages, T + 1
    reach = G[:, :, :W] != 2 ** 31 - 1
    first = torch.where(reach.any(dim=2), reach.int().argmax(dim=2), torch.full((N, S), -1, device=G.device)).long()
    dead = (first < 0).long().cumsum(dim=1) > 0                      # an empty stage kills everything after it
    first = first.clamp(min=0)
    prefix = first.cumsum(dim=1) - first                             # sum over earlier stages
    later = (first.sum(dim=1, keepdim=True) - first.cumsum(dim=1)).clamp(max=W)   # sum over later stages
    t_max = (T - later)[:, 1:]                                       # budget limit of stages 1..S-1
    m = (T - first - prefix)[:, 1:]
    alive = ~dead[:, 1:] & ~dead[:, -1:]                             # an empty later stage: nothing to complete
    useful = int(((m + 1) * (m + 2) // 2 * (m >= 0) * ~dead[:, 1:]).sum())
    m2 = (t_max - first[:, 1:] - prefix[:, 1:])
    needed = int(((m2 + 1) * (m2 + 2) // 2 * (m2 >= 0) * alive).sum())
    R, nhg, extra = packed_launch_shape(W, tile)
    n_tiles = nhg * 16
    Tc = n_tiles * R
    n_dummy = max(0, Tc - W) // R
    n_extra = max(0, W - Tc) if extra else 0
    q_lo = (first[:, 1:] // R) & ~1
    q_shift = ((prefix[:, 1:] // R) + n_dummy) & ~1
    ends = torch.arange(nhg, device=G.device).long() * 16 + 15       # tile | 15 of every half-group
    used = torch.where(t_max < 0, torch.zeros_like(t_max), ((n_dummy + t_max.clamp(min=0) // R) // 16 + 1).clamp(max=nhg))
    in_use = torch.arange(nhg, device=G.device).view(1, 1, -1) < used.unsqueeze(2)
    steps = (ends.view(1, 1, -1) - q_shift.unsqueeze(2) - q_lo.unsqueeze(2) + 1).clamp(min=0)
    steps = steps * in_use * (~dead[:, 1:]).unsqueeze(2)
    executed = int(steps.sum()) * 16 * R * R
    executed += int((alive & (t_max >= Tc)).sum()) * sum(Tc + e + 1 for e in range(n_extra))
    return {"nominal": N * wl.minplus_cells, "useful": useful, "needed": needed, "executed": executed}


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2407_14843_b200 import build as _build

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world == 1 and args.gpus > 1:
        # not under a launcher: start one rank per GPU ourselves
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", "29533", os.path.abspath(__file__)] + sys.argv[1:]
        sys.exit(subprocess.call(cmd))

    from paper_2407_14843_b200 import sharding, workloads
    strong = args.scaling == "strong"
    # weak scaling: every rank its own batch (seeds offset by rank); strong: one batch, split
    wl_all = workloads.make_workload(args.config, args.instances, seed_offset=0 if strong else rank)
    if strong:
        a, b = sharding.shard_range(wl_all.n_instances, rank, world)
        wl = wl_all.take(b - a, a)
    else:
        wl = wl_all
    cpu = None
    if rank == 0:
        _build.build_library()
        if not args.no_cpu_baseline:
            import oracle
            oracle.build()                       # before the first GPU call
            cpu = cpu_baseline(wl_all)
    torch.cuda.set_device(local_rank)
    # Under a launcher (RANK set) the process group is brought up even for one rank, so that
    # the barrier / max-over-ranks path is the same code at every N.
    use_dist = world > 1 or "RANK" in os.environ
    if use_dist:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    from paper_2407_14843_b200 import solver

    def barrier():
        torch.cuda.synchronize()
        if use_dist:
            dist.barrier()
            torch.cuda.synchronize()

    def max_over_ranks(values):
        t = torch.tensor(values, dtype=torch.float64, device="cuda")
        if use_dist:
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return t.tolist()

    mk = lambda: torch.cuda.Event(enable_timing=True)
    packed = args.minplus_mode == 0
    main_kernel = solver.KERNEL_PACKED16 if packed else solver.KERNEL_WIDE32

    def time_dense(w, dev, ws, out, kernel, tile, steps, warmup):
        """`steps` timed steps (scoring launch + recurrence launch) after `warmup` untimed ones."""
        prob = solver.Problem.of_workload(w, kernel, tile)

        def step(ev=None):
            if ev:
                ev[0].record()
            solver.themis_score_batch(prob, dev["lat_us"], dev["profile_id"], dev["lambda_mrps"], dev["replicas"], ws)
            if ev:
                ev[1].record()
            solver.themis_minplus_batch(prob, dev["replicas"], out, ws)
            if ev:
                ev[2].record()

        for _ in range(max(warmup, 1)):
            step()
        evs = [[mk(), mk(), mk()] for _ in range(steps)]
        barrier()
        for k in range(steps):
            step(evs[k])
        barrier()
        total, score, minplus = max_over_ranks([
            evs[0][0].elapsed_time(evs[-1][2]), sum(e[0].elapsed_time(e[1]) for e in evs) / steps,
            sum(e[1].elapsed_time(e[2]) for e in evs) / steps])
        per_step = sorted(e[0].elapsed_time(e[2]) for e in evs)
        return {"total_ms": total, "score_ms": score, "minplus_ms": minplus, "per_step_ms": per_step}

    def time_sparse(w, dev, ws, out, steps):
        prob = solver.Problem.of_workload(w, solver.KERNEL_SPARSE)

        def call():
            if w.vertical:
                solver.themis_solve_vertical_batch(prob, dev["lat_us"], dev["profile_id"], dev["lambda_mrps"],
                                                   dev["replicas"], out, ws)
            else:
                solver.themis_solve_batch(prob, dev["lat_us"], dev["profile_id"], dev["lambda_mrps"], out, ws)

        call()
        barrier()
        a, b = mk(), mk()
        a.record()
        for _ in range(steps):
            call()
        b.record()
        barrier()
        return max_over_ranks([a.elapsed_time(b)])[0] / steps

    def dense_rooflines(w, t, is_packed, probe, counts=None):
        """The recurrence kernel against the integer-ALU peak and the scoring kernel against HBM."""
        cells = w.n_instances * w.minplus_cells
        tops = 2.0 * cells / (t["minplus_ms"] * 1e-3) / 1e12
        derived = ALU_PEAK_TOPS_INT16X2 if is_packed else ALU_PEAK_TOPS_INT32
        measured = probe["int16x2" if is_packed else "int32"] if probe else None
        lay = solver.themis_workspace_layout(solver.Problem.of_workload(w), w.vertical)
        score_bytes = 6.0 * lay.row_pitch * w.n_instances * w.n_stages
        score_gbs = score_bytes / (t["score_ms"] * 1e-3) / 1e9
        r = {"minplus_ms": t["minplus_ms"], "score_ms": t["score_ms"], "achieved_tops": tops,
             "frac_of_derived_peak": tops / derived, "frac_of_probe_peak": tops / measured if measured else None,
             "score_gbs": score_gbs, "score_frac_of_hbm": score_gbs / hbm_peak, "score_bytes": score_bytes}
        if counts:
            r["frac_useful"] = r["frac_of_derived_peak"] * counts["useful"] / counts["nominal"]
            r["frac_executed"] = r["frac_of_derived_peak"] * counts["executed"] / counts["nominal"]
        return r

    hbm_peak, hbm_kind = measured_hbm_peak()
    prob = solver.Problem.of_workload(wl, main_kernel, args.minplus_tile)
    dev = solver.workload_to_device(wl)
    ws = solver.alloc_workspace(prob, wl.vertical, host_variant=True)
    out = solver.alloc_result(wl.n_instances, wl.n_stages)

    # warm-up of the headline step, then the ALU probe (its rate is the measured roofline denominator)
    warm = time_dense(wl, dev, ws, out, main_kernel, args.minplus_tile, 1, args.warmup)
    del warm
    probe = {"int32": probe_alu_peak(solver, torch, 1), "int16x2": probe_alu_peak(solver, torch, 3)}
    probe = dict(zip(probe, max_over_ranks(list(probe.values()))))      # one figure per form for the line
    barrier()

    uuid = str(getattr(torch.cuda.get_device_properties(local_rank), "uuid", ""))
    sampler = ClockSampler(uuid) if rank == 0 else None
    if sampler:
        sampler.start()
        time.sleep(0.25)
    main = time_dense(wl, dev, ws, out, main_kernel, args.minplus_tile, args.steps, 1)
    clocks = sampler.stop() if sampler else None
    total_ms, score_ms, minplus_ms, step_ms = main["total_ms"], main["score_ms"], main["minplus_ms"], main["per_step_ms"]
    dense_out = {k: v.clone() for k, v in out.items()}
    status = out["status"].cpu()
    n_infeasible, n_error = int((status == 1).sum()), int((status < 0).sum())
    counts = None
    if packed:       # the tables of the last timed step are still in the workspace
        counts = cell_update_counts(torch, wl, solver.workspace_tables(prob, wl.vertical, ws), args.minplus_tile)

    # the other dense kernel on the same batch, a few steps
    other_kernel = solver.KERNEL_WIDE32 if packed else solver.KERNEL_PACKED16
    other = time_dense(wl, dev, ws, out, other_kernel, args.minplus_tile, max(1, args.other_kernel_steps), 1) \
        if args.other_kernel_steps > 0 else None
    other_same = all(bool((out[k] == dense_out[k]).all()) for k in out) if other else None

    # The same batch through the solver restricted to undominated entries (one warp per
    # instance on sorted fronts; identical results, a small fraction of the cell updates):
    # reported beside the dense figures, not as them.
    pruned = None
    if args.pruned_steps > 0:
        p_ms = time_sparse(wl, dev, ws, out, args.pruned_steps)
        pruned = {"value": wl.n_instances * world / (p_ms * 1e-3), "unit": UNIT, "ms_per_step": p_ms,
                  "steps": args.pruned_steps,
                  "kernel": "stage_fronts_kernel + prefix_fronts_kernel (+ solve_sparse_kernel for listed "
                            "instances): a 4-byte memset and 3 launches per step",
                  "same_results_as_dense": all(bool((out[k] == dense_out[k]).all()) for k in out),
                  "note": "THEMIS_KERNEL_SPARSE: scoring, fronts and recurrence on undominated entries only"}

    # end to end through the host-buffer entry point: pinned host inputs in,
    # host results out, copies inside the timed region
    pin = lambda a: None if a is None else torch.from_numpy(a).pin_memory()
    h_in = {"lat": pin(wl.lat_us), "pid": pin(wl.profile_id), "lam": pin(wl.lambda_mrps),
            "rep": pin(wl.replicas) if wl.vertical else None}
    h_out = solver.alloc_result(wl.n_instances, wl.n_stages, device="cpu", pin=True)
    e2e_call = lambda: solver.themis_solve_batch_host(prob, h_in["lat"], h_in["pid"], h_in["lam"], h_in["rep"],
                                                      h_out, ws)
    e2e_call()
    barrier()
    t0 = time.perf_counter()
    for _ in range(args.e2e_steps):
        e2e_call()
    torch.cuda.synchronize()
    e2e_s = max_over_ranks([time.perf_counter() - t0])[0]
    h2d = sum(x.numel() * x.element_size() for x in h_in.values() if x is not None)
    d2h = sum(x.numel() * x.element_size() for x in h_out.values())
    same = all(bool((h_out[k] == dense_out[k].cpu()).all()) for k in h_out)

    # strong scaling: the gathered answer of the split batch against the one-GPU answer
    sharded_check = None
    if strong and use_dist:
        full = sharding.solve_sharded(wl_all, lambda block: solver.solve(block)[0])
        if rank == 0:
            one, _ = solver.solve(wl_all)
            torch.cuda.synchronize()
            sharded_check = {k: bool((full[k] == one[k]).all()) for k in full}
            del one
        del full

    # the other benchmark configurations at full size, one after the other (rank 0 of a
    # one-GPU run only: they are context for the headline figure, not part of it)
    others = {}
    if args.other_configs and world == 1:
        del dev, ws, out, dense_out, h_in, h_out
        torch.cuda.empty_cache()
        for cfg in args.other_configs:
            if cfg == args.config:
                continue
            w = workloads.make_workload(cfg)
            d = solver.workload_to_device(w)
            pr = solver.Problem.of_workload(w)
            wsp = solver.alloc_workspace(pr, w.vertical)
            o = solver.alloc_result(w.n_instances, w.n_stages)
            steps = args.other_config_steps
            t16 = time_dense(w, d, wsp, o, solver.KERNEL_PACKED16, 0, steps, 3)
            ref = {k: v.clone() for k, v in o.items()}
            cnt = cell_update_counts(torch, w, solver.workspace_tables(pr, w.vertical, wsp))
            t32 = time_dense(w, d, wsp, o, solver.KERNEL_WIDE32, 0, max(2, steps // 2), 1)
            same32 = all(bool((o[k] == ref[k]).all()) for k in o)
            sp_ms = time_sparse(w, d, wsp, o, steps)
            same_sp = all(bool((o[k] == ref[k]).all()) for k in o)
            others[str(cfg)] = {
                "workload": w.name, "instances": w.n_instances, "stages": w.n_stages, "T": w.T, "steps": steps,
                "ms_per_step": t16["total_ms"] / steps, "instances_per_s": w.n_instances * steps / (t16["total_ms"] * 1e-3),
                "packed16": dense_rooflines(w, t16, True, probe, cnt),
                "wide32": dict(dense_rooflines(w, t32, False, probe), same_results=same32),
                "sparse": {"ms_per_step": sp_ms, "instances_per_s": w.n_instances / (sp_ms * 1e-3), "same_results": same_sp,
                           "roofline": sparse_issue_roofline(
                               cfg, w.n_instances / (sp_ms * 1e-3),
                               (clocks or {}).get("sm_mhz") or (clocks or {}).get("sm_max_mhz") or 1965.0,
                               torch.cuda.get_device_properties(local_rank).multi_processor_count)},
                "cell_updates": cnt, "infeasible_instances": int((ref["status"] == 1).sum()),
            }
            del d, wsp, o, ref
            torch.cuda.empty_cache()

    if use_dist:
        dist.barrier()
        dist.destroy_process_group()
    if rank != 0:
        return

    N_total = wl.n_instances * world if not strong else wl_all.n_instances
    # score + min-plus, plus the 32-bit second pass where a total may exceed 15 bits
    second_pass = packed and (wl.vertical or wl.n_stages * wl.h_max * wl.c_max >= 0x7FFF)
    # score_lists_kernel + score_kernel + the recurrence kernel (+ the 32-bit pass over flagged instances)
    launches_per_step = 4 if second_pass else 3
    cells_per_launch = wl.n_instances * wl.minplus_cells
    main_r = dense_rooflines(wl, main, packed, probe, counts)
    kernel_name = ("minplus16_warp_kernel" if wl.T + 1 <= 1900 and args.minplus_tile != 16 else "minplus16_kernel") \
        if packed else ("minplus_warp_kernel" if wl.T + 1 <= 2800 and args.minplus_tile != 16 else "minplus_kernel")
    measured_peak = probe["int16x2" if packed else "int32"]
    derived_peak = ALU_PEAK_TOPS_INT16X2 if packed else ALU_PEAK_TOPS_INT32
    line = {
        "metric": METRIC, "value": N_total * args.steps / (total_ms * 1e-3), "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_ms / args.steps,
        "ms_per_step_best": step_ms[0], "ms_per_step_median": step_ms[len(step_ms) // 2],
        "higher_is_better": True, "scaling": "strong" if strong else "weak", "vs_baseline": None,
        # arithmetic of the dominant kernel: packed pairs of unsigned 16-bit costs, or 32-bit keys
        "dtype": "u16" if packed else "u32",
        "data": "synthetic", "config": workload_config(wl_all if strong else wl, args, world),
        "cell_updates_per_s": world * cells_per_launch * args.steps / (total_ms * 1e-3),
        "minplus_cell_updates_per_s_kernel": cells_per_launch / (minplus_ms * 1e-3),
        "kernels_ms": {"score_kernel": score_ms, kernel_name: minplus_ms},
        "infeasible_instances": n_infeasible, "device_error_instances": n_error,
        "input_checksums": wl.checksums(),
        "device": {"name": torch.cuda.get_device_name(local_rank),
                   "sms": torch.cuda.get_device_properties(local_rank).multi_processor_count},
        "roofline": {
            "kernel": kernel_name, "bound": "alu", "achieved": main_r["achieved_tops"], "peak": measured_peak,
            "unit": "TOP/s (integer add+min, 2 per cell update)", "frac": main_r["achieved_tops"] / measured_peak,
            "traffic": ncu_traffic_bytes("minplus16", args.config, wl.n_instances) if packed else None,
            "peak_kind": "measured in this run: themis_alu_probe, " +
                         ("fused add-min on packed 2 x 16-bit" if packed else "fused 32-bit add-min") +
                         " on registers, all SMs",
            "peak_derived": derived_peak, "frac_of_derived_peak": main_r["frac_of_derived_peak"],
            "peak_derived_kind": ("148 SMs x 64 int lanes x 2 ops x 1.965 GHz"
                                  + (" x 2 half-word cells per lane" if packed else "")),
            "peak_probe": probe, "frac_of_int32_peak": main_r["achieved_tops"] / ALU_PEAK_TOPS_INT32,
            "algorithmic_cells_per_launch": cells_per_launch, "avg_launch_ms": minplus_ms,
        },
        "roofline_score_kernel": {
            "kernel": "score_kernel", "bound": "hbm", "achieved": main_r["score_gbs"], "peak": hbm_peak, "unit": "GB/s",
            "frac": main_r["score_frac_of_hbm"], "traffic": ncu_traffic_bytes("score", args.config, wl.n_instances),
            "peak_kind": f"of {hbm_kind}",
            "algorithmic_bytes_per_launch": main_r["score_bytes"], "avg_launch_ms": score_ms,
        },
        "e2e": {"value": N_total * args.e2e_steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": args.e2e_steps, "matches_device_path": same},
        "gpu_launches": launches_per_step * args.steps,
        "clocks": clocks,
    }
    if counts:
        line["cell_updates_useful_per_s"] = world * counts["useful"] * args.steps / (total_ms * 1e-3)
        line["cell_updates_executed_per_s"] = world * counts["executed"] * args.steps / (total_ms * 1e-3)
        line["roofline"].update({
            "cells_per_launch": counts,
            "frac_useful": main_r["achieved_tops"] / measured_peak * counts["useful"] / counts["nominal"],
            "frac_executed": main_r["achieved_tops"] / measured_peak * counts["executed"] / counts["nominal"],
            "cells_note": "nominal = (S-1)(T+1)(T+2)/2 per instance; useful = cells not unreachable by the stages' "
                          "first reachable entries; needed = useful cells at budgets the later stages can still "
                          "complete; executed = chunk steps the kernel performs x R x R (skips in chunk pairs and "
                          "half-groups, lanes run to their half-group's longest column)"})
    if other:
        o_packed = not packed
        o_r = dense_rooflines(wl, other, o_packed, probe)
        o_peak = probe["int16x2" if o_packed else "int32"]
        line["roofline_int32_kernel" if packed else "roofline_int16_kernel"] = {
            "kernel": "minplus_kernel" if packed else "minplus16_kernel", "bound": "alu",
            "achieved": o_r["achieved_tops"], "peak": o_peak, "unit": "TOP/s (integer add+min, 2 per cell update)",
            "frac": o_r["achieved_tops"] / o_peak, "frac_of_derived_peak": o_r["frac_of_derived_peak"],
            "avg_launch_ms": other["minplus_ms"], "steps": max(1, args.other_kernel_steps),
            "ms_per_step": other["total_ms"] / max(1, args.other_kernel_steps), "same_results": other_same,
            "peak_kind": "measured in this run: themis_alu_probe", "traffic": None}
    if pruned is not None:
        sm_mhz = (clocks or {}).get("sm_mhz") or (clocks or {}).get("sm_max_mhz") or 1965.0
        sms = torch.cuda.get_device_properties(local_rank).multi_processor_count
        pruned["roofline"] = sparse_issue_roofline(args.config, pruned["value"] / world, sm_mhz, sms)
        line["pruned_path"] = pruned
    if sharded_check is not None:
        line["sharded_equals_one_gpu"] = sharded_check
    if others:
        line["other_configs"] = others
    if cpu is not None:
        line["cpu_baseline"] = cpu
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- further entry points

def _timed(torch, fn, steps, warmup):
    """Average milliseconds of fn() over `steps` calls after `warmup` calls (CUDA events on the
    current stream, synchronised on both sides)."""
    for _ in range(max(1, warmup)):
        fn()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(steps):
        fn()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / steps


def run_entry(args):
    """One of the entry points beyond the headline solve: device time per call on resident inputs,
    the oracle's time on a sample of the same inputs, and whether the two agree on that sample."""
    import dataclasses
    import numpy as np
    import torch
    from paper_2407_14843_b200 import build as _build, workloads
    _build.build_library()
    import oracle
    oracle.build()
    cores = os.cpu_count() or 1
    base = {"n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "higher_is_better": True, "data": "synthetic",
            "vs_baseline": None}

    if args.entry == "fit":
        from oracle import profile_fit
        n_models = args.instances or 65536
        c_max, batches = 64, (1, 2, 4, 8, 16, 32, 64)
        sb, sc, lat, _ = workloads.profile_samples(77, n_models)
        n_ref = min(n_models, 2048)
        t = time.perf_counter()
        ref_c, ref_t, ref_s = profile_fit.fit_profiles(sb, sc, lat[:n_ref], c_max, batches)
        cpu_s = time.perf_counter() - t
        torch.cuda.set_device(0)
        from paper_2407_14843_b200 import solver
        dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
        d_sb, d_sc, d_lat, d_b = dev(sb), dev(sc), dev(lat), dev(np.asarray(batches, np.int32))
        coeffs = torch.empty((n_models, 4), dtype=torch.float64, device="cuda")
        tab = torch.empty((n_models, c_max, len(batches)), dtype=torch.int32, device="cuda")
        status = torch.empty(n_models, dtype=torch.int32, device="cuda")
        ms = _timed(torch, lambda: solver.themis_fit_profiles_batch(d_sb, d_sc, d_lat, c_max, d_b, coeffs, tab, status),
                    args.steps, args.warmup)
        diff = np.abs(tab[:n_ref].cpu().numpy().astype(np.int64) - ref_t)
        same = bool(np.allclose(coeffs[:n_ref].cpu().numpy(), ref_c, rtol=1e-8, atol=1e-10) and diff.max() <= 1
                    and np.array_equal(status[:n_ref].cpu().numpy(), ref_s))
        table_bytes = tab.numel() * 4 + lat.nbytes
        hbm_peak, hbm_kind = measured_hbm_peak()
        line = dict(base, metric="profile_fits_per_s", value=n_models / (ms * 1e-3), unit="models/s", ms_per_step=ms,
                    dtype="f64", scaling="weak",
                    config={"workload": f"Eq. 1 fit: {n_models} models x {lat.shape[1]} profiled (b, c) points, tables "
                                        f"{c_max} x {len(batches)}"},
                    roofline={"kernel": "fit_profiles_kernel", "bound": "hbm", "achieved": table_bytes / (ms * 1e-3) / 1e9,
                              "peak": hbm_peak, "unit": "GB/s", "frac": table_bytes / (ms * 1e-3) / 1e9 / hbm_peak,
                              "traffic": None, "peak_kind": f"of {hbm_kind}",
                              "algorithmic_bytes_per_launch": table_bytes},
                    cpu_baseline={"value": n_ref / cpu_s, "unit": "models/s", "cores": 1, "kind": "oracle",
                                  "sample": f"first {n_ref} models, {cpu_s:.2f} s (numpy lstsq per model)"},
                    matches_oracle_on_sample=same, gpu_launches=args.steps)
        print(json.dumps(line), flush=True)
        return

    if args.entry == "fallback":
        wl = workloads.make_workload(3, args.instances)
        res = 1000                                               # search points every 1 request/s
        n_ref = min(wl.n_instances, 4096)
        # the sample: the busiest seconds (where the last branch is taken) and a stride of quiet ones
        hot = np.argsort(wl.lambda_mrps)[-n_ref // 2:]
        pick = np.unique(np.concatenate([hot, np.arange(0, wl.n_instances, max(1, 2 * wl.n_instances // n_ref))]))
        sub = dataclasses.replace(wl, n_instances=len(pick), profile_id=wl.profile_id[pick].copy(),
                                  lambda_mrps=wl.lambda_mrps[pick].copy(), replicas=wl.replicas[pick].copy())
        t = time.perf_counter()
        ref = oracle.vertical_fallback_batch(sub, res)
        cpu_s = time.perf_counter() - t
        torch.cuda.set_device(0)
        from paper_2407_14843_b200 import solver
        prob = solver.Problem.of_workload(wl)
        dev = solver.workload_to_device(wl)
        ws = torch.empty(solver.themis_fallback_workspace_bytes(prob), dtype=torch.uint8, device="cuda")
        out = solver.alloc_result(wl.n_instances, wl.n_stages)
        lam_v = torch.empty(wl.n_instances, dtype=torch.uint32, device="cuda")
        extra = torch.empty((wl.n_instances, wl.n_stages), dtype=torch.int32, device="cuda")
        lam_max = int(wl.lambda_mrps.max())
        call = lambda: solver.themis_vertical_fallback_batch(prob, dev["lat_us"], dev["profile_id"], dev["lambda_mrps"],
                                                             dev["replicas"], res, lam_max, out, lam_v, extra, ws)
        ms = _timed(torch, call, args.steps, args.warmup)
        ms_plain = _timed(torch, lambda: solver.themis_solve_vertical_batch(
            prob, dev["lat_us"], dev["profile_id"], dev["lambda_mrps"], dev["replicas"], out, ws), args.steps, 1)
        call()
        torch.cuda.synchronize()
        st = out["status"].cpu().numpy()
        same = all(np.array_equal(out[k].cpu().numpy()[pick], ref[k]) for k in out) \
            and np.array_equal(lam_v.cpu().numpy()[pick], ref["lambda_vertical"]) \
            and np.array_equal(extra.cpu().numpy()[pick], ref["extra_replicas"])
        rounds = max(0, int(np.ceil(np.log2(max(1, (lam_max + res - 1) // res)))))
        line = dict(base, metric="fallback_instances_per_s", value=wl.n_instances / (ms * 1e-3), unit=UNIT,
                    ms_per_step=ms, dtype="u16", scaling="weak",
                    config={"workload": f"config 3 ({wl.name}): every second of the day, Algorithm 1 with its last "
                                        f"branch, search points every {res} mrps",
                            "instances": wl.n_instances, "stages": wl.n_stages, "T": wl.T,
                            "bisection_rounds": rounds, "split_instances": int((st == 2).sum()),
                            "served_in_place": int((st == 0).sum())},
                    ms_plain_vertical_solve=ms_plain, ms_search_and_second_solve=ms - ms_plain,
                    cpu_baseline={"value": len(pick) / cpu_s, "unit": UNIT, "cores": cores, "kind": "oracle",
                                  "sample": f"{len(pick)} seconds of the trace (the busiest {len(hot)} and a stride of "
                                            f"the rest), {cpu_s:.1f} s"},
                    matches_oracle_on_sample=bool(same), gpu_launches=None)
        print(json.dumps(line), flush=True)
        return

    # horizontal: Algorithm 2 at the current and at the predicted rate, then the stability test
    full = workloads.make_workload(2, args.instances)
    h_max = 256
    wl = dataclasses.replace(full, c_max=1, h_max=h_max, lat_us=np.ascontiguousarray(full.lat_us[:, :, :1, :]))
    growth = 1.0 + 0.3 * workloads.rand_uniform(7501, 1, np.arange(wl.n_instances, dtype=np.uint64))
    pred = dataclasses.replace(wl, lambda_mrps=(wl.lambda_mrps * growth).astype(np.uint32))
    t = time.perf_counter()
    a, b = oracle.solve_batch(wl, horizontal=True), oracle.solve_batch(pred, horizontal=True)
    cpu_s = time.perf_counter() - t
    expect = (a["status"] == 0) & (b["status"] == 0) & np.all(a["h"] == b["h"], axis=1) \
        & np.all(a["b"] == b["b"], axis=1) & np.all(a["c"] == b["c"], axis=1)
    torch.cuda.set_device(0)
    from paper_2407_14843_b200 import solver
    prob = solver.Problem.of_workload(wl)
    d_now, d_pred = solver.workload_to_device(wl), solver.workload_to_device(pred)
    ws = solver.alloc_workspace(prob, False)
    o_now, o_pred = (solver.alloc_result(wl.n_instances, wl.n_stages) for _ in range(2))
    stable = torch.empty(wl.n_instances, dtype=torch.int32, device="cuda")

    def call():
        solver.themis_solve_horizontal_batch(prob, d_now["lat_us"], d_now["profile_id"], d_now["lambda_mrps"], o_now, ws)
        solver.themis_solve_horizontal_batch(prob, d_pred["lat_us"], d_pred["profile_id"], d_pred["lambda_mrps"], o_pred, ws)
        solver.themis_configs_equal_batch(o_now, o_pred, stable)

    ms = _timed(torch, call, args.steps, args.warmup)
    same = bool(np.array_equal(stable.cpu().numpy().astype(bool), expect)
                and all(np.array_equal(o_now[k].cpu().numpy(), a[k]) for k in o_now))
    line = dict(base, metric="stability_tests_per_s", value=wl.n_instances / (ms * 1e-3), unit=UNIT, ms_per_step=ms,
                dtype="u16", scaling="weak",
                config={"workload": f"config 2 shapes with one-core replicas (Algorithm 2, up to {h_max} replicas): two "
                                    "solves (current rate, predicted rate up to 30 % higher) and the comparison",
                        "instances": wl.n_instances, "stages": wl.n_stages, "T": wl.T,
                        "batch_sizes": list(wl.batch_sizes), "stable_instances": int(expect.sum()),
                        "infeasible_now": int((a["status"] == 1).sum())},
                cpu_baseline={"value": wl.n_instances / cpu_s, "unit": UNIT, "cores": cores, "kind": "oracle",
                              "sample": f"all {wl.n_instances} instances, both rates, {cpu_s:.1f} s"},
                matches_oracle_on_sample=same, gpu_launches=5 * args.steps)
    print(json.dumps(line), flush=True)


def run_alu_probe():
    """Rates of themis_alu_probe in all its forms (updates per SM per clock at the boost
    clock, and TOP/s counting two operations per cell update).  Forms 0-4 keep their
    operands in registers; form 5 is the packed kernel's inner step with its operand
    loads from shared memory."""
    import torch
    from paper_2407_14843_b200 import build as _build
    _build.build_library()
    from paper_2407_14843_b200 import solver
    torch.cuda.set_device(0)
    forms = {0: "32-bit add, then unsigned min", 1: "fused 32-bit add-min", 2: "two adds + one three-input min per two updates",
             3: "fused add-min on packed 2 x 16-bit", 4: "single-precision add, then min",
             5: "inner step of the packed recurrence kernel (operands from shared memory)"}
    threads = 256
    out = {}
    for mode, what in forms.items():
        # form 5: 4 blocks per SM as the recurrence kernel runs, 256 steps x 64 cells per iteration
        blocks, warm, iters = (N_SMS * 4, 2, 300) if mode == 5 else (N_SMS * 8, 50, 20000)
        sink = torch.empty(blocks * threads, dtype=torch.uint32, device="cuda")
        solver.themis_alu_probe(mode, blocks, threads, warm, sink)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        solver.themis_alu_probe(mode, blocks, threads, iters, sink)
        b.record()
        torch.cuda.synchronize()
        per_iter = 256 * 64 if mode == 5 else (128 if mode == 3 else 64)
        cells = blocks * threads * iters * per_iter
        rate = cells / (a.elapsed_time(b) * 1e-3)
        out[f"mode{mode}"] = {"form": what, "ms": a.elapsed_time(b), "cell_updates_per_s": rate,
                              "tops": 2.0 * rate / 1e12,
                              "cell_updates_per_sm_per_clock_at_1965mhz": rate / N_SMS / (SM_GHZ * 1e9)}
    print(json.dumps({"alu_probe": out, "derived_peak_tops": {"int32": ALU_PEAK_TOPS_INT32,
                                                              "int16x2": ALU_PEAK_TOPS_INT16X2}}), flush=True)


def main():
    args = parse_args()
    if args.alu_probe:
        run_alu_probe()
    elif args.impl == "reference":
        run_reference(args)
    elif args.entry != "solve":
        run_entry(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
