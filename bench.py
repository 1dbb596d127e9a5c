#!/usr/bin/env python
"""Benchmark of the batched pipeline-scaling solver.

A "step" is one pass of the whole hot path (candidate scoring, min-plus
recurrence, final scan, backtrack) over one batch of synthetic instances.
Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1..5] [--impl reference]

With N > 1 launch under ``python -m torch.distributed.run`` (one rank per GPU);
the batch is replicated per rank with independent seeds (weak scaling, no
collective on the solve path).  ``--impl reference`` times the CPU oracle
instead (rank 0 only).
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

# DRAM bytes (read + write) of one min-plus launch from the ncu capture summarised
# under profiles/, per instance of the captured workload.  Traffic is proportional
# to the instance count (one block per instance, no reuse across blocks).  The
# figure is only reported while the kernel sources still have the recorded hash.
NCU_TRAFFIC = {
    "config": 4, "bytes_per_instance": (315.842304e6 + 156.111616e6) / 2368,
    "sources": ("paper_2407_14843_b200/csrc/themis_minplus16.cu",
                "paper_2407_14843_b200/csrc/themis_minplus16_step.cuh"),
    "sha256_16": "1a1de2cc92ace9e8",
}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=4, help="benchmark configuration 1..5 (default 4: large joint DP)")
    ap.add_argument("--instances", type=int, default=None, help="override the batch size (debugging)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=5)
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


def ncu_traffic_bytes(cfg: int, n_instances: int):
    import hashlib
    try:
        h = hashlib.sha256()
        for src in NCU_TRAFFIC["sources"]:
            with open(os.path.join(ROOT, src), "rb") as f:
                h.update(f.read())
        if h.hexdigest()[:16] != NCU_TRAFFIC["sha256_16"]:
            return None
    except OSError:
        return None
    return NCU_TRAFFIC["bytes_per_instance"] * n_instances if cfg == NCU_TRAFFIC["config"] else None


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

    from paper_2407_14843_b200 import workloads
    wl = workloads.make_workload(args.config, args.instances, seed_offset=rank)
    cpu = None
    if rank == 0:
        _build.build_library()
        if not args.no_cpu_baseline:
            import oracle
            oracle.build()                       # before the first GPU call
            cpu = cpu_baseline(wl)
    torch.cuda.set_device(local_rank)
    # Under a launcher (RANK set) the process group is brought up even for one rank, so that
    # the barrier / max-over-ranks path is the same code at every N.
    use_dist = world > 1 or "RANK" in os.environ
    if use_dist:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    from paper_2407_14843_b200 import solver

    packed = args.minplus_mode == 0
    prob = solver.Problem.of_workload(wl, solver.KERNEL_PACKED16 if packed else solver.KERNEL_WIDE32, args.minplus_tile)
    prob_sparse = solver.Problem.of_workload(wl, solver.KERNEL_SPARSE)
    dev = solver.workload_to_device(wl)
    ws = solver.alloc_workspace(prob, wl.vertical, host_variant=True)
    out = solver.alloc_result(wl.n_instances, wl.n_stages)

    def step(events=None):
        if events:
            events[0].record()
        solver.themis_score_batch(prob, dev["lat_us"], dev["profile_id"], dev["lambda_mrps"], dev["replicas"], ws)
        if events:
            events[1].record()
        solver.themis_minplus_batch(prob, dev["replicas"], out, ws)
        if events:
            events[2].record()

    def barrier():
        torch.cuda.synchronize()
        if use_dist:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(max(args.warmup, 1)):
        step()
    alu_probe_tops = {"int32": probe_alu_peak(solver, torch, 1), "int16x2": probe_alu_peak(solver, torch, 3)} \
        if rank == 0 else None
    barrier()

    uuid = str(getattr(torch.cuda.get_device_properties(local_rank), "uuid", ""))
    sampler = ClockSampler(uuid) if rank == 0 else None
    if sampler:
        sampler.start()
        time.sleep(0.25)
    mk = lambda: torch.cuda.Event(enable_timing=True)
    evs = [[mk(), mk(), mk()] for _ in range(args.steps)]
    barrier()
    for k in range(args.steps):
        step(evs[k])
    barrier()
    clocks = sampler.stop() if sampler else None

    step_ms = sorted(e[0].elapsed_time(e[2]) for e in evs)
    total_ms = evs[0][0].elapsed_time(evs[-1][2])
    score_ms = sum(e[0].elapsed_time(e[1]) for e in evs) / args.steps
    minplus_ms = sum(e[1].elapsed_time(e[2]) for e in evs) / args.steps
    t = torch.tensor([total_ms, score_ms, minplus_ms], dtype=torch.float64, device="cuda")
    if use_dist:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    total_ms, score_ms, minplus_ms = t.tolist()

    # The same batch through the solver restricted to undominated entries (mode 3: one fused
    # kernel; identical results, a small fraction of the cell updates): reported beside the
    # dense figures, not as them.
    pruned = None
    if args.pruned_steps > 0:
        dense_out = {k: v.clone() for k, v in out.items()}

        def sparse_step():
            if wl.vertical:
                solver.themis_solve_vertical_batch(prob_sparse, dev["lat_us"], dev["profile_id"], dev["lambda_mrps"],
                                                   dev["replicas"], out, ws)
            else:
                solver.themis_solve_batch(prob_sparse, dev["lat_us"], dev["profile_id"], dev["lambda_mrps"], out, ws)

        sparse_step()
        barrier()
        pe = [mk() for _ in range(args.pruned_steps + 1)]
        pe[0].record()
        for k in range(args.pruned_steps):
            sparse_step()
            pe[k + 1].record()
        barrier()
        tp = torch.tensor([pe[0].elapsed_time(pe[-1])], dtype=torch.float64, device="cuda")
        if use_dist:
            dist.all_reduce(tp, op=dist.ReduceOp.MAX)
        p_total = float(tp.item())
        pruned = {"value": wl.n_instances * world * args.pruned_steps / (p_total * 1e-3), "unit": UNIT,
                  "ms_per_step": p_total / args.pruned_steps, "steps": args.pruned_steps,
                  "kernel": "solve_front_kernel + solve_sparse_kernel for listed instances (memset + 2 launches per step)",
                  "same_results_as_dense": all(bool((out[k] == dense_out[k]).all()) for k in out),
                  "note": "THEMIS_KERNEL_SPARSE: scoring, fronts and recurrence on undominated "
                          "entries in one kernel, one warp per instance"}

    status = out["status"].cpu()
    n_infeasible = int((status == 1).sum())
    n_error = int((status < 0).sum())

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
    e2e_s = time.perf_counter() - t0
    t = torch.tensor([e2e_s], dtype=torch.float64, device="cuda")
    if use_dist:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    e2e_s = float(t.item())
    h2d = sum(x.numel() * x.element_size() for x in h_in.values() if x is not None)
    d2h = sum(x.numel() * x.element_size() for x in h_out.values())
    same = all(bool((h_out[k] == out[k].cpu()).all()) for k in h_out)

    if use_dist:
        dist.barrier()
        dist.destroy_process_group()
    if rank != 0:
        return

    N_total = wl.n_instances * world
    # score + min-plus, plus the 32-bit second pass where a total may exceed 15 bits
    second_pass = packed and (wl.vertical or wl.n_stages * wl.h_max * wl.c_max >= 0x7FFF)
    launches_per_step = 3 if second_pass else 2
    cells_per_launch = wl.n_instances * wl.minplus_cells
    achieved_tops = 2.0 * cells_per_launch / (minplus_ms * 1e-3) / 1e12
    alu_peak = ALU_PEAK_TOPS_INT16X2 if packed else ALU_PEAK_TOPS_INT32
    lay = solver.themis_workspace_layout(prob, wl.vertical)
    score_bytes = 6.0 * lay.row_pitch * wl.n_instances * wl.n_stages
    hbm_peak, hbm_kind = measured_hbm_peak()
    score_gbs = score_bytes / (score_ms * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": N_total * args.steps / (total_ms * 1e-3), "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_ms / args.steps,
        "ms_per_step_best": step_ms[0], "ms_per_step_median": step_ms[len(step_ms) // 2],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        # arithmetic of the dominant kernel: packed pairs of unsigned 16-bit costs, or 32-bit keys
        "dtype": "u16" if packed else "u32",
        "data": "synthetic", "config": workload_config(wl, args, world),
        "cell_updates_per_s": world * cells_per_launch * args.steps / (total_ms * 1e-3),
        "minplus_cell_updates_per_s_kernel": cells_per_launch / (minplus_ms * 1e-3),
        "kernels_ms": {"score_kernel": score_ms, ("minplus16_kernel" if packed else "minplus_kernel"): minplus_ms},
        "infeasible_instances": n_infeasible, "device_error_instances": n_error,
        "input_checksums": wl.checksums(),
        "device": {"name": torch.cuda.get_device_name(local_rank),
                   "sms": torch.cuda.get_device_properties(local_rank).multi_processor_count},
        "roofline": {
            "kernel": "minplus16_kernel" if packed else "minplus_kernel", "bound": "alu",
            "achieved": achieved_tops, "peak": alu_peak,
            "unit": "TOP/s (integer add+min, 2 per cell update)", "frac": achieved_tops / alu_peak,
            "traffic": ncu_traffic_bytes(args.config, wl.n_instances) if packed else None,
            "peak_kind": ("derived: 148 SMs x 64 int lanes x 2 ops x 1.965 GHz"
                          + (" x 2 half-word cells per lane (packed 16-bit add-min)" if packed else "")),
            "peak_probe": alu_probe_tops, "frac_of_int32_peak": achieved_tops / ALU_PEAK_TOPS_INT32,
            "algorithmic_cells_per_launch": cells_per_launch, "avg_launch_ms": minplus_ms,
        },
        "roofline_score_kernel": {
            "kernel": "score_kernel", "bound": "hbm", "achieved": score_gbs, "peak": hbm_peak, "unit": "GB/s",
            "frac": score_gbs / hbm_peak, "traffic": None, "peak_kind": f"of {hbm_kind}",
            "algorithmic_bytes_per_launch": score_bytes, "avg_launch_ms": score_ms,
        },
        "e2e": {"value": N_total * args.e2e_steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": args.e2e_steps, "matches_device_path": same},
        "gpu_launches": launches_per_step * args.steps,
        "clocks": clocks,
    }
    if pruned is not None:
        line["pruned_path"] = pruned
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
