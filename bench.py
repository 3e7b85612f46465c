"""Benchmark of the per-epoch scheduling path: jobs scheduled per second at 100,000 jobs.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

One step = one whole scheduling epoch (normalise, fit, predict, allocate) over the
100,000-job synthetic workload (config 3: ragged histories of 3..1000 losses stored
packed with a CSR offsets array, 400,000 cores, at most 64 per job, T = 1 s).
Prints one JSON line.  With N > 1 (under torchrun) every rank schedules its own
100,000-job cluster partition; there is no exchange on the data path.
"""

from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

from workloads import make_workload, true_curve  # noqa: E402

CFG = 3
METRIC = "jobs_scheduled_per_second"
UNIT = "jobs/s"
WARM_TRIALS = 5   # trials per epoch of the warm-started loop reported beside the headline
# algorithmic fp64 work of the fit, per stored point: one sweep of family I, one of family II, set-up
FLOP_SWEEP_I, FLOP_SWEEP_II, FLOP_SETUP = 40.0, 25.0, 40.0
FP64_LANES_PER_SM = 64          # fp64 FMA lanes per SM on B200
# The sweep of the fit issues 43 fp64 arithmetic instructions per point for its 65 algorithmic flop: 86 cycles per
# warp row of 32 points and sub-partition at the pipe's 2 cycles per instruction, 90 with the 4 fused multiply-adds on
# three different registers, which take 3 (measured with bench_probes/fp64_issue_probe)
SWEEP_FLOP_PER_POINT, SWEEP_ISSUE_CYCLES_PER_ROW = FLOP_SWEEP_I + FLOP_SWEEP_II, 90.0
SUBPARTITIONS_PER_SM = 4
MIN_TIMED_SECONDS = 1.0   # the block of --steps steps is repeated until the timed region is at least this long
# DRAM bytes per stored loss moved by the fit kernel (ncu: dram__bytes_read.sum + dram__bytes_write.sum =
# 166.16 MB + 13.31 MB on a 20,068,408-loss cut of this workload, profiles/fit_kernel_40k_jobs.md; traffic grows
# with the stored losses)
NCU_FIT_DRAM_BYTES_PER_LOSS = (166.16e6 + 13.31e6) / 20_068_408


from paper_1802_04819_b200.partition import max_over_ranks, partition_seed_offset, rank_info, whole_job_rate  # noqa: E402


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.rows.append((time.perf_counter(), [c.strip() for c in line.split(",")]))

    def stop(self, t_from=0.0, t_to=float("inf")):
        """Summary of the samples that arrived within [t_from, t_to] (perf_counter seconds)."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for stamp, row in self.rows:
            if len(row) < 7 or not (t_from <= stamp <= t_to + 0.15):
                continue
            try:
                sm.append(float(row[0]))
                mx.append(float(row[1]))
            except ValueError:
                continue
            for name, val in zip(names, row[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def next_losses(wl, step: int, rng):
    """The loss each job would report `step + 1` iterations after its stored window (same generator law)."""
    k = (wl.k_last + 1 + step).astype(np.float64)
    clean = true_curve(wl.family, wl.params, k)
    return clean * np.exp(wl.sigma * rng.standard_normal(wl.n_jobs))


def measured_peaks():
    path = ROOT / "MEASURED_PEAKS.json"
    if path.exists():
        return json.loads(path.read_text()), "measured"
    return {"hbm_gbs": 6650.0, "sm_max_mhz": 1965.0}, "fallback"


def measured_fp64_peak():
    """Best fused multiply-add rate of the fp64 pipe on this GPU, measured now with bench_probes/fp64_issue_probe
    (12 independent accumulators per thread, 16 warps per SM).  Returns (TFLOP/s, note) or (None, why)."""
    exe = ROOT / "bench_probes" / "fp64_issue_probe"
    try:
        if not exe.exists():
            sys.path.insert(0, str(ROOT / "bench_probes"))
            import build_probes as probe_build   # bench_probes/build_probes.py
            probe_build.build_probes()
        out = subprocess.run([str(exe)], capture_output=True, text=True, timeout=120, check=True).stdout
    except (OSError, subprocess.SubprocessError, ImportError) as err:
        return None, f"fp64_issue_probe did not run: {err}"
    best = 0.0
    for row in out.splitlines():
        cols = row.split()
        if len(cols) == 4 and cols[0].startswith("fma"):
            best = max(best, float(cols[3]))
    return (best, "best fused multiply-add rate of bench_probes/fp64_issue_probe, run before the timed region") \
        if best > 0 else (None, "fp64_issue_probe printed no rate")


def host_threads() -> int:
    """Host cores this process may use (launchers often set OMP_NUM_THREADS=1: the oracle is told explicitly)."""
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return max(1, os.cpu_count() or 1)


def run_reference(args):
    """The CPU oracle, as it stands, on a bounded sample of the same workload.

    The sample (the first jobs of the config-3 generator) is sized from one calibration step so that the
    whole --steps/--warmup run stays within about two minutes."""
    rank, _, world = rank_info()
    if rank != 0:
        return
    import oracle
    oracle.build()
    cores = host_threads()

    def step(wl):
        return oracle.schedule(wl.offsets, wl.losses, wl.m_seen, wl.s, wl.w, wl.epoch_seconds, wl.total_cores,
                               wl.max_cores_per_job, threads=cores)

    probe = make_workload(CFG, n_jobs=1000)
    step(probe)
    t0 = time.perf_counter()
    step(probe)
    per_job = (time.perf_counter() - t0) / probe.n_jobs
    budget = 120.0 / (args.steps + args.warmup)
    sample_jobs = int(min(20_000, max(500, budget / per_job)))
    wl = make_workload(CFG, n_jobs=sample_jobs)
    for _ in range(args.warmup):
        step(wl)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step(wl)
    dt = (time.perf_counter() - t0) / args.steps
    value = sample_jobs / dt
    sample = (f"first {sample_jobs} jobs of the config-3 generator ({int(wl.offsets[-1])} stored losses), "
              f"one epoch per step")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "config3_100k_jobs_400k_cores_cap64_hist3-1000_csr", "sample_jobs": sample_jobs},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_gpu(args):
    import torch
    rank, local_rank, world = rank_info()
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU path)"
    torch.cuda.set_device(local_rank)
    import paper_1802_04819_b200 as slaq
    slaq.build()

    wl = make_workload(args.cfg, n_jobs=args.jobs, seed_offset=partition_seed_offset(rank))   # each rank: its own partition
    J, cap = wl.n_jobs, wl.max_cores_per_job
    ids = np.arange(J, dtype=np.int32)
    stream = torch.cuda.current_stream()
    sched = slaq.Scheduler(J, wl.max_hist, cap, stream=stream)
    sched.load_histories(ids, wl.offsets, wl.losses, wl.k_last, wl.m_seen, packed=args.cfg == CFG)   # config 4: rings
    sched.set_time_model(ids, wl.s, wl.w)
    if args.selection is not None:
        sched.set_param(slaq.binding.P_SELECTION, args.selection)
    d_alloc = torch.zeros(J, dtype=torch.int32, device="cuda")

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident throughput ----
    sampler = ClockSampler(local_rank)
    sampler.start()                      # nvidia-smi needs a moment to start: the warm-up covers it
    for _ in range(args.warmup):
        sched.schedule_device(wl.epoch_seconds, wl.total_cores, d_alloc)
    torch.cuda.synchronize()
    pred = sched.get_predictions(want_gain=False)
    fitted = pred["status"] == 0
    H = wl.hist_len.astype(np.float64)
    fit_flops = float((H[fitted] * (FLOP_SWEEP_I * pred["evals"][fitted, 0] + FLOP_SWEEP_II * pred["evals"][fitted, 1]
                                    + FLOP_SETUP)).sum())
    fp64_peak_measured, fp64_peak_note = measured_fp64_peak() if rank == 0 else (None, "")
    barrier()
    # The timed block is exactly --steps epochs between a barrier + synchronise on both sides.  It is repeated
    # until the region lasts MIN_TIMED_SECONDS (a clock excursion then shows in the sampled clocks and in the
    # spread of the blocks); the reported step time is the median block's.
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    fit_ms, stage_ms, launches, block_ms = [], [], 0, []
    t_from = time.perf_counter()
    while True:
        barrier()
        ev0.record(stream)
        for _ in range(args.steps):
            sched.schedule_device(wl.epoch_seconds, wl.total_cores, d_alloc)
            st = sched.get_stats()                 # reads the library's own per-stage CUDA events (same stream)
            fit_ms.append(st.ms_fit)
            stage_ms.append((st.ms_fit, st.ms_gain, st.ms_alloc))
            if not block_ms:
                launches += st.launches            # kernels of one block of --steps steps
        ev1.record(stream)
        barrier()
        block_ms.append(ev0.elapsed_time(ev1))
        enough = time.perf_counter() - t_from >= args.min_seconds
        if world > 1:                              # every rank runs the same number of blocks
            flag = torch.tensor([1.0 if enough else 0.0], device="cuda")
            dist.all_reduce(flag, op=dist.ReduceOp.MIN)
            enough = bool(flag.item() > 0)
        if enough or len(block_ms) >= 1000:
            break
    clocks = sampler.stop(t_from, time.perf_counter())
    ms_step = float(np.median(block_ms)) / args.steps
    alloc_dev = d_alloc.cpu().numpy()
    assert int(alloc_dev.sum()) == wl.total_cores

    # ---- end to end through the host-pointer calls: append one new loss per job, schedule, read the allocation ----
    rng = np.random.default_rng(99 + rank)
    pin = lambda n, dt: torch.empty(n, dtype=dt).pin_memory().numpy()   # noqa: E731
    h_ids, h_time = pin(J, torch.int32), pin(J, torch.float64)
    h_alloc = pin(J, torch.int32)
    h_ids[:] = ids
    e2e_steps = max(1, args.steps)
    # every step's input (one new loss per job and the seconds its iteration took) waits in pinned host memory
    feeds = []
    for s in range(2 * (args.warmup + e2e_steps)):
        buf = pin(J, torch.float64)
        buf[:] = next_losses(wl, s, rng)
        feeds.append(buf)
    h_time[:] = wl.s + wl.w / np.maximum(alloc_dev.astype(np.float64), 1.0)

    def e2e_step(k):
        sched.append_losses(h_ids, feeds[k], h_time)
        sched.schedule(wl.epoch_seconds, wl.total_cores, out_alloc=h_alloc)

    for k in range(args.warmup):
        e2e_step(k)
    barrier()
    t0 = time.perf_counter()
    for k in range(e2e_steps):
        e2e_step(args.warmup + k)
    torch.cuda.synchronize()
    e2e_s = (time.perf_counter() - t0) / e2e_steps
    assert int(h_alloc.sum()) == wl.total_cores

    # ---- the same loop with warm-started refits: 5 trials per epoch from last epoch's curves (reported beside
    # the headline, not instead of it: the headline fits every job from its first guess with 20 trials) ----
    sched.set_param(slaq.binding.P_WARM_START, 1)
    sched.set_param(slaq.binding.P_LM_TRIALS, WARM_TRIALS)
    base = args.warmup + e2e_steps
    for k in range(args.warmup):
        e2e_step(base + k)
    barrier()
    t0 = time.perf_counter()
    warm_fit_ms = []
    for k in range(e2e_steps):
        e2e_step(base + args.warmup + k)
        warm_fit_ms.append(sched.get_stats().ms_total)
    torch.cuda.synchronize()
    warm_s = (time.perf_counter() - t0) / e2e_steps
    assert int(h_alloc.sum()) == wl.total_cores

    # ---- one cluster sharded over several handles (the multi-GPU protocol: a histogram sum per radix pass and one
    # exchange of tie counts).  With one GPU: the same 100,000 jobs as two shards of 50,000 on this GPU, sums done
    # locally - the protocol's overhead against the single handle.  With N GPUs: the N partitions as ONE cluster of
    # N x 100,000 jobs, one shard per rank, sums over NCCL.  Reported beside the headline, never instead of it. ----
    sharded = None
    try:
        if world > 1 and not args.sharded:
            raise RuntimeError("not run: with several GPUs this leg needs --sharded (its NCCL path has never run on "
                               "hardware; a rank that failed inside it would leave the others waiting)")
        sched.set_param(slaq.binding.P_WARM_START, 0)
        sched.set_param(slaq.binding.P_LM_TRIALS, 20)
        reps = max(3, min(args.steps, 20))
        if world == 1:
            half = J // 2
            shards = []
            for lo, hi in ((0, half), (half, J)):
                sh = slaq.Scheduler(hi - lo, wl.max_hist, cap, stream=stream)
                sh.load_histories(np.arange(hi - lo, dtype=np.int32), wl.offsets[lo:hi + 1] - wl.offsets[lo],
                                  wl.losses[wl.offsets[lo]:wl.offsets[hi]], wl.k_last[lo:hi], wl.m_seen[lo:hi],
                                  packed=args.cfg == CFG)
                sh.set_time_model(np.arange(hi - lo, dtype=np.int32), wl.s[lo:hi], wl.w[lo:hi])
                shards.append(sh)
            exchange, cluster_cores = slaq.LocalExchange(), wl.total_cores
        else:
            shards, exchange, cluster_cores = [sched], slaq.ProcessGroupExchange(), world * wl.total_cores
        for _ in range(args.warmup):
            parts = slaq.schedule_sharded(shards, exchange, wl.epoch_seconds, cluster_cores)
        barrier()
        t0 = time.perf_counter()
        for _ in range(reps):
            parts = slaq.schedule_sharded(shards, exchange, wl.epoch_seconds, cluster_cores)
        torch.cuda.synchronize()
        shard_ms = (time.perf_counter() - t0) / reps * 1e3
        handed = sum(int(p.sum()) for p in parts)
        same = bool(world > 1 or np.array_equal(np.concatenate(parts), alloc_dev))
        sharded = {"ms_per_epoch": max_over_ranks([shard_ms], device="cuda")[0], "shards": len(shards) * world,
                   "jobs_in_the_cluster": J * world, "epochs_timed": reps, "cores_handed_out_by_this_rank": handed,
                   "equals_single_handle": same if world == 1 else None,
                   "what": "wall clock per epoch of schedule_sharded (host waits once, for the allocation); with one GPU "
                           "two local shards of the benchmark's jobs, with N GPUs one shard per rank over NCCL"}
        if world == 1:
            for sh in shards:
                sh.close()
    except Exception as err:   # the headline must not depend on this leg
        sharded = {"error": f"{type(err).__name__}: {err}"}

    ms_step, e2e_ms, warm_ms = max_over_ranks([ms_step, e2e_s * 1e3, warm_s * 1e3], device="cuda")

    if rank == 0:
        peaks, peak_kind = measured_peaks()
        sm_max = float(peaks.get("sm_max_mhz", 1965.0))
        sm_count = torch.cuda.get_device_properties(local_rank).multi_processor_count
        peak_tflops = sm_count * FP64_LANES_PER_SM * 2 * sm_max * 1e6 / 1e12
        issue_bound = (SWEEP_FLOP_PER_POINT * 32 / SWEEP_ISSUE_CYCLES_PER_ROW) * SUBPARTITIONS_PER_SM * sm_count * sm_max * 1e6 / 1e12
        fit_ms_avg = float(np.mean(fit_ms))
        achieved = fit_flops / (fit_ms_avg * 1e-3) / 1e12
        stage = np.mean(np.array(stage_ms), axis=0)
        line = {
            "metric": METRIC, "value": whole_job_rate(J, world, ms_step), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "config3_100k_jobs_400k_cores_cap64_hist3-1000_csr"
                       if args.jobs is None and args.cfg == CFG
                       else f"config {args.cfg} generator at {J} jobs (profiling run, not the benchmark)",
                       "jobs_per_gpu": J,
                       "stored_losses_per_gpu": int(wl.offsets[-1]), "total_cores_per_gpu": wl.total_cores,
                       "max_cores_per_job": cap, "epoch_seconds": wl.epoch_seconds,
                       "l2": f"inputs larger than L2 ({int(wl.offsets[-1]) * 8 / 1e6:.0f} MB of losses read per step)",
                       "parallelism": f"{world} independent cluster partition(s), one per GPU"},
            "clocks": clocks,
            "timed_blocks": {"blocks": len(block_ms), "steps_per_block": args.steps, "ms_per_step_median": ms_step,
                             "ms_per_step_min": float(np.min(block_ms)) / args.steps,
                             "ms_per_step_max": float(np.max(block_ms)) / args.steps,
                             "what": "the block of --steps epochs, repeated until the timed region lasts one second; "
                                     "value and ms_per_step come from the median block"},
            "e2e": {"value": whole_job_rate(J, world, e2e_ms), "unit": UNIT, "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": int(J * (4 + 8 + 8)), "d2h_bytes_per_step": int(J * 4 + 4),
                    "steps": e2e_steps,
                    "what": "slaq_append_losses (host arrays, one new loss per job) + slaq_schedule (host out_alloc)"},
            "warm_refit": {"value": whole_job_rate(J, world, warm_ms), "unit": UNIT, "ms_per_step": warm_ms,
                           "device_ms_per_epoch": float(np.mean(warm_fit_ms)), "lm_trials": WARM_TRIALS,
                           "steps": e2e_steps,
                           "what": "the end-to-end loop with SLAQ_P_WARM_START = 1: every family starts from the "
                                   "curve it ended with last epoch and runs 5 trials instead of 20"},
            "sharded_cluster": sharded,
            "gpu_launches": launches,
            "stage_ms": {"fit": float(stage[0]), "gain": float(stage[1]), "alloc": float(stage[2])},
            "roofline": {"bound": "alu", "kernel": "fit_kernel", "achieved": achieved, "peak": peak_tflops,
                         "unit": "TFLOP/s", "frac": achieved / peak_tflops,
                         "traffic": NCU_FIT_DRAM_BYTES_PER_LOSS * int(wl.offsets[-1]),
                         "traffic_note": "bytes per launch, scaled by stored losses from the ncu capture of a 40,000-job cut",
                         "algorithmic_flops_per_launch": fit_flops, "ms_per_launch": fit_ms_avg,
                         "issue_bound_peak": issue_bound, "frac_of_issue_bound": achieved / issue_bound,
                         "issue_bound_note": "a loop of nothing but the fit's sweeps at the measured issue rates: 65 flop "
                                             "per point on 43 fp64 instructions, 90 cycles per warp row of 32 points",
                         "peak_is": f"{sm_count} SMs x {FP64_LANES_PER_SM} fp64 FMA lanes x 2 x {sm_max:.0f} MHz "
                                    f"(clock from MEASURED_PEAKS.json: {peak_kind}; that file holds no fp64 figure)",
                         "peak_measured": fp64_peak_measured,
                         "frac_of_peak_measured": achieved / fp64_peak_measured if fp64_peak_measured else None,
                         "peak_measured_is": fp64_peak_note},
        }
        if args.cpu_baseline:
            import oracle
            oracle.build()
            cores = host_threads()
            t0 = time.perf_counter()
            oracle.schedule(wl.offsets, wl.losses, wl.m_seen, wl.s, wl.w, wl.epoch_seconds, wl.total_cores, cap,
                            threads=cores)
            dt = time.perf_counter() - t0
            line["cpu_baseline"] = {"value": J / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
                                    "sample": f"the whole workload of this line ({J} jobs), one epoch, run once", "seconds": dt}
        print(json.dumps(line), flush=True)
    sched.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", dest="cpu_baseline", action="store_false")
    ap.add_argument("--cfg", type=int, default=CFG, choices=[2, 3, 4],
                    help="profiling aid: another workload generator (the reported line is then not the benchmark)")
    ap.add_argument("--sharded", action="store_true",
                    help="with --gpus N > 1: also time the N partitions as ONE cluster sharded over the ranks (NCCL)")
    ap.add_argument("--min-seconds", type=float, default=MIN_TIMED_SECONDS,
                    help="the block of --steps steps is repeated until the timed region lasts this long (0: one block; "
                         "for runs under a profiler)")
    ap.add_argument("--selection", type=int, default=None, choices=[0, 1],
                    help="profiling aid: threshold selection over the gain table (0) or without a table (1)")
    ap.add_argument("--jobs", type=int, default=None,
                    help="profiling aid: a smaller cut of the same generator (the reported line is then not the benchmark)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
