"""Where the warps of the fit kernel spend their time: phase clocks on the benchmark workload.

    python bench_probes/fit_phase_split.py [--jobs N] [--cfg 3]

Builds the "clocks" variant of the library (the same sources with -DSLAQ_PHASE_CLOCKS: lane 0 of
every warp reads clock64() at the phase boundaries, nothing is skipped), schedules the workload
with it and with the ordinary library, and prints per phase the share of the warps' cycles and
that share of the ordinary library's fit time.  Also prints the cycles a sub-partition spends per
warp row of a trial sweep inside the kernel: (cycles in phase 3 / warps per sub-partition) / rows
swept, to set beside fit_sweep_probe's figure for the sweep alone.
"""

from __future__ import annotations

import argparse
import sys
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent.parent
sys.path.insert(0, str(ROOT))

PHASES = ["staging + normalisation", "first guesses + first sweep", "solver steps", "trial sweeps + reductions",
          "winner + record", "queue + statistics"]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--cfg", type=int, default=3)
    ap.add_argument("--jobs", type=int, default=None)
    args = ap.parse_args()
    import torch
    assert torch.cuda.is_available(), "needs a CUDA device"
    import paper_1802_04819_b200 as slaq
    from paper_1802_04819_b200.build import build_variant
    from workloads import make_workload
    slaq.build()
    build_variant("clocks")
    wl = make_workload(args.cfg, n_jobs=args.jobs)
    ids = np.arange(wl.n_jobs, dtype=np.int32)
    result = {}
    for variant in (None, "clocks"):
        sched = slaq.Scheduler(wl.n_jobs, wl.max_hist, wl.max_cores_per_job, variant=variant)
        sched.load_histories(ids, wl.offsets, wl.losses, wl.k_last, wl.m_seen, packed=args.cfg == 3)
        sched.set_time_model(ids, wl.s, wl.w)
        ms = []
        for _ in range(8):
            sched.schedule_device(wl.epoch_seconds, wl.total_cores)
            ms.append(sched.get_stats().ms_fit)
        result[variant] = (float(np.median(ms[3:])), sched.get_fit_phase_cycles(), sched.get_predictions(want_gain=False))
        sched.close()
    ms_plain, _, pred = result[None]
    ms_clocked, cycles, _ = result["clocks"]
    total = cycles.sum()
    print(f"config {args.cfg}, {wl.n_jobs} jobs, {int(wl.offsets[-1])} stored losses")
    print(f"fit stage: {ms_plain:.3f} ms (ordinary library), {ms_clocked:.3f} ms (with phase clocks)")
    print(f"{'phase':34s} {'share of warp cycles':>22s} {'of the fit stage, ms':>22s}")
    for name, c in zip(PHASES, cycles):
        print(f"{name:34s} {c / total:22.3f} {ms_plain * c / total:22.3f}")
    fitted = pred["status"] == 0
    H = wl.hist_len[fitted].astype(np.float64)
    trial_rows = float((H * (pred["evals"][fitted].max(axis=1) - 1)).sum()) / 32.0   # rows of 32 points, both families in one sweep
    print(f"trial sweeps: about {trial_rows:.3e} warp rows; phase 3 = {cycles[3] / 4.0 / trial_rows:.1f} cycles per "
          f"warp row and sub-partition (4 warps per sub-partition share it)")


if __name__ == "__main__":
    main()
