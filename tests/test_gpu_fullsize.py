"""Parity at the benchmark's full size and launch configuration (100,000 jobs, packed histories)."""

import numpy as np
import pytest

from workloads import make_workload
from gpu_common import compare_epoch, make_scheduler, oracle_epoch

pytestmark = pytest.mark.gpu


def test_config3_full_size_all_jobs(oracle_mod):
    import paper_1802_04819_b200 as slaq
    slaq.build()
    wl = make_workload(3)
    sched = make_scheduler(wl, packed=True)
    alloc, rc = sched.schedule(wl.epoch_seconds, wl.total_cores)
    assert rc == 0
    pred = sched.get_predictions()
    ref = oracle_epoch(oracle_mod, wl)            # OpenMP over jobs on the host cores
    info = compare_epoch(alloc, pred, ref, wl.total_cores, wl.max_cores_per_job)
    print("config 3 full size:", info, sched.get_stats().as_dict())
    assert alloc.sum() == wl.total_cores
