"""Parity at the benchmark's full size and launch configuration (100,000 jobs, packed histories)."""

import numpy as np
import pytest

from workloads import make_workload
from gpu_common import compare_epoch, make_scheduler, oracle_epoch, oracle_spread, tolerance_widths

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
    width = tolerance_widths(pred, ref)
    print("config 3 full size:", info, sched.get_stats().as_dict())
    print("distance from the oracle in tolerances, quantiles 50 / 99 / 99.9 / 100 %:",
          np.round(np.quantile(width, [0.5, 0.99, 0.999, 1.0]), 4))
    assert width.max() <= 1.0             # measured: 0.78 at worst, 99.9 % of the jobs within 0.02
    assert alloc.sum() == wl.total_cores


def test_config4_full_size_every_job(oracle_mod):
    """1,000,000 jobs, ring of 64, 128 cores per job: the predictions of every job against the oracle one by one,
    and the allocation entry by entry - against the oracle's greedy loop fed the GPU's gain table (bit for bit), and
    against the oracle's own whole epoch (equal except within rounding of the threshold).
    A job may miss the tolerance on R(n) only where the oracle's own result moves as much when its losses are
    perturbed by 1e-13 (unfinished fits of nearly flat windows; measured: 9 of the 1,000,000)."""
    import paper_1802_04819_b200 as slaq
    slaq.build()
    wl = make_workload(4)
    sched = make_scheduler(wl)
    alloc, rc = sched.schedule(wl.epoch_seconds, wl.total_cores)
    assert rc == 0
    pred = sched.get_predictions()
    cap = wl.max_cores_per_job
    ref = oracle_mod.predict(wl.offsets, wl.losses, wl.m_seen, wl.s, wl.w, wl.epoch_seconds, cap)
    np.testing.assert_array_equal(pred["status"], ref["status"])
    np.testing.assert_array_equal(pred["M"], ref["M"])
    tied = pred["family"] != ref["family"]          # flat windows: both families end as the same constant
    S = ref["S"][tied]
    assert (np.abs(S[:, 0] - S[:, 1]) <= 1e-9 * np.abs(S).max(axis=1)).all()
    misses = []
    for lo in range(0, wl.n_jobs, 100_000):          # in blocks, to bound the memory of the cumulative sums
        hi = lo + 100_000
        Rg, Rc = np.cumsum(pred["gain"][lo:hi], axis=1), np.cumsum(ref["gain"][lo:hi], axis=1)
        tol = 1e-6 * np.abs(Rc) + 1e-9
        width = (np.abs(Rg - Rc) / tol).max(axis=1)
        for j in np.nonzero((width > 1.0) & ~tied[lo:hi])[0]:
            spread = oracle_spread(oracle_mod, wl, lo + j, cap)
            assert (np.abs(Rg[j] - Rc[j]) <= 4.0 * spread + tol[j]).all(), f"job {lo + j}: {width[j]:.2f} tolerances off"
            misses.append((int(lo + j), float(width[j])))
    print("config 4 full size: misses", misses, "tied winners", int(tied.sum()))
    assert len(misses) <= wl.n_jobs // 25_000
    # allocation: all cores handed out, floor and cap respected, and it is a top-C selection of the GPU's own gains:
    # every gain taken beyond the floor is at least as large as every gain left
    assert alloc.sum() == wl.total_cores and alloc.min() >= 1 and alloc.max() <= cap
    g = pred["gain"]
    cols = np.arange(cap)[None, :]
    taken = (cols < alloc[:, None]) & (cols >= 1)
    left = cols >= alloc[:, None]
    tau = g[taken].min()
    assert g[left].max() <= tau
    # ties at the threshold go to the lowest job ids
    at_tau_taken = np.nonzero(((g == tau) & taken).any(axis=1))[0]
    at_tau_left = np.nonzero(((g == tau) & left).any(axis=1))[0]
    if at_tau_taken.size and at_tau_left.size:
        assert at_tau_taken.max() <= at_tau_left.min()
    dst = np.nonzero(wl.clone_of >= 0)[0]
    np.testing.assert_array_equal(g[dst], g[wl.clone_of[dst]])
    # bit for bit the allocation of the literal greedy loop (a heap of one offer per job, one core per pop) run
    # on the CPU over the same 1,000,000 x 128 gain table, exact ties of the clones included
    active = np.ones(wl.n_jobs, np.uint8)
    np.testing.assert_array_equal(alloc, oracle_mod.allocate(g, active, wl.total_cores))
    # and the oracle's own epoch (its own gains): different only where a deciding gain is within rounding of the threshold
    own = oracle_mod.allocate(ref["gain"], active, wl.total_cores)
    for j in np.nonzero(own != alloc)[0]:
        a, b = sorted((int(own[j]), int(alloc[j])))
        assert np.all(np.abs(ref["gain"][j, a:b] - tau) <= 1e-9 + 1e-6 * tau)
    R_direct = np.where(cols < alloc[:, None], g, 0.0).sum(axis=1)
    np.testing.assert_allclose(pred["R"], R_direct, rtol=1e-12, atol=1e-15)
