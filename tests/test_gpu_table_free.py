"""Selection without a gain table (SLAQ_P_SELECTION = 1): binary searches over each job's falling gains instead of a
written table.  Same tolerances against the oracle as the table path; against the table path itself the allocation
may differ only where a deciding gain sits within rounding of the threshold."""

import numpy as np
import pytest

from workloads import make_workload
from gpu_common import compare_epoch, make_scheduler, oracle_epoch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def slaq():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import paper_1802_04819_b200 as mod
    mod.build()
    return mod


def _both_ways(slaq, wl, C, packed=False):
    sched = make_scheduler(wl, packed=packed)
    sched.set_param(slaq.binding.P_EPOCH_GRAPH, 0)
    table, rc_t = sched.schedule(wl.epoch_seconds, C)
    pred_t = sched.get_predictions()
    sched.set_param(slaq.binding.P_SELECTION, 1)
    free, rc_f = sched.schedule(wl.epoch_seconds, C)
    stats = sched.get_stats()
    pred_f = sched.get_predictions()          # the gain rows are written on request
    assert rc_t == rc_f
    return sched, table, pred_t, free, pred_f, stats


@pytest.mark.parametrize("cfg,n_jobs,packed", [(0, None, False), (1, None, False), (2, None, True), (3, 3000, True),
                                               (4, 20000, False), (4, 30000, False)])
def test_table_free_epoch_matches_the_oracle_and_the_table(slaq, oracle_mod, cfg, n_jobs, packed):
    wl = make_workload(cfg, n_jobs=n_jobs)
    ref = oracle_epoch(oracle_mod, wl)
    sched, table, pred_t, free, pred_f, stats = _both_ways(slaq, wl, wl.total_cores, packed)
    compare_epoch(free, pred_f, ref, wl.total_cores, wl.max_cores_per_job)
    assert free.sum() == wl.total_cores == stats.cores_handed_out
    assert free.min() >= 1 and free.max() <= wl.max_cores_per_job
    np.testing.assert_array_equal(pred_f["gain"], pred_t["gain"])       # the rows written on request are the table's
    diff = np.nonzero(free != table)[0]
    assert diff.size <= max(2, wl.n_jobs // 2000)
    tau = stats.threshold
    for j in diff:                              # only gains within rounding of the threshold may change hands
        lo, hi = sorted((free[j], table[j]))
        assert np.all(np.abs(pred_t["gain"][j, lo:hi] - tau) <= 1e-12 * tau + 1e-300)
    same = free == table
    np.testing.assert_allclose(pred_f["R"][same], pred_t["R"][same], rtol=1e-13, atol=0)


def test_table_free_edge_cases(slaq, oracle_mod):
    wl = make_workload(2, n_jobs=900)
    J, cap = wl.n_jobs, wl.max_cores_per_job
    for C in (0, 1, J - 1, J, J + 1, 3 * J + 5, J * cap - 1, J * cap, J * cap + 9):
        sched, table, pred_t, free, pred_f, stats = _both_ways(slaq, wl, C)
        ref = oracle_epoch(oracle_mod, wl, total_cores=C)
        compare_epoch(free, pred_f, ref, C, cap)
        assert free.sum() == min(C, J * cap)
        sched.close()
    # inactive ids, jobs that predict nothing (flat, no time law) and one-point jobs beside ordinary ones
    sched = slaq.Scheduler(40, 16, 8)
    ref = oracle_mod.OracleScheduler(40, 16, 8)
    rng = np.random.default_rng(2)
    for step in range(12):
        ids = [j for j in range(0, 40, 2) if step < 1 + j % 13]
        vals = [5.0 / (1 + 0.3 * step + 0.01 * j) + 0.01 * rng.random() if j % 8 else 3.0 for j in ids]
        times = [1.0 + 0.05 * j for j in ids]
        for side in (sched, ref):
            side.append_losses(ids, vals, times if step % 2 == 0 else None)
    sched.set_param(slaq.binding.P_SELECTION, 1)
    for C in (7, 20, 61, 400):
        alloc, rc = sched.schedule(2.0, C)
        compare_epoch(alloc, sched.get_predictions(), ref.schedule(2.0, C), C, 8)
        assert (alloc[1::2] == 0).all()


def test_identical_jobs_share_by_job_id_without_a_table(slaq):
    base = make_workload(2, n_jobs=1)
    J = 500
    H = int(base.hist_len[0])
    offsets = np.arange(J + 1, dtype=np.int64) * H
    sched = slaq.Scheduler(J, base.max_hist, 8)
    ids = np.arange(J, dtype=np.int32)
    sched.load_histories(ids, offsets, np.tile(base.losses, J), np.repeat(base.k_last, J), np.repeat(base.m_seen, J))
    sched.set_time_model(ids, np.repeat(base.s, J), np.repeat(base.w, J))
    for C in (J + 1, J + 499, 2 * J + 7, 5 * J - 1, 8 * J):
        table, _ = sched.schedule(3.0, C)
        sched.set_param(slaq.binding.P_SELECTION, 1)
        free, _ = sched.schedule(3.0, C)
        sched.set_param(slaq.binding.P_SELECTION, 0)
        np.testing.assert_array_equal(free, table)          # every gain ties with its copies: lowest ids first
        assert (np.diff(free) <= 0).all() and free.sum() == C


def test_options_that_need_the_table_still_get_it(slaq, oracle_mod):
    wl = make_workload(4, n_jobs=5000)
    sched = make_scheduler(wl)
    sched.set_param(slaq.binding.P_SELECTION, 1)
    sched.set_param(slaq.binding.P_GAIN_ENVELOPE, 1)
    alloc, _ = sched.schedule(wl.epoch_seconds, wl.total_cores)
    ref = oracle_mod.schedule(wl.offsets, wl.losses, wl.m_seen, wl.s, wl.w, wl.epoch_seconds, wl.total_cores,
                              wl.max_cores_per_job, envelope=True)
    # this cut of config 4 holds one of the rare jobs whose unfinished fit ends 1.15 tolerances from the oracle's
    # (see test_unseen_cuts_survey): allowed here, at the looser bound of compare_epoch
    compare_epoch(alloc, sched.get_predictions(), ref, wl.total_cores, wl.max_cores_per_job, allow_unstable=1)
    sched.set_param(slaq.binding.P_GAIN_ENVELOPE, 0)
    newest = wl.losses[wl.offsets[1:] - 1]
    target = np.full(wl.n_jobs, np.nan)
    target[::4] = newest[::4] * 0.999
    sched.set_target_loss(np.arange(0, wl.n_jobs, 4), target[::4])
    alloc, _ = sched.schedule(wl.epoch_seconds, wl.total_cores)
    ref = oracle_mod.schedule(wl.offsets, wl.losses, wl.m_seen, wl.s, wl.w, wl.epoch_seconds, wl.total_cores,
                              wl.max_cores_per_job, target_loss=target)
    compare_epoch(alloc, sched.get_predictions(), ref, wl.total_cores, wl.max_cores_per_job, allow_unstable=1)


@pytest.mark.parametrize("cap", [1, 2, 33, 1024])
def test_extreme_caps_with_every_way_of_predicting(slaq, oracle_mod, cap):
    """One core per job at most, two, a row that is one entry longer than a warp step, and the largest cap the
    library takes: table and table-free selection, envelope rows and target hints against the oracle."""
    wl = make_workload(4, n_jobs=600)
    J = wl.n_jobs
    newest = wl.losses[wl.offsets[1:] - 1]
    target = np.full(J, np.nan)
    target[::3] = newest[::3] * 0.9995
    for C in (J // 2, J, 3 * J, J * cap):
        for selection, envelope, hints in ((0, 0, False), (1, 0, False), (0, 1, False), (0, 0, True), (1, 1, True)):
            sched = slaq.Scheduler(J, wl.max_hist, cap)
            ids = np.arange(J, dtype=np.int32)
            sched.load_histories(ids, wl.offsets, wl.losses, wl.k_last, wl.m_seen)
            sched.set_time_model(ids, wl.s, wl.w)
            sched.set_param(slaq.binding.P_SELECTION, selection)
            sched.set_param(slaq.binding.P_GAIN_ENVELOPE, envelope)
            if hints:
                sched.set_target_loss(ids[::3], target[::3])
            alloc, rc = sched.schedule(wl.epoch_seconds, C)
            ref = oracle_mod.schedule(wl.offsets, wl.losses, wl.m_seen, wl.s, wl.w, wl.epoch_seconds, C, cap,
                                      envelope=bool(envelope), target_loss=target if hints else None)
            compare_epoch(alloc, sched.get_predictions(), ref, C, cap)
            assert alloc.sum() == min(C, J * cap) and alloc.max() <= cap
            sched.close()
