"""The two options of the prediction step against their oracle twins: gain rows as slopes of the concave envelope of
R(n) (SLAQ_P_GAIN_ENVELOPE), and target-loss hints that cap a job's predicted reduction (slaq_set_target_loss)."""

import numpy as np
import pytest

from workloads import make_workload
from gpu_common import compare_epoch, make_scheduler

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def slaq():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import paper_1802_04819_b200 as mod
    mod.build()
    return mod


@pytest.mark.parametrize("cfg,n_jobs,cap", [(4, 20000, None), (2, None, None), (4, 3000, 700)])
def test_envelope_rows_match_the_oracle(slaq, oracle_mod, cfg, n_jobs, cap):
    wl = make_workload(cfg, n_jobs=n_jobs)
    if cap:                                   # rows longer than one warp step, up to the stack's size class
        wl.max_cores_per_job = cap
    sched = make_scheduler(wl)
    plain, _ = sched.schedule(wl.epoch_seconds, wl.total_cores)
    first = sched.get_predictions()
    g_plain = first["gain"]
    # the statistics count the fits that are not convex ahead: family I with b^2 < a c (typed here from the curve)
    p = first["params"]
    typed = int(((first["status"] == 0) & (first["family"] == 0) & (p[:, 1] ** 2 < p[:, 0] * p[:, 2])).sum())
    assert sched.get_stats().nonconvex_fits == typed > 0
    sched.set_param(slaq.binding.P_GAIN_ENVELOPE, 1)
    assert sched.get_param(slaq.binding.P_GAIN_ENVELOPE) == 1
    alloc, rc = sched.schedule(wl.epoch_seconds, wl.total_cores)
    pred = sched.get_predictions()
    ref = oracle_mod.schedule(wl.offsets, wl.losses, wl.m_seen, wl.s, wl.w, wl.epoch_seconds, wl.total_cores,
                              wl.max_cores_per_job, envelope=True)
    compare_epoch(alloc, pred, ref, wl.total_cores, wl.max_cores_per_job)
    g = pred["gain"]
    assert (g >= 0).all() and (np.diff(g, axis=1) <= 0).all()
    changed = (g != g_plain).any(axis=1)
    assert changed.sum() >= 5 and (pred["family"][changed] == 0).all()
    # the envelope keeps each curve's whole drop at the last core: no less than the running minimum's
    assert (g.sum(axis=1) >= g_plain.sum(axis=1) * (1 - 1e-12)).all()
    sched.set_param(slaq.binding.P_GAIN_ENVELOPE, 0)
    again, _ = sched.schedule(wl.epoch_seconds, wl.total_cores)
    np.testing.assert_array_equal(again, plain)


@pytest.mark.parametrize("envelope", [0, 1])
def test_target_loss_hints_match_the_oracle(slaq, oracle_mod, envelope):
    wl = make_workload(2, n_jobs=1500)
    T = 30.0                                               # a long epoch, so that the caps bite
    newest = wl.losses[wl.offsets[1:] - 1]
    target = np.full(wl.n_jobs, np.nan)
    target[::2] = newest[::2] * 0.97
    target[1::10] = newest[1::10] * 1.5                    # already below the target: no gain
    sched = make_scheduler(wl, packed=True)
    sched.set_param(slaq.binding.P_GAIN_ENVELOPE, envelope)
    hinted = np.nonzero(np.isfinite(target))[0].astype(np.int32)
    sched.set_target_loss(hinted, target[hinted])
    alloc, rc = sched.schedule(T, wl.total_cores)
    pred = sched.get_predictions()
    ref = oracle_mod.schedule(wl.offsets, wl.losses, wl.m_seen, wl.s, wl.w, T, wl.total_cores, wl.max_cores_per_job,
                              envelope=bool(envelope), target_loss=target)
    compare_epoch(alloc, pred, ref, wl.total_cores, wl.max_cores_per_job)
    cap_R = np.maximum(newest - target, 0.0) / pred["M"]
    R = pred["gain"].sum(axis=1)
    fits = np.isfinite(target) & (pred["status"] == slaq.JOB_FITTED)
    assert (R[fits] <= cap_R[fits] * (1 + 1e-12) + 1e-15).all()
    assert (np.abs(R[fits] - cap_R[fits]) <= 1e-12 * cap_R[fits] + 1e-15).sum() > 100      # many sit exactly on their cap
    assert (pred["gain"][1::10] == 0).all()
    # removing the hints brings the plain prediction back; a removed job forgets its hint
    sched.set_target_loss(hinted, np.full(hinted.size, np.nan))
    alloc2, _ = sched.schedule(T, wl.total_cores)
    ref2 = oracle_mod.schedule(wl.offsets, wl.losses, wl.m_seen, wl.s, wl.w, T, wl.total_cores, wl.max_cores_per_job,
                               envelope=bool(envelope))
    compare_epoch(alloc2, sched.get_predictions(), ref2, wl.total_cores, wl.max_cores_per_job)
    with pytest.raises(slaq.SlaqError):
        sched.set_target_loss([0], [np.inf])


def test_hints_in_the_streaming_loop_and_the_state_blob(slaq, oracle_mod):
    wl = make_workload(1)
    J, cap = wl.n_jobs, wl.max_cores_per_job
    ids = np.arange(J, dtype=np.int32)
    sched = slaq.Scheduler(J, wl.max_hist, cap)
    ref = oracle_mod.OracleScheduler(J, wl.max_hist, cap)
    for side in (sched, ref):
        side.load_histories(ids, wl.offsets, wl.losses, wl.k_last, wl.m_seen)
        side.set_time_model(ids, wl.s, wl.w)
    newest = wl.losses[wl.offsets[1:] - 1]
    sched.set_target_loss(ids[::3], newest[::3] * 0.9)
    ref.set_target_loss(ids[::3], newest[::3] * 0.9)
    alloc, _ = sched.schedule(20.0, wl.total_cores)
    compare_epoch(alloc, sched.get_predictions(), ref.schedule(20.0, wl.total_cores), wl.total_cores, cap)
    twin = slaq.Scheduler(J, wl.max_hist, cap)
    twin.import_state(sched.export_state())                 # the hints travel with the state
    np.testing.assert_array_equal(twin.schedule(20.0, wl.total_cores)[0], alloc)
    sched.remove_jobs(ids[:6])
    ref.remove_jobs(ids[:6])
    alloc, _ = sched.schedule(20.0, wl.total_cores)
    compare_epoch(alloc, sched.get_predictions(), ref.schedule(20.0, wl.total_cores), wl.total_cores, cap)
