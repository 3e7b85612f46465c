"""Warm-started refits on the GPU against the oracle's: both sides keep their own fitted curves
between epochs and start each family from them (SLAQ_P_WARM_START)."""

import functools

import numpy as np
import pytest

import gpu_common
from workloads import make_workload, true_curve

pytestmark = pytest.mark.gpu

# a warm-started fit continues an unfinished iteration: single jobs stay within the per-job tolerance, but not
# a thousand times inside it as the cold path's do, so the total is compared at a tenth of that tolerance
compare_epoch = functools.partial(gpu_common.compare_epoch, total_rtol=1e-7)


@pytest.fixture(scope="module")
def slaq():
    import paper_1802_04819_b200 as slaq
    return slaq


def _pair(slaq, oracle_mod, wl, max_hist, lm_trials, warm=True):
    J, cap = wl.n_jobs, wl.max_cores_per_job
    sched = slaq.Scheduler(J, max_hist, cap)
    sched.set_param(slaq.binding.P_LM_TRIALS, lm_trials)
    sched.set_param(slaq.binding.P_WARM_START, 1 if warm else 0)
    ref = oracle_mod.OracleScheduler(J, max_hist, cap, lm_trials=lm_trials)
    ref.warm_start = warm
    ids = np.arange(J, dtype=np.int32)
    sched.set_time_model(ids, wl.s, wl.w)
    ref.set_time_model(ids, wl.s, wl.w)
    return sched, ref


def _load_prefix(wl, sched, ref, keep):
    """Both sides start with the first keep[j] points of every job's history."""
    J = wl.n_jobs
    ids = np.arange(J, dtype=np.int32)
    offs = np.zeros(J + 1, np.int64)
    np.cumsum(keep, out=offs[1:])
    rows = np.concatenate([wl.losses[wl.offsets[j]:wl.offsets[j] + keep[j]] for j in range(J)])
    k_last = wl.k_last - (wl.hist_len - keep)
    sched.load_histories(ids, offs, rows, k_last)
    ref.load_histories(ids, offs, rows, k_last)


def _append_next(wl, sched, ref, pos, steps):
    ids = np.arange(wl.n_jobs, dtype=np.int32)
    for _ in range(steps):
        live = ids[pos < wl.hist_len]
        if live.size == 0:
            return
        vals = wl.losses[wl.offsets[live] + pos[live]]
        sched.append_losses(live, vals)
        ref.append_losses(live, vals)
        pos[live] += 1


def _oracle_state(ref):
    """The oracle's fitted curves in the layout slaq_set_fit_state takes."""
    st = {k: v.copy() for k, v in ref.fitted.items()}
    none = st["valid"] == 0
    st["span"][none], st["M"][none] = 1.0, 1.0
    return st


@pytest.mark.parametrize("lm_trials,free_running", [(20, False), (5, False), (20, True), (5, True)])
def test_warm_started_epochs_match_the_oracle(slaq, oracle_mod, lm_trials, free_running):
    """The cluster experiment's shape (4,000 jobs' worth of window lengths, here 1,500 jobs): six epochs,
    three new losses per job and epoch, every epoch compared element by element.

    Not free running: after each comparison the library continues from the oracle's fitted curves, so every
    epoch tests one warm-started fit from identical starting points, at the cold path's tolerance.
    Free running: each side continues from its own curves; rounding differences then compound in the few jobs
    whose residual is flat along a direction, so a few per thousand may miss the tolerance (by a bounded factor)."""
    wl = make_workload(2, n_jobs=1500)
    epochs, step = 6, 3
    sched, ref = _pair(slaq, oracle_mod, wl, int(wl.max_hist), lm_trials)
    keep = np.maximum(wl.hist_len - (epochs - 1) * step, np.minimum(wl.hist_len, 4))
    _load_prefix(wl, sched, ref, keep)
    pos = keep.copy()
    sweeps = []
    for epoch in range(epochs):
        got, _ = sched.schedule(wl.epoch_seconds, wl.total_cores)
        out = ref.schedule(wl.epoch_seconds, wl.total_cores)
        compare_epoch(got, sched.get_predictions(), out, wl.total_cores, wl.max_cores_per_job,
                      allow_unstable=(wl.n_jobs * 3) // 1000 if free_running and epoch > 0 else 0)
        st = sched.get_fit_state()
        np.testing.assert_array_equal(st["valid"], out["mask"])
        fitted = out["mask"] != 0
        np.testing.assert_array_equal(st["K"][fitted], ref.k_last[fitted])
        np.testing.assert_array_equal(st["span"][fitted], ref.fitted["span"][fitted])
        np.testing.assert_array_equal(st["M"][fitted], ref.fitted["M"][fitted])
        sweeps.append((int(sched.get_stats().model_sweeps), int((out["evals"].sum(axis=1) * wl_points(ref)).sum())))
        if not free_running:      # both sides: the call also resets the starting points of jobs that get no new loss
            state = _oracle_state(ref)
            sched.set_fit_state(state)
            ref.set_fit_state(state)
        _append_next(wl, sched, ref, pos, step)
    for mine, theirs in sweeps:       # same work on both sides, up to early-stop jitter
        assert abs(mine - theirs) <= 0.15 * theirs


def wl_points(ref):
    return np.array([len(w) for w in ref.window], dtype=np.int64)


def test_warm_start_through_a_wrapping_ring_and_a_change_of_scale(slaq, oracle_mod):
    """A short ring wraps during the run, and half of the jobs show, late, a larger one-step reduction than any
    before (a bump followed by a drop), so the scale M the window is normalised by changes between two epochs.
    Both sides run freely from their own earlier results: after the first epoch one job per epoch
    may leave the tolerance, within the loose one (a 24-point window whose twenty trials end unfinished; which job
    and epoch depends on the seed and on the order of the kernel's sums: measured 1.1 tolerances with seed 7 and
    the sums multiplied out, 16 with seed 5 and the running sums)."""
    wl = make_workload(1)
    J, cap, max_hist = wl.n_jobs, wl.max_cores_per_job, 24
    sched, ref = _pair(slaq, oracle_mod, wl, max_hist, 20)
    rng = np.random.default_rng(5)
    ids = np.arange(J, dtype=np.int32)
    k_next = np.zeros(J, dtype=np.int64)
    scale_changed = 0
    for epoch in range(8):
        for step in range(5):
            losses = true_curve(wl.family, wl.params, k_next.astype(np.float64)) * np.exp(0.01 * rng.standard_normal(J))
            if epoch == 4 and step == 1:
                losses[::2] *= 4.0                      # the bump: the next iteration drops by more than ever before
            sched.append_losses(ids, losses)
            ref.append_losses(ids, losses)
            k_next += 1
        before = ref.fitted["M"].copy()
        got, _ = sched.schedule(wl.epoch_seconds, wl.total_cores)
        out = ref.schedule(wl.epoch_seconds, wl.total_cores)
        compare_epoch(got, sched.get_predictions(), out, wl.total_cores, cap, allow_unstable=1 if epoch > 0 else 0)
        if epoch > 0:
            scale_changed += int(np.sum(out["M"] > before))
    assert scale_changed >= J // 4
    assert (k_next > max_hist).all()


def test_an_epoch_repeated_without_new_losses_is_identical(slaq, oracle_mod):
    wl = make_workload(1)
    sched, ref = _pair(slaq, oracle_mod, wl, int(wl.max_hist), 5)
    keep = np.maximum(wl.hist_len - 3, np.minimum(wl.hist_len, 4))
    _load_prefix(wl, sched, ref, keep)
    pos = keep.copy()
    sched.schedule(wl.epoch_seconds, wl.total_cores)
    ref.schedule(wl.epoch_seconds, wl.total_cores)
    _append_next(wl, sched, ref, pos, 3)
    a, _ = sched.schedule(wl.epoch_seconds, wl.total_cores)
    pa, sa = sched.get_predictions(), sched.get_fit_state()
    b, _ = sched.schedule(wl.epoch_seconds, wl.total_cores)
    pb, sb = sched.get_predictions(), sched.get_fit_state()
    np.testing.assert_array_equal(a, b)
    np.testing.assert_array_equal(pa["gain"], pb["gain"])
    np.testing.assert_array_equal(sa["p"][sa["valid"] == 3], sb["p"][sb["valid"] == 3])
    compare_epoch(b, pb, ref.schedule(wl.epoch_seconds, wl.total_cores), wl.total_cores, wl.max_cores_per_job)


def test_an_unusable_carried_point_falls_back_to_the_first_guess(slaq, oracle_mod):
    """Fit state written from outside: family I's point has a negative denominator, family II's is not a number
    (even job ids), or only one of the two is unusable (odd ids).  Those families start from their first guesses."""
    wl = make_workload(1)
    J = wl.n_jobs
    sched, ref = _pair(slaq, oracle_mod, wl, int(wl.max_hist), 20)
    cold, cold_ref = _pair(slaq, oracle_mod, wl, int(wl.max_hist), 20, warm=False)
    ids = np.arange(J, dtype=np.int32)
    for s in (sched, ref, cold, cold_ref):
        s.load_histories(ids, wl.offsets, wl.losses, wl.k_last, wl.m_seen)
    # a proper state to spoil: one epoch on the oracle's side
    ref.schedule(wl.epoch_seconds, wl.total_cores)
    state = {k: v.copy() for k, v in ref.fitted.items()}
    has = state["valid"] == 3
    state["valid"][~has] = 0
    spoil_I = has & ((ids % 2 == 0) | (ids % 4 == 1))
    spoil_II = has & ((ids % 2 == 0) | (ids % 4 == 3))
    state["p"][spoil_I, 2] = -5.0
    state["p"][spoil_II, 4] = np.nan
    state["p"][~has] = 0.0
    state["span"][~has] = 1.0
    state["M"][~has] = 1.0
    sched.set_fit_state(state)
    ref.set_fit_state(state)
    got, _ = sched.schedule(wl.epoch_seconds, wl.total_cores)
    out = ref.schedule(wl.epoch_seconds, wl.total_cores)
    compare_epoch(got, sched.get_predictions(), out, wl.total_cores, wl.max_cores_per_job)
    # where both families were spoilt the result is the cold one, and the wasted sweeps are counted
    both = spoil_I & spoil_II
    got_cold, _ = cold.schedule(wl.epoch_seconds, wl.total_cores)
    np.testing.assert_array_equal(sched.get_predictions()["gain"][both], cold.get_predictions()["gain"][both])
    np.testing.assert_array_equal(sched.get_predictions()["evals"][both], cold.get_predictions()["evals"][both] + 1)
    assert both.sum() > 10 and (spoil_I ^ spoil_II).sum() > 10


def test_fit_state_round_trip_and_argument_checks(slaq, oracle_mod):
    wl = make_workload(1)
    J = wl.n_jobs
    sched, ref = _pair(slaq, oracle_mod, wl, int(wl.max_hist), 5)
    ids = np.arange(J, dtype=np.int32)
    sched.load_histories(ids, wl.offsets, wl.losses, wl.k_last, wl.m_seen)
    ref.load_histories(ids, wl.offsets, wl.losses, wl.k_last, wl.m_seen)
    sched.schedule(wl.epoch_seconds, wl.total_cores)
    state = sched.get_fit_state()
    # a second scheduler restored from the first one's state continues exactly like it
    twin = slaq.Scheduler(J, int(wl.max_hist), wl.max_cores_per_job)
    twin.set_param(slaq.binding.P_LM_TRIALS, 5)
    twin.set_param(slaq.binding.P_WARM_START, 1)
    twin.set_time_model(ids, wl.s, wl.w)
    twin.load_histories(ids, wl.offsets, wl.losses, wl.k_last, wl.m_seen)
    twin.set_fit_state(state)
    new = wl.losses[wl.offsets[1:] - 1] * 0.99
    sched.append_losses(ids, new)
    twin.append_losses(ids, new)
    a, _ = sched.schedule(wl.epoch_seconds, wl.total_cores)
    b, _ = twin.schedule(wl.epoch_seconds, wl.total_cores)
    np.testing.assert_array_equal(a, b)
    np.testing.assert_array_equal(sched.get_predictions()["gain"], twin.get_predictions()["gain"])
    # argument checks
    bad = {k: v.copy() for k, v in state.items()}
    bad["valid"][0] = 7
    with pytest.raises(slaq.SlaqError):
        twin.set_fit_state(bad)
    bad = {k: v.copy() for k, v in state.items()}
    j = int(np.nonzero(state["valid"])[0][0])
    bad["span"][j] = 0.0
    with pytest.raises(slaq.SlaqError):
        twin.set_fit_state(bad)
    empty = slaq.Scheduler(J, int(wl.max_hist), wl.max_cores_per_job)
    with pytest.raises(slaq.SlaqError):
        empty.set_fit_state(state)          # no job has losses yet


def test_replacing_a_history_forgets_its_fit(slaq, oracle_mod):
    wl = make_workload(1)
    J = wl.n_jobs
    sched, ref = _pair(slaq, oracle_mod, wl, int(wl.max_hist), 20)
    ids = np.arange(J, dtype=np.int32)
    for s in (sched, ref):
        s.load_histories(ids, wl.offsets, wl.losses, wl.k_last, wl.m_seen)
    sched.schedule(wl.epoch_seconds, wl.total_cores)
    ref.schedule(wl.epoch_seconds, wl.total_cores)
    # every other job gets its history replaced (same data): its next fit is a cold one again
    some = ids[::2]
    offs = np.zeros(some.size + 1, np.int64)
    np.cumsum(wl.hist_len[some], out=offs[1:])
    rows = np.concatenate([wl.losses[wl.offsets[j]:wl.offsets[j + 1]] for j in some])
    for s in (sched, ref):
        s.load_histories(some, offs, rows, wl.k_last[some], wl.m_seen[some])
    new = wl.losses[wl.offsets[1:] - 1] * 0.995
    sched.append_losses(ids, new)
    ref.append_losses(ids, new)
    assert (sched.get_fit_state()["valid"][some] == 0).all()
    got, _ = sched.schedule(wl.epoch_seconds, wl.total_cores)
    out = ref.schedule(wl.epoch_seconds, wl.total_cores)
    compare_epoch(got, sched.get_predictions(), out, wl.total_cores, wl.max_cores_per_job)


@pytest.mark.parametrize("warm", [False, True])
def test_the_fitted_curves_are_recorded_with_and_without_warm_start(slaq, oracle_mod, warm):
    """After an epoch the scheduler state holds both families' end points, the iteration index they belong to
    and the window's span and scale, whether or not the next fit will start from them: the recorded curve of
    the winning family is the one the predictions were made from, bit for bit, and the record agrees with the
    oracle's in which families ended with a finite residual."""
    wl = make_workload(2, n_jobs=1200)
    sched, ref = _pair(slaq, oracle_mod, wl, int(wl.max_hist), 20, warm=warm)
    ids = np.arange(wl.n_jobs, dtype=np.int32)
    sched.load_histories(ids, wl.offsets, wl.losses, wl.k_last)
    ref.load_histories(ids, wl.offsets, wl.losses, wl.k_last)
    sched.schedule(wl.epoch_seconds, wl.total_cores)
    out = ref.schedule(wl.epoch_seconds, wl.total_cores)
    st, pred = sched.get_fit_state(), sched.get_predictions(want_gain=False)
    np.testing.assert_array_equal(st["valid"], out["mask"])
    fitted = out["mask"] != 0
    assert fitted.sum() > 1000
    np.testing.assert_array_equal(st["K"][fitted], wl.k_last[fitted])
    np.testing.assert_array_equal(st["span"][fitted], np.maximum(wl.hist_len[fitted] - 1, 1).astype(np.float64))
    np.testing.assert_array_equal(st["M"][fitted], pred["M"][fitted])
    for fam in (0, 1):
        won = fitted & (pred["family"] == fam)
        assert won.sum() > 50
        width = 4 if fam == 0 else 3
        np.testing.assert_array_equal(st["p"][won, 4 * fam:4 * fam + width], pred["params"][won, :width])
    sched.close()
