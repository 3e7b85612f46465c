"""Pins for the oracle's warm start: a family may start from the parameters the job's last epoch
ended with, carried into the new window coordinates.  Pinned against what the mathematics fixes:
the carried parameters describe the same curve (substitution identity), a noise-free curve is a
fixed point, the solver never ends above the residual of its starting point (evaluated here in
numpy from the families' definitions), and an unusable carried point changes nothing."""

import numpy as np
import pytest

from workloads import true_curve


def curve(family, p, x):
    """The two families of "Predicting Quality Improvement", written out."""
    x = np.asarray(x, dtype=np.float64)
    if family == 0:
        return 1.0 / (p[0] * x * x + p[1] * x + p[2]) + p[3]
    return np.exp(p[0] - p[1] * x) + p[2]


@pytest.mark.parametrize("family", [0, 1])
def test_carried_parameters_describe_the_same_curve(oracle_mod, family):
    rng = np.random.default_rng(11 + family)
    checked = 0
    for _ in range(50):
        if family == 0:
            p = np.array([rng.uniform(0, 3), rng.uniform(0, 3), rng.uniform(0.2, 3), rng.uniform(-0.5, 0.5)])
        else:
            p = np.array([rng.uniform(-2, 1), rng.uniform(0, 4), rng.uniform(-0.2, 0.5), 0.0])
        t, r, sigma = rng.uniform(0, 2), rng.uniform(0.5, 2.5), rng.uniform(0.05, 1.0)
        x = np.linspace(-1.0, 0.5, 13)          # the new window and a stretch ahead of it
        x_old = t + r * x
        if family == 0 and (p[0] * x_old * x_old + p[1] * x_old + p[2]).min() < 0.1:
            continue                            # the curve has a pole in reach: not a fitted curve
        q = oracle_mod.carry(family, p, t, r, sigma)
        want = sigma * curve(family, p, x_old)
        np.testing.assert_allclose(curve(family, q, x), want, rtol=1e-11, atol=1e-13)
        for xi, wi in zip(x, want):             # and through the oracle's own evaluation of the family
            ok, f, _ = oracle_mod.family_eval(family, q, float(xi))
            assert ok and abs(f - wi) <= 1e-11 * abs(wi) + 1e-13
        checked += 1
    assert checked >= 20


def _exact_job(family):
    params = np.array([[2e-3, 0.15, 1.1, 0.05]]) if family == 0 else np.array([[0.93, 2.0, 0.04, 0.0]])
    fam = np.array([family], dtype=np.int8)
    return lambda k: true_curve(fam, params, np.asarray([k], dtype=np.float64))[0]


@pytest.mark.parametrize("family", [0, 1])
def test_a_noise_free_curve_is_a_fixed_point_of_the_warm_start(oracle_mod, family):
    loss_at = _exact_job(family)
    warm = oracle_mod.OracleScheduler(1, 64, 16)
    cold = oracle_mod.OracleScheduler(1, 64, 16)
    warm.warm_start = True
    for sched in (warm, cold):
        sched.set_time_model([0], [0.1], [4.0])
    k = 0
    for sched in (warm, cold):
        for i in range(30):
            sched.append_losses([0], [loss_at(i)])
    k = 30
    first_w, first_c = warm.schedule(3.0, 8), cold.schedule(3.0, 8)
    np.testing.assert_array_equal(first_w["gain"], first_c["gain"])      # nothing to start from yet
    assert first_w["family"][0] == family
    for sched in (warm, cold):
        for i in range(k, k + 6):
            sched.append_losses([0], [loss_at(i)])
    k += 6
    out_w, out_c = warm.schedule(3.0, 8), cold.schedule(3.0, 8)
    assert out_w["status"][0] == 0 and out_w["family"][0] == family
    M, span = out_w["M"][0], k - 1
    assert out_w["S"][0, family] <= 1e-18
    # the prediction is the true curve's drop over the epoch
    for n in (1, 4, 16):
        m = 3.0 * n / (0.1 * n + 4.0)
        want = (loss_at(k - 1) - loss_at(k - 1 + m)) / M
        got = out_w["gain"][0, :n].sum()
        assert abs(got - want) <= 1e-6 * want
    assert span == warm.fitted["span"][0] and warm.fitted["K"][0] == k - 1


def _noisy_scheduler(oracle_mod, warm_start, n_jobs=40, seed=3, lm_trials=20):
    from workloads import make_workload
    wl = make_workload(1, n_jobs=n_jobs)
    sched = oracle_mod.OracleScheduler(n_jobs, 48, wl.max_cores_per_job, lm_trials=lm_trials)
    sched.warm_start = warm_start
    sched.set_time_model(np.arange(n_jobs), wl.s, wl.w)
    return wl, sched, np.random.default_rng(seed)


def _advance(wl, scheds, rng, k_next, steps):
    J = wl.n_jobs
    ids = np.arange(J)
    for _ in range(steps):
        losses = true_curve(wl.family, wl.params, k_next.astype(np.float64)) * np.exp(0.01 * rng.standard_normal(J))
        for s in scheds:
            s.append_losses(ids, losses)
        k_next += 1


def test_the_solver_never_ends_above_its_carried_starting_point(oracle_mod):
    wl, sched, rng = _noisy_scheduler(oracle_mod, True)
    J = wl.n_jobs
    k_next = np.zeros(J, dtype=np.int64)
    _advance(wl, [sched], rng, k_next, 12)
    sched.schedule(wl.epoch_seconds, wl.total_cores)
    checked = 0
    for epoch in range(4):
        _advance(wl, [sched], rng, k_next, 5)     # the ring of 48 wraps in the last epochs
        start = {k: v.copy() for k, v in sched.warm.items()}
        out = sched.schedule(wl.epoch_seconds, wl.total_cores)
        for j in range(J):
            y = np.array(sched.window[j]) / out["M"][j]
            H = y.size
            span = max(H - 1, 1)
            x = (np.arange(H) - (H - 1)) / span
            w = 0.9 ** (H - 1 - np.arange(H))
            t = (sched.k_last[j] - start["K"][j]) / start["span"][j]
            r, sigma = span / start["span"][j], start["M"][j] / out["M"][j]
            for family in (0, 1):
                if not (start["valid"][j] >> family) & 1:
                    continue
                p0 = start["p"][j, 4 * family:4 * family + 4]
                # the carried curve, evaluated from the OLD parameters at the old coordinates
                S_start = float(np.sum(w * (y - sigma * curve(family, p0, t + r * x)) ** 2))
                assert out["S"][j, family] <= S_start * (1 + 1e-9) + 1e-30, (epoch, j, family)
                checked += 1
    assert checked > 200


def test_an_epoch_repeated_without_new_losses_is_identical(oracle_mod):
    wl, sched, rng = _noisy_scheduler(oracle_mod, True, lm_trials=5)
    k_next = np.zeros(wl.n_jobs, dtype=np.int64)
    _advance(wl, [sched], rng, k_next, 10)
    sched.schedule(wl.epoch_seconds, wl.total_cores)
    _advance(wl, [sched], rng, k_next, 3)
    a = sched.schedule(wl.epoch_seconds, wl.total_cores)
    b = sched.schedule(wl.epoch_seconds, wl.total_cores)
    np.testing.assert_array_equal(a["gain"], b["gain"])
    np.testing.assert_array_equal(a["both"], b["both"])


def test_fewer_trials_per_epoch_catch_up_over_the_epochs(oracle_mod):
    # 5 trials per epoch from a warm start reach, within a few epochs, the residual that 20 trials
    # from the first guess reach: the iterations of a fit are spread over the epochs
    wl, warm, rng = _noisy_scheduler(oracle_mod, True, n_jobs=120, lm_trials=5)
    _, cold, _ = _noisy_scheduler(oracle_mod, False, n_jobs=120, lm_trials=20)
    k_next = np.zeros(wl.n_jobs, dtype=np.int64)
    _advance(wl, [warm, cold], rng, k_next, 10)
    ratio = []
    for epoch in range(8):
        a, b = warm.schedule(wl.epoch_seconds, wl.total_cores), cold.schedule(wl.epoch_seconds, wl.total_cores)
        Sa, Sb = a["S"].min(axis=1), b["S"].min(axis=1)
        ratio.append(float(np.median(Sa / Sb)))
        sweeps = (int(a["evals"].sum()), int(b["evals"].sum()))
        _advance(wl, [warm, cold], rng, k_next, 3)
    assert ratio[-1] <= 1.02, ratio
    assert sweeps[0] * 2 < sweeps[1]


def test_an_unusable_carried_point_falls_back_to_the_first_guess(oracle_mod):
    wl, warm, rng = _noisy_scheduler(oracle_mod, True, n_jobs=12)
    _, cold, _ = _noisy_scheduler(oracle_mod, False, n_jobs=12)
    J = wl.n_jobs
    k_next = np.zeros(J, dtype=np.int64)
    _advance(wl, [warm, cold], rng, k_next, 15)
    bad = dict(valid=np.full(J, 3, np.uint8), p=np.zeros((J, 8)), K=warm.k_last.copy(),
               span=np.full(J, 14.0), M=np.ones(J))
    bad["p"][:, 2] = -5.0            # family I: negative denominator at the newest point
    bad["p"][:, 4] = np.nan          # family II: no finite residual
    warm.set_fit_state(bad)
    a, b = warm.schedule(wl.epoch_seconds, wl.total_cores), cold.schedule(wl.epoch_seconds, wl.total_cores)
    np.testing.assert_array_equal(a["gain"], b["gain"])
    np.testing.assert_array_equal(a["evals"], b["evals"] + 1)      # the wasted sweep at the carried point is counted


def test_replacing_or_removing_a_history_forgets_its_fit(oracle_mod):
    wl, sched, rng = _noisy_scheduler(oracle_mod, True, n_jobs=6)
    k_next = np.zeros(wl.n_jobs, dtype=np.int64)
    _advance(wl, [sched], rng, k_next, 10)
    sched.schedule(wl.epoch_seconds, wl.total_cores)
    _advance(wl, [sched], rng, k_next, 1)
    assert (sched.warm["valid"] == 3).all()
    sched.remove_jobs([1])
    sched.load_histories([2], np.array([0, 5]), np.array([5.0, 4.0, 3.5, 3.2, 3.1]), [4])
    assert sched.warm["valid"][1] == 0 and sched.warm["valid"][2] == 0 and sched.warm["valid"][0] == 3
