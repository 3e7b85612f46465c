"""Pins for the oracle's prediction step: loss reduction over one epoch per core count
(the objective Loss_j(a_j, t) - Loss_j(a_j, t+T) of "Scheduling Based on Quality Improvements")."""

import numpy as np

from workloads import make_workload, make_time_samples


def fitted_curve(family, p, x):
    if family == 0:
        return 1.0 / (p[0] * x * x + p[1] * x + p[2]) + p[3]
    return np.exp(p[0] - p[1] * x) + p[2]


def test_gains_telescope_to_the_curve_drop(oracle_mod):
    # sum_{n<=N} g(n) must equal f(0) - f(m(N)/span) of the fitted curve, with
    # m(n) = T n / (s n + w) iterations in the epoch, wherever no clamp was active
    wl = make_workload(2)
    out = oracle_mod.predict(wl.offsets, wl.losses, wl.m_seen, wl.s, wl.w, wl.epoch_seconds, wl.max_cores_per_job)
    cap = wl.max_cores_per_job
    n = np.arange(1, cap + 1)
    checked = 0
    for j in np.nonzero(out["status"] == 0)[0][:1500]:
        g = out["gain"][j]
        if not ((g > 0).all() and (np.diff(g) < 0).all()):
            continue                      # a clamp or the running minimum touched this row
        H = wl.hist_len[j]
        m = wl.epoch_seconds * n / (wl.s[j] * n + wl.w[j])
        X = m / (H - 1)
        fam, p = int(out["family"][j]), out["params"][j]
        drop = fitted_curve(fam, p, 0.0) - fitted_curve(fam, p, X)
        scale = abs(fitted_curve(fam, p, 0.0)) + abs(p[3 if fam == 0 else 2])
        np.testing.assert_allclose(np.cumsum(g), drop, rtol=1e-9, atol=1e-13 * scale)
        checked += 1
    assert checked > 500


def test_gains_are_nonnegative_and_nonincreasing(oracle_mod):
    for cfg in (1, 2):
        wl = make_workload(cfg)
        out = oracle_mod.predict(wl.offsets, wl.losses, wl.m_seen, wl.s, wl.w, wl.epoch_seconds,
                                 wl.max_cores_per_job)
        g = out["gain"]
        assert np.isfinite(g).all()
        assert (g >= 0).all()
        assert (np.diff(g, axis=1) <= 0).all()


def test_convex_fits_need_no_clamp(oracle_mod):
    # an exponential fit is convex and decreasing, and iterations per epoch are concave in
    # the core count, so its raw marginal gains already fall with n: strictly, while positive
    wl = make_workload(2)
    out = oracle_mod.predict(wl.offsets, wl.losses, wl.m_seen, wl.s, wl.w, wl.epoch_seconds, wl.max_cores_per_job)
    rows = (out["status"] == 0) & (out["family"] == 1) & (out["params"][:, 1] > 1e-6)
    g = out["gain"][rows]
    pos = g[:, :-1] > 1e-300
    assert (np.diff(g, axis=1)[pos] < 0).all()


def test_time_units_cancel(oracle_mod):
    # (T, s, w) -> (2T, 2s, 2w) is a change of time unit: iterations per epoch are unchanged, bit for bit
    wl = make_workload(1)
    a = oracle_mod.predict(wl.offsets, wl.losses, wl.m_seen, wl.s, wl.w, wl.epoch_seconds, wl.max_cores_per_job)
    b = oracle_mod.predict(wl.offsets, wl.losses, wl.m_seen, 2 * wl.s, 2 * wl.w, 2 * wl.epoch_seconds,
                           wl.max_cores_per_job)
    np.testing.assert_array_equal(a["gain"], b["gain"])


def test_more_time_per_epoch_never_predicts_less(oracle_mod):
    wl = make_workload(1)
    a = oracle_mod.predict(wl.offsets, wl.losses, wl.m_seen, wl.s, wl.w, 1.0, wl.max_cores_per_job)
    b = oracle_mod.predict(wl.offsets, wl.losses, wl.m_seen, wl.s, wl.w, 2.0, wl.max_cores_per_job)
    Ra, Rb = a["gain"].sum(1), b["gain"].sum(1)
    assert (Rb >= Ra * (1 - 1e-12)).all()


def test_jobs_without_time_model_get_no_gain(oracle_mod):
    wl = make_workload(0)
    s = wl.s.copy()
    s[2] = np.nan
    out = oracle_mod.predict(wl.offsets, wl.losses, wl.m_seen, s, wl.w, wl.epoch_seconds, wl.max_cores_per_job)
    assert out["status"][2] == oracle_mod.ST_NO_TIME
    assert (out["gain"][2] == 0).all()


def test_time_model_recovered_from_samples(oracle_mod):
    # t(n) = s + w/n sampled without noise at n = 1, 2, 4, 8: least squares returns (s, w)
    wl = make_workload(1)
    cores, secs = make_time_samples(wl, 8)
    sched = oracle_mod.OracleScheduler(wl.n_jobs, wl.max_hist, wl.max_cores_per_job)
    ids = np.arange(wl.n_jobs)
    for i in range(8):
        sched.append_losses(ids, np.full(wl.n_jobs, 1.0 / (i + 1)), secs[i], cores[i])
    s, w = sched.time_model()
    np.testing.assert_allclose(s, wl.s, rtol=1e-9)
    np.testing.assert_allclose(w, wl.w, rtol=1e-9)
    # one core count only: all time is taken as parallel work
    sched = oracle_mod.OracleScheduler(4, 8, 4)
    sched.append_losses([0, 1], [1.0, 1.0], [2.0, 3.0], [4, 4])
    sched.append_losses([0, 1], [0.5, 0.5], [2.0, 3.0], [4, 4])
    s, w = sched.time_model()
    np.testing.assert_allclose(s[:2], [0.0, 0.0])
    np.testing.assert_allclose(w[:2], [8.0, 12.0])
    assert np.isnan(s[2]) and np.isnan(w[2])


def _envelope_by_definition(R):
    """Upper concave envelope of the points (n, R[n]) straight from its definition: at n it is the largest
    value any chord between two of the points (one at or left of n, one at or right of n) reaches at n."""
    N = len(R)
    env = np.array(R, dtype=float)
    for n in range(N):
        for i in range(n + 1):
            for j in range(n, N):
                if j > i:
                    env[n] = max(env[n], R[i] + (R[j] - R[i]) * (n - i) / (j - i))
    return env


def test_concave_envelope_equals_its_definition(oracle_mod):
    rng = np.random.default_rng(8)
    for trial in range(200):
        cap = int(rng.integers(1, 14))
        steps = rng.uniform(0, 1, cap) * rng.integers(0, 2, cap)          # some zero steps, rises and falls
        if trial % 3 == 0:
            steps = -np.sort(-steps)                                       # already non-increasing
        R = np.concatenate([[0.0], np.cumsum(steps)])
        slopes = oracle_mod.envelope(R)
        env = np.concatenate([[0.0], np.cumsum(slopes)])
        np.testing.assert_allclose(env, _envelope_by_definition(R), rtol=1e-12, atol=1e-14)
        assert (np.diff(slopes) <= 1e-15).all() and (slopes >= 0).all()   # concave and non-decreasing
        assert (env >= R - 1e-14).all() and abs(env[-1] - R[-1]) <= 1e-14  # nowhere below R, same end point
        if trial % 3 == 0:
            np.testing.assert_allclose(slopes, steps, rtol=1e-12, atol=1e-15)


def test_envelope_option_changes_only_rows_that_rise(oracle_mod):
    """Convex fits give concave R(n): the envelope is the row itself.  Where the fitted curve is not convex ahead
    of the newest point the raw differences rise with n; there the default flattens them with a running minimum
    (it never predicts more than the curve's drop) and the envelope option keeps the whole drop."""
    wl = make_workload(4, n_jobs=4000)
    kw = dict(offsets=wl.offsets, losses=wl.losses, m_seen=wl.m_seen, s=wl.s, w=wl.w, epoch_seconds=wl.epoch_seconds,
              cap=wl.max_cores_per_job)
    a = oracle_mod.predict(**kw)
    b = oracle_mod.predict(**kw, envelope=True)
    differs = (a["gain"] != b["gain"]).any(axis=1)
    assert 50 < differs.sum() < wl.n_jobs // 2
    assert (a["family"][differs] == 0).all()                 # the exponential family is convex everywhere
    assert (b["gain"] >= 0).all() and (np.diff(b["gain"], axis=1) <= 1e-18).all()
    cap = wl.max_cores_per_job
    n = np.arange(1, cap + 1)
    for j in np.nonzero(differs)[0][:200]:
        H = wl.hist_len[j]
        X = wl.epoch_seconds * n / (wl.s[j] * n + wl.w[j]) / (H - 1)
        p = a["params"][j]
        drop = fitted_curve(0, p, 0.0) - fitted_curve(0, p, X)          # typed: f(0) - f(X_n)
        if (np.diff(drop, prepend=0.0) > 0).all():                       # no clamp at zero was needed
            env = np.cumsum(b["gain"][j])
            fuzz = 1e-13 * (abs(fitted_curve(0, p, 0.0)) + abs(p[3]))    # the typed drop is a difference of two levels
            assert (env >= drop * (1 - 1e-9) - fuzz).all()               # never below the curve's own drop
            np.testing.assert_allclose(env[-1], drop[-1], rtol=1e-9, atol=fuzz)   # and equal to it at the last core
            assert np.cumsum(a["gain"][j])[-1] <= env[-1] * (1 + 1e-12)  # the running minimum predicts no more


def test_target_loss_hint_caps_the_predicted_reduction(oracle_mod):
    """A hint of the loss a job will end at: nothing is predicted below it.  Expected from the rule itself:
    cumulative gains = min(default cumulative gains, (newest loss - target) / M)."""
    wl = make_workload(2, n_jobs=300)
    kw = dict(offsets=wl.offsets, losses=wl.losses, m_seen=wl.m_seen, s=wl.s, w=wl.w, epoch_seconds=30.0,
              cap=wl.max_cores_per_job)
    newest = wl.losses[wl.offsets[1:] - 1]
    target = np.full(wl.n_jobs, np.nan)
    target[::2] = newest[::2] * 0.97                       # every other job: 3 % below where it is now
    target[1::10] = newest[1::10] * 1.5                    # some already below their target: nothing to gain
    a = oracle_mod.predict(**kw)
    b = oracle_mod.predict(**kw, target_loss=target)
    hinted = np.isfinite(target)
    np.testing.assert_array_equal(a["gain"][~hinted], b["gain"][~hinted])
    cap_R = np.maximum(newest - target, 0.0) / a["M"]
    Ra, Rb = np.cumsum(a["gain"], axis=1), np.cumsum(b["gain"], axis=1)
    fits = hinted & (a["status"] != oracle_mod.ST_FLAT)
    np.testing.assert_allclose(Rb[fits], np.minimum(Ra[fits], cap_R[fits, None]), rtol=1e-12, atol=1e-15)
    assert (Rb[fits][:, -1] < Ra[fits][:, -1]).sum() > 20           # the cap bites for a good share of them
    assert (b["gain"][1::10] == 0).all()
    assert (np.diff(b["gain"], axis=1) <= 0).all() and (b["gain"] >= 0).all()
