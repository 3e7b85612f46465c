"""Pins for the oracle's curve fit (Design, "Predicting Quality Improvement").

The two families are the paper's: f(k) = 1/(a k^2 + b k + c) + d and f(k) = mu^(k-b) + c.
Everything typed here (model values, objective, closed-form regression) is typed from
those formulas and from textbook definitions, not from the oracle's source.
"""

import numpy as np
import pytest
from scipy.optimize import least_squares

from workloads import make_workload, true_curve

GAMMA = 0.9


def local_problem(loss, m_seen=-np.inf):
    """Normalised levels, local coordinates and weights of one history."""
    H = loss.size
    M = max(m_seen, (loss[:-1] - loss[1:]).max())
    x = (np.arange(H) - (H - 1)) / (H - 1)
    w = GAMMA ** np.arange(H - 1, -1, -1)
    return x, loss / M, w, M


def model(family, p, x):
    if family == 0:
        return 1.0 / (p[0] * x * x + p[1] * x + p[2]) + p[3]
    return np.exp(p[0] - p[1] * x) + p[2]


def objective(family, p, x, y, w):
    r = y - model(family, p, x)
    return float(np.sum(w * r * r))


def test_solver_on_a_line_is_weighted_linear_regression(oracle_mod):
    # With no damping the first trial solves the normal equations exactly, so on a model
    # that is linear in its parameters one step must land on the closed-form solution.
    rng = np.random.default_rng(3)
    for H in (4, 9, 57):
        x = np.sort(rng.uniform(-1, 0, H))
        y = 2.0 - 3.0 * x + 0.1 * rng.standard_normal(H)
        w = GAMMA ** np.arange(H - 1, -1, -1)
        p, S, evals = oracle_mod.lm_line(x, y, w, trials=1, lambda0=0.0, p0=[0.3, -0.2])
        sw, swx, swy = w.sum(), (w * x).sum(), (w * y).sum()
        swxx, swxy = (w * x * x).sum(), (w * x * y).sum()
        slope = (sw * swxy - swx * swy) / (sw * swxx - swx * swx)
        icpt = (swy - slope * swx) / sw
        np.testing.assert_allclose(p, [icpt, slope], rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(S, np.sum(w * (y - icpt - slope * x) ** 2), rtol=1e-10)
        # and numpy's own weighted polynomial fit agrees
        np.testing.assert_allclose(p[::-1], np.polyfit(x, y, 1, w=np.sqrt(w)), rtol=1e-9)
        # damped trials still converge to it
        p20, _, _ = oracle_mod.lm_line(x, y, w, trials=20, lambda0=1e-3, p0=[0.3, -0.2])
        np.testing.assert_allclose(p20, [icpt, slope], rtol=1e-7)


@pytest.mark.parametrize("family,p", [(0, [0.7, 1.3, 2.1, -0.2]), (0, [0.0, 0.4, 1.0, 0.3]),
                                      (1, [-0.5, 1.7, 0.2, 0.0]), (1, [0.3, 0.0, -0.1, 0.0])])
def test_jacobians_match_central_differences(oracle_mod, family, p):
    p = np.array(p, dtype=float)
    n = 4 if family == 0 else 3
    for x in (-1.0, -0.37, 0.0, 0.8):
        ok, f, jac = oracle_mod.family_eval(family, p, x)
        assert ok
        assert f == pytest.approx(model(family, p, x), rel=1e-14)
        for a in range(n):
            h = 1e-6
            up, dn = p.copy(), p.copy()
            up[a] += h
            dn[a] -= h
            fd = (model(family, up, x) - model(family, dn, x)) / (2 * h)
            assert jac[a] == pytest.approx(fd, rel=1e-7, abs=1e-9)


def test_sublinear_rejects_nonpositive_denominator(oracle_mod):
    ok, _, _ = oracle_mod.family_eval(0, np.array([0.0, 2.0, 1.0, 0.0]), -0.75)
    assert not ok


def test_fit_never_raises_the_objective_and_ends_at_a_local_minimum(oracle_mod):
    # The end point must be no worse than the starting guess under an independently typed
    # objective, and where the solver stopped by itself inside the feasible set, no
    # coordinate move may lower the objective (a wrong sign or a dropped term in the
    # oracle's normal equations would stop it somewhere else).
    wl = make_workload(2)
    checked = 0
    for j in range(0, 600):
        loss = wl.history(j)
        if loss.size < 8:
            continue
        x, y, w, _ = local_problem(loss, wl.m_seen[j])
        for family in (0, 1):
            r = oracle_mod.fit_family(family, loss, wl.m_seen[j])
            n = 4 if family == 0 else 3
            S_end = objective(family, r["p"], x, y, w)
            assert S_end == pytest.approx(r["S"], rel=1e-9)
            assert S_end <= objective(family, r["p0"], x, y, w) * (1 + 1e-12)
            interior = (r["p"][:2] > 0).all() if family == 0 else r["p"][1] > 0
            if r["evals"] < 21 and interior:
                checked += 1
                for a in range(n):
                    for sgn in (-1, 1):
                        q = r["p"].copy()
                        q[a] += sgn * 1e-4 * max(abs(q[a]), 1e-3)
                        assert objective(family, q, x, y, w) >= S_end * (1 - 1e-9)
    assert checked > 100


def test_optimum_agrees_with_library_solver(oracle_mod):
    # Where the oracle's solver stopped by itself strictly inside the bounds, a trust-region
    # solver from scipy started at the oracle's end point must not find a better weighted
    # residual: the end point is a local minimum of the paper's objective.
    wl = make_workload(2)
    compared = 0
    for j in range(0, 400):
        loss = wl.history(j)
        if loss.size < 10:
            continue
        x, y, w, _ = local_problem(loss, wl.m_seen[j])
        for family in (0, 1):
            r = oracle_mod.fit_family(family, loss, wl.m_seen[j])
            interior = (r["p"][:2] > 0).all() if family == 0 else r["p"][1] > 0
            if r["evals"] >= 21 or not interior:
                continue
            n = 4 if family == 0 else 3
            lo = [0, 0, 1e-12, -np.inf] if family == 0 else [-np.inf, 0, -np.inf]
            sw = np.sqrt(w)

            def resid(p):
                with np.errstate(all="ignore"):
                    f = model(family, p, x)
                return np.where(np.isfinite(f), sw * (y - f), 1e6)

            sol = least_squares(resid, r["p"][:n], bounds=(lo, np.inf), xtol=1e-15, ftol=1e-15, gtol=1e-15,
                                max_nfev=2000)
            S_lib = float(np.sum(sol.fun ** 2))
            compared += 1
            assert r["S"] <= S_lib * (1 + 1e-9) or r["S"] - S_lib < 1e-15
    assert compared > 50


def _global_params(family, p, M, K, span):
    if family == 0:
        a, b, c, d = p
        ag = a / (M * span ** 2)
        bg = b / (M * span) - 2 * ag * K
        cg = c / M - bg * K - ag * K * K
        return np.array([ag, bg, cg, M * d])
    alpha, beta, c = p[:3]
    return np.array([np.exp(-beta / span), K + span * (alpha + np.log(M)) / beta, M * c, 0.0])


def test_exact_recovery_of_noise_free_curves(oracle_mod):
    # Histories drawn from either family without noise: given enough trials the fit must
    # return the generating curve (residual at rounding level, parameters mapped back to
    # global iteration numbers, predictions up to 60 iterations ahead).
    rng = np.random.default_rng(11)
    exact = {0: 0, 1: 0}
    total = {0: 0, 1: 0}
    for t in range(120):
        family = t % 2
        H = int(rng.integers(8, 60))
        k0 = int(rng.integers(0, 30))
        if family == 0:
            p_true = np.array([rng.uniform(1e-4, 1e-2), rng.uniform(0.01, 1), rng.uniform(0.5, 2), rng.uniform(0, 0.1)])
        else:
            p_true = np.array([rng.uniform(0.8, 0.99), rng.uniform(0, 5), rng.uniform(0, 0.1), 0.0])
        k = np.arange(k0, k0 + H)
        loss = true_curve(np.int8(family), p_true, k)
        x, y, w, M = local_problem(loss)
        r = oracle_mod.fit_family(family, loss, trials=400)
        total[family] += 1
        if r["S"] <= 1e-24 * np.sum(w * y * y):
            exact[family] += 1
            K, span = k0 + H - 1, H - 1
            pg = _global_params(family, r["p"], M, K, span)
            n = 4 if family == 0 else 3
            np.testing.assert_allclose(pg[:n], p_true[:n], rtol=1e-6, atol=1e-9)
            ahead = K + np.arange(1, 61)
            pred = M * model(family, r["p"], (ahead - K) / span)
            np.testing.assert_allclose(pred, true_curve(np.int8(family), p_true, ahead), rtol=1e-9)
    assert exact[1] >= 0.9 * total[1]
    assert exact[0] >= 0.6 * total[0]


def test_winner_is_the_generating_family_on_clean_data(oracle_mod):
    rng = np.random.default_rng(5)
    wins = 0
    n = 60
    for t in range(n):
        family = t % 2
        H = int(rng.integers(12, 50))
        if family == 0:
            p_true = np.array([rng.uniform(1e-4, 1e-2), rng.uniform(0.01, 1), rng.uniform(0.5, 2), rng.uniform(0, 0.1)])
        else:
            p_true = np.array([rng.uniform(0.8, 0.95), rng.uniform(0, 5), rng.uniform(0, 0.1), 0.0])
        loss = true_curve(np.int8(family), p_true, np.arange(H))
        out = oracle_mod.predict(np.array([0, H]), loss, None, np.array([0.2]), np.array([10.0]), 3.0, 8,
                                 lm_trials=200)
        wins += int(out["family"][0] == family)
    assert wins >= 0.9 * n


def test_prediction_ten_iterations_ahead(oracle_mod):
    # The paper reports under 5 % error when predicting the 10th next iteration; with the
    # standard 20 trials on the noisy synthetic jobs the median error must be well inside that.
    wl = make_workload(2)
    errs = []
    for j in range(0, 1500):
        loss = wl.history(j)
        H = loss.size
        if H < 30:
            continue
        hist, future = loss[:H - 10], true_curve(wl.family[j], wl.params[j], float(H - 1))
        out = oracle_mod.predict(np.array([0, H - 10]), hist, None, np.array([0.2]), np.array([10.0]), 3.0, 4)
        if out["status"][0] != 0:
            continue
        fam, p = int(out["family"][0]), out["params"][0]
        span = H - 11
        pred = out["M"][0] * model(fam, p, 10.0 / span)
        errs.append(abs(pred - future) / future)
    errs = np.array(errs)
    assert np.median(errs) < 0.05
    assert np.mean(errs < 0.05) > 0.7


def test_short_histories_use_linear_extrapolation(oracle_mod):
    # Fewer than four points: no curve is fitted.  One point: one normalised unit per
    # iteration, at most 1 in total.  Two or three: the weighted mean normalised reduction.
    s, w, T, cap = np.array([0.1]), np.array([4.0]), 3.0, 6
    n = np.arange(1, cap + 1)
    m = T * n / (s[0] * n + w[0])
    out = oracle_mod.predict(np.array([0, 1]), np.array([5.0]), None, s, w, T, cap)
    assert out["status"][0] == oracle_mod.ST_NEW
    R = np.minimum(m, 1.0)
    expect = np.minimum.accumulate(np.maximum(np.diff(np.concatenate([[0.0], R])), 0.0))
    np.testing.assert_allclose(out["gain"][0], expect, rtol=1e-13, atol=1e-15)

    loss = np.array([10.0, 7.0, 6.0])      # reductions 3, 1 -> normalised 1, 1/3; weights 0.9, 1
    out = oracle_mod.predict(np.array([0, 3]), loss, None, s, w, T, cap)
    assert out["status"][0] == oracle_mod.ST_SHORT
    rho = (0.9 * 1.0 + 1.0 / 3.0) / 1.9
    R = np.minimum(rho * m, 6.0 / 3.0)
    expect = np.minimum.accumulate(np.maximum(np.diff(np.concatenate([[0.0], R])), 0.0))
    np.testing.assert_allclose(out["gain"][0], expect, rtol=1e-12, atol=1e-15)

    out = oracle_mod.predict(np.array([0, 3]), np.array([1.0, 2.0, 3.0]), None, s, w, T, cap)
    assert out["status"][0] == oracle_mod.ST_FLAT   # the loss never fell
    assert (out["gain"][0] == 0).all()


def test_windows_on_which_no_family_can_start_use_the_mean_normalised_change(oracle_mod):
    """Four or more points, yet neither family has a usable starting point: the prediction falls back to
    the weighted mean normalised reduction per iteration (the rule for short windows), capped by the
    newest normalised level.  The expected figures are typed from that rule, not taken from the oracle."""
    from workloads import make_unfittable_histories
    s, w, T, cap = 0.25, 6.0, 3.0, 8
    n = np.arange(1, cap + 1)
    m = T * n / (s * n + w)
    lengths = [4, 5, 6, 9, 33, 64, 83, 205, 409, 817, 1000]
    J = len(lengths)
    # staircase: every fall is exactly the largest one, so the normalised changes are 1 at the falls and 0 elsewhere
    offsets, losses, m_seen, drops = make_unfittable_histories(lengths, "staircase")
    out = oracle_mod.predict(offsets, losses, m_seen, np.full(J, s), np.full(J, w), T, cap)
    assert (out["status"] == oracle_mod.ST_FIT_FAILED).all()
    assert (out["family"] == -1).all() and np.isinf(out["S"]).all()
    np.testing.assert_array_equal(out["M"], np.full(J, 2.0 ** -53))
    for j, H in enumerate(lengths):
        i = np.arange(1, H)                          # the changes belong to iterations 1 .. H-1
        weight = GAMMA ** (H - 1 - i)
        change = np.isin(i, drops[j]).astype(float)
        rho = (weight * change).sum() / weight.sum()
        assert 0.0 < rho <= 1.0
        R = rho * m                                  # far below the cap: the newest level is about 2^53
        expect = np.diff(np.concatenate([[0.0], R]))
        np.testing.assert_allclose(out["gain"][j], expect, rtol=1e-12, atol=0)
    # flat windows under a tiny largest-reduction-seen: nothing ever fell inside the window, so no gain is predicted
    offsets, losses, m_seen, _ = make_unfittable_histories(lengths, "flat")
    out = oracle_mod.predict(offsets, losses, m_seen, np.full(J, s), np.full(J, w), T, cap)
    assert (out["status"] == oracle_mod.ST_FIT_FAILED).all()
    np.testing.assert_array_equal(out["M"], np.full(J, 1e-300))
    assert (out["gain"] == 0.0).all()


def test_the_cap_of_the_fallback_is_the_newest_normalised_level(oracle_mod):
    # Three points falling 8 -> 4 -> 3: M = 4, newest level 3/4.  The weighted mean change is
    # (0.9 * 1 + 1 * 0.25) / 1.9 per iteration; one core stays below the cap, two reach it.
    s, w, T, cap = np.array([0.0]), np.array([1.0]), 1.0, 5
    out = oracle_mod.predict(np.array([0, 3]), np.array([8.0, 4.0, 3.0]), None, s, w, T, cap)
    rho = (0.9 * 1.0 + 0.25) / 1.9
    R = np.minimum(rho * T * np.arange(1, cap + 1), 0.75)
    expect = np.minimum.accumulate(np.maximum(np.diff(np.concatenate([[0.0], R])), 0.0))
    assert R[-1] == 0.75 and R[0] < 0.75
    np.testing.assert_allclose(out["gain"][0], expect, rtol=1e-13, atol=1e-16)
