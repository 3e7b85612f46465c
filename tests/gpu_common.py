"""Helpers shared by the GPU parity tests: build a scheduler from a workload, compare with the oracle."""

import numpy as np

R_RTOL, R_ATOL = 1e-6, 1e-9          # predicted reductions: |gpu - cpu| <= 1e-6 |cpu| + 1e-9
THRESHOLD_BAND = 1e-9                # allocations may differ where a deciding gain lies this close to the threshold


def make_scheduler(wl, packed=False, max_hist=None, workspace=None, m_seen=None):
    """m_seen: the largest reduction seen that the handle is told (default: the workload's, which already
    includes the stored window's own largest reduction)."""
    import paper_1802_04819_b200 as slaq
    sched = slaq.Scheduler(wl.n_jobs, max_hist or wl.max_hist, wl.max_cores_per_job, workspace=workspace)
    ids = np.arange(wl.n_jobs, dtype=np.int32)
    sched.load_histories(ids, wl.offsets, wl.losses, wl.k_last, wl.m_seen if m_seen is None else m_seen, packed=packed)
    sched.set_time_model(ids, wl.s, wl.w)
    return sched


def oracle_epoch(oracle, wl, total_cores=None, threads=0):
    return oracle.schedule(wl.offsets, wl.losses, wl.m_seen, wl.s, wl.w, wl.epoch_seconds,
                           wl.total_cores if total_cores is None else total_cores, wl.max_cores_per_job,
                           threads=threads)


def compare_epoch(gpu_alloc, pred, ref, total_cores, cap, allow_unstable=0, loose=(1e-4, 1e-7), total_rtol=1e-9):
    """Element-by-element comparison of one epoch.  Returns a dict of counts for reporting.

    allow_unstable: how many jobs may miss the tolerance on R(n); those must still meet the
    `loose` (relative, absolute) one.  Zero everywhere except where the fits of both sides run
    freely over several epochs from their own earlier results, so that rounding differences
    compound in the few jobs whose residual is flat along a direction.
    total_rtol: tolerance on the sum of the predicted reductions at the allocation (the per-job
    tolerance is R_RTOL; the sum of the cold path's fits agrees a thousand times better)."""
    status_g, status_c = pred["status"], ref["status"]
    np.testing.assert_array_equal(status_g, status_c)
    fitted = status_c == 0
    # largest reduction: exactly rounded operations only, so bit-exact
    both = np.isfinite(ref["M"])
    np.testing.assert_array_equal(pred["M"][both], ref["M"][both])
    assert (np.isnan(pred["M"]) == np.isnan(ref["M"])).all()
    # winner: may differ only where the two residuals tie to rounding
    fam_diff = np.nonzero(pred["family"] != ref["family"])[0]
    for j in fam_diff:
        S = ref["S"][j]
        assert abs(S[0] - S[1]) <= 1e-9 * max(abs(S[0]), abs(S[1])), f"job {j}: family differs, residuals {S}"
    # R(n) for every n: cumulative gains
    Rg, Rc = np.cumsum(pred["gain"], axis=1), np.cumsum(ref["gain"], axis=1)
    bad = np.abs(Rg - Rc) > R_RTOL * np.abs(Rc) + R_ATOL
    bad_jobs = np.nonzero(bad.any(axis=1))[0]
    bad_jobs = np.setdiff1d(bad_jobs, fam_diff)    # a tied winner may predict differently: judged separately
    assert bad_jobs.size <= allow_unstable, (
        f"{bad_jobs.size} jobs exceed the tolerance on R(n): first {bad_jobs[:5]}, "
        f"worst {np.abs(Rg - Rc)[bad_jobs].max() if bad_jobs.size else 0}")
    if bad_jobs.size:
        np.testing.assert_allclose(Rg[bad_jobs], Rc[bad_jobs], rtol=loose[0], atol=loose[1])
    # allocation: equal except where the deciding gains lie within the band around the threshold
    ca = ref["alloc"]
    assert gpu_alloc.sum() == ca.sum()
    diff = np.nonzero(gpu_alloc != ca)[0]
    if diff.size:
        active = status_c != -1
        floor = 1 if total_cores >= active.sum() else 0
        g = ref["gain"]
        taken = np.arange(cap)[None, :] < ca[:, None]
        beyond = taken & (np.arange(cap)[None, :] >= floor)
        tau = g[beyond].min() if beyond.any() else 0.0
        for j in diff:
            lo, hi = sorted((gpu_alloc[j], ca[j]))
            contested = np.concatenate([ref["gain"][j, lo:hi], pred["gain"][j, lo:hi]])
            assert np.all(np.abs(contested - tau) <= THRESHOLD_BAND + 1e-6 * tau), (
                f"job {j}: alloc {gpu_alloc[j]} vs {ca[j]} but gains {contested} are not near threshold {tau}")
    # predicted reduction at the allocation, and its total
    same = gpu_alloc == ca
    same[bad_jobs] = False
    same[fam_diff] = False
    np.testing.assert_allclose(pred["R"][same], ref["R"][same], rtol=R_RTOL, atol=R_ATOL)
    tot_c = ref["R"].sum()
    slack = np.abs(pred["R"] - ref["R"])[np.union1d(bad_jobs, fam_diff).astype(np.int64)].sum()
    assert abs(pred["R"].sum() - tot_c) <= total_rtol * abs(tot_c) + 1e-9 * max(1, diff.size) + slack
    return dict(jobs=int(status_c.size), fitted=int(fitted.sum()), family_ties=int(fam_diff.size),
                unstable=int(bad_jobs.size), alloc_diff=int(diff.size))


def tolerance_widths(pred, ref):
    """Per job the largest |R_gpu(n) - R_cpu(n)| over n in units of the tolerance (1 = at the tolerance); jobs whose
    winner differs are left out (judged separately by compare_epoch)."""
    Rg, Rc = np.cumsum(pred["gain"], axis=1), np.cumsum(ref["gain"], axis=1)
    width = (np.abs(Rg - Rc) / (R_RTOL * np.abs(Rc) + R_ATOL)).max(axis=1)
    return width[pred["family"] == ref["family"]]


def oracle_spread(oracle_mod, wl, j, cap, n_trials=24):
    """How far the oracle's own R(n) of job j moves when its losses are perturbed by 1e-13 relative: per n the
    largest distance from the unperturbed result.  Zero to rounding for a fit that has finished; large where the
    twenty trials end on a path-dependent point."""
    h = wl.history(j)
    off = np.array([0, h.size])
    one = lambda a: np.array([a[j]])     # noqa: E731
    base = np.cumsum(oracle_mod.predict(off, h, one(wl.m_seen), one(wl.s), one(wl.w), wl.epoch_seconds, cap)["gain"][0])
    rng = np.random.default_rng(1000 + j)
    spread = np.zeros_like(base)
    for _ in range(n_trials):
        hp = h * (1.0 + 1e-13 * rng.standard_normal(h.size))
        R = np.cumsum(oracle_mod.predict(off, hp, one(wl.m_seen), one(wl.s), one(wl.w), wl.epoch_seconds, cap)["gain"][0])
        spread = np.maximum(spread, np.abs(R - base))
    return spread
