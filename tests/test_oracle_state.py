"""The oracle's between-epoch state (window, largest reduction seen, time sums) and the
workload generator's invariants."""

import numpy as np

from workloads import CONFIGS, make_workload, make_time_samples


def test_append_path_equals_bulk_path(oracle_mod):
    # feeding a job's losses one at a time must leave the same window and the same
    # "largest change seen so far" as loading the whole history at once
    wl = make_workload(1)
    J = wl.n_jobs
    a = oracle_mod.OracleScheduler(J, wl.max_hist, wl.max_cores_per_job)
    b = oracle_mod.OracleScheduler(J, wl.max_hist, wl.max_cores_per_job)
    ids = np.arange(J)
    b.load_histories(ids, wl.offsets, wl.losses, wl.k_last, wl.m_seen)
    b.set_time_model(ids, wl.s, wl.w)
    fresh = wl.k_last + 1 == wl.hist_len            # jobs whose whole life is in the window
    H = wl.hist_len
    for step in range(int(H.max())):
        live = np.nonzero((step < H) & fresh)[0]
        a.append_losses(live, wl.losses[wl.offsets[live] + step])
    a.set_time_model(ids, wl.s, wl.w)
    ra = a.schedule(wl.epoch_seconds, wl.total_cores)
    rb = b.schedule(wl.epoch_seconds, wl.total_cores)
    np.testing.assert_array_equal(ra["gain"][fresh], rb["gain"][fresh])
    np.testing.assert_array_equal(a.k_last[fresh], wl.k_last[fresh])
    assert (ra["alloc"][~fresh] == 0).all()


def test_ring_forgets_points_but_not_the_largest_reduction(oracle_mod):
    sched = oracle_mod.OracleScheduler(1, 4, 4)
    losses = [10.0, 4.0, 3.5, 3.2, 3.0, 2.9]
    for v in losses:
        sched.append_losses([0], [v], [1.0])
    assert list(sched.window[0]) == losses[-4:]
    assert sched.m_seen[0] == 6.0                    # 10 -> 4 happened before the stored window
    assert sched.k_last[0] == 5
    out = sched.schedule(3.0, 4)
    assert out["M"][0] == 6.0
    sched.remove_jobs([0])
    assert sched.schedule(3.0, 4)["alloc"][0] == 0


def test_default_core_count_is_last_allocation(oracle_mod):
    wl = make_workload(0)
    sched = oracle_mod.OracleScheduler(wl.n_jobs, wl.max_hist, wl.max_cores_per_job)
    ids = np.arange(wl.n_jobs)
    sched.load_histories(ids, wl.offsets, wl.losses, wl.k_last, wl.m_seen)
    sched.set_time_model(ids, wl.s, wl.w)
    alloc = sched.schedule(wl.epoch_seconds, wl.total_cores)["alloc"]
    t = wl.s + wl.w / alloc
    sched.append_losses(ids, wl.losses[wl.offsets[1:] - 1] * 0.99, t)
    np.testing.assert_allclose(sched.tm[:, 5], t * alloc)     # sum of t * n used the allocation


def test_workload_shapes_follow_the_configs():
    for cfg, n in ((0, None), (1, None), (2, None), (3, 3000), (4, 5000)):
        wl = make_workload(cfg, n_jobs=n)
        spec = CONFIGS[cfg]
        J = spec["J"] if n is None else n
        assert wl.n_jobs == J and wl.total_cores == spec["cores_per_job"] * J
        H = wl.hist_len
        assert H.min() >= 3 and H.max() <= spec["hmax"]
        assert np.isfinite(wl.losses).all() and (wl.losses > 0).all()
        again = make_workload(cfg, n_jobs=n)
        np.testing.assert_array_equal(wl.losses, again.losses)
    wl = make_workload(4, n_jobs=5000)
    H = wl.hist_len
    assert 0.15 < (H < 64).mean() < 0.25                        # new jobs hold 3-5 points
    conv = wl.k_last >= 10_000
    assert 0.15 < conv.mean() < 0.25
    for j in np.nonzero(conv)[0][:200]:
        h = wl.history(j)
        assert np.abs(h[:-1] - h[1:]).max() / wl.m_seen[j] < 1e-4   # converged: normalised change < 1e-4
    dst = np.nonzero(wl.clone_of >= 0)[0]
    assert dst.size == 50
    for j in dst:
        np.testing.assert_array_equal(wl.history(j), wl.history(wl.clone_of[j]))
    cores, secs = make_time_samples(wl, 4, np.arange(3))
    assert cores[:, 0].tolist() == [1, 2, 4, 8]
