"""Pins for the oracle's normalisation step (Design, "Normalizing Quality Metrics")."""

import numpy as np

from workloads import make_workload


def test_hand_worked_example(oracle_mod):
    # losses 10, 7, 6, 6.5, 5: reductions 3, 1, -0.5, 1.5; the largest is 3.
    losses = np.array([10.0, 7.0, 6.0, 6.5, 5.0])
    offsets = np.array([0, 5])
    M, dn, y = oracle_mod.normalise(offsets, losses)
    assert M[0] == 3.0
    np.testing.assert_array_equal(dn, np.array([0.0, 1.0, 1.0 / 3.0, -0.5 / 3.0, 1.5 / 3.0]))
    np.testing.assert_array_equal(y, losses / 3.0)
    # a larger reduction seen before the stored window wins
    M, dn, y = oracle_mod.normalise(offsets, losses, np.array([4.0]))
    assert M[0] == 4.0
    np.testing.assert_array_equal(dn[1:], np.array([3.0, 1.0, -0.5, 1.5]) / 4.0)
    # a smaller one does not
    M, _, _ = oracle_mod.normalise(offsets, losses, np.array([2.0]))
    assert M[0] == 3.0


def test_changes_fall_from_one(oracle_mod):
    # "normalized to decrease from 1 to 0": the largest normalised change of a window that
    # holds the job's whole life is exactly 1 and nothing exceeds it.
    wl = make_workload(2)
    M, dn, _ = oracle_mod.normalise(wl.offsets, wl.losses)
    for j in range(0, wl.n_jobs, 7):
        seg = dn[wl.offsets[j] + 1:wl.offsets[j + 1]]
        if M[j] > 0:
            assert seg.max() == 1.0
            assert (seg <= 1.0).all()


def test_power_of_two_scaling_is_exact(oracle_mod):
    # multiplying a job's losses by 2^m scales M by 2^m exactly and leaves the normalised
    # values, and with them everything downstream, bit-identical
    wl = make_workload(1)
    a = oracle_mod.schedule(wl.offsets, wl.losses, wl.m_seen, wl.s, wl.w, wl.epoch_seconds, wl.total_cores,
                            wl.max_cores_per_job)
    b = oracle_mod.schedule(wl.offsets, wl.losses * 2.0 ** 7, wl.m_seen * 2.0 ** 7, wl.s, wl.w, wl.epoch_seconds,
                            wl.total_cores, wl.max_cores_per_job)
    np.testing.assert_array_equal(a["M"] * 2.0 ** 7, b["M"])
    np.testing.assert_array_equal(a["gain"], b["gain"])
    np.testing.assert_array_equal(a["params"], b["params"])
    np.testing.assert_array_equal(a["alloc"], b["alloc"])


def test_window_shift_invariance(oracle_mod):
    # the fit sees only positions relative to the newest point: the iteration index of the
    # window does not enter (the CSR interface has no k at all), so a job and its copy with a
    # different past give identical predictions when the largest reduction seen is the same
    wl = make_workload(0)
    a = oracle_mod.predict(wl.offsets, wl.losses, wl.m_seen, wl.s, wl.w, wl.epoch_seconds, wl.max_cores_per_job)
    b = oracle_mod.predict(wl.offsets, wl.losses, None, wl.s, wl.w, wl.epoch_seconds, wl.max_cores_per_job)
    np.testing.assert_array_equal(a["gain"], b["gain"])  # config 0 starts at k = 0: m_seen is the window's own
