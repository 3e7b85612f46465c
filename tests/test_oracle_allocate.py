"""Pins for the oracle's greedy allocation ("Scheduling Based on Quality Improvements")."""

import itertools

import numpy as np

from workloads import make_workload


def brute_force(gain, total):
    """Best total predicted reduction over every allocation with a_j >= 1 and sum a_j <= total."""
    J, cap = gain.shape
    R = np.concatenate([np.zeros((J, 1)), np.cumsum(gain, axis=1)], axis=1)
    best, arg = -1.0, []
    for a in itertools.product(range(1, cap + 1), repeat=J):
        if sum(a) > total:
            continue
        val = sum(R[j, a[j]] for j in range(J))
        if val > best + 1e-15:
            best, arg = val, [a]
        elif abs(val - best) <= 1e-15:
            arg.append(a)
    return best, arg


def test_greedy_equals_brute_force_on_tiny_clusters(oracle_mod):
    # max sum_j [Loss_j(a_j, t) - Loss_j(a_j, t+T)] s.t. sum a_j <= C, every a_j >= 1
    rng = np.random.default_rng(2)
    for trial in range(40):
        J = int(rng.integers(2, 5))
        cap = int(rng.integers(2, 6))
        C = int(rng.integers(J, 13))
        raw = rng.uniform(0, 1, (J, cap)) * rng.uniform(0.1, 3, (J, 1))
        gain = -np.sort(-raw, axis=1)                    # non-increasing rows
        alloc = oracle_mod.allocate(gain, np.ones(J, np.uint8), C)
        assert alloc.sum() == min(C, J * cap)
        R = oracle_mod.reduction_at(gain, alloc)
        best, arg = brute_force(gain, C)
        assert abs(R.sum() - best) <= 1e-12 * max(best, 1.0)
        if len(arg) == 1:
            assert tuple(alloc) == arg[0]


def test_greedy_on_fitted_gains_matches_brute_force(oracle_mod):
    wl = make_workload(0)
    out = oracle_mod.predict(wl.offsets, wl.losses, wl.m_seen, wl.s, wl.w, wl.epoch_seconds, 4)
    gain = out["gain"][:4]
    for C in (4, 7, 12):
        alloc = oracle_mod.allocate(gain, np.ones(4, np.uint8), C)
        best, _ = brute_force(gain, C)
        assert abs(oracle_mod.reduction_at(gain, alloc).sum() - best) <= 1e-12 * best


def test_capacity_and_floor(oracle_mod):
    for cfg in (0, 1, 2):
        wl = make_workload(cfg)
        out = oracle_mod.schedule(wl.offsets, wl.losses, wl.m_seen, wl.s, wl.w, wl.epoch_seconds, wl.total_cores,
                                  wl.max_cores_per_job)
        a = out["alloc"]
        assert a.sum() == wl.total_cores
        assert a.min() >= 1 and a.max() <= wl.max_cores_per_job


def test_ties_go_to_the_lowest_job_id(oracle_mod):
    gain = np.tile(np.array([[0.5, 0.25, 0.25, 0.1]]), (3, 1))
    active = np.ones(3, np.uint8)
    # 3 floor cores, then the 0.25s in job order, each job's second 0.25 before the next job's first
    np.testing.assert_array_equal(oracle_mod.allocate(gain, active, 4), [2, 1, 1])
    np.testing.assert_array_equal(oracle_mod.allocate(gain, active, 5), [3, 1, 1])
    np.testing.assert_array_equal(oracle_mod.allocate(gain, active, 6), [3, 2, 1])
    np.testing.assert_array_equal(oracle_mod.allocate(gain, active, 9), [3, 3, 3])
    np.testing.assert_array_equal(oracle_mod.allocate(gain, active, 10), [4, 3, 3])
    # all-zero gains are still handed out, lowest ids first
    np.testing.assert_array_equal(oracle_mod.allocate(np.zeros((3, 4)), active, 6), [4, 1, 1])


def test_fewer_cores_than_jobs_and_more_cores_than_slots(oracle_mod):
    gain = np.array([[0.1, 0.05], [0.9, 0.5], [0.3, 0.2], [0.0, 0.0]])
    active = np.array([1, 1, 1, 1], np.uint8)
    # no floor when there are fewer cores than jobs: the best first units win
    np.testing.assert_array_equal(oracle_mod.allocate(gain, active, 3), [0, 2, 1, 0])
    # more cores than slots: everyone is filled to the cap, the rest stays idle
    np.testing.assert_array_equal(oracle_mod.allocate(gain, active, 100), [2, 2, 2, 2])
    # inactive ids never receive cores
    np.testing.assert_array_equal(oracle_mod.allocate(gain, np.array([1, 0, 1, 0], np.uint8), 3), [1, 0, 2, 0])
    np.testing.assert_array_equal(oracle_mod.allocate(gain, active, 0), [0, 0, 0, 0])


def test_clones_split_ties_by_id(oracle_mod):
    wl = make_workload(4, n_jobs=3000)
    out = oracle_mod.schedule(wl.offsets, wl.losses, wl.m_seen, wl.s, wl.w, wl.epoch_seconds, wl.total_cores,
                              wl.max_cores_per_job)
    dst = np.nonzero(wl.clone_of >= 0)[0]
    src = wl.clone_of[dst]
    assert dst.size > 0
    np.testing.assert_array_equal(out["gain"][dst], out["gain"][src])
    lo, hi = np.minimum(src, dst), np.maximum(src, dst)
    diff = out["alloc"][lo] - out["alloc"][hi]
    assert (diff >= 0).all()                     # the lower id is never behind
    assert out["alloc"].sum() == wl.total_cores
