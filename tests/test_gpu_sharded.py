"""One cluster split over several shards must be scheduled exactly like the same cluster on one handle.

Only one GPU is available to these tests, so the shards live in one process on one GPU and their
histograms are summed locally (``LocalExchange``): the calls, their order and the exchanged data are
those of the multi-GPU protocol; with one shard per process only the transport differs."""

import numpy as np
import pytest

from workloads import make_workload

pytestmark = pytest.mark.gpu


def _build(slaq, wl, lo, hi):
    ids = np.arange(hi - lo, dtype=np.int32)
    sched = slaq.Scheduler(hi - lo, wl.max_hist, wl.max_cores_per_job)
    off = wl.offsets[lo:hi + 1] - wl.offsets[lo]
    sched.load_histories(ids, off, wl.losses[wl.offsets[lo]:wl.offsets[hi]], wl.k_last[lo:hi], wl.m_seen[lo:hi])
    sched.set_time_model(ids, wl.s[lo:hi], wl.w[lo:hi])
    return sched


@pytest.mark.parametrize("cfg,n_jobs,cuts", [(1, None, [0, 70, 160]), (2, None, [0, 1000, 1001, 2900, 4000]),
                                             (4, 12000, [0, 5000, 12000])])
def test_sharded_cluster_equals_one_handle(cfg, n_jobs, cuts):
    import paper_1802_04819_b200 as slaq
    slaq.build()
    wl = make_workload(cfg, n_jobs=n_jobs)
    whole = _build(slaq, wl, 0, wl.n_jobs)
    shards = [_build(slaq, wl, lo, hi) for lo, hi in zip(cuts[:-1], cuts[1:])]
    for C in (wl.total_cores, wl.n_jobs - 3, wl.n_jobs, 2 * wl.n_jobs + 1, wl.n_jobs * wl.max_cores_per_job + 5):
        ref, _ = whole.schedule(wl.epoch_seconds, C)
        parts = slaq.schedule_sharded(shards, slaq.LocalExchange(), wl.epoch_seconds, C)
        np.testing.assert_array_equal(np.concatenate(parts), ref)        # integer work: bit-exact
        gains = np.concatenate([s.get_predictions()["gain"] for s in shards])
        np.testing.assert_array_equal(gains, whole.get_predictions()["gain"])
        R = np.concatenate([s.get_predictions(want_gain=False)["R"] for s in shards])
        np.testing.assert_array_equal(R, whole.get_predictions(want_gain=False)["R"])


def test_sharded_ties_cross_shard_boundaries():
    import paper_1802_04819_b200 as slaq
    slaq.build()
    # identical jobs everywhere: every gain ties with its copies in all shards, lowest global id first
    base = make_workload(2, n_jobs=1)
    J = 300
    reps = lambda a: np.repeat(a, J, axis=0)      # noqa: E731
    H = int(base.hist_len[0])
    offsets = np.arange(J + 1, dtype=np.int64) * H
    losses = np.tile(base.losses, J)

    def build(lo, hi):
        ids = np.arange(hi - lo, dtype=np.int32)
        s = slaq.Scheduler(hi - lo, base.max_hist, 8)
        s.load_histories(ids, offsets[lo:hi + 1] - offsets[lo], losses[offsets[lo]:offsets[hi]],
                         reps(base.k_last)[lo:hi], reps(base.m_seen)[lo:hi])
        s.set_time_model(ids, reps(base.s)[lo:hi], reps(base.w)[lo:hi])
        return s

    whole = build(0, J)
    shards = [build(0, 100), build(100, 101), build(101, 300)]
    for C in (J + 1, J + 150, 2 * J + 7, 5 * J - 1):
        ref, _ = whole.schedule(3.0, C)
        parts = np.concatenate(slaq.schedule_sharded(shards, slaq.LocalExchange(), 3.0, C))
        np.testing.assert_array_equal(parts, ref)
        assert (np.diff(ref) <= 0).all()          # identical jobs: extra units go to the lowest ids
