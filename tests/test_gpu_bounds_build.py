"""The bounds-checking build of the library (-DSLAQ_DEBUG_BOUNDS, the stand-in for a memory checker): every index
into a ring, the packed pool, a shared-memory slice, the gain table, a candidate segment or a histogram is compared
with its extent before the access, a bad one sets a bit of the device error word and is skipped.  Run over the
workloads whose shapes stress the index arithmetic, the word must stay zero (slaq_schedule reports a non-zero word
as an error) and the results must equal the ordinary library's bit for bit."""

import numpy as np
import pytest

from workloads import make_workload

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def slaq():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import paper_1802_04819_b200 as mod
    from paper_1802_04819_b200.build import build_variant
    mod.build()
    build_variant("bounds")
    return mod


def _epoch(slaq, wl, variant, packed, params=()):
    sched = slaq.Scheduler(wl.n_jobs, wl.max_hist, wl.max_cores_per_job, variant=variant)
    ids = np.arange(wl.n_jobs, dtype=np.int32)
    sched.load_histories(ids, wl.offsets, wl.losses, wl.k_last, wl.m_seen, packed=packed)
    sched.set_time_model(ids, wl.s, wl.w)
    for key, value in params:
        sched.set_param(key, value)
    alloc, rc = sched.schedule(wl.epoch_seconds, wl.total_cores)      # raises if the error word is set
    pred = sched.get_predictions()
    norm = sched.get_normalised(ids[: min(wl.n_jobs, 300)])
    sched.close()
    return alloc, pred, norm


CLASS_EDGES = [4, 5, 7, 8, 9, 15, 16, 17, 31, 32, 33, 62, 63, 64, 65, 66, 82, 83, 124, 125, 126, 127, 128, 129, 204, 205,
               249, 250, 251, 252, 255, 256, 257, 408, 409, 499, 500, 501, 502, 511, 512, 513, 816, 817, 998, 999, 1000]


@pytest.mark.parametrize("case", ["cfg0", "cfg1", "cfg2", "cfg2-packed", "edges", "edges-as-a-large-cluster", "long",
                                  "cfg4-ring", "small-slices"])
def test_no_index_leaves_its_extent(slaq, case):
    params, packed = (), False
    if case in ("cfg0", "cfg1", "cfg2", "cfg2-packed"):
        wl = make_workload(int(case[3]))
        packed = case.endswith("packed")
    elif case.startswith("edges"):
        wl = make_workload(3, hist_lengths=CLASS_EDGES * 2)
        packed = True
        if case.endswith("cluster"):
            params = ((slaq.binding.P_FIT_CLUSTER_JOBS, 10_000_000),)     # as few lanes per job as the windows allow
    elif case == "long":
        wl = make_workload(3, hist_lengths=[6000, 5999, 4097, 3001, 3000, 1501, 1500, 751, 750, 400, 100, 20, 4, 3])
        packed = True
    elif case == "cfg4-ring":
        wl = make_workload(4, n_jobs=20000)
    else:
        wl = make_workload(3, n_jobs=1500)
        packed = True
        params = ((slaq.binding.P_FIT_SLICE_BYTES, 8192),)
    checked = _epoch(slaq, wl, "bounds", packed, params)
    plain = _epoch(slaq, wl, None, packed, params)
    np.testing.assert_array_equal(checked[0], plain[0])
    for key in ("gain", "params", "S", "R", "status", "M"):
        np.testing.assert_array_equal(checked[1][key], plain[1][key])
    for a, b in zip(checked[2], plain[2]):
        np.testing.assert_array_equal(a, b)


def test_appends_through_a_wrapping_ring_and_the_sharded_steps(slaq):
    from paper_1802_04819_b200 import LocalExchange, schedule_sharded
    from workloads import true_curve
    wl = make_workload(1)
    J, cap, max_hist = wl.n_jobs, wl.max_cores_per_job, 12
    sched = slaq.Scheduler(J, max_hist, cap, variant="bounds")
    ids = np.arange(J, dtype=np.int32)
    rng = np.random.default_rng(3)
    for step in range(30):                                  # the ring of 12 wraps twice
        k = np.full(J, float(step))
        losses = true_curve(wl.family, wl.params, k) * np.exp(0.01 * rng.standard_normal(J))
        sched.append_losses(ids, losses, wl.s + wl.w / (1 + step % 3), np.full(J, 1 + step % 3, np.int32))
        if step % 7 == 6:
            alloc, rc = sched.schedule(wl.epoch_seconds, wl.total_cores)
            assert rc == 0 and alloc.sum() == wl.total_cores
    sched.remove_jobs(ids[::5])
    alloc, rc = sched.schedule(wl.epoch_seconds, wl.total_cores)
    assert alloc[::5].sum() == 0
    sched.close()
    # the step-by-step calls of a sharded cluster run the same kernels: two shards of the bounds build
    wl = make_workload(2, n_jobs=1200)
    cut = 500
    shards = []
    for lo, hi in ((0, cut), (cut, wl.n_jobs)):
        n = hi - lo
        sh = slaq.Scheduler(n, wl.max_hist, wl.max_cores_per_job, variant="bounds")
        off = wl.offsets[lo:hi + 1] - wl.offsets[lo]
        sh.load_histories(np.arange(n, dtype=np.int32), off, wl.losses[wl.offsets[lo]:wl.offsets[hi]], wl.k_last[lo:hi],
                          wl.m_seen[lo:hi])
        sh.set_time_model(np.arange(n, dtype=np.int32), wl.s[lo:hi], wl.w[lo:hi])
        shards.append(sh)
    allocs = schedule_sharded(shards, LocalExchange(), wl.epoch_seconds, wl.total_cores)
    assert sum(int(a.sum()) for a in allocs) == wl.total_cores
