"""Checkpoint and resume: a handle that imported another handle's exported state continues bit for bit like it."""

import numpy as np
import pytest

from workloads import make_workload, true_curve

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def slaq():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import paper_1802_04819_b200 as mod
    mod.build()
    return mod


def _advance(sched, wl, rng_seed, steps, k0):
    """`steps` rounds of one new loss per job (with an iteration time booked at the last allocation) and an epoch."""
    rng = np.random.default_rng(rng_seed)
    J = wl.n_jobs
    ids = np.arange(J, dtype=np.int32)
    out = []
    for step in range(steps):
        k = (k0 + step).astype(np.float64)
        losses = true_curve(wl.family, wl.params, k) * np.exp(0.01 * rng.standard_normal(J))
        sched.append_losses(ids, losses, wl.s + wl.w / (1 + step % 4), np.full(J, 1 + step % 4, np.int32))
        alloc, rc = sched.schedule(wl.epoch_seconds, wl.total_cores)
        pred = sched.get_predictions()
        out.append((alloc.copy(), pred["gain"].copy(), pred["params"].copy(), pred["status"].copy()))
    return out


@pytest.mark.parametrize("warm", [0, 1])
@pytest.mark.parametrize("packed", [False, True])
def test_an_imported_state_continues_like_the_exporting_handle(slaq, warm, packed):
    wl = make_workload(2, n_jobs=700)
    J, cap = wl.n_jobs, wl.max_cores_per_job
    ids = np.arange(J, dtype=np.int32)
    a = slaq.Scheduler(J, wl.max_hist, cap)
    a.set_param(slaq.binding.P_WARM_START, warm)
    a.load_histories(ids, wl.offsets, wl.losses, wl.k_last, wl.m_seen, packed=packed)
    a.set_time_model(ids[::3], wl.s[::3], wl.w[::3])           # a fixed law for a third, sampled laws for the rest
    a.remove_jobs(ids[5::50])                                   # some inactive ids
    live = np.ones(J, bool)
    live[5::50] = False
    k_next = wl.k_last + 1
    _advance(a, wl, 1, 3, k_next)                               # appends to removed ids start them anew at iteration 0
    blob = a.export_state()
    b = slaq.Scheduler(J, wl.max_hist, cap)
    b.set_param(slaq.binding.P_WARM_START, warm)
    b.import_state(blob)
    c = slaq.Scheduler(J, wl.max_hist + 9, cap)                 # longer rings are allowed: the same epoch until
    c.set_param(slaq.binding.P_WARM_START, warm)                # appends let its windows grow beyond the exporter's
    c.import_state(blob)
    np.testing.assert_array_equal(c.schedule(wl.epoch_seconds, wl.total_cores)[0],
                                  a.schedule(wl.epoch_seconds, wl.total_cores)[0])
    c.close()
    assert b.get_active_count() == a.get_active_count()
    np.testing.assert_array_equal(b.export_state()[64:], blob[64:])    # the same state again (header: longest window)
    sa, wa = a.get_time_model()
    sb, wb = b.get_time_model()
    np.testing.assert_array_equal(sa, sb)
    np.testing.assert_array_equal(wa, wb)
    if packed:      # a packed row keeps the length it was loaded with, the importer's ring grows: equal only until appends
        np.testing.assert_array_equal(b.schedule(wl.epoch_seconds, wl.total_cores)[0],
                                      a.schedule(wl.epoch_seconds, wl.total_cores)[0])
        np.testing.assert_array_equal(a.get_predictions()["gain"], b.get_predictions()["gain"])
        return
    ra = _advance(a, wl, 2, 4, k_next + 3)
    rb = _advance(b, wl, 2, 4, k_next + 3)
    for (alloc_a, gain_a, par_a, st_a), (alloc_b, gain_b, par_b, st_b) in zip(ra, rb):
        np.testing.assert_array_equal(alloc_a, alloc_b)
        np.testing.assert_array_equal(gain_a, gain_b)
        np.testing.assert_array_equal(par_a, par_b)
        np.testing.assert_array_equal(st_a, st_b)
    fa, fb = a.get_fit_state(), b.get_fit_state()
    for key in fa:
        np.testing.assert_array_equal(fa[key], fb[key])


def test_blobs_that_do_not_fit_are_refused_and_leave_the_handle_alone(slaq):
    wl = make_workload(1)
    J, cap = wl.n_jobs, wl.max_cores_per_job
    ids = np.arange(J, dtype=np.int32)
    a = slaq.Scheduler(J, wl.max_hist, cap)
    a.load_histories(ids, wl.offsets, wl.losses, wl.k_last, wl.m_seen)
    a.set_time_model(ids, wl.s, wl.w)
    before, _ = a.schedule(wl.epoch_seconds, wl.total_cores)
    blob = a.export_state()
    bad_magic = blob.copy()
    bad_magic[0] ^= 0xFF
    other_jobs = slaq.Scheduler(J + 1, wl.max_hist, cap)
    short_ring = slaq.Scheduler(J, max(4, int(wl.hist_len.max()) - 1), cap)
    for target, data, code in ((a, bad_magic, -1), (a, blob[:-8], -1), (a, blob[:40], -1), (other_jobs, blob, -2),
                               (short_ring, blob, -2)):
        with pytest.raises(slaq.SlaqError) as err:
            target.import_state(data)
        assert err.value.code == code
    after, _ = a.schedule(wl.epoch_seconds, wl.total_cores)
    np.testing.assert_array_equal(before, after)
    a.import_state(blob)                                        # and the good blob still goes in
    again, _ = a.schedule(wl.epoch_seconds, wl.total_cores)
    np.testing.assert_array_equal(before, again)
    empty = slaq.Scheduler(8, 16, 4)
    empty.import_state(empty.export_state())
    assert empty.get_active_count() == 0
    # a handle that holds a packed pool (other jobs, other seed) gives it up when it imports
    other = make_workload(1, seed_offset=3)
    packed = slaq.Scheduler(J, wl.max_hist, cap)
    packed.load_histories(ids, other.offsets, other.losses, other.k_last, other.m_seen, packed=True)
    packed.set_time_model(ids, other.s, other.w)
    packed.set_target_loss(ids[:5], other.losses[other.offsets[1:6] - 1] * 0.5)
    packed.schedule(wl.epoch_seconds, wl.total_cores)
    packed.import_state(blob)
    np.testing.assert_array_equal(packed.schedule(wl.epoch_seconds, wl.total_cores)[0], before)
    np.testing.assert_array_equal(packed.export_state()[64:], blob[64:])
    packed.append_losses(ids, wl.losses[wl.offsets[1:] - 1] * 0.98, wl.s + wl.w)       # its rings take new losses
    a.append_losses(ids, wl.losses[wl.offsets[1:] - 1] * 0.98, wl.s + wl.w)
    np.testing.assert_array_equal(packed.schedule(wl.epoch_seconds, wl.total_cores)[0],
                                  a.schedule(wl.epoch_seconds, wl.total_cores)[0])
