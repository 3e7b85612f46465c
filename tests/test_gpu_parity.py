"""GPU-vs-oracle parity, element by element, through the C ABI."""

import numpy as np
import pytest

from workloads import make_workload, make_time_samples
from gpu_common import compare_epoch, make_scheduler, oracle_epoch, oracle_spread

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def slaq():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    import paper_1802_04819_b200 as mod
    mod.build()
    return mod


# ---------------------------------------------------------------- normalisation: bit-exact
@pytest.mark.parametrize("own_maximum", [False, True])
@pytest.mark.parametrize("cfg,n_jobs,packed", [(1, None, False), (2, None, True), (4, 3000, False), (3, 2000, True)])
def test_normalisation_is_bit_exact(slaq, oracle_mod, cfg, n_jobs, packed, own_maximum):
    """own_maximum: both sides are told only the largest reduction BEFORE the stored window (nothing for a window
    that starts at iteration 0), so the largest reduction inside the window is found by the kernel itself; the
    workload's m_seen already contains it."""
    wl = make_workload(cfg, n_jobs=n_jobs)
    seen = wl.m_past if own_maximum else wl.m_seen
    if own_maximum:
        assert (seen < wl.m_seen).any()          # the window's own maximum decides for some jobs
    sched = make_scheduler(wl, packed=packed, m_seen=seen)
    ids = np.arange(wl.n_jobs)
    offsets, changes, levels, largest = sched.get_normalised(ids, capacity=int(wl.offsets[-1]))
    M, dn, y = oracle_mod.normalise(wl.offsets, wl.losses, seen)
    if own_maximum:                              # typed here: the window's largest one-step reduction joined with the past
        for j in range(0, wl.n_jobs, max(1, wl.n_jobs // 200)):
            h = wl.history(j)
            assert largest[j] == max(seen[j], (h[:-1] - h[1:]).max())
    np.testing.assert_array_equal(offsets, wl.offsets)
    np.testing.assert_array_equal(largest, M)
    usable = np.repeat(M > 0, wl.hist_len)
    np.testing.assert_array_equal(changes[usable], dn[usable])
    np.testing.assert_array_equal(levels[usable], y[usable])
    assert np.isnan(levels[~usable]).all()
    # the paper's property: normalised changes never exceed 1
    assert (changes[usable] <= 1.0).all()


# ---------------------------------------------------------------- allocation alone: bit-exact
def _alloc_case(slaq, oracle_mod, gain, active, C):
    J, cap = gain.shape
    sched = slaq.Scheduler(J, 8, cap)
    live = np.nonzero(active)[0].astype(np.int32)
    if live.size:
        sched.append_losses(live, np.ones(live.size))
    sched.set_gains(gain)
    got, rc = sched.allocate_only(C)
    want = oracle_mod.allocate(gain, active, C)
    np.testing.assert_array_equal(got, want)
    n_act = int(active.sum())
    if n_act and C < n_act:
        assert rc == 1
    elif C > n_act * cap:
        assert rc == 2
    return got


def test_allocation_matches_greedy_on_oracle_gains(slaq, oracle_mod):
    for cfg, n in ((1, None), (2, None), (4, 6000)):
        wl = make_workload(cfg, n_jobs=n)
        ref = oracle_mod.predict(wl.offsets, wl.losses, wl.m_seen, wl.s, wl.w, wl.epoch_seconds,
                                 wl.max_cores_per_job)
        active = np.ones(wl.n_jobs, np.uint8)
        for C in (wl.total_cores, wl.n_jobs, wl.n_jobs + 1, 2 * wl.n_jobs + 7, wl.n_jobs * wl.max_cores_per_job - 3):
            _alloc_case(slaq, oracle_mod, ref["gain"], active, C)


def test_allocation_degenerate_gain_tables(slaq, oracle_mod):
    rng = np.random.default_rng(4)
    J, cap = 700, 12
    active = np.ones(J, np.uint8)
    zero = np.zeros((J, cap))
    equal = np.full((J, cap), 0.125)
    few = -np.sort(-rng.integers(0, 4, (J, cap)).astype(float) / 8.0, axis=1)   # many exact ties at 4 levels
    for gain in (zero, equal, few):
        for C in (0, 1, J - 1, J, J + 1, 3 * J, J * cap - 1, J * cap, J * cap + 5):
            _alloc_case(slaq, oracle_mod, gain, active, C)
    # inactive rows never receive cores, even with the largest gains
    some = (rng.random(J) < 0.6).astype(np.uint8)
    raw = -np.sort(-rng.uniform(0, 1, (J, cap)), axis=1)
    for C in (int(some.sum()) - 3, int(some.sum()), 2 * J, J * cap):
        got = _alloc_case(slaq, oracle_mod, raw, some, C)
        assert (got[some == 0] == 0).all()
    # tiny and huge magnitudes, denormals included, order like their bit patterns
    wide = -np.sort(-(10.0 ** rng.uniform(-320, 300, (J, cap))), axis=1)
    for C in (J + 5, 4 * J):
        _alloc_case(slaq, oracle_mod, wide, active, C)


# ---------------------------------------------------------------- whole epoch
@pytest.mark.parametrize("cfg,n_jobs,packed", [(0, None, False), (1, None, False), (2, None, True),
                                               (3, 3000, True), (4, 20000, False)])
def test_epoch_matches_oracle(slaq, oracle_mod, cfg, n_jobs, packed):
    wl = make_workload(cfg, n_jobs=n_jobs)
    sched = make_scheduler(wl, packed=packed)
    alloc, rc = sched.schedule(wl.epoch_seconds, wl.total_cores)
    assert rc == 0
    pred = sched.get_predictions()
    ref = oracle_epoch(oracle_mod, wl)
    info = compare_epoch(alloc, pred, ref, wl.total_cores, wl.max_cores_per_job)
    assert alloc.sum() == wl.total_cores
    assert alloc.min() >= 1 and alloc.max() <= wl.max_cores_per_job
    g = pred["gain"]
    assert (g >= 0).all() and (np.diff(g, axis=1) <= 0).all()
    stats = sched.get_stats()
    assert stats.cores_handed_out == wl.total_cores
    assert stats.points == wl.offsets[-1]
    assert stats.fitted_jobs == info["fitted"]
    sweeps = (ref["evals"].sum(axis=1) * wl.hist_len)[ref["status"] == 0].sum()
    assert abs(stats.model_sweeps - sweeps) <= 0.15 * sweeps      # same algorithm: about the same number of sweeps
    if cfg == 0:
        import json
        from pathlib import Path
        doc = json.loads((Path(__file__).parent / "golden" / "config0_oracle.json").read_text())
        assert alloc.tolist() == doc["alloc"]


def test_epoch_is_deterministic_and_repeatable(slaq):
    wl = make_workload(2)
    sched = make_scheduler(wl, packed=True)
    a1, _ = sched.schedule(wl.epoch_seconds, wl.total_cores)
    p1 = sched.get_predictions()
    a2, _ = sched.schedule(wl.epoch_seconds, wl.total_cores)
    p2 = sched.get_predictions()
    np.testing.assert_array_equal(a1, a2)
    for key in ("gain", "params", "S", "R"):
        np.testing.assert_array_equal(p1[key], p2[key])
    # and a second handle in ring layout gives the same bits as the packed one
    other = make_scheduler(wl, packed=False)
    a3, _ = other.schedule(wl.epoch_seconds, wl.total_cores)
    np.testing.assert_array_equal(a1, a3)
    np.testing.assert_array_equal(p1["gain"], other.get_predictions()["gain"])


def test_clones_get_identical_gains_and_ordered_ties(slaq, oracle_mod):
    wl = make_workload(4, n_jobs=30000)
    sched = make_scheduler(wl)
    alloc, _ = sched.schedule(wl.epoch_seconds, wl.total_cores)
    gain = sched.get_predictions()["gain"]
    dst = np.nonzero(wl.clone_of >= 0)[0]
    src = wl.clone_of[dst]
    np.testing.assert_array_equal(gain[dst], gain[src])
    lo, hi = np.minimum(src, dst), np.maximum(src, dst)
    assert (alloc[lo] >= alloc[hi]).all()


# ---------------------------------------------------------------- state: append path, ring, time law
def test_append_path_matches_oracle_scheduler(slaq, oracle_mod):
    wl = make_workload(1)
    J, max_hist, cap = wl.n_jobs, 16, wl.max_cores_per_job     # ring shorter than many histories: it wraps
    sched = slaq.Scheduler(J, max_hist, cap)
    ref = oracle_mod.OracleScheduler(J, max_hist, cap)
    H = wl.hist_len
    cores, secs = make_time_samples(wl, int(H.max()))
    for step in range(int(H.max())):
        live = np.nonzero(step < H)[0]
        losses = wl.losses[wl.offsets[live] + step]
        sched.append_losses(live, losses, secs[step, live], cores[step, live])
        ref.append_losses(live, losses, secs[step, live], cores[step, live])
        if step in (0, 1, 2, 5, 17, int(H.max()) - 1):
            alloc, _ = sched.schedule(wl.epoch_seconds, wl.total_cores)
            out = ref.schedule(wl.epoch_seconds, wl.total_cores)
            compare_epoch(alloc, sched.get_predictions(), out, wl.total_cores, cap)
    s, w = sched.get_time_model()
    rs, rw = ref.time_model()
    np.testing.assert_array_equal(s, rs)
    np.testing.assert_array_equal(w, rw)
    np.testing.assert_allclose(s, wl.s, rtol=1e-9)
    # default core count of a sample = the last allocation
    last = alloc.copy()
    t = wl.s + wl.w / last
    ids = np.arange(J)
    newest = wl.losses[wl.offsets[1:] - 1] * 0.97
    sched.append_losses(ids, newest, t)
    ref.append_losses(ids, newest, t)
    s2, w2 = sched.get_time_model()
    r2s, r2w = ref.time_model()
    np.testing.assert_array_equal(s2, r2s)
    np.testing.assert_array_equal(w2, r2w)


def test_short_flat_new_and_removed_jobs(slaq, oracle_mod):
    J, max_hist, cap = 12, 8, 6
    sched = slaq.Scheduler(J, max_hist, cap)
    ref = oracle_mod.OracleScheduler(J, max_hist, cap)
    histories = {
        0: [5.0],                                  # one point
        1: [5.0, 4.0],                             # two
        2: [5.0, 4.0, 3.5],                        # three
        3: [1.0, 2.0, 3.0, 4.0, 5.0],              # never fell
        4: [3.0, 3.0, 3.0, 3.0],                   # constant
        5: [9.0, 6.0, 4.5, 3.6, 3.0, 2.6, 2.3],    # ordinary
        6: [9.0, 6.0, 4.5, 3.6, 3.0, 2.6, 2.3, 2.1, 1.95, 1.85],   # longer than the ring
        7: [2.0, 1.0, 1.5, 0.7],                   # a rebound
    }
    for step in range(10):
        ids = [j for j, h in histories.items() if step < len(h)]
        vals = [histories[j][step] for j in ids]
        times = [1.0 + 0.1 * j for j in ids]
        cs = [1 + (step + j) % 3 for j in ids]
        sched.append_losses(ids, vals, times, cs)
        ref.append_losses(ids, vals, times, cs)
    for C in (3, 8, 20, 200):
        alloc, rc = sched.schedule(2.0, C)
        out = ref.schedule(2.0, C)
        compare_epoch(alloc, sched.get_predictions(), out, C, cap)
        assert (alloc[8:] == 0).all()
    status = sched.get_predictions()["status"]
    assert status[0] == slaq.JOB_NEW and status[1] == slaq.JOB_SHORT and status[3] == slaq.JOB_FLAT
    assert status[4] == slaq.JOB_FLAT and status[5] == slaq.JOB_FITTED and status[9] == slaq.JOB_INACTIVE
    sched.remove_jobs([5, 6])
    ref.remove_jobs([5, 6])
    alloc, _ = sched.schedule(2.0, 20)
    out = ref.schedule(2.0, 20)
    compare_epoch(alloc, sched.get_predictions(), out, 20, cap)
    assert alloc[5] == 0 and alloc[6] == 0
    # a job without any time sample predicts nothing
    sched.append_losses([10], [4.0])
    sched.append_losses([10], [3.0])
    ref.append_losses([10], [4.0])
    ref.append_losses([10], [3.0])
    alloc, _ = sched.schedule(2.0, 20)
    compare_epoch(alloc, sched.get_predictions(), ref.schedule(2.0, 20), 20, cap)
    assert sched.get_predictions()["status"][10] == slaq.JOB_NO_TIME


def test_empty_scheduler_and_argument_errors(slaq):
    sched = slaq.Scheduler(16, 8, 4)
    alloc, rc = sched.schedule(1.0, 10)
    assert (alloc == 0).all() and rc == 2
    with pytest.raises(slaq.SlaqError) as e:
        sched.append_losses([16], [1.0])
    assert e.value.code == -2
    with pytest.raises(slaq.SlaqError) as e:
        sched.append_losses([1, 1], [1.0, 2.0])
    assert e.value.code == -1
    with pytest.raises(slaq.SlaqError) as e:
        sched.append_losses([1], [float("nan")])
    assert e.value.code == -3
    with pytest.raises(slaq.SlaqError):
        sched.schedule(0.0, 10)
    with pytest.raises(slaq.SlaqError):
        sched.schedule(1.0, -1)
    with pytest.raises(slaq.SlaqError):
        sched.set_param(3, 5)                       # beyond the 4 cores per job the handle was made for
    with pytest.raises(slaq.SlaqError):
        sched.set_time_model([0], [0.1], [0.0])
    # nothing was applied by the failed calls
    alloc, _ = sched.schedule(1.0, 10)
    assert (alloc == 0).all()
    with pytest.raises(slaq.SlaqError):
        slaq.Scheduler(4, 100000, 4)                # window too long for one warp's shared memory


def test_a_rejected_append_leaves_the_state_untouched(slaq):
    """The library copies an append's arrays to the device while it checks them on the host; a batch that
    fails a check (a value that is not finite, an id listed twice, an id out of range) must change nothing."""
    wl = make_workload(1)
    sched = make_scheduler(wl)
    before, _ = sched.schedule(wl.epoch_seconds, wl.total_cores)
    gains = sched.get_predictions()["gain"].copy()
    ids = np.arange(wl.n_jobs, dtype=np.int32)
    good = 0.9 * wl.losses[wl.offsets[1:] - 1]
    for bad_ids, bad_losses, code in ((ids, np.where(ids == 77, np.inf, good), -3),
                                      (np.where(ids == 5, 4, ids).astype(np.int32), good, -1),
                                      (np.where(ids == 9, wl.n_jobs, ids).astype(np.int32), good, -2)):
        with pytest.raises(slaq.SlaqError) as e:
            sched.append_losses(bad_ids, bad_losses, np.ones(wl.n_jobs))
        assert e.value.code == code
        after, _ = sched.schedule(wl.epoch_seconds, wl.total_cores)
        np.testing.assert_array_equal(after, before)
        np.testing.assert_array_equal(sched.get_predictions()["gain"].view(np.int64), gains.view(np.int64))
    sched.append_losses(ids, good, np.ones(wl.n_jobs))        # and a clean batch is still taken
    sched.schedule(wl.epoch_seconds, wl.total_cores)
    assert not np.array_equal(sched.get_predictions()["gain"].view(np.int64), gains.view(np.int64))
    sched.close()


def test_caller_owned_workspace_and_stream(slaq, oracle_mod):
    import torch
    wl = make_workload(1)
    need = slaq.workspace_bytes(wl.n_jobs, wl.max_hist, wl.max_cores_per_job)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.Stream()
    sched = make_scheduler(wl, workspace=ws)
    sched.set_stream(stream)
    d_alloc = torch.zeros(wl.n_jobs, dtype=torch.int32, device="cuda")
    sched.schedule_device(wl.epoch_seconds, wl.total_cores, d_alloc)
    stream.synchronize()
    ref = oracle_epoch(oracle_mod, wl)
    compare_epoch(d_alloc.cpu().numpy(), sched.get_predictions(), ref, wl.total_cores, wl.max_cores_per_job)
    with pytest.raises(slaq.SlaqError):
        slaq.Scheduler(wl.n_jobs, wl.max_hist, wl.max_cores_per_job, workspace=ws[: need // 2])


def test_parameters_change_the_fit(slaq, oracle_mod):
    wl = make_workload(1)
    sched = make_scheduler(wl)
    sched.set_param(1, 0.8)      # gamma
    sched.set_param(2, 7)        # trials
    sched.set_param(3, 16)       # cores per job
    alloc, _ = sched.schedule(wl.epoch_seconds, wl.total_cores)
    ref = oracle_mod.schedule(wl.offsets, wl.losses, wl.m_seen, wl.s, wl.w, wl.epoch_seconds, wl.total_cores, 16,
                              gamma=0.8, lm_trials=7)
    compare_epoch(alloc, sched.get_predictions(), ref, wl.total_cores, 16)


# ---------------------------------------------------------------- window lengths at every class edge
def test_window_lengths_at_class_boundaries(slaq, oracle_mod):
    lengths = [4, 5, 7, 8, 9, 15, 16, 17, 31, 32, 33, 62, 63, 64, 65, 66, 124, 125, 126, 127, 128, 129, 249, 250, 251,
               252, 255, 256, 257, 499, 500, 501, 502, 511, 512, 513, 998, 999, 1000] * 3
    wl = make_workload(3, hist_lengths=lengths)
    for packed in (False, True):
        sched = make_scheduler(wl, packed=packed)
        alloc, _ = sched.schedule(wl.epoch_seconds, wl.total_cores)
        compare_epoch(alloc, sched.get_predictions(), oracle_epoch(oracle_mod, wl), wl.total_cores,
                      wl.max_cores_per_job)


def test_longest_supported_windows(slaq, oracle_mod):
    lengths = [6000, 5999, 4097, 3001, 3000, 1501, 1500, 751, 750, 400, 100, 20, 4, 3]
    wl = make_workload(3, hist_lengths=lengths)
    assert wl.max_hist == 6000
    sched = make_scheduler(wl, packed=True)
    alloc, _ = sched.schedule(wl.epoch_seconds, wl.total_cores)
    compare_epoch(alloc, sched.get_predictions(), oracle_epoch(oracle_mod, wl), wl.total_cores, wl.max_cores_per_job)
    ids = np.arange(wl.n_jobs)
    offsets, changes, levels, largest = sched.get_normalised(ids, capacity=int(wl.offsets[-1]))
    M, dn, y = oracle_mod.normalise(wl.offsets, wl.losses, wl.m_seen)
    np.testing.assert_array_equal(levels, y)
    np.testing.assert_array_equal(changes, dn)


@pytest.mark.parametrize("slice_bytes", [8192, 12288, 32768, 65536, 200 * 1024])
def test_lanes_per_job_do_not_change_results_beyond_rounding(slaq, oracle_mod, slice_bytes):
    wl = make_workload(3, n_jobs=1500)
    sched = make_scheduler(wl, packed=True)
    sched.set_param(5, slice_bytes)          # shared memory per warp: decides how many lanes share a job
    alloc, _ = sched.schedule(wl.epoch_seconds, wl.total_cores)
    compare_epoch(alloc, sched.get_predictions(), oracle_epoch(oracle_mod, wl), wl.total_cores, wl.max_cores_per_job)


@pytest.mark.parametrize("cluster_jobs", [0, 3000, 40000, 10_000_000])
def test_lanes_chosen_for_the_number_of_active_jobs_do_not_change_results_beyond_rounding(slaq, oracle_mod,
                                                                                          cluster_jobs):
    """With few active jobs a job gets up to a whole warp; a handle told that it is a shard of a large
    cluster uses as few lanes as its windows allow.  Either way the epoch matches the oracle."""
    wl = make_workload(3, n_jobs=1500)
    sched = make_scheduler(wl, packed=True)
    sched.set_param(slaq.binding.P_FIT_CLUSTER_JOBS, cluster_jobs)
    assert sched.get_param(slaq.binding.P_FIT_CLUSTER_JOBS) == cluster_jobs
    alloc, _ = sched.schedule(wl.epoch_seconds, wl.total_cores)
    compare_epoch(alloc, sched.get_predictions(), oracle_epoch(oracle_mod, wl), wl.total_cores, wl.max_cores_per_job)


@pytest.mark.parametrize("gamma", [1.0, 0.5, 0.99])
def test_other_weight_bases(slaq, oracle_mod, gamma):
    wl = make_workload(2, n_jobs=1200)
    sched = make_scheduler(wl)
    sched.set_param(1, gamma)
    alloc, _ = sched.schedule(wl.epoch_seconds, wl.total_cores)
    ref = oracle_mod.schedule(wl.offsets, wl.losses, wl.m_seen, wl.s, wl.w, wl.epoch_seconds, wl.total_cores,
                              wl.max_cores_per_job, gamma=gamma)
    compare_epoch(alloc, sched.get_predictions(), ref, wl.total_cores, wl.max_cores_per_job)


def test_other_seeds(slaq, oracle_mod):
    for seed in (1, 2, 3):
        wl = make_workload(2, seed_offset=seed)
        sched = make_scheduler(wl, packed=True)
        alloc, _ = sched.schedule(wl.epoch_seconds, wl.total_cores)
        compare_epoch(alloc, sched.get_predictions(), oracle_epoch(oracle_mod, wl), wl.total_cores,
                      wl.max_cores_per_job)


# ---------------------------------------------------------------- a packed load replaced by another
def test_a_second_packed_load_keeps_time_laws_and_drops_unlisted_jobs(slaq, oracle_mod):
    """Jobs listed again in a second packed load keep their time law, time sums and core count (a bulk load
    replaces histories only); jobs of the first load that are not listed again become inactive."""
    wl = make_workload(2, n_jobs=900)
    J, cap = wl.n_jobs, wl.max_cores_per_job
    ids = np.arange(J, dtype=np.int32)
    sched = slaq.Scheduler(J, wl.max_hist, cap)
    fixed = ids[: J // 2]                                    # a fixed law for the first half
    sched.set_time_model(fixed, wl.s[fixed], wl.w[fixed])
    sched.load_histories(ids, wl.offsets, wl.losses, wl.k_last, wl.m_seen, packed=True)
    sampled = ids[J // 2:]                                   # time samples for the second half: 2 and then 4 cores
    for n_cores in (2, 4):
        k = wl.k_last[sampled] + (1 if n_cores == 2 else 2)
        sched.append_losses(sampled, wl.losses[wl.offsets[sampled + 1] - 1] * 0.99,
                            wl.s[sampled] + wl.w[sampled] / n_cores, np.full(sampled.size, n_cores, np.int32))
    s_before, w_before = sched.get_time_model()
    assert np.isfinite(s_before).all() and np.isfinite(w_before).all()
    # second load: every third job is left out, the others get another seed's histories
    other = make_workload(2, n_jobs=J, seed_offset=4)
    keep = ids[ids % 3 != 0]
    H = other.hist_len[keep]
    off = np.concatenate([[0], np.cumsum(H)]).astype(np.int64)
    ls = np.concatenate([other.history(j) for j in keep])
    sched.load_histories(keep, off, ls, other.k_last[keep], other.m_seen[keep], packed=True)
    assert sched.get_active_count() == keep.size
    s_after, w_after = sched.get_time_model()
    np.testing.assert_array_equal(s_after[keep], s_before[keep])
    np.testing.assert_array_equal(w_after[keep], w_before[keep])
    gone = ids[ids % 3 == 0]
    assert np.isnan(s_after[gone]).all()
    C = 4 * keep.size
    alloc, rc = sched.schedule(wl.epoch_seconds, C)
    pred = sched.get_predictions()
    assert rc == 0 and (alloc[gone] == 0).all() and (pred["status"][gone] == slaq.JOB_INACTIVE).all()
    assert (pred["status"][keep] != slaq.JOB_NO_TIME).all()
    # oracle on the same state: all J ids, the dropped ones with empty histories
    H_all = np.zeros(J, np.int64)
    H_all[keep] = H
    off_all = np.concatenate([[0], np.cumsum(H_all)]).astype(np.int64)
    m_all = np.full(J, -np.inf)
    m_all[keep] = other.m_seen[keep]
    ref = oracle_mod.schedule(off_all, ls, m_all, s_before, w_before, wl.epoch_seconds, C, cap)
    compare_epoch(alloc, pred, ref, C, cap)
    # a third load into rings releases the packed pool's jobs that it lists, and later appends extend them
    sched.load_histories(keep[:10], off[:11], ls[:off[10]], other.k_last[keep[:10]], other.m_seen[keep[:10]])
    assert sched.get_active_count() == keep.size


# ---------------------------------------------------------------- four or more points, yet no curve can be started
@pytest.mark.parametrize("cluster_jobs", [0, 10_000_000])
@pytest.mark.parametrize("packed", [False, True])
def test_windows_without_a_usable_start_take_the_fallback(slaq, oracle_mod, packed, cluster_jobs):
    """Both families fail at their first guess (levels that are integers near 2^53 a few units apart; or a flat
    window scaled by a tiny largest-reduction-seen, whose squares overflow): the job is predicted from its weighted
    mean normalised change, capped by its newest level.  The failing windows sit between ordinary ones, at
    lengths of every class of lanes per job (cluster_jobs = 10^7: as few lanes per job as the window allows, so the
    short ones share a warp with fifteen other jobs; 0: a whole warp each)."""
    from workloads import make_unfittable_histories
    lengths = [4, 5, 6, 9, 33, 64, 82, 83, 204, 205, 408, 409, 816, 817, 1000]
    o1, l1, m1, drops = make_unfittable_histories(lengths, "staircase", seed=1)
    o2, l2, m2, _ = make_unfittable_histories(lengths, "flat", seed=2)
    wl = make_workload(3, hist_lengths=[7, 40, 90, 300, 600, 950] * 12)
    n_bad = len(lengths)
    # interleave: ordinary jobs first and last, the failing ones in the middle of the id range
    half = wl.n_jobs // 2
    pieces = [(wl.offsets[:half + 1], wl.losses[:wl.offsets[half]], wl.m_seen[:half]), (o1, l1, m1), (o2, l2, m2),
              (wl.offsets[half:] - wl.offsets[half], wl.losses[wl.offsets[half]:], wl.m_seen[half:])]
    H = np.concatenate([np.diff(o) for o, _, _ in pieces])
    offsets = np.concatenate([[0], np.cumsum(H)]).astype(np.int64)
    losses = np.concatenate([l for _, l, _ in pieces])
    m_seen = np.concatenate([m for _, _, m in pieces])
    J, cap, T = H.size, 16, 1.0
    rng = np.random.default_rng(5)
    s, w = rng.uniform(0.05, 0.5, J), rng.uniform(1.0, 100.0, J)
    C = 4 * J
    sched = slaq.Scheduler(J, 1000, cap)
    ids = np.arange(J, dtype=np.int32)
    sched.load_histories(ids, offsets, losses, H.astype(np.int64) - 1, m_seen, packed=packed)
    sched.set_time_model(ids, s, w)
    sched.set_param(slaq.binding.P_FIT_CLUSTER_JOBS, cluster_jobs)
    alloc, rc = sched.schedule(T, C)
    pred = sched.get_predictions()
    ref = oracle_mod.schedule(offsets, losses, m_seen, s, w, T, C, cap)
    compare_epoch(alloc, pred, ref, C, cap)
    stair = np.arange(half, half + n_bad)
    flat = np.arange(half + n_bad, half + 2 * n_bad)
    assert (pred["status"][stair] == slaq.JOB_FIT_FAILED).all() and (pred["status"][flat] == slaq.JOB_FIT_FAILED).all()
    assert (pred["family"][stair] == -1).all() and np.isinf(pred["S"][stair]).all()
    ordinary = np.setdiff1d(ids, np.concatenate([stair, flat]))
    assert (pred["status"][ordinary] == slaq.JOB_FITTED).all()
    # expected from the rule itself: changes are 1 at the falls and 0 elsewhere, weights 0.9^(H-1-i)
    n = np.arange(1, cap + 1)
    for k, j in enumerate(stair):
        i = np.arange(1, lengths[k])
        weight = 0.9 ** (lengths[k] - 1 - i)
        rho = (weight * np.isin(i, drops[k])).sum() / weight.sum()
        R = rho * T * n / (s[j] * n + w[j])
        np.testing.assert_allclose(np.cumsum(pred["gain"][j]), R, rtol=1e-12, atol=0)
        assert pred["params"][j, 1] == losses[offsets[j + 1] - 1] / 2.0 ** -53      # the cap: the newest level
    assert (pred["gain"][flat] == 0.0).all()
    assert sched.get_stats().fallback_jobs == 2 * n_bad


def test_unseen_cuts_survey(slaq, oracle_mod):
    """Cuts and seeds no other test uses, 100,000 jobs in all: how often does a job miss the tolerance on R(n), and
    why.  Twenty solver trials do not finish every fit.  Where the residual is nearly flat along a direction
    (converged jobs of config 4: sixty-four points of noise around a level), the end point of the unfinished
    iteration depends on rounding, for the oracle too: perturbing such a job's losses by 1e-13 moves the ORACLE'S
    OWN prediction by more than the tolerance.  Measured over 333,000 jobs of 40 unseen cuts: 5 jobs outside the
    tolerance (by factors 1.005 to 15.8), all in config 4, each within the oracle's own spread under that
    perturbation.  Asserted: every miss is explained that way (within 4 spreads), and there is at most one per
    25,000 jobs."""
    total, misses = 0, []
    for cfg, sizes in ((4, (9000, 23000, 31000)), (3, (2500, 6500)), (2, (2000, 3000)), (1, (160,))):
        for n in sizes:
            for seed in (5, 6) if n < 20000 else (5,):
                wl = make_workload(cfg, n_jobs=n, seed_offset=seed)
                cap = wl.max_cores_per_job
                sched = make_scheduler(wl, packed=cfg == 3)
                sched.schedule(wl.epoch_seconds, wl.total_cores)
                pred = sched.get_predictions()
                ref = oracle_mod.predict(wl.offsets, wl.losses, wl.m_seen, wl.s, wl.w, wl.epoch_seconds, cap)
                np.testing.assert_array_equal(pred["status"], ref["status"])
                Rg, Rc = np.cumsum(pred["gain"], axis=1), np.cumsum(ref["gain"], axis=1)
                tol = 1e-6 * np.abs(Rc) + 1e-9
                width = (np.abs(Rg - Rc) / tol).max(axis=1)
                tied = pred["family"] != ref["family"]
                for j in np.nonzero(tied)[0]:
                    S = ref["S"][j]
                    assert abs(S[0] - S[1]) <= 1e-9 * max(abs(S[0]), abs(S[1]))
                for j in np.nonzero((width > 1.0) & ~tied)[0]:
                    spread = oracle_spread(oracle_mod, wl, j, cap)
                    assert (np.abs(Rg[j] - Rc[j]) <= 4.0 * spread + tol[j]).all(), (
                        f"config {cfg}, {n} jobs, seed {seed}, job {j}: {width[j]:.2f} tolerances off, and the oracle's "
                        f"own result is stable ({(spread / tol[j]).max():.2f} tolerances under perturbation)")
                    misses.append((cfg, n, seed, int(j), float(width[j]), float((spread / tol[j]).max())))
                total += wl.n_jobs
                sched.close()
    print(f"survey: {total} jobs, misses (config, jobs, seed, job, tolerances off, oracle's own spread): {misses}")
    assert total >= 100_000
    assert len(misses) <= total // 25_000


# ---------------------------------------------------------------- streaming: append -> schedule with the allocation fed back
def test_streaming_epochs_with_allocation_feedback(slaq, oracle_mod):
    """Several epochs in a row: each job runs as many iterations as its allocation allows in the epoch, reports
    their losses and times (booked at the allocation), and is scheduled again.  Both sides carry their own state."""
    from workloads import true_curve
    wl = make_workload(1)
    J, cap, max_hist = wl.n_jobs, wl.max_cores_per_job, 24          # short ring: it wraps within the run
    sched = slaq.Scheduler(J, max_hist, cap)
    ref = oracle_mod.OracleScheduler(J, max_hist, cap)
    rng = np.random.default_rng(77)
    k_next = np.zeros(J, dtype=np.int64)
    alloc = np.ones(J, dtype=np.int32)
    T = wl.epoch_seconds
    for epoch in range(7):
        # iterations each job completes this epoch on its current cores (at least one, so every job reports)
        iters = np.maximum(1, np.floor(T * alloc / (wl.s * alloc + wl.w)).astype(np.int64))
        iters = np.minimum(iters, 6)
        for step in range(int(iters.max())):
            live = np.nonzero(step < iters)[0]
            k = k_next[live].astype(np.float64)
            losses = true_curve(wl.family[live], wl.params[live], k) * np.exp(0.01 * rng.standard_normal(live.size))
            times = wl.s[live] + wl.w[live] / alloc[live]
            sched.append_losses(live, losses, times)             # booked at the last allocation on both sides
            ref.append_losses(live, losses, times)
            k_next[live] += 1
        got, rc = sched.schedule(T, wl.total_cores)
        out = ref.schedule(T, wl.total_cores)
        compare_epoch(got, sched.get_predictions(), out, wl.total_cores, cap)
        s, w = sched.get_time_model()
        np.testing.assert_array_equal(s, out["s"])
        np.testing.assert_array_equal(w, out["w"])
        alloc = got.copy()
    assert (k_next >= 7).all()


def test_appends_from_device_memory(slaq, oracle_mod):
    """slaq_append_losses_device: the same update as the host call, from CUDA tensors and without a host wait; what
    the host call would refuse is skipped on the device and reported by the next epoch."""
    import torch
    wl = make_workload(1)
    J, cap, max_hist = wl.n_jobs, wl.max_cores_per_job, 24
    sched = slaq.Scheduler(J, max_hist, cap)
    ref = oracle_mod.OracleScheduler(J, max_hist, cap)
    ids = np.arange(J, dtype=np.int32)
    rng = np.random.default_rng(12)
    d_ids = torch.arange(J, dtype=torch.int32, device="cuda")
    first = wl.losses[wl.offsets[:-1]]
    sched.append_losses(ids, first, wl.s + wl.w)                  # the first loss activates a job: host call
    ref.append_losses(ids, first, wl.s + wl.w)
    for step in range(1, 40):                                    # the ring of 24 wraps
        losses = first / (1.0 + 0.2 * step) * np.exp(0.01 * rng.standard_normal(J))
        cores = np.full(J, 1 + step % 4, np.int32)
        times = wl.s + wl.w / cores
        sched.append_losses_device(d_ids, torch.from_numpy(losses).cuda(), torch.from_numpy(times).cuda(),
                                   torch.from_numpy(cores).cuda())
        ref.append_losses(ids, losses, times, cores)
        if step % 13 == 0:
            alloc, rc = sched.schedule(wl.epoch_seconds, wl.total_cores)
            out = ref.schedule(wl.epoch_seconds, wl.total_cores)
            compare_epoch(alloc, sched.get_predictions(), out, wl.total_cores, cap)
            s, w = sched.get_time_model()
            np.testing.assert_array_equal(s, out["s"])
            np.testing.assert_array_equal(w, out["w"])
    good, _ = sched.schedule(wl.epoch_seconds, wl.total_cores)
    # entries the host call would refuse: skipped, reported once, and the state is as before
    bad_ids = torch.tensor([0, 1, J + 5, 2], dtype=torch.int32, device="cuda")
    bad_losses = torch.tensor([float("nan"), float("inf"), 1.0, 1.0], dtype=torch.float64, device="cuda")
    bad_times = torch.tensor([1.0, 1.0, 1.0, float("nan")], dtype=torch.float64, device="cuda")
    sched.append_losses_device(bad_ids, bad_losses, bad_times)
    with pytest.raises(slaq.SlaqError) as err:
        sched.schedule(wl.epoch_seconds, wl.total_cores)
    assert err.value.code == -5 and "slaq_append_losses_device" in str(err.value)
    again, rc = sched.schedule(wl.epoch_seconds, wl.total_cores)
    assert rc == 0
    np.testing.assert_array_equal(again, good)
    fresh = slaq.Scheduler(4, 8, 2)                               # a job's first loss cannot come this way
    fresh.append_losses_device(torch.zeros(1, dtype=torch.int32, device="cuda"),
                               torch.ones(1, dtype=torch.float64, device="cuda"))
    with pytest.raises(slaq.SlaqError):
        fresh.schedule(1.0, 4)
    assert fresh.get_active_count() == 0
    with pytest.raises(slaq.SlaqError):
        sched.append_losses_device(d_ids, torch.ones(J, dtype=torch.float64, device="cuda"), None,
                                   torch.ones(J, dtype=torch.int32, device="cuda"))
