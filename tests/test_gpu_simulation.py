"""Closed loop: arrivals, appends, epochs, removals - the scheduling path driven the way a cluster would.

Shaped after the paper's cluster experiment (Poisson arrivals, comparison with a fair share); the jobs are
synthetic, so only the direction of the effect is checked: giving cores to the jobs with the largest predicted
loss reduction lowers the average normalised loss of the running jobs."""

import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def test_quality_driven_beats_fair_share_on_a_synthetic_trace():
    import paper_1802_04819_b200 as slaq
    slaq.build()
    from paper_1802_04819_b200.simulate import compare
    out = compare(n_jobs=60, horizon=400.0, total_cores=240, seed=3)
    print(out)
    assert out["mean_loss_slaq"] < 0.9 * out["mean_loss_fair"]      # measured: 0.171 against 0.217
    assert out["t90_slaq"] < 0.85 * out["t90_fair"]                 # measured: 35 s against 57 s to 90 % reduction
    # cores follow the loss: the quarter of the jobs with the highest normalised loss gets more than its head count
    # (the paper's cluster: 60 % to that quarter, 22 % to the lower half; a fair share gives 25 % / 50 % by count)
    assert out["core_share_top_quarter_slaq"] > out["core_share_top_quarter_fair"] + 0.05
    assert out["core_share_lower_half_slaq"] < out["core_share_lower_half_fair"] - 0.05


def test_the_simulated_cluster_is_the_same_under_the_oracle(oracle_mod):
    """The closed loop driven once by the library and once by the CPU oracle's scheduler on the same trace and the
    same noise: every epoch's allocation is identical, hence every reported figure."""
    import paper_1802_04819_b200 as slaq
    slaq.build()
    from paper_1802_04819_b200.simulate import draw_trace, run

    class OracleDriven:
        def __init__(self, max_jobs, max_hist, cap):
            self.inner = oracle_mod.OracleScheduler(max_jobs, max_hist, cap)

        def append_losses(self, ids, losses, times=None, cores=None):
            self.inner.append_losses(list(ids), list(losses), None if times is None else list(times),
                                     None if cores is None else list(cores))

        def schedule(self, epoch, total_cores):
            return self.inner.schedule(epoch, total_cores)["alloc"], 0

        def remove_jobs(self, ids):
            self.inner.remove_jobs(list(ids))

        def close(self):
            pass

    trace = draw_trace(40, mean_gap=6.0, seed=5)
    kw = dict(total_cores=160, max_cores_per_job=32, horizon=420.0, keep_allocations=True)
    gpu = run(trace, "slaq", **kw)
    cpu = run(trace, "slaq", scheduler_factory=OracleDriven, **kw)
    assert len(gpu["allocations"]) == len(cpu["allocations"]) > 100
    for epoch, (a, b) in enumerate(zip(gpu["allocations"], cpu["allocations"])):
        np.testing.assert_array_equal(a, b, err_msg=f"epoch {epoch}")
    np.testing.assert_array_equal(gpu["avg_loss"], cpu["avg_loss"])
    np.testing.assert_array_equal(gpu["t90"], cpu["t90"])
    for key in ("core_share_top_quarter", "core_share_next_quarter", "core_share_lower_half", "finished"):
        assert gpu[key] == cpu[key]
    assert gpu["finished"] >= 1 and np.isfinite(gpu["t90"]).sum() > 20


def test_prediction_ten_iterations_ahead_on_the_gpu():
    """The paper reports under 5 % error when predicting the 10th next iteration; here on the noisy synthetic
    jobs, with the fit done by the GPU library on histories cut 10 iterations short."""
    import paper_1802_04819_b200 as slaq
    from workloads import make_workload, true_curve
    wl = make_workload(2, n_jobs=3000)
    H = wl.hist_len
    keep = np.nonzero(H >= 30)[0]
    cut = H[keep] - 10
    off = np.zeros(keep.size + 1, np.int64)
    np.cumsum(cut, out=off[1:])
    losses = np.concatenate([wl.history(j)[:c] for j, c in zip(keep, cut)])
    ids = np.arange(keep.size, dtype=np.int32)
    with slaq.Scheduler(keep.size, wl.max_hist, 4) as sched:
        sched.load_histories(ids, off, losses, cut - 1)
        sched.set_time_model(ids, wl.s[keep], wl.w[keep])
        sched.schedule(3.0, keep.size)
        pred = sched.get_predictions(want_gain=False)
    ok = pred["status"] == slaq.JOB_FITTED
    x = 10.0 / (cut - 1)
    p = pred["params"]
    f = np.where(pred["family"] == 0, 1.0 / (p[:, 0] * x * x + p[:, 1] * x + p[:, 2]) + p[:, 3],
                 np.exp(p[:, 0] - p[:, 1] * x) + p[:, 2]) * pred["M"]
    truth = true_curve(wl.family[keep], wl.params[keep], (H[keep] - 1).astype(float))
    err = np.abs(f - truth)[ok] / truth[ok]
    print("median error 10 ahead:", np.median(err), "share under 5 %:", np.mean(err < 0.05))
    assert np.median(err) < 0.05
    assert np.mean(err < 0.05) > 0.7


def test_prediction_accuracy_by_family_and_noise_level():
    """The accuracy table's figures: clean curves are predicted closely, the error grows with the noise,
    and at the benchmark's noise level the median stays under the paper's 5 %."""
    import paper_1802_04819_b200 as slaq
    slaq.build()
    from paper_1802_04819_b200.accuracy import measure
    rows = measure(n_jobs=600)
    by = {(r["family"], r["sigma"]): r for r in rows}
    for family in ("sublinear", "exponential"):
        # twenty trials do not finish every clean sublinear fit: 0.7 % there, 1e-5 on clean exponentials
        assert by[(family, 0.0)]["median_error"] < (0.02 if family == "sublinear" else 1e-3)
        assert by[(family, 0.01)]["median_error"] < 0.05 and by[(family, 0.01)]["under_5_percent"] > 0.7
        errs = [by[(family, s)]["median_error"] for s in (0.0, 0.01, 0.02, 0.05)]
        assert errs == sorted(errs), errs
        assert all(r["fitted"] == 600 for r in rows)
    print(rows)
