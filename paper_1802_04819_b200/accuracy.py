"""How well the fitted curves predict ahead: error of the loss predicted `ahead` iterations after the newest
point, per curve family and noise level.

The paper reports under 5 % error ten iterations ahead on its own jobs (Design, "Predicting Quality
Improvement"); those jobs are not available, so this measures the same quantity on synthetic jobs of the two
families (parameter ranges of the benchmark workloads, multiplicative lognormal noise of width sigma).  Every
history is cut `ahead` iterations short, fitted by the library on the GPU, and the fitted curve is evaluated
`ahead` iterations past the cut against the noise-free generating curve.

    python -m paper_1802_04819_b200.accuracy            # needs a GPU; prints a table
"""

from __future__ import annotations

import numpy as np

SIGMAS = (0.0, 0.01, 0.02, 0.05)


def _curve(family, p, k):
    k = np.asarray(k, dtype=np.float64)
    sub = 1.0 / (p[:, 0] * k * k + p[:, 1] * k + p[:, 2]) + p[:, 3]
    expo = np.power(np.where(family == 1, p[:, 0], 0.5), k - p[:, 1]) + p[:, 2]
    return np.where(family == 0, sub, expo)


def draw_jobs(n_jobs, family, sigma, seed, hmin=30, hmax=200):
    """Histories of one family (0 sublinear, 1 exponential) from iteration 0, lengths uniform in [hmin, hmax]."""
    rng = np.random.default_rng(seed)
    p = np.zeros((n_jobs, 4))
    if family == 0:
        p[:] = np.stack([rng.uniform(1e-4, 1e-2, n_jobs), rng.uniform(0.01, 1.0, n_jobs), rng.uniform(0.5, 2.0, n_jobs),
                         rng.uniform(0.0, 0.1, n_jobs)], axis=1)
    else:
        p[:] = np.stack([rng.uniform(0.80, 0.99, n_jobs), rng.uniform(0.0, 5.0, n_jobs), rng.uniform(0.0, 0.1, n_jobs),
                         np.zeros(n_jobs)], axis=1)
    H = rng.integers(hmin, hmax + 1, n_jobs).astype(np.int64)
    fam = np.full(n_jobs, family, np.int8)
    offsets = np.zeros(n_jobs + 1, np.int64)
    np.cumsum(H, out=offsets[1:])
    job = np.repeat(np.arange(n_jobs), H)
    k = (np.arange(int(offsets[-1])) - np.repeat(offsets[:-1], H)).astype(np.float64)
    clean = _curve(fam[job], p[job], k)
    losses = clean * np.exp(sigma * rng.standard_normal(clean.size))
    return fam, p, H, offsets, losses


def measure(n_jobs=2000, ahead=10, sigmas=SIGMAS, seed=0):
    """Rows of (family, sigma, jobs fitted, median relative error, share of jobs under 5 %, share won by the
    generating family)."""
    import paper_1802_04819_b200 as slaq
    rows = []
    for family in (0, 1):
        for sigma in sigmas:
            fam, p, H, offsets, losses = draw_jobs(n_jobs, family, sigma, seed + 17 * family + int(1000 * sigma))
            cut = H - ahead
            off = np.zeros(n_jobs + 1, np.int64)
            np.cumsum(cut, out=off[1:])
            kept = np.concatenate([losses[offsets[j]:offsets[j] + cut[j]] for j in range(n_jobs)])
            ids = np.arange(n_jobs, dtype=np.int32)
            with slaq.Scheduler(n_jobs, int(H.max()), 4) as sched:
                sched.load_histories(ids, off, kept, cut - 1)
                sched.set_time_model(ids, np.full(n_jobs, 0.1), np.full(n_jobs, 10.0))
                sched.schedule(1.0, n_jobs)
                pred = sched.get_predictions(want_gain=False)
            ok = pred["status"] == slaq.JOB_FITTED
            x = ahead / (cut - 1.0)
            q = pred["params"]
            with np.errstate(all="ignore"):
                f = np.where(pred["family"] == 0, 1.0 / (q[:, 0] * x * x + q[:, 1] * x + q[:, 2]) + q[:, 3],
                             np.exp(q[:, 0] - q[:, 1] * x) + q[:, 2]) * pred["M"]
            truth = _curve(fam, p, (H - 1).astype(np.float64))
            err = (np.abs(f - truth) / truth)[ok]
            rows.append(dict(family="sublinear" if family == 0 else "exponential", sigma=sigma, fitted=int(ok.sum()),
                             median_error=float(np.median(err)), under_5_percent=float(np.mean(err < 0.05)),
                             generating_family_wins=float(np.mean(pred["family"][ok] == family))))
    return rows


if __name__ == "__main__":
    print(f"{'family':12s} {'sigma':>6s} {'fitted':>7s} {'median error':>13s} {'under 5 %':>10s} {'own family wins':>16s}")
    for r in measure():
        print(f"{r['family']:12s} {r['sigma']:6.2f} {r['fitted']:7d} {r['median_error']:13.4f} {r['under_5_percent']:10.3f} "
              f"{r['generating_family_wins']:16.3f}")
