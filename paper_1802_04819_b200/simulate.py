"""Closed-loop trace simulation: jobs arrive over time, report losses, and are re-scheduled every epoch.

The shape follows the paper's cluster experiment (Evaluation, "Scheduler Quality and Runtime
Improvement": 160 jobs, Poisson arrivals with a mean of 15 s, an 800 s window, compared with a
work-conserving fair scheduler), with simulated jobs and workers as in its scalability experiment.
Jobs are synthetic convergence curves; nothing here reproduces the paper's numbers, which need its
jobs and datasets - the simulation shows the scheduling path working in a loop:
``append_losses`` -> ``schedule`` -> run an epoch at the allocation -> ``append_losses`` ...

    python -m paper_1802_04819_b200.simulate            # needs a GPU
"""

from __future__ import annotations

import numpy as np


def _curve(family, p, k):
    k = np.asarray(k, dtype=np.float64)
    if family == 0:
        return 1.0 / (p[0] * k * k + p[1] * k + p[2]) + p[3]
    return np.power(p[0], k - p[1]) + p[2]


def draw_trace(n_jobs=160, mean_gap=15.0, seed=0):
    """Arrival times and per-job curves / time laws (same parameter ranges as the benchmark workloads)."""
    rng = np.random.default_rng(seed)
    arrive = np.cumsum(rng.exponential(mean_gap, n_jobs))
    family = (rng.random(n_jobs) < 0.5).astype(np.int8)
    params = np.zeros((n_jobs, 4))
    for j in range(n_jobs):
        if family[j] == 0:
            params[j] = [rng.uniform(1e-4, 1e-2), rng.uniform(0.01, 1.0), rng.uniform(0.5, 2.0), rng.uniform(0, 0.1)]
        else:
            params[j] = [rng.uniform(0.80, 0.99), rng.uniform(0, 5.0), rng.uniform(0, 0.1), 0.0]
    s = rng.uniform(0.05, 0.5, n_jobs)
    w = rng.uniform(1.0, 100.0, n_jobs)
    return dict(arrive=arrive, family=family, params=params, s=s, w=w)


def loss_groups(norm_loss):
    """Positions (into `norm_loss`) of the quarter of the jobs with the highest normalised loss, of the next
    quarter, and of the lower half - the three groups of the paper's allocation-by-loss-group figure."""
    order = np.argsort(-np.asarray(norm_loss), kind="stable")
    n = order.size
    q = (n + 3) // 4
    return order[:q], order[q:min(2 * q, n)], order[min(2 * q, n):]


def run(trace, policy="slaq", total_cores=640, max_cores_per_job=64, epoch=3.0, horizon=800.0, max_hist=64,
        sigma=0.01, target=0.99, seed=1, scheduler_factory=None, keep_allocations=False):
    """Simulate one policy ("slaq" or "fair").  Returns per-epoch average normalised loss of the running
    jobs, per job the time from arrival to 90 % and 95 % loss reduction (NaN if not reached), and the share
    of the handed-out cores that went to the running jobs' top quarter / next quarter / lower half by
    normalised loss, averaged over the epochs with at least four running jobs.

    scheduler_factory(max_jobs, max_hist, max_cores_per_job): what schedules under policy "slaq" (default:
    this library's ``Scheduler``); it needs append_losses, schedule -> (alloc, status), remove_jobs and close.
    keep_allocations: also return every epoch's allocation vector."""
    J = trace["arrive"].size
    rng = np.random.default_rng(seed)
    if policy != "slaq":
        sched = None
    elif scheduler_factory is not None:
        sched = scheduler_factory(J, max_hist, max_cores_per_job)
    else:
        import paper_1802_04819_b200 as slaq
        sched = slaq.Scheduler(J, max_hist, max_cores_per_job)
    fam, par, s, w = trace["family"], trace["params"], trace["s"], trace["w"]
    first = np.array([_curve(fam[j], par[j], 0.0) for j in range(J)])
    last = np.array([_curve(fam[j], par[j], 1e9) for j in range(J)])
    k_done = np.zeros(J, dtype=np.int64)          # iterations completed
    credit = np.zeros(J)                          # fraction of an iteration carried over
    alloc = np.zeros(J, dtype=np.int64)
    state = np.zeros(J, dtype=np.int8)            # 0 not arrived, 1 running, 2 finished
    reached = {0.90: np.full(J, np.nan), 0.95: np.full(J, np.nan)}
    avg_loss, t = [], 0.0
    shares, allocations = [], []

    def norm_loss(j):
        return (_curve(fam[j], par[j], float(k_done[j])) - last[j]) / (first[j] - last[j])

    while t < horizon:
        # arrivals: a new job reports its initial loss (normalised loss 1.0)
        for j in np.nonzero((state == 0) & (trace["arrive"] <= t))[0]:
            state[j] = 1
            if sched is not None:
                # the initial loss costs one pass over the data on the single core the job starts with:
                # that pass is the job's first iteration-time sample (without one it would predict nothing)
                sched.append_losses([j], [first[j] * np.exp(sigma * rng.standard_normal())], [s[j] + w[j]], [1])
        running = np.nonzero(state == 1)[0]
        if running.size:
            if policy == "slaq":
                a, _ = sched.schedule(epoch, total_cores)
                alloc[:] = a
            else:   # work-conserving fair share
                share = min(max_cores_per_job, total_cores // running.size)
                alloc[:] = 0
                alloc[running] = max(share, 1) if total_cores >= running.size else 0
                extra = total_cores - int(alloc.sum())
                for j in running[:max(0, extra)]:
                    if alloc[j] < max_cores_per_job:
                        alloc[j] += 1
            if keep_allocations:
                allocations.append(alloc.copy())
            if running.size >= 4 and alloc[running].sum() > 0:
                before = np.array([norm_loss(j) for j in running])
                handed = float(alloc[running].sum())
                shares.append([alloc[running][g].sum() / handed for g in loss_groups(before)])
            # run the epoch: iterations each job completes on its cores, reported one by one
            n = np.maximum(alloc[running], 0)
            per_iter = s[running] + w[running] / np.maximum(n, 1)
            progress = np.where(n > 0, epoch / per_iter, 0.0) + credit[running]
            iters = np.floor(progress).astype(np.int64)
            credit[running] = progress - iters
            for step in range(int(iters.max()) if iters.size else 0):
                live = running[step < iters]
                k_done[live] += 1
                if sched is not None:
                    losses = np.array([_curve(fam[j], par[j], float(k_done[j])) for j in live])
                    losses *= np.exp(sigma * rng.standard_normal(live.size))
                    sched.append_losses(live, losses, s[live] + w[live] / np.maximum(alloc[live], 1))
            nl = np.array([norm_loss(j) for j in running])
            avg_loss.append(float(nl.mean()))
            for frac, store in reached.items():
                hit = running[(1.0 - nl >= frac) & np.isnan(store[running])]
                store[hit] = t + epoch - trace["arrive"][hit]
            done = running[1.0 - nl >= target]
            state[done] = 2
            if sched is not None and done.size:
                sched.remove_jobs(done)
        else:
            avg_loss.append(float("nan"))
        t += epoch
    if sched is not None:
        sched.close()
    share = np.mean(np.array(shares), axis=0) if shares else np.full(3, np.nan)
    out = dict(avg_loss=np.array(avg_loss), t90=reached[0.90], t95=reached[0.95], finished=int((state == 2).sum()),
               core_share_top_quarter=float(share[0]), core_share_next_quarter=float(share[1]),
               core_share_lower_half=float(share[2]))
    if keep_allocations:
        out["allocations"] = allocations
    return out


def compare(n_jobs=160, horizon=800.0, total_cores=320, seed=1):
    trace = draw_trace(n_jobs, seed=seed)
    a = run(trace, "slaq", total_cores=total_cores, horizon=horizon)
    b = run(trace, "fair", total_cores=total_cores, horizon=horizon)
    both = ~np.isnan(a["avg_loss"]) & ~np.isnan(b["avg_loss"])
    return dict(
        mean_loss_slaq=float(a["avg_loss"][both].mean()), mean_loss_fair=float(b["avg_loss"][both].mean()),
        t90_slaq=float(np.nanmean(a["t90"])), t90_fair=float(np.nanmean(b["t90"])),
        t95_slaq=float(np.nanmean(a["t95"])), t95_fair=float(np.nanmean(b["t95"])),
        finished_slaq=a["finished"], finished_fair=b["finished"],
        # share of the cores by loss group (the paper's cluster: 60 % to the top quarter, 22 % to the lower half)
        core_share_top_quarter_slaq=a["core_share_top_quarter"], core_share_lower_half_slaq=a["core_share_lower_half"],
        core_share_top_quarter_fair=b["core_share_top_quarter"], core_share_lower_half_fair=b["core_share_lower_half"],
    )


if __name__ == "__main__":
    import json
    print(json.dumps(compare()))
