"""Seeded generators for the five scheduler workloads.

Every workload is a set of simulated training jobs, as in the paper's
scalability experiment (Evaluation, "Scalability and efficiency": jobs and
workers are both simulated).  A job is one of the paper's two convergence
families (Design, "Predicting Quality Improvement"),

    sublinear:   L(k) = 1 / (a k^2 + b k + c) + d
    exponential: L(k) = mu^(k - b0) + c0

sampled at consecutive iterations with multiplicative lognormal noise, plus an
iteration-time law t(n) = s + w / n on n cores.

Nothing here normalises, fits, predicts or allocates: this module only draws
numbers.  `numpy.random.default_rng(180204819 + cfg)` seeds every draw.
"""

from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

SEED_BASE = 180204819

# J jobs, C cores, cap = max cores per job, history length range, noise, epoch T.
CONFIGS = {
    0: dict(J=8, cores_per_job=8, cap=16, hmin=5, hmax=20, sigma=0.01, T=3.0),
    1: dict(J=160, cores_per_job=4, cap=32, hmin=3, hmax=40, sigma=0.01, T=3.0,
            converged_frac=0.10),
    2: dict(J=4000, cores_per_job=4, cap=64, hmin=3, hmax=200, sigma=0.02, T=3.0,
            outlier_frac=0.05),
    3: dict(J=100_000, cores_per_job=4, cap=64, hmin=3, hmax=1000, sigma=0.01, T=1.0,
            w_loguniform=True),
    4: dict(J=1_000_000, cores_per_job=4, cap=128, hmin=64, hmax=64, sigma=0.01, T=1.0,
            stages=True, clone_frac=0.01),
}

FAMILY_SUBLINEAR = 0
FAMILY_EXPONENTIAL = 1


@dataclass
class Workload:
    """One scheduling epoch's inputs, histories stored ragged (CSR)."""

    cfg: int
    n_jobs: int
    total_cores: int
    max_cores_per_job: int
    max_hist: int
    epoch_seconds: float
    offsets: np.ndarray        # int64 [J+1]; job j owns losses[offsets[j]:offsets[j+1]], oldest first
    losses: np.ndarray         # float64 [sum H]
    k_last: np.ndarray         # int64 [J]; iteration index of each job's newest loss (first ever = 0)
    m_seen: np.ndarray         # float64 [J]; largest one-step loss reduction over the job's whole life
    s: np.ndarray              # float64 [J]; serial seconds per iteration
    w: np.ndarray              # float64 [J]; parallel core-seconds per iteration
    family: np.ndarray         # int8 [J]; generating family (ground truth, tests only)
    params: np.ndarray         # float64 [J,4]; (a,b,c,d) or (mu,b0,c0,0) (ground truth, tests only)
    sigma: np.ndarray          # float64 [J]; noise level actually used
    m_past: np.ndarray = field(default_factory=lambda: np.zeros(0))   # float64 [J]; largest one-step reduction
                               # BEFORE the stored window only (-inf for a job whose window starts at iteration 0)
    clone_of: np.ndarray = field(default_factory=lambda: np.zeros(0, np.int64))  # int64 [J]; -1 or source id

    @property
    def hist_len(self) -> np.ndarray:
        return np.diff(self.offsets)

    def history(self, j: int) -> np.ndarray:
        return self.losses[self.offsets[j]:self.offsets[j + 1]]


def true_curve(family, params, k):
    """Noise-free loss of the generating curve at iteration(s) k (broadcasts)."""
    family = np.asarray(family)
    params = np.asarray(params, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    p0, p1, p2, p3 = (params[..., i] for i in range(4))
    sub = 1.0 / (p0 * k * k + p1 * k + p2) + p3
    with np.errstate(under="ignore"):
        # mu in (0, 1); only used where family == exponential
        mu = np.where(family == FAMILY_EXPONENTIAL, p0, 0.5)
        expo = np.power(mu, k - p1) + p2
    return np.where(family == FAMILY_SUBLINEAR, sub, expo)


def _past_max_reduction(family, params, k0):
    """Largest one-step reduction L(k-1)-L(k) of the noise-free curve for k = 1..k0.

    Both families peak early (the sublinear one no later than its inflection,
    k ~ sqrt(c / 3a) < 100 for the parameter ranges drawn here), so a scan of
    the first 200 steps is exhaustive.  Returns -inf where k0 == 0.
    """
    n = family.shape[0]
    out = np.full(n, -np.inf)
    idx = np.nonzero(k0 > 0)[0]
    chunk = 100_000
    for lo in range(0, idx.size, chunk):
        sel = idx[lo:lo + chunk]
        kmax = int(min(200, k0[sel].max()))
        k = np.arange(0, kmax + 1, dtype=np.float64)[None, :]
        vals = true_curve(family[sel, None], params[sel, None, :], k)
        red = vals[:, :-1] - vals[:, 1:]                       # red[:, i] is the step i -> i+1
        steps = np.arange(1, kmax + 1)[None, :]
        red = np.where(steps <= k0[sel, None], red, -np.inf)
        out[sel] = red.max(axis=1)
    return out


def make_workload(cfg: int, n_jobs: int | None = None, seed_offset: int = 0, hist_lengths=None) -> Workload:
    """Draw workload `cfg` (0..4).  `n_jobs` overrides J (cores scale with it); `hist_lengths`
    (one entry per job) replaces the drawn history lengths, for tests that need exact lengths."""
    spec = CONFIGS[cfg]
    if hist_lengths is not None:
        n_jobs = len(hist_lengths)
    J = int(spec["J"] if n_jobs is None else n_jobs)
    rng = np.random.default_rng(SEED_BASE + cfg + 1000 * seed_offset)
    cap = spec["cap"]
    C = spec["cores_per_job"] * J

    family = (rng.random(J) < 0.5).astype(np.int8)             # 1 = exponential
    params = np.zeros((J, 4))
    a = rng.uniform(1e-4, 1e-2, J)
    b = rng.uniform(0.01, 1.0, J)
    c = rng.uniform(0.5, 2.0, J)
    d = rng.uniform(0.0, 0.1, J)
    mu = rng.uniform(0.80, 0.99, J)
    b0 = rng.uniform(0.0, 5.0, J)
    c0 = rng.uniform(0.0, 0.1, J)
    sub = family == FAMILY_SUBLINEAR
    params[sub] = np.stack([a, b, c, d], axis=1)[sub]
    params[~sub] = np.stack([mu, b0, c0, np.zeros(J)], axis=1)[~sub]

    s = rng.uniform(0.05, 0.5, J)
    if spec.get("w_loguniform"):
        w = np.exp(rng.uniform(np.log(1.0), np.log(1000.0), J))
    else:
        w = rng.uniform(1.0, 100.0, J)

    H = rng.integers(spec["hmin"], spec["hmax"] + 1, J).astype(np.int64)
    if hist_lengths is not None:
        H = np.asarray(hist_lengths, dtype=np.int64).copy()
    k0 = np.zeros(J, dtype=np.int64)
    sigma = np.full(J, spec["sigma"])
    converged = np.zeros(J, dtype=bool)

    if spec.get("converged_frac"):
        converged = rng.random(J) < spec["converged_frac"]
        k0[converged] = 10_000
    if spec.get("stages"):
        u = rng.random(J)
        new = u < 0.2
        converged = u >= 0.8
        mid = ~new & ~converged
        H[new] = rng.integers(3, 6, int(new.sum()))
        k0[mid] = rng.integers(0, 501, int(mid.sum()))
        k0[converged] = 10_000

    past = _past_max_reduction(family, params, k0)
    if spec.get("stages"):
        # converged jobs must show normalised one-step changes below 1e-4: shrink their
        # noise so that a 5-sigma step of the noisy level stays under 1e-4 of the largest
        # reduction of their earlier life.
        level = true_curve(family, params, k0.astype(np.float64))
        quiet = 1e-4 * past / (level * np.sqrt(2.0) * 5.0)
        sigma = np.where(converged, np.minimum(sigma, quiet), sigma)

    offsets = np.zeros(J + 1, dtype=np.int64)
    np.cumsum(H, out=offsets[1:])
    total = int(offsets[-1])
    losses = np.empty(total)
    chunk = 20_000
    for lo in range(0, J, chunk):
        hi = min(J, lo + chunk)
        h = H[lo:hi]
        job = np.repeat(np.arange(lo, hi), h)
        pos = np.arange(int(h.sum())) - np.repeat(offsets[lo:hi] - offsets[lo], h)
        k = (k0[job] + pos).astype(np.float64)
        clean = true_curve(family[job], params[job], k)
        z = rng.standard_normal(job.size)
        losses[offsets[lo]:offsets[hi]] = clean * np.exp(sigma[job] * z)

    if spec.get("outlier_frac"):
        hit = np.nonzero(rng.random(J) < spec["outlier_frac"])[0]
        where = offsets[hit] + rng.integers(0, H[hit])
        losses[where] *= 1.5

    clone_of = np.full(J, -1, dtype=np.int64)
    if spec.get("clone_frac"):
        n_clone = int(round(spec["clone_frac"] * J))
        full = np.nonzero(H == spec["hmax"])[0]
        picks = rng.choice(full, size=2 * n_clone, replace=False)
        src, dst = picks[:n_clone], picks[n_clone:]
        for arr in (family, params, s, w, k0, sigma, past):
            arr[dst] = arr[src]
        hh = spec["hmax"]
        rows = losses.reshape(-1)  # view
        src_idx = offsets[src][:, None] + np.arange(hh)[None, :]
        dst_idx = offsets[dst][:, None] + np.arange(hh)[None, :]
        rows[dst_idx] = rows[src_idx]
        clone_of[dst] = src

    # largest reduction seen over the whole life = unseen past joined with the stored window
    starts = offsets[:-1]
    diffs = losses[:-1] - losses[1:]
    diffs_valid = np.ones(total - 1, dtype=bool)
    diffs_valid[offsets[1:-1] - 1] = False                      # steps that straddle two jobs
    diffs = np.where(diffs_valid, diffs, -np.inf)
    # every job holds at least two points, and each straddling step is -inf, so reducing from
    # one job's start to the next job's start covers exactly that job's own steps
    assert H.min() >= 2
    win = np.maximum.reduceat(np.append(diffs, -np.inf), starts)
    m_seen = np.maximum(past, win)

    return Workload(
        cfg=cfg, n_jobs=J, total_cores=C, max_cores_per_job=cap, max_hist=int(max(spec["hmax"], H.max())),
        epoch_seconds=float(spec["T"]), offsets=offsets, losses=losses,
        k_last=k0 + H - 1, m_seen=m_seen, s=s, w=w, family=family, params=params,
        sigma=sigma, clone_of=clone_of, m_past=past,
    )


def make_time_samples(wl: Workload, n_samples: int, jobs: np.ndarray | None = None):
    """Noise-free iteration-time samples t = s + w / n with n cycling 1, 2, 4, 8.

    Returns (cores int32 [n_samples, len(jobs)], seconds float64 [n_samples, len(jobs)]).
    """
    jobs = np.arange(wl.n_jobs) if jobs is None else np.asarray(jobs)
    cyc = np.array([1, 2, 4, 8], dtype=np.int32)
    cores = np.tile(cyc[np.arange(n_samples) % 4][:, None], (1, jobs.size)).astype(np.int32)
    secs = wl.s[jobs][None, :] + wl.w[jobs][None, :] / cores
    return cores, secs


def make_unfittable_histories(lengths, kind: str, seed: int = 0):
    """Histories of at least four points on which neither curve family can be started.

    kind "staircase": the loss sits just below 1 and falls by exactly one unit in the last place
    (2^-53) at one to four randomly chosen iterations and stays put otherwise.  Scaled by its
    largest one-step reduction such a window holds integers near 2^53 that span at most four
    units, so an offset placed a tenth of that span below the smallest level rounds back onto it.
    kind "flat": a constant loss; together with a tiny positive largest-reduction-seen (returned as
    m_seen = 1e-300) the scaled levels are of the order 1e300 and their squares overflow.

    Returns (offsets int64 [n+1], losses float64, m_seen float64 [n], drops: list of index arrays,
    the iterations i >= 1 at which history j fell).  Only numbers are drawn here.
    """
    rng = np.random.default_rng(SEED_BASE + 7000 + seed)
    lengths = np.asarray(lengths, dtype=np.int64)
    assert lengths.min() >= 4
    offsets = np.zeros(lengths.size + 1, dtype=np.int64)
    np.cumsum(lengths, out=offsets[1:])
    losses = np.empty(int(offsets[-1]))
    m_seen = np.full(lengths.size, -np.inf)
    drops = []
    unit = 2.0 ** -53
    for j, H in enumerate(lengths):
        if kind == "staircase":
            n_drops = int(rng.integers(1, 5))
            where = np.sort(rng.choice(np.arange(1, H), size=min(n_drops, H - 1), replace=False))
            fallen = np.zeros(H)
            fallen[where] = 1.0
            losses[offsets[j]:offsets[j + 1]] = 1.0 - np.cumsum(fallen) * unit   # exact: multiples of 2^-53 in [0.5, 1]
        elif kind == "flat":
            where = np.zeros(0, dtype=np.int64)
            losses[offsets[j]:offsets[j + 1]] = rng.uniform(0.5, 4.0)
            m_seen[j] = 1e-300
        else:
            raise ValueError(kind)
        drops.append(where)
    return offsets, losses, m_seen, drops
