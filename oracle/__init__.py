"""CPU oracle of the scheduling path: build, load and call `slaq_oracle.cpp`.

TEST INFRASTRUCTURE ONLY.  Nothing in the product package imports this module;
tests, the smoke check and the benchmark's CPU-baseline leg do.  The arithmetic
lives in `slaq_oracle.cpp`; this file marshals numpy arrays into it and keeps the
per-job state (stored window, largest reduction seen, iteration-time sums) that a
scheduler carries between epochs, in plain numpy.
"""

from __future__ import annotations

import ctypes
import os
import subprocess
from collections import deque
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "slaq_oracle.cpp"
_LIB = _HERE / "libslaq_oracle.so"

ST_INACTIVE, ST_FITTED, ST_SHORT, ST_NEW, ST_FIT_FAILED, ST_FLAT, ST_NONFINITE, ST_NO_TIME = -1, 0, 1, 2, 3, 4, 5, 6


def build(force: bool = False) -> Path:
    """Compile the oracle with g++ (no fused multiply-add contraction, OpenMP over jobs)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        cmd = ["g++", "-std=c++17", "-O2", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared",
               "-o", str(_LIB), str(_SRC)]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def _bind(lib):
    """Declare the argument types of every entry point of an oracle library."""
    c_i64, c_i32, c_f64, vp = ctypes.c_int64, ctypes.c_int32, ctypes.c_double, ctypes.c_void_p
    lib.oracle_max_threads.restype = ctypes.c_int
    lib.oracle_normalise.argtypes = [c_i64, vp, vp, vp, vp, vp, vp]
    lib.oracle_predict.argtypes = [c_i64, vp, vp, vp, vp, vp, c_f64, c_i32, c_f64, c_i32, c_i32,
                                   vp, vp, vp, vp, vp, vp, vp]
    lib.oracle_predict_warm.argtypes = [c_i64, vp, vp, vp, vp, vp, c_f64, c_i32, c_f64, c_i32, c_i32,
                                        vp, vp, vp, vp, vp, vp, vp] + [vp] * 8 + [c_i32, vp]
    lib.oracle_envelope.argtypes = [c_i32, vp, vp]
    lib.oracle_envelope.restype = None
    lib.oracle_carry.argtypes = [c_i32, vp, c_f64, c_f64, c_f64, vp]
    lib.oracle_carry.restype = None
    lib.oracle_allocate.argtypes = [c_i64, c_i32, vp, vp, c_i64, vp]
    lib.oracle_allocate.restype = c_i64
    lib.oracle_reduction_at.argtypes = [c_i64, c_i32, vp, vp, vp]
    lib.oracle_reduction_at.restype = None
    lib.oracle_time_model.argtypes = [c_i64] + [vp] * 10
    lib.oracle_time_model.restype = None
    lib.oracle_family_eval.argtypes = [c_i32, vp, c_f64, vp, vp]
    lib.oracle_lm_line.argtypes = [c_i64, vp, vp, vp, c_i32, c_f64, vp, vp]
    lib.oracle_fit_family.argtypes = [c_i32, c_i64, vp, c_f64, c_f64, c_i32, vp, vp, vp, vp]
    return lib


def _load():
    global _lib
    if _lib is not None:
        return _lib
    build()
    _lib = _bind(ctypes.CDLL(str(_LIB)))
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _i64(a):
    return np.ascontiguousarray(a, dtype=np.int64)


def max_threads() -> int:
    return int(_load().oracle_max_threads())


def normalise(offsets, losses, m_seen=None):
    """Step 1.  Returns (M [J], dnorm [sum H], y [sum H])."""
    lib = _load()
    offsets, losses = _i64(offsets), _f64(losses)
    J = offsets.size - 1
    m_seen = None if m_seen is None else _f64(m_seen)
    M = np.empty(J)
    dn = np.empty(losses.size)
    y = np.empty(losses.size)
    lib.oracle_normalise(J, _p(offsets), _p(losses), _p(m_seen), _p(M), _p(dn), _p(y))
    return M, dn, y


def predict(offsets, losses, m_seen, s, w, epoch_seconds, cap, gamma=0.9, lm_trials=20, threads=0,
            want_gain=True, k_last=None, warm=None, envelope=False, target_loss=None):
    """Steps 1-3.  Returns a dict with family, params, S, status, evals, M, gain [J, cap], and both
    families' final parameters (`both` [J, 8], `mask`).

    warm: dict(valid uint8 [J], p [J, 8], K int64 [J], span [J], M [J]) from an earlier epoch; the
    families it covers start from those parameters carried into this epoch's coordinates
    (k_last = index of each job's newest iteration now).
    envelope: rows become the slopes of the upper concave envelope of R(n) instead of a running minimum.
    target_loss: per job a loss below which nothing is predicted (NaN: no hint)."""
    lib = _load()
    offsets, losses = _i64(offsets), _f64(losses)
    J = offsets.size - 1
    m_seen = None if m_seen is None else _f64(m_seen)
    s, w = _f64(s), _f64(w)
    out = dict(
        family=np.empty(J, np.int8), params=np.empty((J, 4)), S=np.empty((J, 2)),
        status=np.empty(J, np.int32), evals=np.empty((J, 2), np.int32), M=np.empty(J),
        gain=np.empty((J, cap)) if want_gain else None,
        both=np.empty((J, 8)), mask=np.empty(J, np.uint8),
    )
    wv = wp = wK = wS = wM = None
    if warm is not None:
        wv = np.ascontiguousarray(warm["valid"], dtype=np.uint8)
        wp, wK, wS, wM = _f64(warm["p"]), _i64(warm["K"]), _f64(warm["span"]), _f64(warm["M"])
        k_last = _i64(k_last)
    lib.oracle_predict_warm(J, _p(offsets), _p(losses), _p(m_seen), _p(s), _p(w), float(epoch_seconds), int(cap),
                            float(gamma), int(lm_trials), int(threads), _p(out["family"]), _p(out["params"]),
                            _p(out["S"]), _p(out["status"]), _p(out["evals"]), _p(out["M"]), _p(out["gain"]),
                            _p(k_last) if warm is not None else None, _p(wv), _p(wp), _p(wK), _p(wS), _p(wM),
                            _p(out["both"]), _p(out["mask"]), int(bool(envelope)),
                            None if target_loss is None else _p(_f64(target_loss)))
    return out


def envelope(R):
    """Slopes of the upper concave envelope of the points (n, R[n]), n = 0..len(R)-1."""
    lib = _load()
    R = _f64(R)
    out = np.empty(R.size - 1)
    lib.oracle_envelope(R.size - 1, _p(R), _p(out))
    return out


def carry(family, p, t, r, sigma):
    """A family's parameters in window coordinates shifted by t, stretched by r, levels scaled by sigma."""
    lib = _load()
    p = _f64(p)
    out = np.empty(4)
    lib.oracle_carry(int(family), _p(p), float(t), float(r), float(sigma), _p(out))
    return out


def allocate(gain, active, total_cores):
    """Step 4: the literal greedy loop on gain rows [J, cap].  Returns alloc int32 [J]."""
    lib = _load()
    gain = _f64(gain)
    J, cap = gain.shape
    active = np.ascontiguousarray(active, dtype=np.uint8)
    alloc = np.empty(J, np.int32)
    lib.oracle_allocate(J, cap, _p(gain), _p(active), int(total_cores), _p(alloc))
    return alloc


def reduction_at(gain, alloc):
    """Predicted normalised loss reduction of each job at its allocation."""
    lib = _load()
    gain = _f64(gain)
    J, cap = gain.shape
    alloc = np.ascontiguousarray(alloc, dtype=np.int32)
    R = np.empty(J)
    lib.oracle_reduction_at(J, cap, _p(gain), _p(alloc), _p(R))
    return R


def time_model(cnt, su, suu, st, sut, stn, umin, umax):
    lib = _load()
    arrs = [_f64(a) for a in (cnt, su, suu, st, sut, stn, umin, umax)]
    J = arrs[0].size
    s = np.empty(J)
    w = np.empty(J)
    lib.oracle_time_model(J, *[_p(a) for a in arrs], _p(s), _p(w))
    return s, w


def schedule(offsets, losses, m_seen, s, w, epoch_seconds, total_cores, cap, gamma=0.9, lm_trials=20, threads=0,
             k_last=None, warm=None, envelope=False, target_loss=None):
    """One whole epoch on CSR histories.  Returns dict(alloc, R, gain, ...fit record)."""
    out = predict(offsets, losses, m_seen, s, w, epoch_seconds, cap, gamma, lm_trials, threads,
                  k_last=k_last, warm=warm, envelope=envelope, target_loss=target_loss)
    active = (np.diff(_i64(offsets)) > 0)
    out["alloc"] = allocate(out["gain"], active, total_cores)
    out["R"] = reduction_at(out["gain"], out["alloc"])
    return out


def family_eval(family, p, x):
    lib = _load()
    p = _f64(p)
    f = np.empty(1)
    jac = np.empty(4)
    ok = lib.oracle_family_eval(int(family), _p(p), float(x), _p(f), _p(jac))
    return bool(ok), float(f[0]), jac


def lm_line(x, y, w, trials, lambda0, p0):
    lib = _load()
    x, y, w = _f64(x), _f64(y), _f64(w)
    p = _f64(p0).copy()
    S = np.empty(1)
    evals = lib.oracle_lm_line(x.size, _p(x), _p(y), _p(w), int(trials), float(lambda0), _p(p), _p(S))
    return p, float(S[0]), evals


def fit_family(family, loss, m_seen=-np.inf, gamma=0.9, trials=20):
    """Fit one family on one history.  Returns dict(p, S, grad, p0, evals)."""
    lib = _load()
    loss = _f64(loss)
    p, S, g, p0 = np.empty(4), np.empty(1), np.empty(4), np.empty(4)
    evals = lib.oracle_fit_family(int(family), loss.size, _p(loss), float(m_seen), float(gamma), int(trials),
                                  _p(p), _p(S), _p(g), _p(p0))
    return dict(p=p, S=float(S[0]), grad=g, p0=p0, evals=evals)


class OracleScheduler:
    """The state a scheduler keeps between epochs, in plain numpy, with the oracle's arithmetic.

    Mirrors the library's calls (create / append_losses / load_histories / set_time_model /
    remove_jobs / schedule) so that a test can drive both with the same inputs.
    """

    def __init__(self, max_jobs: int, max_hist: int, max_cores_per_job: int, gamma=0.9, lm_trials=20):
        self.max_jobs, self.max_hist, self.cap = max_jobs, max_hist, max_cores_per_job
        self.gamma, self.lm_trials = gamma, lm_trials
        self.window = [deque(maxlen=max_hist) for _ in range(max_jobs)]
        self.k_last = np.full(max_jobs, -1, np.int64)
        self.m_seen = np.full(max_jobs, -np.inf)
        self.tm = np.zeros((max_jobs, 6))                 # count, sum u, sum u^2, sum t, sum u t, sum t n
        self.umin = np.full(max_jobs, np.inf)
        self.umax = np.full(max_jobs, -np.inf)
        self.s_set = np.full(max_jobs, np.nan)
        self.w_set = np.full(max_jobs, np.nan)
        self.last_alloc = np.ones(max_jobs, np.int32)
        # warm start: `fitted` is what the last epoch found, `warm` what the next fit starts from.
        # A job's `warm` is refreshed from `fitted` when its history changes, so an epoch repeated
        # without new losses starts from the same point and gives the same result.
        self.warm_start = False
        self.envelope = False                              # rows as slopes of the concave envelope of R(n)
        self.target = np.full(max_jobs, np.nan)            # target-loss hints (NaN: none)
        self.fitted = self._no_fit(max_jobs)
        self.warm = self._no_fit(max_jobs)

    @staticmethod
    def _no_fit(n):
        return dict(valid=np.zeros(n, np.uint8), p=np.full((n, 8), np.nan), K=np.zeros(n, np.int64),
                    span=np.ones(n), M=np.full(n, np.nan))

    def _carry_over(self, j):
        for key in self.warm:
            self.warm[key][j] = self.fitted[key][j]

    def _forget_fit(self, j):
        self.fitted["valid"][j] = 0
        self.warm["valid"][j] = 0

    def set_fit_state(self, state):
        """Make `state` (dict valid, p, K, span, M) the starting point of every job's next fit."""
        self.fitted = {k: np.array(state[k]) for k in ("valid", "p", "K", "span", "M")}
        self.warm = {k: np.array(state[k]) for k in ("valid", "p", "K", "span", "M")}

    def append_losses(self, job_ids, losses, iter_times=None, cores_used=None):
        for i, j in enumerate(job_ids):
            loss = float(losses[i])
            win = self.window[j]
            if len(win) > 0:
                self.m_seen[j] = max(self.m_seen[j], win[-1] - loss)
            win.append(loss)
            self.k_last[j] += 1
            self._carry_over(j)
            if iter_times is not None:
                n = int(cores_used[i]) if cores_used is not None else max(int(self.last_alloc[j]), 1)
                t = float(iter_times[i])
                u = 1.0 / n
                self.tm[j] += np.array([1.0, u, u * u, t, u * t, t * n])
                self.umin[j] = min(self.umin[j], u)
                self.umax[j] = max(self.umax[j], u)

    def load_histories(self, job_ids, offsets, losses, k_last, m_seen=None):
        for i, j in enumerate(job_ids):
            rows = losses[offsets[i]:offsets[i + 1]]
            self.window[j] = deque((float(v) for v in rows[-self.max_hist:]), maxlen=self.max_hist)
            self.k_last[j] = int(k_last[i])
            self.m_seen[j] = -np.inf if m_seen is None else float(m_seen[i])
            self._forget_fit(j)

    def set_time_model(self, job_ids, s, w):
        for i, j in enumerate(job_ids):
            self.s_set[j], self.w_set[j] = float(s[i]), float(w[i])

    def set_target_loss(self, job_ids, targets):
        for i, j in enumerate(job_ids):
            self.target[j] = float(targets[i])

    def remove_jobs(self, job_ids):
        for j in job_ids:
            self.target[j] = np.nan
            self.window[j].clear()
            self.k_last[j] = -1
            self.m_seen[j] = -np.inf
            self.tm[j] = 0.0
            self.umin[j], self.umax[j] = np.inf, -np.inf
            self.s_set[j] = self.w_set[j] = np.nan
            self.last_alloc[j] = 1
            self._forget_fit(j)

    def time_model(self):
        s, w = time_model(*(self.tm[:, i] for i in range(6)), self.umin, self.umax)
        have = np.isfinite(self.s_set)
        return np.where(have, self.s_set, s), np.where(have, self.w_set, w)

    def csr(self):
        H = np.array([len(win) for win in self.window], np.int64)
        offsets = np.zeros(self.max_jobs + 1, np.int64)
        np.cumsum(H, out=offsets[1:])
        losses = np.fromiter((v for win in self.window for v in win), dtype=np.float64, count=int(offsets[-1]))
        return offsets, losses

    def schedule(self, epoch_seconds, total_cores, threads=0):
        offsets, losses = self.csr()
        s, w = self.time_model()
        out = schedule(offsets, losses, self.m_seen, s, w, epoch_seconds, total_cores, self.cap,
                       self.gamma, self.lm_trials, threads, k_last=self.k_last,
                       warm=self.warm if self.warm_start else None, envelope=self.envelope,
                       target_loss=self.target if np.isfinite(self.target).any() else None)
        H = np.diff(offsets)
        self.fitted = dict(valid=out["mask"].copy(), p=out["both"].copy(), K=self.k_last.copy(),
                           span=np.maximum(H - 1, 1).astype(np.float64), M=out["M"].copy())
        active = H > 0
        self.last_alloc = np.where(active, out["alloc"], self.last_alloc).astype(np.int32)
        out["s"], out["w"] = s, w
        return out
