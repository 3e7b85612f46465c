"""ctypes binding of libslaq.so: same names as the C ABI, argument marshalling only."""

from __future__ import annotations

import ctypes
from ctypes import POINTER, c_double, c_float, c_int, c_int8, c_int32, c_int64, c_size_t, c_void_p, c_char_p

import numpy as np

from .build import LIB, variant_path

JOB_INACTIVE, JOB_FITTED, JOB_SHORT, JOB_NEW, JOB_FIT_FAILED, JOB_FLAT, JOB_NONFINITE, JOB_NO_TIME = -1, 0, 1, 2, 3, 4, 5, 6
P_GAMMA, P_LM_TRIALS, P_MAX_CORES_PER_JOB, P_MIN_FIT_POINTS, P_FIT_SLICE_BYTES, P_WARM_START = 1, 2, 3, 4, 5, 6
P_FIT_CLUSTER_JOBS = 7
P_EPOCH_GRAPH = 8
P_GAIN_ENVELOPE = 9
P_SELECTION = 10
W_OVERSUBSCRIBED, W_UNDERFILLED = 1, 2

EXPORTED_SYMBOLS = [
    "slaq_create", "slaq_create_in", "slaq_workspace_bytes", "slaq_destroy", "slaq_last_error", "slaq_set_stream",
    "slaq_set_param", "slaq_get_param", "slaq_append_losses", "slaq_append_losses_ex", "slaq_append_losses_device",
    "slaq_load_histories",
    "slaq_load_histories_packed", "slaq_set_time_model", "slaq_set_target_loss", "slaq_remove_jobs", "slaq_schedule",
    "slaq_schedule_device",
    "slaq_get_predictions", "slaq_get_normalised", "slaq_get_time_model", "slaq_get_fit_state",
    "slaq_set_fit_state", "slaq_set_gains", "slaq_allocate_only",
    "slaq_get_stats", "slaq_get_fit_phase_cycles", "slaq_export_state_bytes", "slaq_export_state",
    "slaq_import_state", "slaq_allocate_static", "slaq_get_active_count", "slaq_shard_predict", "slaq_shard_histogram",
    "slaq_shard_pick", "slaq_shard_pass", "slaq_shard_count", "slaq_shard_finalise", "slaq_shard_count_device",
    "slaq_shard_finalise_device",
]


class Stats(ctypes.Structure):
    _fields_ = [
        ("ms_total", c_float), ("ms_fit", c_float), ("ms_gain", c_float), ("ms_alloc", c_float),
        ("launches", c_int32), ("active_jobs", c_int32), ("cores_handed_out", c_int64), ("points", c_int64),
        ("model_sweeps", c_int64), ("tie_units", c_int64), ("threshold", c_double), ("fitted_jobs", c_int32),
        ("sublinear_wins", c_int32), ("exponential_wins", c_int32), ("fallback_jobs", c_int32),
        ("nonconvex_fits", c_int32),
    ]

    def as_dict(self):
        return {name: getattr(self, name) for name, _ in self._fields_}


class SlaqError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__(f"slaq error {code}: {message}")
        self.code = code


_libs = {}


def load_library(variant: str | None = None):
    """Load libslaq.so (must have been built: ``python -m paper_1802_04819_b200.build``), or with
    ``variant`` an instrumented build of the same sources (``build.build_variant(variant)``)."""
    if variant in _libs:
        return _libs[variant]
    path = LIB if variant is None else variant_path(variant)
    if not path.exists():
        raise FileNotFoundError(f"{path} is missing: build the CUDA library first (paper_1802_04819_b200.build())")
    lib = ctypes.CDLL(str(path))
    vp = c_void_p
    sig = {
        "slaq_create": (c_int, [c_int32, c_int32, POINTER(vp)]),
        "slaq_create_in": (c_int, [vp, c_size_t, c_int32, c_int32, c_int32, POINTER(vp)]),
        "slaq_workspace_bytes": (c_size_t, [c_int32, c_int32, c_int32]),
        "slaq_destroy": (c_int, [vp]),
        "slaq_last_error": (c_char_p, [vp]),
        "slaq_set_stream": (c_int, [vp, vp]),
        "slaq_set_param": (c_int, [vp, c_int, c_double]),
        "slaq_get_param": (c_int, [vp, c_int, POINTER(c_double)]),
        "slaq_append_losses": (c_int, [vp, c_int32, vp, vp, vp]),
        "slaq_append_losses_ex": (c_int, [vp, c_int32, vp, vp, vp, vp]),
        "slaq_append_losses_device": (c_int, [vp, c_int32, vp, vp, vp, vp]),
        "slaq_load_histories": (c_int, [vp, c_int32, vp, vp, vp, vp, vp]),
        "slaq_load_histories_packed": (c_int, [vp, c_int32, vp, vp, vp, vp, vp]),
        "slaq_set_time_model": (c_int, [vp, c_int32, vp, vp, vp]),
        "slaq_set_target_loss": (c_int, [vp, c_int32, vp, vp]),
        "slaq_remove_jobs": (c_int, [vp, c_int32, vp]),
        "slaq_schedule": (c_int, [vp, c_double, c_int64, vp]),
        "slaq_schedule_device": (c_int, [vp, c_double, c_int64, vp]),
        "slaq_get_predictions": (c_int, [vp] * 9),
        "slaq_get_normalised": (c_int, [vp, c_int32, vp, c_int64, vp, vp, vp, vp]),
        "slaq_get_time_model": (c_int, [vp, vp, vp]),
        "slaq_get_fit_state": (c_int, [vp, vp, vp, vp, vp, vp]),
        "slaq_set_fit_state": (c_int, [vp, vp, vp, vp, vp, vp]),
        "slaq_set_gains": (c_int, [vp, vp]),
        "slaq_allocate_only": (c_int, [vp, c_int64, vp]),
        "slaq_get_stats": (c_int, [vp, POINTER(Stats)]),
        "slaq_get_fit_phase_cycles": (c_int, [vp, vp]),
        "slaq_export_state_bytes": (c_int, [vp, POINTER(c_size_t)]),
        "slaq_export_state": (c_int, [vp, vp, c_size_t]),
        "slaq_import_state": (c_int, [vp, vp, c_size_t]),
        "slaq_allocate_static": (c_int, [vp, c_int32, c_int32, c_int64, vp, vp, vp]),
        "slaq_get_active_count": (c_int, [vp, POINTER(c_int32)]),
        "slaq_shard_predict": (c_int, [vp, c_double, c_int32]),
        "slaq_shard_histogram": (c_int, [vp, c_int32, vp, c_int32]),
        "slaq_shard_pick": (c_int, [vp, c_int32, c_int64]),
        "slaq_shard_pass": (c_int, [vp, c_int32]),
        "slaq_shard_count": (c_int, [vp, POINTER(c_int64)]),
        "slaq_shard_finalise": (c_int, [vp, c_int64, vp]),
        "slaq_shard_count_device": (c_int, [vp, vp]),
        "slaq_shard_finalise_device": (c_int, [vp, vp, vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    _libs[variant] = lib
    return lib


def workspace_bytes(max_jobs: int, max_hist: int, max_cores_per_job: int) -> int:
    return int(load_library().slaq_workspace_bytes(max_jobs, max_hist, max_cores_per_job))


STATIC_MAX_JOBS = 32768


def allocate_static(d_gain, total_cores: int, d_out_alloc, d_out_reduction, stream=None) -> int:
    """slaq_allocate_static on torch CUDA tensors: gain float64 [n_jobs, cap], outputs int32 / float64 [n_jobs].

    Allocates nothing on the device; asynchronous on ``stream`` (a torch stream, a raw
    cudaStream_t or None).  Returns 0 or a warning code; raises SlaqError on an error code.
    """
    lib = load_library()
    n_jobs, cap = d_gain.shape
    assert d_gain.is_contiguous() and d_out_alloc.is_contiguous() and d_out_reduction.is_contiguous()
    raw = getattr(stream, "cuda_stream", stream)
    rc = lib.slaq_allocate_static(c_void_p(d_gain.data_ptr()), n_jobs, cap, int(total_cores),
                                  c_void_p(d_out_alloc.data_ptr()), c_void_p(d_out_reduction.data_ptr()),
                                  c_void_p(raw))
    if rc < 0:
        messages = {-1: "bad argument", -2: f"size beyond the static scratch (n_jobs <= {STATIC_MAX_JOBS}, cap <= 1024)",
                    -5: "a CUDA call failed"}
        raise SlaqError(rc, messages.get(rc, "error"))
    return rc


def _arr(a, dtype):
    return None if a is None else np.ascontiguousarray(a, dtype=dtype)


def _ptr(a):
    return None if a is None else a.ctypes.data_as(c_void_p)


class Scheduler:
    """One scheduler handle.  Methods mirror the C calls of the same name (without ``slaq_``)."""

    def __init__(self, max_jobs: int, max_hist: int, max_cores_per_job: int = 64, workspace=None, stream=None,
                 variant: str | None = None):
        """``workspace``: optional torch uint8 CUDA tensor of at least ``workspace_bytes(...)`` bytes
        (device memory owned by the caller); ``stream``: optional ``torch.cuda.Stream``;
        ``variant``: an instrumented build of the library (``build.VARIANTS``) instead of libslaq.so."""
        self._lib = load_library(variant)
        self._h = c_void_p()
        self.max_jobs, self.max_hist, self.max_cores_per_job = int(max_jobs), int(max_hist), int(max_cores_per_job)
        self._workspace = workspace
        if workspace is not None:
            rc = self._lib.slaq_create_in(c_void_p(workspace.data_ptr()), workspace.numel() * workspace.element_size(),
                                          max_jobs, max_hist, max_cores_per_job, ctypes.byref(self._h))
        else:
            rc = self._lib.slaq_create_in(None, 0, max_jobs, max_hist, max_cores_per_job, ctypes.byref(self._h))
        if rc < 0 or not self._h:
            raise SlaqError(rc, "slaq_create failed (is a CUDA device present?)")
        if stream is not None:
            self.set_stream(stream)

    # -- plumbing --
    def _check(self, rc: int) -> int:
        if rc < 0:
            raise SlaqError(rc, self._lib.slaq_last_error(self._h).decode())
        return rc

    def close(self):
        if getattr(self, "_h", None):
            self._lib.slaq_destroy(self._h)
            self._h = c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    # -- the C calls --
    def set_stream(self, stream):
        raw = getattr(stream, "cuda_stream", stream)
        return self._check(self._lib.slaq_set_stream(self._h, c_void_p(raw)))

    def set_param(self, key: int, value: float):
        rc = self._check(self._lib.slaq_set_param(self._h, key, float(value)))
        if key == P_MAX_CORES_PER_JOB:
            self.max_cores_per_job = int(value)
        return rc

    def get_param(self, key: int) -> float:
        out = c_double()
        self._check(self._lib.slaq_get_param(self._h, key, ctypes.byref(out)))
        return out.value

    def append_losses(self, job_ids, losses, iter_times=None, cores_used=None):
        ids, ls = _arr(job_ids, np.int32), _arr(losses, np.float64)
        ts, cs = _arr(iter_times, np.float64), _arr(cores_used, np.int32)
        if cs is None:
            return self._check(self._lib.slaq_append_losses(self._h, ids.size, _ptr(ids), _ptr(ls), _ptr(ts)))
        return self._check(self._lib.slaq_append_losses_ex(self._h, ids.size, _ptr(ids), _ptr(ls), _ptr(ts), _ptr(cs)))

    def append_losses_device(self, d_job_ids, d_losses, d_iter_times=None, d_cores_used=None):
        """One new iteration per listed job from torch CUDA tensors (int32 ids, float64 losses and times, int32
        cores), asynchronous on the handle's stream; only for jobs that already have a loss."""
        ptr = lambda t: None if t is None else c_void_p(t.data_ptr())   # noqa: E731
        assert d_job_ids.is_contiguous() and d_losses.is_contiguous() and d_job_ids.numel() == d_losses.numel()
        return self._check(self._lib.slaq_append_losses_device(self._h, d_job_ids.numel(), ptr(d_job_ids), ptr(d_losses),
                                                               ptr(d_iter_times), ptr(d_cores_used)))

    def load_histories(self, job_ids, offsets, losses, k_last, m_seen=None, packed=False):
        ids, off = _arr(job_ids, np.int32), _arr(offsets, np.int64)
        ls, kl, ms = _arr(losses, np.float64), _arr(k_last, np.int64), _arr(m_seen, np.float64)
        fn = self._lib.slaq_load_histories_packed if packed else self._lib.slaq_load_histories
        return self._check(fn(self._h, ids.size, _ptr(ids), _ptr(off), _ptr(ls), _ptr(kl), _ptr(ms)))

    def set_time_model(self, job_ids, s, w):
        ids, s, w = _arr(job_ids, np.int32), _arr(s, np.float64), _arr(w, np.float64)
        return self._check(self._lib.slaq_set_time_model(self._h, ids.size, _ptr(ids), _ptr(s), _ptr(w)))

    def set_target_loss(self, job_ids, targets):
        ids, t = _arr(job_ids, np.int32), _arr(targets, np.float64)
        return self._check(self._lib.slaq_set_target_loss(self._h, ids.size, _ptr(ids), _ptr(t)))

    def remove_jobs(self, job_ids):
        ids = _arr(job_ids, np.int32)
        return self._check(self._lib.slaq_remove_jobs(self._h, ids.size, _ptr(ids)))

    def schedule(self, epoch_seconds: float, total_cores: int, out_alloc=None):
        """Returns (alloc int32 [max_jobs], status) with status 0 or a warning code."""
        out = np.empty(self.max_jobs, np.int32) if out_alloc is None else out_alloc
        rc = self._check(self._lib.slaq_schedule(self._h, float(epoch_seconds), int(total_cores), _ptr(out)))
        return out, rc

    def schedule_device(self, epoch_seconds: float, total_cores: int, d_out_alloc=None):
        """Asynchronous epoch; ``d_out_alloc``: optional torch int32 CUDA tensor [max_jobs]."""
        ptr = None if d_out_alloc is None else c_void_p(d_out_alloc.data_ptr())
        return self._check(self._lib.slaq_schedule_device(self._h, float(epoch_seconds), int(total_cores), ptr))

    def get_predictions(self, want_gain=True):
        J, cap = self.max_jobs, self.max_cores_per_job
        out = dict(
            R=np.empty(J), gain=np.empty((J, cap)) if want_gain else None, family=np.empty(J, np.int8),
            params=np.empty((J, 4)), S=np.empty((J, 2)), status=np.empty(J, np.int32),
            evals=np.empty((J, 2), np.int32), M=np.empty(J),
        )
        self._check(self._lib.slaq_get_predictions(
            self._h, _ptr(out["R"]), _ptr(out["gain"]), _ptr(out["family"]), _ptr(out["params"]), _ptr(out["S"]),
            _ptr(out["status"]), _ptr(out["evals"]), _ptr(out["M"])))
        return out

    def get_normalised(self, job_ids, capacity=None):
        ids = _arr(job_ids, np.int32)
        cap = int(capacity if capacity is not None else ids.size * self.max_hist)
        offsets = np.empty(ids.size + 1, np.int64)
        changes, levels, largest = np.empty(cap), np.empty(cap), np.empty(ids.size)
        self._check(self._lib.slaq_get_normalised(self._h, ids.size, _ptr(ids), cap, _ptr(offsets), _ptr(changes),
                                                  _ptr(levels), _ptr(largest)))
        total = int(offsets[-1])
        return offsets, changes[:total], levels[:total], largest

    def get_time_model(self):
        s, w = np.empty(self.max_jobs), np.empty(self.max_jobs)
        self._check(self._lib.slaq_get_time_model(self._h, _ptr(s), _ptr(w)))
        return s, w

    def get_fit_state(self):
        """Both families' end points of the last epoch: dict(p [J, 8], valid uint8 [J], K int64 [J], span, M)."""
        J = self.max_jobs
        st = dict(p=np.empty((J, 8)), valid=np.empty(J, np.uint8), K=np.empty(J, np.int64), span=np.empty(J),
                  M=np.empty(J))
        self._check(self._lib.slaq_get_fit_state(self._h, _ptr(st["p"]), _ptr(st["valid"]), _ptr(st["K"]),
                                                 _ptr(st["span"]), _ptr(st["M"])))
        return st

    def set_fit_state(self, state):
        """Make `state` (as returned by get_fit_state) the starting point of every job's next fit."""
        J = self.max_jobs
        p, valid = _arr(state["p"], np.float64), _arr(state["valid"], np.uint8)
        K, span, M = _arr(state["K"], np.int64), _arr(state["span"], np.float64), _arr(state["M"], np.float64)
        assert p.shape == (J, 8) and valid.shape == (J,) and K.shape == (J,) and span.shape == (J,) and M.shape == (J,)
        return self._check(self._lib.slaq_set_fit_state(self._h, _ptr(p), _ptr(valid), _ptr(K), _ptr(span), _ptr(M)))

    def set_gains(self, gain):
        g = _arr(gain, np.float64)
        assert g.shape == (self.max_jobs, self.max_cores_per_job)
        return self._check(self._lib.slaq_set_gains(self._h, _ptr(g)))

    def allocate_only(self, total_cores: int):
        out = np.empty(self.max_jobs, np.int32)
        rc = self._check(self._lib.slaq_allocate_only(self._h, int(total_cores), _ptr(out)))
        return out, rc

    # -- one cluster sharded over several GPUs: the steps between which histograms are summed --
    def get_active_count(self) -> int:
        out = c_int32()
        self._check(self._lib.slaq_get_active_count(self._h, ctypes.byref(out)))
        return out.value

    def shard_predict(self, epoch_seconds: float, with_floor: bool):
        return self._check(self._lib.slaq_shard_predict(self._h, float(epoch_seconds), int(bool(with_floor))))

    def shard_histogram(self, pass_index: int, d_hist, import_it: bool):
        """``d_hist``: torch int64 CUDA tensor of 2048 entries (the counts stay far below 2^63)."""
        return self._check(self._lib.slaq_shard_histogram(self._h, pass_index, c_void_p(d_hist.data_ptr()),
                                                          int(bool(import_it))))

    def shard_pick(self, pass_index: int, want: int):
        return self._check(self._lib.slaq_shard_pick(self._h, pass_index, int(want)))

    def shard_pass(self, pass_index: int):
        return self._check(self._lib.slaq_shard_pass(self._h, pass_index))

    def shard_count(self) -> int:
        out = c_int64()
        self._check(self._lib.slaq_shard_count(self._h, ctypes.byref(out)))
        return out.value

    def shard_finalise(self, ties_before: int):
        out = np.empty(self.max_jobs, np.int32)
        self._check(self._lib.slaq_shard_finalise(self._h, int(ties_before), _ptr(out)))
        return out

    def export_state(self) -> np.ndarray:
        """The whole per-job state of the handle as one blob (uint8 array)."""
        n = c_size_t()
        self._check(self._lib.slaq_export_state_bytes(self._h, ctypes.byref(n)))
        blob = np.zeros(n.value, np.uint8)
        self._check(self._lib.slaq_export_state(self._h, _ptr(blob), blob.size))
        return blob

    def import_state(self, blob):
        blob = np.ascontiguousarray(blob, dtype=np.uint8)
        return self._check(self._lib.slaq_import_state(self._h, _ptr(blob), blob.size))

    def get_fit_phase_cycles(self):
        """SM cycles the fit kernel's warps spent per phase (zeros unless the "clocks" variant is loaded)."""
        out = np.zeros(6, np.int64)
        self._check(self._lib.slaq_get_fit_phase_cycles(self._h, _ptr(out)))
        return out

    def shard_count_device(self, d_ties):
        """``d_ties``: torch int64 CUDA tensor of one entry that receives this shard's tie count (no host wait)."""
        return self._check(self._lib.slaq_shard_count_device(self._h, c_void_p(d_ties.data_ptr())))

    def shard_finalise_device(self, d_ties_before):
        """``d_ties_before``: torch int64 CUDA tensor of one entry, ordered on the handle's stream."""
        out = np.empty(self.max_jobs, np.int32)
        self._check(self._lib.slaq_shard_finalise_device(self._h, c_void_p(d_ties_before.data_ptr()), _ptr(out)))
        return out

    def get_stats(self) -> Stats:
        st = Stats()
        self._check(self._lib.slaq_get_stats(self._h, ctypes.byref(st)))
        return st
